"""Seeded synthetic workloads: shapes, device tables and random tensors.

This module serves both the CUDA library's callers and the CPU oracle's tests,
so it holds no arithmetic of the method itself: only the workload tables and
calls to the seeded normal / uniform generators.  Tensors take LLaMA FFN
*shapes*; values are i.i.d. draws as each workload states.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple

import numpy as np
import torch

SHARE_ONE = 65536  # integer weight that stands for a capacity share of 1.0


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    d_model: int
    d_ffn: int
    group_size: int
    pred_rank: int
    dtype: str                      # "f32" | "bf16": storage type of weights and activations
    loss_rate: Tuple[float, ...]    # per virtual device
    share_weight: Tuple[int, ...]   # integer capacity weights per virtual device
    keep_permille: int              # critical (master-held) share of the groups, in 1/1000
    steps: int
    n_tok: int = 1
    seed: int = 0
    weight_std: float = 0.02
    pred_std: float = 0.05

    @property
    def n_groups(self) -> int:
        return self.d_ffn // self.group_size

    @property
    def n_dev(self) -> int:
        return len(self.loss_rate)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def group_bytes(self) -> int:
        return 3 * self.group_size * self.d_model * self.elem_bytes

    @property
    def layer_bytes(self) -> int:
        return self.n_groups * self.group_bytes

    @property
    def pred_bytes(self) -> int:
        return (self.d_model * self.pred_rank + self.pred_rank * self.n_groups) * self.elem_bytes


def _hetero_devices(n: int, seed: int):
    """Capacity shares ~ U(0.5, 2) and loss rates ~ U(0, 0.3) from a seeded host generator."""
    rng = np.random.Generator(np.random.PCG64(seed * 1000003 + 77))
    shares = rng.uniform(0.5, 2.0, size=n)
    loss = rng.uniform(0.0, 0.3, size=n)
    return tuple(float(v) for v in loss), tuple(int(round(s * SHARE_ONE)) for s in shares)


_L13, _S13 = _hetero_devices(8, 0)

WORKLOADS = {
    "tiny": Workload("tiny", 1, 256, 688, 16, 32, "f32", (0.0, 0.3), (SHARE_ONE,) * 2, 500, 1),
    "tinyllama-1.1b-decode": Workload("tinyllama-1.1b-decode", 22, 2048, 5632, 64, 128, "bf16",
                                      (0.0, 0.0, 0.05, 0.2), (SHARE_ONE,) * 4, 500, 256),
    "llama2-7b-decode": Workload("llama2-7b-decode", 32, 4096, 11008, 128, 256, "bf16",
                                 (0.0, 0.01, 0.1, 0.3), (SHARE_ONE,) * 4, 500, 256),
    "llama2-13b-decode": Workload("llama2-13b-decode", 40, 5120, 13824, 128, 512, "bf16", _L13, _S13, 500, 128),
    "llama2-7b-prefill": Workload("llama2-7b-prefill", 32, 4096, 11008, 128, 256, "bf16",
                                  (0.0, 0.01, 0.1, 0.3), (SHARE_ONE,) * 4, 500, 1, n_tok=512),
}


def workload(name: str, **overrides) -> Workload:
    wl = WORKLOADS[name]
    return replace(wl, **overrides) if overrides else wl


def small_variant(wl: Workload, n_layers: int, steps: int) -> Workload:
    """Same per-layer shapes, fewer layers / steps (what a CPU check can afford)."""
    return replace(wl, n_layers=n_layers, steps=steps)


# tensor ids inside one layer's seed space
_T_GATE, _T_UP, _T_DOWN, _T_PACKED, _T_W1, _T_W2 = range(6)


def _gen(seed: int, tensor_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + tensor_id) % (2**63 - 1))
    return g


def _normal(shape, std, dtype, gen, device):
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=gen)
    return t.to(dtype)


def ffn_matrices(wl: Workload, layer: int, device="cpu"):
    """Conventional matrices Wgate[F][d], Wup[F][d], Wdown[d][F]."""
    base = 100 * (layer + 1)
    d, F = wl.d_model, wl.d_ffn
    wg = _normal((F, d), wl.weight_std, wl.torch_dtype, _gen(wl.seed, base + _T_GATE, device), device)
    wu = _normal((F, d), wl.weight_std, wl.torch_dtype, _gen(wl.seed, base + _T_UP, device), device)
    wd = _normal((d, F), wl.weight_std, wl.torch_dtype, _gen(wl.seed, base + _T_DOWN, device), device)
    return wg, wu, wd


def packed_layer(wl: Workload, layer: int, device="cpu", out: torch.Tensor | None = None) -> torch.Tensor:
    """One layer drawn directly in the packed layout W[G][3][S][d] (i.i.d., so the
    distribution equals packing the conventional matrices)."""
    base = 100 * (layer + 1)
    shape = (wl.n_groups, 3, wl.group_size, wl.d_model)
    t = _normal(shape, wl.weight_std, wl.torch_dtype, _gen(wl.seed, base + _T_PACKED, device), device)
    if out is not None:
        out.copy_(t)
        return out
    return t


def predictor(wl: Workload, layer: int, device="cpu"):
    """Predictor factors W1[r][d], W2[G][r]."""
    base = 100 * (layer + 1)
    w1 = _normal((wl.pred_rank, wl.d_model), wl.pred_std, wl.torch_dtype, _gen(wl.seed, base + _T_W1, device), device)
    w2 = _normal((wl.n_groups, wl.pred_rank), wl.pred_std, wl.torch_dtype, _gen(wl.seed, base + _T_W2, device), device)
    return w1, w2


def stream_input(wl: Workload, step: int, device="cpu") -> torch.Tensor:
    """Fresh residual-stream input h_0 ~ N(0,1), fp32 [n_tok][d], one per step."""
    g = _gen(wl.seed, 10_000_000 + step, device)
    t = torch.empty((wl.n_tok, wl.d_model), dtype=torch.float32, device=device)
    t.normal_(0.0, 1.0, generator=g)
    return t


def activation(wl: Workload, tag: int, device="cpu", n_tok: int | None = None) -> torch.Tensor:
    """x ~ N(0,1) in the workload's storage dtype, [n_tok][d]."""
    g = _gen(wl.seed, 20_000_000 + tag, device)
    t = torch.empty((n_tok or wl.n_tok, wl.d_model), dtype=torch.float32, device=device)
    t.normal_(0.0, 1.0, generator=g)
    return t.to(wl.torch_dtype)


def host_bits(t: torch.Tensor) -> np.ndarray:
    """Byte copy of a tensor for the oracle: fp32 stays float32, bf16 becomes its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def structured_layer(wl: Workload, layer: int, device="cpu", scale_sigma: float = 0.8, coherence: float = 1.5,
                     latent: int = 32):
    """A packed layer whose groups are NOT exchangeable, plus a matching input distribution, for calibrating and
    evaluating a predictor without any trained checkpoint.  Every group gets (i) a log-normal overall scale on
    its down rows, so that some groups matter more than others whatever the input, and (ii) a direction shared by
    all of its gate rows, so that inputs aligned with it switch the whole group on.  The directions live in a
    `latent`-dimensional subspace spanned by the columns of A ("topics"); semantic_inputs() draws inputs that mix
    topic content with noise.  Values are i.i.d. Gaussian apart from these terms.
    Returns (W[G][3][S][d] in the workload dtype, A[d][latent] fp32)."""
    base = 100 * (layer + 1)
    G, S, d = wl.n_groups, wl.group_size, wl.d_model
    gen = _gen(wl.seed, base + 50, device)
    W = torch.empty((G, 3, S, d), dtype=torch.float32, device=device).normal_(0.0, wl.weight_std, generator=gen)
    scale = torch.empty((G,), dtype=torch.float32, device=device).normal_(0.0, scale_sigma, generator=gen).exp()
    A = torch.empty((d, latent), dtype=torch.float32, device=device).normal_(0.0, latent ** -0.5, generator=gen)
    C = torch.empty((latent, G), dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    C = C / C.norm(dim=0, keepdim=True)
    direction = (A @ C).T * (wl.weight_std * latent ** 0.5)          # [G][d], entries ~ weight_std
    W[:, 0] += coherence * direction[:, None, :]
    W[:, 2] *= scale[:, None, None]
    return W.to(wl.torch_dtype), A


def semantic_inputs(wl: Workload, tag: int, A: torch.Tensor, n: int, topic_share: float = 0.5) -> torch.Tensor:
    """n input vectors with unit-variance coordinates: sqrt(topic_share) * (A t) + sqrt(1 - topic_share) * noise,
    t ~ N(0, I): inputs that carry content in the subspace the structured layer's groups listen to."""
    device = A.device
    gen = _gen(wl.seed, 30_000_000 + tag, device)
    t = torch.empty((n, A.shape[1]), dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    noise = torch.empty((n, A.shape[0]), dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    x = (topic_share ** 0.5) * (t @ A.T) + ((1.0 - topic_share) ** 0.5) * noise
    return x.to(wl.torch_dtype)


def mha_matrices(wl: Workload, layer: int, n_heads: int, device="cpu"):
    """Attention projections of one block: Wq, Wk, Wv [H*dh][d] and Wo [d][H*dh], N(0, weight_std)."""
    base = 100 * (layer + 1) + 60
    d = wl.d_model
    mk = lambda i, shape: _normal(shape, wl.weight_std, wl.torch_dtype, _gen(wl.seed, base + i, device), device)
    return mk(0, (d, d)), mk(1, (d, d)), mk(2, (d, d)), mk(3, (d, d))
