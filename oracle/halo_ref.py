"""ctypes front end of the CPU fp64 oracle (``halo_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never touches CUDA and imports nothing from
the CUDA package.  Arrays go in as numpy arrays holding the raw element bytes
(``float32``, or ``uint16`` for bf16) and results come back as numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int32, c_uint8, c_uint32, c_uint64, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "halo_ref.c")
_LIB = os.path.join(_HERE, "libhalo_ref.so")

F32, BF16 = 0, 1
SEL_TOPK, SEL_THRESHOLD = 0, 1
ACT_RELU, ACT_NONE = 0, 1
STATUS_NONFINITE = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over groups)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
             _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.halo_ref_loss_threshold.restype = c_uint64
        _lib.halo_ref_loss_threshold.argtypes = [c_double]
        _lib.halo_ref_arrival.restype = c_int
        _lib.halo_ref_arrival.argtypes = [c_uint64, c_uint32, c_uint32, c_uint32, c_double]
    return _lib


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle arrays are float32 or uint16 (bf16 bits), got {a.dtype}")


def _c(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a)


def _p(a):
    return None if a is None else a.ctypes.data_as(c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with status {rc}")


def k_of(wl) -> int:
    """Critical groups kept by the master for a keep ratio given per mille: the smallest integer k with
    k / G >= permille / 1000 (written on its own here; the oracle shares no code with the CUDA package)."""
    k = 0
    while k * 1000 < int(wl.keep_permille) * int(wl.n_groups):
        k += 1
    return k


def set_threads(n: int) -> None:
    """OpenMP thread count for the group loop (the timed baseline states it)."""
    omp = ctypes.CDLL("libgomp.so.1")
    omp.omp_set_num_threads(int(n))


# --- bf16 helpers for tests (exact bit manipulation, no arithmetic) ----------

def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def to_f64(a: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


# --- RNG / arrival ------------------------------------------------------------

def philox4x32_10(ctr, key):
    c = (c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    out = (c_uint32 * 4)()
    lib().halo_ref_philox4x32_10(c, k, out)
    return [int(v) for v in out]


def loss_threshold(rho: float) -> int:
    return int(lib().halo_ref_loss_threshold(float(rho)))


def arrival(seed: int, step: int, layer: int, device: int, rho: float) -> int:
    return int(lib().halo_ref_arrival(int(seed), int(step), int(layer), int(device), float(rho)))


# --- layout -------------------------------------------------------------------

def pack_weights(Wgate: np.ndarray, Wup: np.ndarray, Wdown: np.ndarray, S: int) -> np.ndarray:
    F, d = Wgate.shape
    assert Wup.shape == (F, d) and Wdown.shape == (d, F)
    dt = _dtype_of(Wgate)
    Wgate, Wup, Wdown = _c(Wgate), _c(Wup), _c(Wdown)
    out = np.empty((F // S, 3, S, d), dtype=Wgate.dtype)
    _check(lib().halo_ref_pack_weights(c_int(d), c_int(F), c_int(S), c_int(dt), _p(Wgate), _p(Wup), _p(Wdown),
                                       _p(out)), "pack_weights")
    return out


def unpack_weights(Wpacked: np.ndarray):
    G, three, S, d = Wpacked.shape
    assert three == 3
    F = G * S
    dt = _dtype_of(Wpacked)
    Wpacked = _c(Wpacked)
    wg = np.empty((F, d), dtype=Wpacked.dtype)
    wu = np.empty((F, d), dtype=Wpacked.dtype)
    wd = np.empty((d, F), dtype=Wpacked.dtype)
    _check(lib().halo_ref_unpack_weights(c_int(d), c_int(F), c_int(S), c_int(dt), _p(Wpacked), _p(wg), _p(wu),
                                         _p(wd)), "unpack_weights")
    return wg, wu, wd


# --- a1 -----------------------------------------------------------------------

def predict(W1: np.ndarray, W2: np.ndarray, feat: np.ndarray, act: int = ACT_RELU, mean_pool: bool = False):
    """W1[r][d_in], W2[G][r], feat[n_tok][d_in] (or [d_in]) -> fp32 scores."""
    r, d_in = W1.shape
    G = W2.shape[0]
    assert W2.shape == (G, r)
    feat2 = feat.reshape(-1, d_in)
    n_tok = feat2.shape[0]
    dt = _dtype_of(W1)
    assert _dtype_of(W2) == dt and _dtype_of(feat2) == dt
    W1, W2, feat2 = _c(W1), _c(W2), _c(feat2)
    out = np.empty((G,) if (mean_pool or n_tok == 1) else (n_tok, G), dtype=np.float32)
    _check(lib().halo_ref_predict(c_int(d_in), c_int(r), c_int(G), c_int(dt), c_int(act), _p(W1), _p(W2),
                                  _p(feat2), c_int(n_tok), c_int(1 if (mean_pool and n_tok > 1) else 0),
                                  _p(out)), "predict")
    return out


# --- Algorithm 3 ----------------------------------------------------------------

def plan(loss_rate, share_weight, M: int):
    n = len(loss_rate)
    lr = np.asarray(loss_rate, dtype=np.float64)
    sw = np.asarray(share_weight, dtype=np.uint32)
    order = np.empty(max(n, 1), dtype=np.int32)
    thr = np.empty(max(n, 1), dtype=np.uint64)
    bnd = np.empty(n + 1, dtype=np.int32)
    _check(lib().halo_ref_plan(c_int(n), _p(lr), _p(sw), c_int(M), _p(order), _p(thr), _p(bnd)), "plan")
    return order[:n].copy(), thr[:n].copy(), bnd


# --- a2..a5 ---------------------------------------------------------------------

def select(scores: np.ndarray, loss_rate, share_weight, mode: int, k_critical: int, threshold: float,
           seed: int, step: int, layer: int, force_all: bool = False):
    G = scores.shape[0]
    n = len(loss_rate)
    s = _c(scores.astype(np.float32, copy=False))
    lr = np.asarray(loss_rate, dtype=np.float64)
    sw = np.asarray(share_weight, dtype=np.uint32)
    order = np.empty(G, dtype=np.int32)
    rank = np.empty(G, dtype=np.int32)
    dev = np.empty(G, dtype=np.int32)
    arrived = np.empty(max(n, 1), dtype=np.uint8)
    keep = np.empty(G, dtype=np.uint8)
    keep_list = np.empty(G, dtype=np.int32)
    n_keep = np.zeros(1, dtype=np.int32)
    status = np.zeros(1, dtype=np.uint32)
    _check(lib().halo_ref_select(c_int(G), c_int(n), _p(lr), _p(sw), c_int(mode), c_int(k_critical),
                                 c_float(threshold), c_uint64(seed), _p(s), c_uint32(step), c_uint32(layer),
                                 c_int(1 if force_all else 0), _p(order), _p(rank), _p(dev), _p(arrived),
                                 _p(keep), _p(keep_list), _p(n_keep), _p(status)), "select")
    return dict(order=order, rank=rank, dev_of_group=dev, arrived=arrived[:n].copy(), keep=keep,
                keep_list=keep_list, n_keep=int(n_keep[0]), status=int(status[0]))


# --- a6..a8 ---------------------------------------------------------------------

def group_ffn(Wpacked: np.ndarray, x: np.ndarray, group_list, dev_of_group=None, n_dev: int = 0,
              want_group_partials: bool = False):
    """-> partials float64 [n_dev+1][n_tok][d] (and per-group partials)."""
    G, _, S, d = Wpacked.shape
    dt = _dtype_of(Wpacked)
    x2 = _c(x.reshape(-1, d))
    assert _dtype_of(x2) == dt
    n_tok = x2.shape[0]
    Wpacked = _c(Wpacked)
    lst = np.asarray(group_list, dtype=np.int32).reshape(-1)
    dg = None if dev_of_group is None else _c(np.asarray(dev_of_group, dtype=np.int32))
    P = np.empty((n_dev + 1, n_tok, d), dtype=np.float64)
    gp = np.empty((max(len(lst), 1), n_tok, d), dtype=np.float64) if want_group_partials else None
    _check(lib().halo_ref_group_ffn(c_int(d), c_int(G * S), c_int(S), c_int(dt), _p(Wpacked), _p(x2),
                                    c_int(n_tok), _p(lst), c_int(len(lst)), _p(dg), c_int(n_dev), _p(P),
                                    _p(gp)), "group_ffn")
    if want_group_partials:
        return P, gp[: len(lst)]
    return P


# --- a9 -------------------------------------------------------------------------

def merge(partials: np.ndarray, arrived=None):
    n_slots, n_tok, d = partials.shape
    P = _c(partials.astype(np.float64, copy=False))
    arr = None if arrived is None else _c(np.asarray(arrived, dtype=np.uint8))
    y = np.empty((n_tok, d), dtype=np.float64)
    _check(lib().halo_ref_merge(_p(P), _p(arr), c_int(n_slots - 1), c_int(n_tok), c_int(d), _p(y)), "merge")
    return y


# --- glue -----------------------------------------------------------------------

def glue(h: np.ndarray, y, dtype: int):
    """h' = h + y (y may be None), x = cast(rmsnorm(h')). -> (h', x)"""
    h2 = _c(h.astype(np.float64, copy=False))
    n_tok, d = h2.reshape(-1, h2.shape[-1]).shape
    y2 = None if y is None else _c(np.asarray(y, dtype=np.float64))
    h_out = np.empty((n_tok, d), dtype=np.float64)
    x_out = np.empty((n_tok, d), dtype=np.float32 if dtype == F32 else np.uint16)
    _check(lib().halo_ref_glue(c_int(d), c_int(n_tok), c_int(dtype), _p(h2), _p(y2), _p(h_out), _p(x_out)), "glue")
    return h_out, x_out


# --- a1..a9 for one layer ---------------------------------------------------------

def layer(Wpacked, W1, W2, feat, x, loss_rate, share_weight, mode, k_critical, threshold, seed, step, layer_idx,
          force_all=False, act=ACT_RELU):
    G, _, S, d = Wpacked.shape
    dt = _dtype_of(Wpacked)
    r = W1.shape[0]
    n = len(loss_rate)
    x2 = _c(x.reshape(-1, d))
    f2 = _c(feat.reshape(-1, d))
    n_tok = x2.shape[0]
    Wpacked, W1, W2 = _c(Wpacked), _c(W1), _c(W2)
    lr = np.asarray(loss_rate, dtype=np.float64)
    sw = np.asarray(share_weight, dtype=np.uint32)
    scores = np.empty(G, dtype=np.float32)
    order = np.empty(G, dtype=np.int32)
    rank = np.empty(G, dtype=np.int32)
    dev = np.empty(G, dtype=np.int32)
    arrived = np.empty(max(n, 1), dtype=np.uint8)
    keep = np.empty(G, dtype=np.uint8)
    keep_list = np.empty(G, dtype=np.int32)
    n_keep = np.zeros(1, dtype=np.int32)
    status = np.zeros(1, dtype=np.uint32)
    y = np.empty((n_tok, d), dtype=np.float64)
    _check(lib().halo_ref_layer(c_int(d), c_int(G * S), c_int(S), c_int(dt), _p(Wpacked), c_int(r), c_int(act),
                                _p(W1), _p(W2), c_int(n), _p(lr), _p(sw), c_int(mode), c_int(k_critical),
                                c_float(threshold), c_uint64(seed), c_uint32(step), c_uint32(layer_idx),
                                c_int(1 if force_all else 0), _p(f2), _p(x2), c_int(n_tok), _p(scores), _p(order),
                                _p(rank), _p(dev), _p(arrived), _p(keep), _p(keep_list), _p(n_keep), _p(status),
                                _p(y)), "layer")
    return dict(scores=scores, order=order, rank=rank, dev_of_group=dev, arrived=arrived[:n].copy(), keep=keep,
                keep_list=keep_list, n_keep=int(n_keep[0]), status=int(status[0]), y=y)


# --- Algorithms 1 and 2: workload ratios ---------------------------------------------

def comp_greedy(m, c, Mt: float) -> np.ndarray:
    m = np.asarray(m, dtype=np.float64); c = np.asarray(c, dtype=np.float64)
    r = np.empty(len(m), dtype=np.float64)
    _check(lib().halo_ref_comp_greedy(c_int(len(m)), _p(m), _p(c), c_double(Mt), _p(r)), "comp_greedy")
    return r


def min_max(m, c, Mt: float, eps: float = 1e-3) -> np.ndarray:
    m = np.asarray(m, dtype=np.float64); c = np.asarray(c, dtype=np.float64)
    r = np.empty(len(m), dtype=np.float64)
    _check(lib().halo_ref_min_max(c_int(len(m)), _p(m), _p(c), c_double(Mt), c_double(eps), _p(r)), "min_max")
    return r


def late_devices(units, compute, tau: float, t_comm: float, timeout: float) -> np.ndarray:
    """Sec. III-B.3 + Eq. 1: device i is late (its partial counts as lost) iff tau*units[i]/compute[i] + t_comm
    exceeds the timeout; a device that holds nothing is never late."""
    u = np.asarray(units, dtype=np.int32); c = np.asarray(compute, dtype=np.float64)
    late = np.zeros(len(u), dtype=np.uint8)
    _check(lib().halo_ref_late_devices(c_int(len(u)), _p(u), _p(c), c_double(tau), c_double(t_comm), c_double(timeout),
                                       _p(late)), "late_devices")
    return late


# --- int4 group-quantised weights -----------------------------------------------------------

QBLOCK = 128


def quantize_i4(W: np.ndarray):
    """Packed rows [..., d] (float32 or bf16 bits) -> (codes uint8 [..., d/2], scales bf16 bits [..., d/128]);
    symmetric, s = bf16(amax/7) rounded up to 5 significant bits, q = clamp(rint(w/s), -8, 7), nibble = q + 8, element
    2i in the low half of byte i."""
    d = W.shape[-1]
    n_rows = int(np.prod(W.shape[:-1]))
    dt = _dtype_of(W)
    W = _c(W)
    Q = np.empty(W.shape[:-1] + (d // 2,), dtype=np.uint8)
    Sc = np.empty(W.shape[:-1] + (d // QBLOCK,), dtype=np.uint16)
    _check(lib().halo_ref_quantize_i4(c_int(d), ctypes.c_longlong(n_rows), c_int(dt), _p(W), _p(Q), _p(Sc)), "quantize_i4")
    return Q, Sc


def dequantize_i4(Q: np.ndarray, Sc: np.ndarray) -> np.ndarray:
    """(codes, scales) -> float32 rows [..., d]: (nibble - 8) * scale, exact."""
    d = Q.shape[-1] * 2
    n_rows = int(np.prod(Q.shape[:-1]))
    Q, Sc = _c(Q), _c(Sc)
    W = np.empty(Q.shape[:-1] + (d,), dtype=np.float32)
    _check(lib().halo_ref_dequantize_i4(c_int(d), ctypes.c_longlong(n_rows), _p(Q), _p(Sc), _p(W)), "dequantize_i4")
    return W


def group_ffn_i4(Q: np.ndarray, Sc: np.ndarray, x: np.ndarray, group_list, dev_of_group=None, n_dev: int = 0):
    """The group FFN on int4 weights = the group FFN on their dequantised values (x widened exactly to fp32)."""
    W32 = dequantize_i4(Q, Sc)
    x32 = to_f64(x).astype(np.float32)          # bf16 -> fp32 is exact
    return group_ffn(W32, x32, group_list, dev_of_group, n_dev)


# --- MHA neuron groups --------------------------------------------------------------------

def pack_mha(Wq: np.ndarray, Wo: np.ndarray, H: int) -> np.ndarray:
    """Wq[H*dh][d], Wo[d][H*dh] -> packed [H][2][dh][d]."""
    n, d = Wq.shape
    dh = n // H
    assert Wo.shape == (d, n)
    dt = _dtype_of(Wq)
    Wq, Wo = _c(Wq), _c(Wo)
    out = np.empty((H, 2, dh, d), dtype=Wq.dtype)
    _check(lib().halo_ref_pack_mha(c_int(d), c_int(H), c_int(dh), c_int(dt), _p(Wq), _p(Wo), _p(out)), "pack_mha")
    return out


def mha_kv_append(Wk: np.ndarray, Wv: np.ndarray, x: np.ndarray, pos: int, K_cache: np.ndarray, V_cache: np.ndarray):
    """Writes k, v of this token at `pos` into the caches [H][Lmax][dh] (in place)."""
    H, Lmax, dh = K_cache.shape
    d = Wk.shape[1]
    dt = _dtype_of(Wk)
    assert K_cache.flags.c_contiguous and V_cache.flags.c_contiguous and _dtype_of(K_cache) == dt
    Wk, Wv, x1 = _c(Wk), _c(Wv), _c(x.reshape(-1))
    _check(lib().halo_ref_mha_kv_append(c_int(d), c_int(H), c_int(dh), c_int(Lmax), c_int(dt), _p(Wk), _p(Wv), _p(x1),
                                        c_int(pos), _p(K_cache), _p(V_cache)), "mha_kv_append")


def group_mha(Wpacked: np.ndarray, x: np.ndarray, K_cache: np.ndarray, V_cache: np.ndarray, pos: int, head_list,
              dev_of_group=None, n_dev: int = 0, want_head_partials: bool = False):
    H, _, dh, d = Wpacked.shape
    Lmax = K_cache.shape[1]
    dt = _dtype_of(Wpacked)
    Wpacked, x1, K_cache, V_cache = _c(Wpacked), _c(x.reshape(-1)), _c(K_cache), _c(V_cache)
    lst = np.asarray(head_list, dtype=np.int32).reshape(-1)
    dg = None if dev_of_group is None else _c(np.asarray(dev_of_group, dtype=np.int32))
    P = np.empty((n_dev + 1, d), dtype=np.float64)
    hp = np.empty((max(len(lst), 1), d), dtype=np.float64) if want_head_partials else None
    _check(lib().halo_ref_group_mha(c_int(d), c_int(H), c_int(dh), c_int(Lmax), c_int(dt), _p(Wpacked), _p(x1),
                                    _p(K_cache), _p(V_cache), c_int(pos), _p(lst), c_int(len(lst)), _p(dg),
                                    c_int(n_dev), _p(P), _p(hp)), "group_mha")
    if want_head_partials:
        return P, hp[: len(lst)]
    return P


def _widen32(a: np.ndarray) -> np.ndarray:
    """bf16 bits or float32 -> float32 (exact)."""
    return to_f64(a).astype(np.float32)


def mha_kv_append_i4(Qk, Sk, Qv, Sv, x: np.ndarray, pos: int, K_cache32: np.ndarray, V_cache32: np.ndarray):
    """Keys and values of this token from int4 Wk / Wv (their dequantised values) into float32 caches, unrounded."""
    mha_kv_append(dequantize_i4(Qk, Sk), dequantize_i4(Qv, Sv), _widen32(x), pos, K_cache32, V_cache32)


def group_mha_i4(Qp, Sp, H: int, x: np.ndarray, K_cache: np.ndarray, V_cache: np.ndarray, pos: int, head_list,
                 dev_of_group=None, n_dev: int = 0):
    """halo_group_mha on int4 packed weights: Qp [H*2*dh][d/2], Sp [H*2*dh][d/128] -> dequantised [H][2][dh][d]; x and the
    caches (bf16 bits or float32) widened exactly."""
    W = dequantize_i4(Qp, Sp)
    rows, d = W.shape
    return group_mha(W.reshape(H, 2, rows // (2 * H), d), _widen32(x), _widen32(K_cache), _widen32(V_cache), pos, head_list,
                     dev_of_group, n_dev)


def group_lm_head(W: np.ndarray, x: np.ndarray, group_size: int, group_list=None, fill: float = np.nan):
    """LM-head groups (Sec. II-A, Sec. III-B.3): logits[t][v] = <W[v], x_t> for the rows of the listed groups of
    `group_size` vocabulary rows; the other entries keep `fill`."""
    vocab, d = W.shape
    dt = _dtype_of(W)
    x2 = x.reshape(-1, d)
    n_tok = x2.shape[0]
    n_groups = (vocab + group_size - 1) // group_size
    lst = np.arange(n_groups, dtype=np.int32) if group_list is None else np.asarray(group_list, dtype=np.int32).reshape(-1)
    W, x2 = _c(W), _c(x2)
    out = np.full((n_tok, vocab), fill, dtype=np.float64)
    _check(lib().halo_ref_group_lm_head(c_int(d), c_int(vocab), c_int(group_size), c_int(dt), _p(W), _p(x2),
                                        c_int(n_tok), _p(lst), c_int(len(lst)), _p(out)), "group_lm_head")
    return out


def group_lm_head_i4(Q: np.ndarray, Sc: np.ndarray, x: np.ndarray, group_size: int, group_list=None,
                     fill: float = np.nan):
    """The LM-head groups on int4 rows = the LM-head groups on their dequantised values (x widened exactly to fp32)."""
    W32 = dequantize_i4(Q, Sc)
    x32 = to_f64(x).astype(np.float32)          # bf16 -> fp32 is exact
    return group_lm_head(W32, x32, group_size, group_list, fill)


# --- a transformer-block stack: MHA groups, then FFN groups, per layer; LM-head groups at the end --------------

def block_stack_token(h0, pos, step, blocks, lm_W, lm_group_size, plan_mha, plan_ffn, dtype, act=ACT_RELU):
    """One token through L transformer blocks the way the generation phase runs them (Sec. III-B.3: in every layer
    the MHA block and then the MLP block, each with its own predictor fed one layer ahead; the first layer and the LM
    head are sent reliably).  Free running, every step by the functions above, nothing fused:

        for layer l:   x_a = cast(rmsnorm(h));  K, V caches of layer l get the keys / values of x_a at `pos`
                       heads kept = select(predict(mha predictor of l, x_a of layer l-1)), arrival draw (step, 2l)
                       h += merge(group_mha(kept heads))
                       x_f = cast(rmsnorm(h))
                       groups kept = select(predict(ffn predictor of l, x_f of layer l-1)), arrival draw (step, 2l+1)
                       h += merge(group_ffn(kept groups))
        logits = LM-head groups (all of them) on cast(rmsnorm(h))

    blocks: list of dicts with W_mha (packed [H][2][dh][d]), Wk, Wv, K, V (caches, updated in place), W_ffn (packed),
    and for l >= 1 the predictor factors W1_mha, W2_mha, W1_ffn, W2_ffn.  plan_*: dict(loss_rate, share_weight, mode,
    k, threshold, seed).  Returns (h, logits or None, records per layer)."""
    h = np.asarray(h0, dtype=np.float64).reshape(1, -1)
    recs = []
    xa_prev = xf_prev = None
    for l, b in enumerate(blocks):
        H = b["W_mha"].shape[0]
        G = b["W_ffn"].shape[0]
        _, x_a = glue(h, None, dtype)
        mha_kv_append(b["Wk"], b["Wv"], x_a[0], pos, b["K"], b["V"])
        s_a = np.zeros(H, dtype=np.float32) if l == 0 else predict(b["W1_mha"], b["W2_mha"], xa_prev, act=act)
        sel_a = select(s_a, plan_mha["loss_rate"], plan_mha["share_weight"], plan_mha["mode"], plan_mha["k"],
                       plan_mha["threshold"], plan_mha["seed"], step, 2 * l, force_all=(l == 0))
        n_a = len(plan_mha["loss_rate"])
        P_a = group_mha(b["W_mha"], x_a[0], b["K"], b["V"], pos, sel_a["keep_list"][: sel_a["n_keep"]],
                        sel_a["dev_of_group"], n_a)
        y_a = merge(P_a[:, None, :])
        h, x_f = glue(h, y_a, dtype)
        s_f = np.zeros(G, dtype=np.float32) if l == 0 else predict(b["W1_ffn"], b["W2_ffn"], xf_prev, act=act)
        sel_f = select(s_f, plan_ffn["loss_rate"], plan_ffn["share_weight"], plan_ffn["mode"], plan_ffn["k"],
                       plan_ffn["threshold"], plan_ffn["seed"], step, 2 * l + 1, force_all=(l == 0))
        n_f = len(plan_ffn["loss_rate"])
        P_f = group_ffn(b["W_ffn"], x_f, sel_f["keep_list"][: sel_f["n_keep"]], sel_f["dev_of_group"], n_f)
        y_f = merge(P_f)
        h = h + y_f
        recs.append(dict(x_a=x_a, x_f=x_f, scores_a=s_a, scores_f=s_f, sel_a=sel_a, sel_f=sel_f, y_a=y_a, y_f=y_f))
        xa_prev, xf_prev = x_a, x_f
    logits = None
    if lm_W is not None:
        _, x_o = glue(h, None, dtype)
        logits = group_lm_head(lm_W, x_o, lm_group_size)
    return h, logits, recs
