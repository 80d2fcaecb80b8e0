"""Thin ctypes binding of libhalo.so: same names as include/halo.h, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams are torch's); every
step of the path runs inside the library's kernels.  The library must have been
built (``python -m paper_2601_11676_b200.build``); there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int32, c_longlong, c_size_t, \
    c_uint8, c_uint32, c_uint64, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libhalo.so")

F32, BF16 = 0, 1
SEL_TOPK, SEL_THRESHOLD = 0, 1
ACT_RELU, ACT_NONE = 0, 1
DEV_NONFINITE_SCORE, DEV_BAD_INDEX, DEV_TIMEOUT = 1, 2, 4
STACK_PER_STEP_LAUNCHES, STACK_PRED_SERIAL, STACK_LOAD_SERIAL, STACK_DETERMINISTIC, STACK_PROMPT_ONE_LAUNCH = 1, 2, 4, 8, 16
MAX_DEVICES, MAX_GROUPS = 32, 1024

EXPORTS = [
    "halo_status_string", "halo_status_message", "halo_plan_create", "halo_plan_destroy", "halo_plan_describe",
    "halo_predict_workspace_bytes", "halo_predict_groups", "halo_predict_groups_static", "halo_select_groups", "halo_group_ffn_workspace_bytes",
    "halo_group_ffn", "halo_merge_partials", "halo_pack_weights", "halo_glue", "halo_stack_create",
    "halo_stack_destroy", "halo_stack_decode", "halo_stack_decode_host", "halo_stack_status",
    "halo_stack_last_launches", "halo_stack_set_mode", "halo_stack_set_trace", "halo_stack_trace_width",
    "halo_schedule_comp_greedy", "halo_schedule_min_max", "halo_ratios_to_share_weights",
    "halo_selftest_bounded_wait", "halo_group_importance_workspace_bytes", "halo_group_importance",
    "halo_layer_workspace_bytes", "halo_layer_fused", "halo_read_status",
    "halo_pack_mha_weights", "halo_mha_kv_append", "halo_group_mha_workspace_bytes", "halo_group_mha",
    "halo_group_lm_head", "halo_late_devices", "halo_quantize_weights_i4", "halo_group_ffn_i4", "halo_dequantize_weights_i4", "halo_quantize_rows_i4", "halo_group_lm_head_i4", "halo_mha_block_i4",
    "halo_block_stack_create_i4", "halo_group_ffn_i4_workspace_bytes", "halo_group_ffn_i4_prompt",
    "halo_set_option",
    "halo_block_stack_create", "halo_block_stack_destroy", "halo_block_stack_decode", "halo_block_stack_status",
    "halo_block_stack_last_launches", "halo_stack_create_i4", "halo_mha_block",
]


class FfnShape(Structure):
    _fields_ = [("d_model", c_int), ("d_ffn", c_int), ("group_size", c_int), ("wdtype", c_int)]


class PredShape(Structure):
    _fields_ = [("d_in", c_int), ("rank", c_int), ("n_groups", c_int), ("wdtype", c_int), ("act", c_int)]


class MhaShape(Structure):
    _fields_ = [("d_model", c_int), ("n_heads", c_int), ("head_dim", c_int), ("max_len", c_int), ("wdtype", c_int)]


class LmShape(Structure):
    _fields_ = [("d_model", c_int), ("vocab", c_int), ("group_size", c_int), ("wdtype", c_int)]


class Taps(Structure):
    _fields_ = [("x", c_void_p), ("scores", c_void_p), ("dev_of_group", c_void_p), ("arrived", c_void_p),
                ("keep_list", c_void_p), ("n_keep", c_void_p), ("y", c_void_p)]


class BlockWeights(Structure):
    _fields_ = [(n, POINTER(c_void_p)) for n in ("W_ffn", "W_mha", "Wk", "Wv", "W1_ffn", "W2_ffn", "W1_mha", "W2_mha",
                                                  "K_cache", "V_cache")] + [("W_lm", c_void_p)]


class BlockScales(Structure):
    _fields_ = [(n, POINTER(c_void_p)) for n in ("S_ffn", "S_mha", "Sk", "Sv")] + [("S_lm", c_void_p)]


class BlockTaps(Structure):
    _fields_ = [("mha", Taps), ("ffn", Taps)]


class HaloError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: status {code} ({status_string(code)})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libhalo.so; raises if it is missing (no CPU or eager fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2601_11676_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.halo_status_string.restype = c_char_p
        L.halo_status_string.argtypes = [c_int]
        L.halo_predict_workspace_bytes.restype = c_size_t
        L.halo_predict_workspace_bytes.argtypes = [POINTER(PredShape), c_int]
        L.halo_group_ffn_workspace_bytes.restype = c_size_t
        L.halo_group_ffn_workspace_bytes.argtypes = [POINTER(FfnShape), c_int, c_int]
        L.halo_stack_last_launches.restype = c_longlong
        L.halo_stack_last_launches.argtypes = [c_void_p]
        L.halo_plan_create.argtypes = [POINTER(c_void_p), c_int, c_int, POINTER(c_double), POINTER(c_uint32), c_int,
                                       c_int, c_float, c_uint64]
        L.halo_plan_destroy.argtypes = [c_void_p]
        L.halo_plan_describe.argtypes = [c_void_p, c_int, POINTER(c_int32), POINTER(c_uint64), POINTER(c_int32)]
        L.halo_predict_groups.argtypes = [POINTER(PredShape), c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p,
                                          c_void_p, c_size_t, c_void_p, c_void_p]
        L.halo_predict_groups_static.argtypes = [POINTER(PredShape), c_void_p, c_void_p, c_void_p, c_int, c_int,
                                                 c_void_p, c_void_p, c_void_p]
        L.halo_select_groups.argtypes = [c_void_p, c_void_p, c_uint32, c_uint32, c_int, c_void_p, c_void_p, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_group_ffn.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int,
                                     c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.halo_merge_partials.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p]
        L.halo_pack_weights.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_glue.argtypes = [c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_stack_create.argtypes = [POINTER(c_void_p), POINTER(FfnShape), POINTER(PredShape), c_int, c_int,
                                        c_void_p, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p)]
        L.halo_stack_create_i4.argtypes = [POINTER(c_void_p), POINTER(FfnShape), POINTER(PredShape), c_int, c_int,
                                           c_void_p, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p),
                                           POINTER(c_void_p)]
        L.halo_stack_destroy.argtypes = [c_void_p]
        L.halo_stack_decode.argtypes = [c_void_p, c_void_p, c_int, c_uint32, c_void_p, POINTER(Taps), c_void_p]
        L.halo_stack_decode_host.argtypes = [c_void_p, c_void_p, c_int, c_uint32, c_void_p, c_void_p]
        L.halo_stack_status.argtypes = [c_void_p, POINTER(c_uint32), c_void_p]
        L.halo_stack_set_mode.argtypes = [c_void_p, c_int]
        L.halo_stack_set_trace.argtypes = [c_void_p, c_void_p, c_int]
        L.halo_stack_trace_width.argtypes = [c_void_p]
        L.halo_stack_trace_width.restype = c_int
        L.halo_schedule_comp_greedy.argtypes = [c_int, POINTER(c_double), POINTER(c_double), c_double, POINTER(c_double)]
        L.halo_schedule_min_max.argtypes = [c_int, POINTER(c_double), POINTER(c_double), c_double, c_double,
                                            POINTER(c_double)]
        L.halo_ratios_to_share_weights.argtypes = [c_int, POINTER(c_double), POINTER(c_uint32)]
        L.halo_late_devices.argtypes = [c_int, POINTER(c_int32), POINTER(c_double), c_double, c_double, c_double,
                                        POINTER(c_uint8)]
        L.halo_group_importance_workspace_bytes.restype = c_size_t
        L.halo_group_importance_workspace_bytes.argtypes = [POINTER(FfnShape)]
        L.halo_group_importance.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p,
                                            c_void_p]
        L.halo_layer_workspace_bytes.restype = c_size_t
        L.halo_layer_workspace_bytes.argtypes = [POINTER(FfnShape), POINTER(PredShape), c_int, c_int]
        L.halo_layer_fused.argtypes = [POINTER(FfnShape), POINTER(PredShape), c_void_p] + [c_void_p] * 5 + \
            [c_int, c_uint32, c_uint32, c_int] + [c_void_p] * 6 + [c_size_t, c_void_p, c_void_p]
        L.halo_read_status.argtypes = [POINTER(c_uint32), c_char_p, c_int]
        L.halo_pack_mha_weights.argtypes = [POINTER(MhaShape), c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_mha_kv_append.argtypes = [POINTER(MhaShape), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]
        L.halo_group_mha_workspace_bytes.restype = c_size_t
        L.halo_group_mha_workspace_bytes.argtypes = [POINTER(MhaShape)]
        L.halo_group_mha.argtypes = [POINTER(MhaShape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                     c_void_p, c_int, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.halo_mha_block.argtypes = [POINTER(MhaShape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int,
                                     c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]
        L.halo_mha_block_i4.argtypes = [POINTER(MhaShape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int,
                                        c_void_p, c_void_p, c_void_p]
        L.halo_block_stack_create_i4.argtypes = [POINTER(c_void_p), POINTER(FfnShape), POINTER(MhaShape), POINTER(LmShape),
                                                 POINTER(PredShape), POINTER(PredShape), c_int, c_void_p, c_void_p,
                                                 POINTER(BlockWeights), POINTER(BlockScales)]
        L.halo_group_lm_head.argtypes = [POINTER(LmShape), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                         c_void_p, c_void_p]
        L.halo_quantize_weights_i4.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_group_ffn_i4.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                        c_void_p, c_int, c_void_p, c_void_p, c_void_p]
        L.halo_quantize_rows_i4.argtypes = [c_int, c_longlong, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
        L.halo_group_lm_head_i4.argtypes = [POINTER(LmShape), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_void_p]
        L.halo_group_ffn_i4_workspace_bytes.argtypes = [POINTER(FfnShape), c_int]
        L.halo_group_ffn_i4_workspace_bytes.restype = c_size_t
        L.halo_group_ffn_i4_prompt.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                               c_void_p, c_int, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.halo_dequantize_weights_i4.argtypes = [POINTER(FfnShape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                                 c_void_p, c_void_p]
        L.halo_selftest_bounded_wait.argtypes = [c_void_p, c_longlong, c_void_p, c_void_p, c_void_p]
        L.halo_status_message.argtypes = [c_uint32, c_char_p, c_int]
        L.halo_set_option.argtypes = [c_char_p, c_int]
        L.halo_block_stack_create.argtypes = [POINTER(c_void_p), POINTER(FfnShape), POINTER(MhaShape), POINTER(LmShape),
                                              POINTER(PredShape), POINTER(PredShape), c_int, c_void_p, c_void_p,
                                              POINTER(BlockWeights)]
        L.halo_block_stack_destroy.argtypes = [c_void_p]
        L.halo_block_stack_decode.argtypes = [c_void_p, c_void_p, c_int, c_int, c_uint32, c_void_p, c_void_p,
                                              POINTER(BlockTaps), c_void_p]
        L.halo_block_stack_status.argtypes = [c_void_p, POINTER(c_uint32), c_void_p]
        L.halo_block_stack_last_launches.argtypes = [c_void_p]
        L.halo_block_stack_last_launches.restype = c_longlong
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().halo_status_string(code).decode()


def k_of(wl) -> int:
    """Number of critical groups for a workload's keep ratio: ceil(permille * G / 1000) in integers.  The ABI takes
    k itself; this is the convention the callers in this repository use to derive it."""
    return (int(wl.keep_permille) * int(wl.n_groups) + 999) // 1000


def halo_set_option(name: str, value: int) -> None:
    _chk(lib().halo_set_option(name.encode(), int(value)), "halo_set_option")


def status_message(value: int) -> str:
    buf = ctypes.create_string_buffer(128)
    lib().halo_status_message(value, buf, 128)
    return buf.value.decode()


def _chk(code: int, what: str) -> None:
    if code != 0:
        raise HaloError(code, what)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-contiguous tensor expected"
    return c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


def ffn_shape(d_model: int, d_ffn: int, group_size: int, dtype: int) -> FfnShape:
    return FfnShape(d_model, d_ffn, group_size, dtype)


def pred_shape(d_in: int, rank: int, n_groups: int, dtype: int, act: int = ACT_RELU) -> PredShape:
    return PredShape(d_in, rank, n_groups, dtype, act)


class Plan:
    """halo_plan_create / halo_plan_destroy."""

    def __init__(self, n_groups, loss_rate, share_weight, mode=SEL_TOPK, k_critical=0, threshold=0.0, seed=0):
        n = len(loss_rate)
        self.n_groups, self.n_dev = n_groups, n
        lr = (c_double * max(n, 1))(*[float(v) for v in loss_rate])
        sw = (c_uint32 * max(n, 1))(*[int(v) for v in share_weight])
        self.handle = c_void_p()
        _chk(lib().halo_plan_create(byref(self.handle), n_groups, n, lr, sw, mode, k_critical, threshold, seed),
             "halo_plan_create")

    def describe(self, M: int):
        n = self.n_dev
        order = (c_int32 * max(n, 1))()
        thr = (c_uint64 * max(n, 1))()
        bnd = (c_int32 * (n + 1))()
        _chk(lib().halo_plan_describe(self.handle, M, order, thr, bnd), "halo_plan_describe")
        return list(order)[:n], list(thr)[:n], list(bnd)

    def close(self):
        if self.handle:
            lib().halo_plan_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _darr(v):
    return (c_double * len(v))(*[float(x) for x in v])


def halo_schedule_comp_greedy(mem_budget, compute, model_mem):
    n = len(mem_budget)
    out = (c_double * n)()
    _chk(lib().halo_schedule_comp_greedy(n, _darr(mem_budget), _darr(compute), float(model_mem), out),
         "halo_schedule_comp_greedy")
    return list(out)


def halo_schedule_min_max(mem_budget, compute, model_mem, eps=1e-3):
    n = len(mem_budget)
    out = (c_double * n)()
    _chk(lib().halo_schedule_min_max(n, _darr(mem_budget), _darr(compute), float(model_mem), float(eps), out),
         "halo_schedule_min_max")
    return list(out)


def halo_ratios_to_share_weights(ratio):
    n = len(ratio)
    out = (c_uint32 * n)()
    _chk(lib().halo_ratios_to_share_weights(n, _darr(ratio), out), "halo_ratios_to_share_weights")
    return list(out)


def halo_late_devices(units, compute, tau, t_comm, timeout):
    n = len(units)
    out = (c_uint8 * n)()
    _chk(lib().halo_late_devices(n, (c_int32 * n)(*[int(u) for u in units]), _darr(compute), float(tau), float(t_comm),
                                 float(timeout), out), "halo_late_devices")
    return list(out)


def halo_group_importance(shape: FfnShape, W_packed, x, norms, workspace=None, dev_status=None, stream=None):
    """norms[g] = L2 norm of group g's partial output for the single input vector x.  Allocates the workspace
    with torch when none is given; returns it so that it can be reused."""
    need = int(lib().halo_group_importance_workspace_bytes(byref(shape)))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    _chk(lib().halo_group_importance(byref(shape), _ptr(W_packed), _ptr(x), _ptr(norms), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
         "halo_group_importance")
    return workspace


def halo_layer_fused(ffn: FfnShape, pred: PredShape, plan: Plan, W_packed, W1, W2, feat, x, n_tok, step, layer,
                     force_all, scores, dev_of_group, arrived, keep, y, workspace=None, dev_status=None, stream=None):
    """Steps a1..a9 of one block.  Allocates the workspace with torch when none is given and returns it."""
    need = int(lib().halo_layer_workspace_bytes(byref(ffn), byref(pred), n_tok, plan.n_dev))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    _chk(lib().halo_layer_fused(byref(ffn), byref(pred), plan.handle, _ptr(W_packed), _ptr(W1), _ptr(W2), _ptr(feat),
                                _ptr(x), n_tok, step, layer, int(bool(force_all)), _ptr(scores), _ptr(dev_of_group),
                                _ptr(arrived), _ptr(keep), _ptr(y), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
         "halo_layer_fused")
    return workspace


def halo_read_status(value: int) -> str:
    buf = ctypes.create_string_buffer(128)
    v = c_uint32(value)
    _chk(lib().halo_read_status(byref(v), buf, 128), "halo_read_status")
    return buf.value.decode()


def mha_shape(d_model, n_heads, head_dim, max_len, dtype) -> MhaShape:
    return MhaShape(d_model, n_heads, head_dim, max_len, dtype)


def halo_pack_mha_weights(shape: MhaShape, Wq, Wo, W_packed, stream=None) -> None:
    _chk(lib().halo_pack_mha_weights(byref(shape), _ptr(Wq), _ptr(Wo), _ptr(W_packed), _stream(stream)),
         "halo_pack_mha_weights")


def halo_mha_kv_append(shape: MhaShape, Wk, Wv, x, pos, K_cache, V_cache, stream=None) -> None:
    _chk(lib().halo_mha_kv_append(byref(shape), _ptr(Wk), _ptr(Wv), _ptr(x), pos, _ptr(K_cache), _ptr(V_cache),
                                  _stream(stream)), "halo_mha_kv_append")


def halo_group_mha_workspace_bytes(shape: MhaShape) -> int:
    return int(lib().halo_group_mha_workspace_bytes(byref(shape)))


def halo_group_mha(shape: MhaShape, W_packed, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group, n_dev,
                   partials, workspace, dev_status=None, stream=None) -> None:
    _chk(lib().halo_group_mha(byref(shape), _ptr(W_packed), _ptr(x), _ptr(K_cache), _ptr(V_cache), pos,
                              _ptr(keep_list), _ptr(n_keep), _ptr(dev_of_group), n_dev, _ptr(partials), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
         "halo_group_mha")


def halo_mha_block(shape: MhaShape, W_packed, Wk, Wv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group, n_dev,
                   partials, dev_status=None, stream=None) -> None:
    _chk(lib().halo_mha_block(byref(shape), _ptr(W_packed), _ptr(Wk), _ptr(Wv), _ptr(x), _ptr(K_cache), _ptr(V_cache), pos,
                              _ptr(keep_list), _ptr(n_keep), _ptr(dev_of_group), n_dev, _ptr(partials), _ptr(dev_status),
                              _stream(stream)), "halo_mha_block")


def halo_mha_block_i4(shape: MhaShape, Qp, Sp, Qk, Sk, Qv, Sv, x, K_cache, V_cache, pos, keep_list, n_keep, dev_of_group,
                      n_dev, partials, dev_status=None, stream=None) -> None:
    _chk(lib().halo_mha_block_i4(byref(shape), _ptr(Qp), _ptr(Sp), _ptr(Qk), _ptr(Sk), _ptr(Qv), _ptr(Sv), _ptr(x),
                                 _ptr(K_cache), _ptr(V_cache), pos, _ptr(keep_list), _ptr(n_keep), _ptr(dev_of_group), n_dev,
                                 _ptr(partials), _ptr(dev_status), _stream(stream)), "halo_mha_block_i4")


def lm_shape(d_model, vocab, group_size, dtype) -> LmShape:
    return LmShape(d_model, vocab, group_size, dtype)


def halo_group_lm_head(shape: LmShape, W, x, n_tok, keep_list, n_keep, logits, dev_status=None, stream=None) -> None:
    _chk(lib().halo_group_lm_head(byref(shape), _ptr(W), _ptr(x), n_tok, _ptr(keep_list), _ptr(n_keep), _ptr(logits),
                                  _ptr(dev_status), _stream(stream)), "halo_group_lm_head")


def halo_quantize_weights_i4(shape: FfnShape, W_packed, Q, scales, stream=None) -> None:
    _chk(lib().halo_quantize_weights_i4(byref(shape), _ptr(W_packed), _ptr(Q), _ptr(scales), _stream(stream)),
         "halo_quantize_weights_i4")


def halo_quantize_rows_i4(d_model: int, n_rows: int, wdtype: int, W, Q, scales, stream=None) -> None:
    _chk(lib().halo_quantize_rows_i4(d_model, n_rows, wdtype, _ptr(W), _ptr(Q), _ptr(scales), _stream(stream)),
         "halo_quantize_rows_i4")


def halo_group_lm_head_i4(shape: LmShape, Q, scales, x, n_tok, keep_list, n_keep, logits, dev_status, stream=None) -> None:
    _chk(lib().halo_group_lm_head_i4(byref(shape), _ptr(Q), _ptr(scales), _ptr(x), n_tok, _ptr(keep_list), _ptr(n_keep),
                                     _ptr(logits), _ptr(dev_status), _stream(stream)), "halo_group_lm_head_i4")


def halo_group_ffn_i4_workspace_bytes(shape: FfnShape, n_tok: int) -> int:
    return int(lib().halo_group_ffn_i4_workspace_bytes(byref(shape), n_tok))


def halo_group_ffn_i4_prompt(shape: FfnShape, Q, scales, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                             workspace, dev_status=None, stream=None) -> None:
    _chk(lib().halo_group_ffn_i4_prompt(byref(shape), _ptr(Q), _ptr(scales), _ptr(x), n_tok, _ptr(keep_list), _ptr(n_keep),
                                        _ptr(dev_of_group), n_dev, _ptr(partials), _ptr(workspace),
                                        workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                        _ptr(dev_status), _stream(stream)), "halo_group_ffn_i4_prompt")


def halo_dequantize_weights_i4(shape: FfnShape, Q, scales, keep_list, n_keep, W_packed, dev_status=None,
                               stream=None) -> None:
    _chk(lib().halo_dequantize_weights_i4(byref(shape), _ptr(Q), _ptr(scales), _ptr(keep_list), _ptr(n_keep),
                                          _ptr(W_packed), _ptr(dev_status), _stream(stream)),
         "halo_dequantize_weights_i4")


def halo_group_ffn_i4(shape: FfnShape, Q, scales, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                      dev_status=None, stream=None) -> None:
    _chk(lib().halo_group_ffn_i4(byref(shape), _ptr(Q), _ptr(scales), _ptr(x), n_tok, _ptr(keep_list), _ptr(n_keep),
                                 _ptr(dev_of_group), n_dev, _ptr(partials), _ptr(dev_status), _stream(stream)),
         "halo_group_ffn_i4")


def halo_selftest_bounded_wait(never_set_flag, limit_cycles, report, dev_status, stream=None) -> None:
    _chk(lib().halo_selftest_bounded_wait(_ptr(never_set_flag), int(limit_cycles), _ptr(report), _ptr(dev_status),
                                          _stream(stream)), "halo_selftest_bounded_wait")


def halo_predict_workspace_bytes(shape: PredShape, n_tok: int) -> int:
    return int(lib().halo_predict_workspace_bytes(byref(shape), n_tok))


def halo_predict_groups(shape: PredShape, W1, W2, feat, n_tok, mean_pool, scores, workspace, dev_status=None,
                        stream=None) -> None:
    _chk(lib().halo_predict_groups(byref(shape), _ptr(W1), _ptr(W2), _ptr(feat), n_tok, int(bool(mean_pool)),
                                   _ptr(scores), _ptr(workspace),
                                   workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                   _ptr(dev_status), _stream(stream)), "halo_predict_groups")


STATIC_SCRATCH_FLOATS = 512 * 1024


def halo_predict_groups_static(shape: PredShape, W1, W2, feat, n_tok, mean_pool, scores, dev_status=None,
                               stream=None) -> None:
    """halo_predict_groups without a workspace: the intermediates live in a fixed array inside the library, for
    callers that cannot allocate device memory.  Calls on one device share that array: keep them on one stream."""
    _chk(lib().halo_predict_groups_static(byref(shape), _ptr(W1), _ptr(W2), _ptr(feat), n_tok, int(bool(mean_pool)),
                                          _ptr(scores), _ptr(dev_status), _stream(stream)),
         "halo_predict_groups_static")


def halo_select_groups(plan: Plan, scores, step, layer, force_all, order, dev_of_group, arrived, keep, keep_list,
                       n_keep, dev_status=None, stream=None) -> None:
    _chk(lib().halo_select_groups(plan.handle, _ptr(scores), step, layer, int(bool(force_all)), _ptr(order),
                                  _ptr(dev_of_group), _ptr(arrived), _ptr(keep), _ptr(keep_list), _ptr(n_keep),
                                  _ptr(dev_status), _stream(stream)), "halo_select_groups")


def halo_group_ffn_workspace_bytes(shape: FfnShape, n_tok: int, n_dev: int) -> int:
    return int(lib().halo_group_ffn_workspace_bytes(byref(shape), n_tok, n_dev))


def halo_group_ffn(shape: FfnShape, W_packed, x, n_tok, keep_list, n_keep, dev_of_group, n_dev, partials,
                   workspace=None, dev_status=None, stream=None) -> None:
    _chk(lib().halo_group_ffn(byref(shape), _ptr(W_packed), _ptr(x), n_tok, _ptr(keep_list), _ptr(n_keep),
                              _ptr(dev_of_group), n_dev, _ptr(partials), _ptr(workspace),
                              workspace.numel() * workspace.element_size() if workspace is not None else 0,
                              _ptr(dev_status), _stream(stream)), "halo_group_ffn")


def halo_merge_partials(partials, arrived, n_dev, n_tok, d_model, y, stream=None) -> None:
    _chk(lib().halo_merge_partials(_ptr(partials), _ptr(arrived), n_dev, n_tok, d_model, _ptr(y), _stream(stream)),
         "halo_merge_partials")


def halo_pack_weights(shape: FfnShape, Wgate, Wup, Wdown, W_packed, stream=None) -> None:
    _chk(lib().halo_pack_weights(byref(shape), _ptr(Wgate), _ptr(Wup), _ptr(Wdown), _ptr(W_packed), _stream(stream)),
         "halo_pack_weights")


def halo_glue(d_model, n_tok, xdtype, h, y, h_out, x_out, stream=None) -> None:
    _chk(lib().halo_glue(d_model, n_tok, xdtype, _ptr(h), _ptr(y), _ptr(h_out), _ptr(x_out), _stream(stream)),
         "halo_glue")


class Stack:
    """halo_stack_create / halo_stack_decode / halo_stack_destroy.  Keeps the weight tensors alive."""

    def __init__(self, ffn: FfnShape, pred: PredShape, n_tok: int, plan: Plan, W_packed, W1, W2, i4_scales=None):
        """i4_scales given: W_packed holds the int4 codes of halo_quantize_weights_i4 (halo_stack_create_i4)."""
        L = len(W_packed)
        self._keep = (list(W_packed), list(W1), list(W2), plan, list(i4_scales) if i4_scales is not None else None)
        self.ffn, self.pred, self.n_layers, self.n_tok, self.plan = ffn, pred, L, n_tok, plan
        arr = lambda ts: (c_void_p * L)(*[(t.data_ptr() if t is not None else None) for t in ts])
        self.handle = c_void_p()
        if i4_scales is not None:
            _chk(lib().halo_stack_create_i4(byref(self.handle), byref(ffn), byref(pred), L, n_tok, plan.handle,
                                            arr(W_packed), arr(i4_scales), arr(W1), arr(W2)), "halo_stack_create_i4")
        else:
            _chk(lib().halo_stack_create(byref(self.handle), byref(ffn), byref(pred), L, n_tok, plan.handle,
                                         arr(W_packed), arr(W1), arr(W2)), "halo_stack_create")

    def decode(self, h0, steps, step0, h_out, taps: Taps | None = None, stream=None) -> None:
        _chk(lib().halo_stack_decode(self.handle, _ptr(h0), steps, step0, _ptr(h_out),
                                     byref(taps) if taps is not None else None, _stream(stream)), "halo_stack_decode")

    def decode_host(self, h0_host: torch.Tensor, steps, step0, h_out_host: torch.Tensor, stream=None) -> None:
        assert not h0_host.is_cuda and not h_out_host.is_cuda
        _chk(lib().halo_stack_decode_host(self.handle, c_void_p(h0_host.data_ptr()), steps, step0,
                                          c_void_p(h_out_host.data_ptr()), _stream(stream)), "halo_stack_decode_host")

    def set_mode(self, mode: int) -> None:
        _chk(lib().halo_stack_set_mode(self.handle, mode), "halo_stack_set_mode")

    def set_trace(self, n_blocks: int):
        """Allocates and attaches a trace buffer [n_blocks][width][8] (int64, ns); returns the tensor."""
        width = int(lib().halo_stack_trace_width(self.handle))
        self._trace = torch.zeros((max(n_blocks, 1), width, 8), dtype=torch.int64, device="cuda") if n_blocks else None
        _chk(lib().halo_stack_set_trace(self.handle, _ptr(self._trace) if n_blocks else None, n_blocks),
             "halo_stack_set_trace")
        return self._trace

    def status(self, stream=None) -> int:
        v = c_uint32(0)
        _chk(lib().halo_stack_status(self.handle, byref(v), _stream(stream)), "halo_stack_status")
        return int(v.value)

    def last_launches(self) -> int:
        return int(lib().halo_stack_last_launches(self.handle))

    def close(self):
        if self.handle:
            lib().halo_stack_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class BlockStack:
    """halo_block_stack_create / _decode / _destroy.  Keeps the weight and cache tensors alive.
    blocks: list of dicts with W_ffn, W_mha, Wk, Wv, K, V and (from the second layer on) W1_ffn, W2_ffn, W1_mha, W2_mha.
    int4 stacks (halo_block_stack_create_i4): the four weight entries hold codes, the dicts also have S_ffn, S_mha, Sk,
    Sv, and S_lm comes with W_lm."""

    def __init__(self, ffn: FfnShape, mha: MhaShape, lm, pred_ffn: PredShape, pred_mha: PredShape, plan_ffn: Plan,
                 plan_mha: Plan, blocks, W_lm=None, S_lm=None):
        L = len(blocks)
        self._keep = (blocks, W_lm, S_lm)
        self.plan_ffn, self.plan_mha = plan_ffn, plan_mha
        self.n_layers = L
        arr = lambda key: (c_void_p * L)(*[(b[key].data_ptr() if b.get(key) is not None else None) for b in blocks])
        self._arrays = {k: arr(k) for k in ("W_ffn", "W_mha", "Wk", "Wv", "W1_ffn", "W2_ffn", "W1_mha", "W2_mha", "K", "V")}
        w = BlockWeights()
        for k in ("W_ffn", "W_mha", "Wk", "Wv", "W1_ffn", "W2_ffn", "W1_mha", "W2_mha"):
            setattr(w, k, ctypes.cast(self._arrays[k], POINTER(c_void_p)))
        w.K_cache = ctypes.cast(self._arrays["K"], POINTER(c_void_p))
        w.V_cache = ctypes.cast(self._arrays["V"], POINTER(c_void_p))
        w.W_lm = c_void_p(W_lm.data_ptr()) if W_lm is not None else None
        self.handle = c_void_p()
        if blocks[0].get("S_ffn") is not None:
            self._scale_arrays = {k: arr(k) for k in ("S_ffn", "S_mha", "Sk", "Sv")}
            sc = BlockScales()
            for k in ("S_ffn", "S_mha", "Sk", "Sv"):
                setattr(sc, k, ctypes.cast(self._scale_arrays[k], POINTER(c_void_p)))
            sc.S_lm = c_void_p(S_lm.data_ptr()) if S_lm is not None else None
            _chk(lib().halo_block_stack_create_i4(byref(self.handle), byref(ffn), byref(mha),
                                                  byref(lm) if lm is not None else None, byref(pred_ffn), byref(pred_mha), L,
                                                  plan_ffn.handle, plan_mha.handle, byref(w), byref(sc)),
                 "halo_block_stack_create_i4")
            return
        _chk(lib().halo_block_stack_create(byref(self.handle), byref(ffn), byref(mha), byref(lm) if lm is not None else None,
                                           byref(pred_ffn), byref(pred_mha), L, plan_ffn.handle, plan_mha.handle, byref(w)),
             "halo_block_stack_create")

    def decode(self, h0, steps, pos0, step0, logits=None, h_out=None, taps: BlockTaps | None = None, stream=None) -> None:
        _chk(lib().halo_block_stack_decode(self.handle, _ptr(h0), steps, pos0, step0, _ptr(logits), _ptr(h_out),
                                           byref(taps) if taps is not None else None, _stream(stream)),
             "halo_block_stack_decode")

    def status(self, stream=None) -> int:
        v = c_uint32(0)
        _chk(lib().halo_block_stack_status(self.handle, byref(v), _stream(stream)), "halo_block_stack_status")
        return int(v.value)

    def last_launches(self) -> int:
        return int(lib().halo_block_stack_last_launches(self.handle))

    def close(self):
        if self.handle:
            lib().halo_block_stack_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
