"""Thin ctypes binding over libprox.so (declared in include/prox.h).

Argument marshalling only: every function here has the name of the C entry
point it forwards to, takes raw device pointers (Python ints, e.g.
``tensor.data_ptr()``) or objects exposing ``data_ptr()``, and raises
``ProxError`` when the library returns a non-zero status.  No step of the
path is computed in Python and there is no fallback: if the shared library
is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libprox.so")

STATUS_NAMES = {
    0: "PROX_OK", 1: "PROX_ERR_INVALID_ARG", 2: "PROX_ERR_UNSUPPORTED", 3: "PROX_ERR_NOT_QUANTIZED",
    4: "PROX_ERR_CUDA", 5: "PROX_ERR_OOM", 6: "PROX_ERR_TIMEOUT", 7: "PROX_ERR_IO",
}


class ProxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = _lib.prox_last_cuda_error().decode() if status in (4, 5) else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({prox_status_string(status)})"
                         + (f": {detail}" if detail else ""))


class ProxFFNConfig(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("d_ff", C.c_int32), ("max_batch", C.c_int32),
                ("out_dtype", C.c_int32)]


if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2607_27591_b200.build` "
        "(needs nvcc). There is no fallback implementation.")
_lib = C.CDLL(_LIB_PATH)

_vp, _i, _f, _d = C.c_void_p, C.c_int, C.c_float, C.c_double
_SIGS = {
    "prox_ffn_create": [C.POINTER(ProxFFNConfig), _vp, _vp, _vp, _vp, C.POINTER(_vp)],
    "prox_quantize_proxy": [_vp, _i, _i, _vp],
    "prox_stage1_mask": [_vp, _vp, _i, _i, _i, _vp, _vp, _vp],
    "prox_stage2_ffn": [_vp, _vp, _i, _vp, _i, _vp, _vp],
    "prox_ffn_forward": [_vp, _vp, _i, _i, _i, _vp, _vp],
    "prox_ffn_forward_host": [_vp, _vp, _i, _i, _i, _vp, _vp],
    "prox_stage2_ffn_noalloc": [_vp, _vp, _vp, _vp, _i, _i, _vp, _i, _vp, _i, _vp],
    "prox_stage1_mask_threshold": [_vp, _vp, _i, _f, _f, _vp, _vp, _vp, _vp],
    "prox_stage2_ffn_var": [_vp, _vp, _i, _vp, _vp, _vp, _vp],
    "prox_ffn_forward_threshold": [_vp, _vp, _i, _f, _f, _vp, _vp],
    "prox_ffn_forward_proxy_values": [_vp, _vp, _i, _i, _i, _vp, _vp],
    "prox_ffn_block_forward": [_vp, _vp, _vp, _d, _i, _i, _i, _vp, _vp],
    "prox_ffn_stack_forward": [C.POINTER(_vp), _i, _vp, _d, _vp, _i, _i, _i, _vp, _vp],
    "prox_ffn_block_forward_threshold": [_vp, _vp, _vp, _d, _i, _f, _f, _vp, _vp],
    "prox_ffn_stack_forward_threshold": [C.POINTER(_vp), _i, _vp, _d, _vp, _i, C.POINTER(_f), C.POINTER(_f), _vp, _vp],
    "prox_runtime_sparsity": [_vp, _d, C.POINTER(C.c_int64), C.POINTER(_d), C.POINTER(_d), C.POINTER(_d), _i],
    "prox_allocate_budget": [_d, _d, _d, _d, _d, C.POINTER(_d), C.POINTER(_d)],
    "prox_sparsity_to_k": [_d, _i, C.POINTER(_i)],
    "prox_proxy_export": [_vp, _i, _vp, _vp],
    "prox_input_topk": [_vp, _vp, _i, _i, _vp, _vp],
    "prox_pack_save": [_vp, C.c_char_p],
    "prox_pack_load": [_vp, C.c_char_p, _vp],
    "prox_algorithmic_bytes": [_vp, _i, _i, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                               C.POINTER(C.c_int64), C.POINTER(C.c_int64)],
    "prox_last_device_status": [_vp, C.POINTER(C.c_int32), _vp],
    "prox_launch_count": [_vp, C.POINTER(C.c_int64)],
    "prox_ffn_set_fused": [_vp, _i],
    "prox_ffn_set_union": [_vp, _i],
    "prox_ffn_set_mask_policy": [_vp, _i],
    "prox_fused_trace": [_vp, _i, _vp, _i],
    "prox_fused_kernel_info": [_vp, _i, _i, C.POINTER(C.c_int32)],
    "prox_ffn_last_mask": [_vp, _i, _i, _vp, _vp],
    "prox_ffn_last_stage1": [_vp, _i, _vp, _vp, _vp],
    "prox_debug_set_wait": [_vp, C.c_uint32, C.c_uint32],
    "prox_calib_create": [C.c_int64, C.c_uint64, C.POINTER(_vp)],
    "prox_calib_add": [_vp, _vp, C.c_int64, _i, _vp],
    "prox_calib_threshold": [_vp, _d, C.POINTER(_f)],
    "prox_calib_histogram": [_vp, C.POINTER(C.c_int64), C.POINTER(_f)],
    "prox_calib_seen": [_vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)],
    "prox_rmsnorm": [_vp, _vp, _vp, _d, _i, _vp, _vp],
    "prox_profile_enable": [_vp, _i],
    "prox_profile_read": [_vp, C.POINTER(C.c_int64), C.POINTER(_d)],
}
for _name, _args in _SIGS.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = C.c_int
_lib.prox_ffn_destroy.argtypes = [_vp]
_lib.prox_ffn_destroy.restype = None
_lib.prox_calib_destroy.argtypes = [_vp]
_lib.prox_calib_destroy.restype = None
_lib.prox_status_string.argtypes = [C.c_int]
_lib.prox_status_string.restype = C.c_char_p
_lib.prox_last_cuda_error.argtypes = []
_lib.prox_last_cuda_error.restype = C.c_char_p
_lib.prox_version.argtypes = []
_lib.prox_version.restype = C.c_char_p

EXPORTED = tuple(_SIGS) + ("prox_ffn_destroy", "prox_calib_destroy", "prox_status_string", "prox_version", "prox_last_cuda_error")


def _ptr(obj) -> Optional[int]:
    """Raw address of a device/host buffer: int, None, or anything with data_ptr()."""
    if obj is None:
        return None
    if isinstance(obj, int):
        return obj
    if hasattr(obj, "data_ptr"):
        return obj.data_ptr()
    if hasattr(obj, "ctypes"):                       # numpy array (host memory)
        return obj.ctypes.data
    raise TypeError(f"cannot take the address of {type(obj)}")


def _check(status: int, where: str) -> None:
    if status != 0:
        raise ProxError(status, where)


def prox_status_string(status: int) -> str:
    return _lib.prox_status_string(int(status)).decode()


def prox_version() -> str:
    return _lib.prox_version().decode()


def prox_ffn_create(d_model: int, d_ff: int, max_batch: int, out_dtype: int, w_gate, w_up, w_down,
                    stream=None) -> int:
    cfg = ProxFFNConfig(d_model, d_ff, max_batch, out_dtype)
    out = _vp()
    _check(_lib.prox_ffn_create(C.byref(cfg), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(stream),
                                C.byref(out)), "prox_ffn_create")
    return out.value


def prox_ffn_destroy(handle: int) -> None:
    _lib.prox_ffn_destroy(handle)


def prox_quantize_proxy(handle: int, bits: int, group_size: int, stream=None) -> None:
    _check(_lib.prox_quantize_proxy(handle, bits, group_size, _ptr(stream)), "prox_quantize_proxy")


def prox_stage1_mask(handle: int, x, B: int, k1: int, k2: int, sel, scores=None, stream=None) -> None:
    _check(_lib.prox_stage1_mask(handle, _ptr(x), B, k1, k2, _ptr(sel), _ptr(scores), _ptr(stream)),
           "prox_stage1_mask")


def prox_stage2_ffn(handle: int, x, B: int, sel, k2: int, y, stream=None) -> None:
    _check(_lib.prox_stage2_ffn(handle, _ptr(x), B, _ptr(sel), k2, _ptr(y), _ptr(stream)), "prox_stage2_ffn")


def prox_ffn_forward(handle: int, x, B: int, k1: int, k2: int, y, stream=None) -> None:
    _check(_lib.prox_ffn_forward(handle, _ptr(x), B, k1, k2, _ptr(y), _ptr(stream)), "prox_ffn_forward")


def prox_stage2_ffn_noalloc(x, w_gate, w_up, w_down_t, d_model: int, d_ff: int, sel, k2: int, y,
                            out_dtype: int, stream=None) -> None:
    """Stage 2 without a handle and without any allocation (B = 1): the caller passes
    every tensor, W_down in channel-major [d_ff, d_model] form; the intermediates sit
    in a fixed array inside the library (d_model <= 16384, k2 <= 32768)."""
    _check(_lib.prox_stage2_ffn_noalloc(_ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down_t), d_model, d_ff,
                                        _ptr(sel), k2, _ptr(y), out_dtype, _ptr(stream)),
           "prox_stage2_ffn_noalloc")


def prox_ffn_set_fused(handle: int, on: int) -> None:
    _check(_lib.prox_ffn_set_fused(handle, int(on)), "prox_ffn_set_fused")


def prox_ffn_set_mask_policy(handle: int, policy: int) -> None:
    _check(_lib.prox_ffn_set_mask_policy(handle, int(policy)), "prox_ffn_set_mask_policy")


def prox_ffn_set_union(handle: int, on: int) -> None:
    _check(_lib.prox_ffn_set_union(handle, int(on)), "prox_ffn_set_union")


def prox_fused_kernel_info(handle: int, k1: int, k2: int) -> dict:
    info = (C.c_int32 * 8)()
    _check(_lib.prox_fused_kernel_info(handle, k1, k2, info), "prox_fused_kernel_info")
    keys = ("usable", "grid", "ksplit", "smem_bytes", "ring_slots", "registers", "static_smem", "blocks_per_sm")
    return dict(zip(keys, list(info)))


def prox_fused_trace(handle: int, on: int, stamps_host=None, max_blocks: int = 0) -> None:
    _check(_lib.prox_fused_trace(handle, int(on), _ptr(stamps_host), max_blocks), "prox_fused_trace")


def prox_ffn_last_mask(handle: int, B: int, k2: int, sel, stream=None) -> None:
    _check(_lib.prox_ffn_last_mask(handle, B, k2, _ptr(sel), _ptr(stream)), "prox_ffn_last_mask")


def prox_ffn_forward_host(handle: int, x_host, B: int, k1: int, k2: int, y_host, stream=None) -> None:
    _check(_lib.prox_ffn_forward_host(handle, _ptr(x_host), B, k1, k2, _ptr(y_host), _ptr(stream)),
           "prox_ffn_forward_host")


def prox_stage1_mask_threshold(handle: int, x, B: int, tau_x: float, tau_s: float, sel, count,
                               scores=None, stream=None) -> None:
    _check(_lib.prox_stage1_mask_threshold(handle, _ptr(x), B, tau_x, tau_s, _ptr(sel), _ptr(count),
                                           _ptr(scores), _ptr(stream)), "prox_stage1_mask_threshold")


def prox_stage2_ffn_var(handle: int, x, B: int, sel, count, y, stream=None) -> None:
    _check(_lib.prox_stage2_ffn_var(handle, _ptr(x), B, _ptr(sel), _ptr(count), _ptr(y), _ptr(stream)),
           "prox_stage2_ffn_var")


def prox_ffn_forward_threshold(handle: int, x, B: int, tau_x: float, tau_s: float, y, stream=None) -> None:
    _check(_lib.prox_ffn_forward_threshold(handle, _ptr(x), B, tau_x, tau_s, _ptr(y), _ptr(stream)),
           "prox_ffn_forward_threshold")


def prox_ffn_forward_proxy_values(handle: int, x, B: int, k1: int, k2: int, y, stream=None) -> None:
    _check(_lib.prox_ffn_forward_proxy_values(handle, _ptr(x), B, k1, k2, _ptr(y), _ptr(stream)),
           "prox_ffn_forward_proxy_values")


def prox_ffn_block_forward(handle: int, x_res, norm_w, eps: float, B: int, k1: int, k2: int, x_res_out,
                           stream=None) -> None:
    _check(_lib.prox_ffn_block_forward(handle, _ptr(x_res), _ptr(norm_w), eps, B, k1, k2, _ptr(x_res_out),
                                       _ptr(stream)), "prox_ffn_block_forward")


def prox_ffn_stack_forward(handles, norm_w, eps: float, x_res, B: int, k1: int, k2: int, trace=None,
                           stream=None) -> None:
    arr = (_vp * len(handles))(*handles)
    _check(_lib.prox_ffn_stack_forward(arr, len(handles), _ptr(norm_w), eps, _ptr(x_res), B, k1, k2,
                                       _ptr(trace), _ptr(stream)), "prox_ffn_stack_forward")


def prox_ffn_block_forward_threshold(handle: int, x_res, norm_w, eps: float, B: int, tau_x: float, tau_s: float,
                                     x_res_out, stream=None) -> None:
    _check(_lib.prox_ffn_block_forward_threshold(handle, _ptr(x_res), _ptr(norm_w), eps, B, tau_x, tau_s,
                                                 _ptr(x_res_out), _ptr(stream)), "prox_ffn_block_forward_threshold")


def prox_ffn_stack_forward_threshold(handles, norm_w, eps: float, x_res, B: int, tau_x, tau_s, trace=None,
                                     stream=None) -> None:
    n = len(handles)
    arr = (_vp * n)(*handles)
    tx = (_f * n)(*[float(v) for v in tau_x])
    ts = (_f * n)(*[float(v) for v in tau_s])
    _check(_lib.prox_ffn_stack_forward_threshold(arr, n, _ptr(norm_w), eps, _ptr(x_res), B, tx, ts, _ptr(trace),
                                                 _ptr(stream)), "prox_ffn_stack_forward_threshold")


def prox_calib_create(capacity: int = 200000, seed: int = 0) -> int:
    out = _vp()
    _check(_lib.prox_calib_create(capacity, seed, C.byref(out)), "prox_calib_create")
    return out.value


def prox_calib_destroy(calib: int) -> None:
    _lib.prox_calib_destroy(calib)


def prox_calib_add(calib: int, values, n: int, dtype: int, stream=None) -> None:
    """dtype 0: dev bf16 values, 1: dev fp32 values."""
    _check(_lib.prox_calib_add(calib, _ptr(values), n, dtype, _ptr(stream)), "prox_calib_add")


def prox_calib_threshold(calib: int, s: float) -> float:
    tau = _f()
    _check(_lib.prox_calib_threshold(calib, s, C.byref(tau)), "prox_calib_threshold")
    return tau.value


def prox_calib_histogram(calib: int):
    counts = (C.c_int64 * 4096)()
    hi = _f()
    _check(_lib.prox_calib_histogram(calib, counts, C.byref(hi)), "prox_calib_histogram")
    return list(counts), hi.value


def prox_calib_seen(calib: int):
    seen, held = C.c_int64(), C.c_int64()
    _check(_lib.prox_calib_seen(calib, C.byref(seen), C.byref(held)), "prox_calib_seen")
    return seen.value, held.value


def prox_rmsnorm(handle: int, x_res, norm_w, eps: float, B: int, xn_out, stream=None) -> None:
    _check(_lib.prox_rmsnorm(handle, _ptr(x_res), _ptr(norm_w), eps, B, _ptr(xn_out), _ptr(stream)), "prox_rmsnorm")


def prox_calibrate_stack(handles, d_ff: int, norm_w, eps: float, x_res_tokens, s1: float, s2: float,
                         capacity: int = 200000, seed: int = 0, stream=None):
    """Sequential threshold calibration (Alg. 1) of a stack of FFN sub-blocks, driven through the library:
    per layer, in depth order, on the stream that the finalized rules of the earlier layers produce:
    FFN inputs (prox_rmsnorm) -> tau_x (reservoir quantile at s1) -> proxy scores under that input mask
    (prox_stage1_mask_threshold) -> tau_s (quantile at s2) -> the tokens advance through the layer under
    its finalized rule (prox_ffn_block_forward_threshold).
    handles: one per layer (all of width d_ff); norm_w: dev bf16 [L, d_model]; x_res_tokens: dev fp32 [N, d_model] (left untouched).
    Device buffers come from torch (plumbing); every step of the path is a library call.
    Returns (tau_x list, tau_s list, list of (hist_x, hist_s) with hist = (counts[4096], upper edge))."""
    import torch
    N, D = x_res_tokens.shape
    xs = x_res_tokens.clone()
    nxt = torch.empty_like(xs)
    dev = xs.device
    xn = torch.empty(N, D, dtype=torch.bfloat16, device=dev)
    sc = torch.empty(N, d_ff, dtype=torch.float32, device=dev)
    sel = torch.empty(1, d_ff, dtype=torch.int32, device=dev)
    cnt = torch.empty(1, dtype=torch.int32, device=dev)
    tau_x, tau_s, hists = [], [], []
    for li, h in enumerate(handles):
        cx, cs = prox_calib_create(capacity, seed + 2 * li), prox_calib_create(capacity, seed + 2 * li + 1)
        try:
            for i in range(N):
                prox_rmsnorm(h, xs[i], norm_w[li], eps, 1, xn[i], stream)
            prox_calib_add(cx, xn, N * D, 0, stream)
            tx = prox_calib_threshold(cx, s1)
            for i in range(N):
                prox_stage1_mask_threshold(h, xn[i], 1, tx, 0.0, sel, cnt, sc[i], stream)
            prox_calib_add(cs, sc, sc.numel(), 1, stream)
            ts = prox_calib_threshold(cs, s2)
            for i in range(N):
                prox_ffn_block_forward_threshold(h, xs[i], norm_w[li], eps, 1, tx, ts, nxt[i], stream)
            hists.append((prox_calib_histogram(cx), prox_calib_histogram(cs)))
        finally:
            prox_calib_destroy(cx); prox_calib_destroy(cs)
        tau_x.append(tx); tau_s.append(ts)
        xs, nxt = nxt, xs
    torch.cuda.synchronize(dev)
    return tau_x, tau_s, hists


def prox_runtime_sparsity(handle: int, alpha: float = 1.0 / 3.0, reset: bool = False):
    tok, s1, s2, e = C.c_int64(), _d(), _d(), _d()
    _check(_lib.prox_runtime_sparsity(handle, alpha, C.byref(tok), C.byref(s1), C.byref(s2), C.byref(e),
                                      int(reset)), "prox_runtime_sparsity")
    return tok.value, s1.value, s2.value, e.value


def prox_allocate_budget(e: float, alpha: float = 1.0 / 3.0, s_ref: float = 0.7, s1_min: float = 0.0,
                         s1_max: float = 0.7) -> Tuple[float, float]:
    s1, s2 = _d(), _d()
    _check(_lib.prox_allocate_budget(e, alpha, s_ref, s1_min, s1_max, C.byref(s1), C.byref(s2)),
           "prox_allocate_budget")
    return s1.value, s2.value


def prox_sparsity_to_k(s: float, dim: int) -> int:
    k = _i()
    _check(_lib.prox_sparsity_to_k(s, dim, C.byref(k)), "prox_sparsity_to_k")
    return k.value


def prox_proxy_export(handle: int, which: int, q_host, scale_host) -> None:
    _check(_lib.prox_proxy_export(handle, which, _ptr(q_host), _ptr(scale_host)), "prox_proxy_export")


def prox_input_topk(handle: int, x, B: int, k1: int, idx, stream=None) -> None:
    _check(_lib.prox_input_topk(handle, _ptr(x), B, k1, _ptr(idx), _ptr(stream)), "prox_input_topk")


def prox_pack_save(handle: int, path: str) -> None:
    _check(_lib.prox_pack_save(handle, os.fsencode(path)), "prox_pack_save")


def prox_pack_load(handle: int, path: str, stream=None) -> None:
    _check(_lib.prox_pack_load(handle, os.fsencode(path), _ptr(stream)), "prox_pack_load")


def prox_algorithmic_bytes(handle: int, rows_in: int, rows_ch: int):
    a, b, c, d = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
    _check(_lib.prox_algorithmic_bytes(handle, rows_in, rows_ch, C.byref(a), C.byref(b), C.byref(c),
                                       C.byref(d)), "prox_algorithmic_bytes")
    return a.value, b.value, c.value, d.value


def prox_last_device_status_raw(handle: int, stream=None):
    """(status, code) of prox_last_device_status: status is PROX_ERR_TIMEOUT (6) when bit 4 of code is set."""
    code = C.c_int32()
    status = _lib.prox_last_device_status(handle, C.byref(code), _ptr(stream))
    return status, code.value


def prox_last_device_status(handle: int, stream=None) -> int:
    """The status word (bit 4 = a bounded wait expired; the library has then reset its shared counters)."""
    status, code = prox_last_device_status_raw(handle, stream)
    if status not in (0, 6):
        _check(status, "prox_last_device_status")
    return code


def prox_ffn_last_stage1(handle: int, k1: int, idx=None, scores=None, stream=None) -> None:
    _check(_lib.prox_ffn_last_stage1(handle, k1, _ptr(idx), _ptr(scores), _ptr(stream)), "prox_ffn_last_stage1")


def prox_debug_set_wait(handle: int, spin_limit: int, barrier_bias: int) -> None:
    _check(_lib.prox_debug_set_wait(handle, spin_limit, barrier_bias), "prox_debug_set_wait")


def prox_launch_count(handle: int) -> int:
    n = C.c_int64()
    _check(_lib.prox_launch_count(handle, C.byref(n)), "prox_launch_count")
    return n.value


KERNEL_KINDS = ("input_select", "proxy_gemv", "channel_select", "gateup", "down", "finalize", "prox_fused", "union")


def prox_profile_enable(handle: int, on: int) -> None:
    _check(_lib.prox_profile_enable(handle, int(on)), "prox_profile_enable")


def prox_profile_read(handle: int):
    """{kernel kind: (launches, total milliseconds)} since the last read."""
    n = (C.c_int64 * len(KERNEL_KINDS))()
    ms = (_d * len(KERNEL_KINDS))()
    _check(_lib.prox_profile_read(handle, n, ms), "prox_profile_read")
    return {k: (n[i], ms[i]) for i, k in enumerate(KERNEL_KINDS)}


def raw(name: str):
    """The raw ctypes function (returns the status instead of raising); for tests of error paths."""
    return getattr(_lib, name)
