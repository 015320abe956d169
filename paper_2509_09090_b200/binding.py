"""ctypes binding of ``libsqap.so``: same names as the C ABI (``include/sqap.h``), argument
marshalling only. Tensors are torch CUDA tensors (device memory) or raw integer addresses;
nothing is computed here, and there is no fallback: if the library cannot be loaded the
import of a symbol raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsqap.so")

SQAP_OK, SQAP_ERR_INVALID, SQAP_ERR_RANGE, SQAP_ERR_ALIGN, SQAP_ERR_UNSUPPORTED, SQAP_ERR_NOMEM, \
    SQAP_ERR_CUDA, SQAP_ERR_TIMEOUT, SQAP_ERR_TOO_LARGE = range(9)
SQAP_STATIC_WORKSPACE_BYTES = 4 * 1024 * 1024 + 8192
SQAP_FP16, SQAP_BF16, SQAP_I32 = 0, 1, 2
SQAP_Q_ROTATE = 1
SQAP_Q_PER_TENSOR = 2
SQAP_W_ROTATED = 1
SQAP_L_FORCE_SIMT, SQAP_L_FORCE_TCGEN05, SQAP_L_FORCE_GEMV, SQAP_L_REUSE_EXPANDED, SQAP_L_FORCE_TCGEN05_TS, SQAP_L_FORCE_TCGEN05_PAIR = 1, 2, 4, 8, 16, 32
SQAP_L_FORCE_MMA = 64
SQAP_L_FORCE_TCGEN05_SPLITK = 128


def SQAP_L_KSPLIT(n: int) -> int:
    return n << 8

EXPORTS = ("sqap_pack_weights", "sqap_quantize_weights", "sqap_free_weights", "sqap_weights_info", "sqap_unpack_weights",
           "sqap_quantize_act", "sqap_quantize_act_ex", "sqap_workspace_bytes", "sqap_w4a4_linear", "sqap_w4a4_linear_static",
           "sqap_quantize_linear", "sqap_quantize_linear_workspace_bytes",
           "sqap_prune_tokens", "sqap_prune_select", "sqap_attention_scores",
           "sqap_project_center", "sqap_device_status", "sqap_last_cuda_error", "sqap_status_string",
           "sqap_kernel_launch_count", "sqap_selftest_bounded_wait")


class SqapError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().sqap_status_string(status).decode()
        extra = f" (cudaError {lib().sqap_last_cuda_error()})" if status == SQAP_ERR_CUDA else ""
        super().__init__(f"{where}: {msg}{extra}")


class PruneParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("batch", "rows", "visual_start", "n_visual", "grid_w", "grid_h",
                                            "score_rows", "k_attn", "keep_total", "ring_radius")] + \
               [("flags", ctypes.c_uint32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library (building it with nvcc first if the shared object is absent)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        from . import build as _build
        _build.build()
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32, ctypes.c_size_t
    L.sqap_pack_weights.argtypes = [vp, vp, i32, i32, u32, vp, ctypes.POINTER(vp)]
    L.sqap_quantize_weights.argtypes = [vp, i32, i32, i64, u32, vp, vp, vp, vp]
    L.sqap_quantize_act_ex.argtypes = [vp, i32, i32, i64, vp, u32, vp, vp, vp, vp]
    L.sqap_free_weights.argtypes = [vp]
    L.sqap_weights_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(u32)]
    L.sqap_unpack_weights.argtypes = [vp, vp, vp]
    L.sqap_quantize_act.argtypes = [vp, i32, i32, i64, vp, u32, vp, vp, vp]
    L.sqap_workspace_bytes.argtypes = [i32, i32, i32, u32]
    L.sqap_workspace_bytes.restype = sz
    L.sqap_w4a4_linear.argtypes = [vp, vp, i32, vp, vp, vp, i64, i32, u32, vp, sz, vp]
    L.sqap_w4a4_linear_static.argtypes = [vp, vp, i32, vp, vp, vp, i64, i32, u32, vp]
    L.sqap_quantize_linear_workspace_bytes.argtypes = [i32, i32, i32]
    L.sqap_quantize_linear_workspace_bytes.restype = sz
    L.sqap_quantize_linear.argtypes = [vp, i32, i64, vp, u32, vp, vp, vp, i64, i32, u32, vp, sz, vp]
    L.sqap_prune_tokens.argtypes = [ctypes.POINTER(PruneParams), vp, vp, vp, i64, i32, vp, i64, i32, vp, vp, vp]
    L.sqap_prune_select.argtypes = [ctypes.POINTER(PruneParams), vp, vp, i32, vp, vp, vp, vp]
    L.sqap_attention_scores.argtypes = [vp, i64, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp]
    L.sqap_project_center.argtypes = [ctypes.POINTER(ctypes.c_double)] * 3 + [ctypes.c_double, ctypes.c_double,
                                                                              ctypes.POINTER(ctypes.c_int32),
                                                                              ctypes.POINTER(i32)]
    L.sqap_device_status.argtypes = [vp]
    L.sqap_selftest_bounded_wait.argtypes = [i64, vp]
    L.sqap_last_cuda_error.restype = i32
    L.sqap_status_string.argtypes = [i32]
    L.sqap_status_string.restype = ctypes.c_char_p
    L.sqap_kernel_launch_count.restype = i64
    for name in EXPORTS:
        getattr(L, name)  # raises AttributeError if the library lacks a declared entry point
    _lib = L
    return L


def _ptr(t):
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(f"cannot take the address of {type(t)}")


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(st: int, where: str):
    if st != SQAP_OK:
        raise SqapError(st, where)


class Weights:
    """Owner of a ``sqap_weights*``; freed on ``close()`` or garbage collection."""

    def __init__(self, handle: int, N: int, K: int):
        self.handle, self.N, self.K = handle, N, K

    def close(self):
        if self.handle:
            lib().sqap_free_weights(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sqap_pack_weights(codes, scales_fp16, N: int, K: int, flags: int = 0, stream=None) -> Weights:
    """codes: int8 [N, K] (numpy on the host or torch on the device); scales_fp16: fp16 [N]."""
    out = ctypes.c_void_p()
    st = lib().sqap_pack_weights(_ptr(codes), _ptr(scales_fp16), N, K, flags, _stream(stream), ctypes.byref(out))
    _check(st, "sqap_pack_weights")
    return Weights(out.value, N, K)


def sqap_quantize_weights(w_fp16, N: int, K: int, ldw: int, flags: int, channel_mul, codes_out, scales_out_fp16,
                          stream=None):
    """fp16 weights [N, ldw] (device) -> int8 codes [N, K] and fp16 scales [N] (device), see include/sqap.h."""
    _check(lib().sqap_quantize_weights(_ptr(w_fp16), N, K, ldw, flags, _ptr(channel_mul), _ptr(codes_out),
                                       _ptr(scales_out_fp16), _stream(stream)), "sqap_quantize_weights")


def sqap_quantize_act_ex(x, M: int, K: int, ldx: int, row_index, flags: int, channel_mul, q_packed, scales, stream=None):
    _check(lib().sqap_quantize_act_ex(_ptr(x), M, K, ldx, _ptr(row_index), flags, _ptr(channel_mul), _ptr(q_packed),
                                      _ptr(scales), _stream(stream)), "sqap_quantize_act_ex")


def sqap_free_weights(w: Weights):
    w.close()


def sqap_weights_info(w: Weights):
    n, k, f = ctypes.c_int(), ctypes.c_int(), ctypes.c_uint32()
    _check(lib().sqap_weights_info(w.handle, ctypes.byref(n), ctypes.byref(k), ctypes.byref(f)), "sqap_weights_info")
    return n.value, k.value, f.value


def sqap_unpack_weights(w: Weights):
    import numpy as np
    codes = np.empty((w.N, w.K), np.int8)
    scales = np.empty((w.N,), np.uint16)
    _check(lib().sqap_unpack_weights(w.handle, _ptr(codes), _ptr(scales)), "sqap_unpack_weights")
    return codes, scales.view(np.float16)


def sqap_quantize_act(x, M: int, K: int, ldx: int, row_index, flags: int, q_packed, scales, stream=None):
    _check(lib().sqap_quantize_act(_ptr(x), M, K, ldx, _ptr(row_index), flags, _ptr(q_packed), _ptr(scales),
                                   _stream(stream)), "sqap_quantize_act")


def sqap_workspace_bytes(M: int, N: int, K: int, flags: int = 0) -> int:
    return int(lib().sqap_workspace_bytes(M, N, K, flags))


def sqap_w4a4_linear(q_packed, act_scales, M: int, w: Weights, w_up, out, ldo: int, out_dtype: int, flags: int,
                     workspace, workspace_bytes: int, stream=None):
    _check(lib().sqap_w4a4_linear(_ptr(q_packed), _ptr(act_scales), M, w.handle, w_up.handle if w_up else None,
                                  _ptr(out), ldo, out_dtype, flags, _ptr(workspace), workspace_bytes,
                                  _stream(stream)), "sqap_w4a4_linear")


def sqap_quantize_linear_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().sqap_quantize_linear_workspace_bytes(M, N, K))


def sqap_quantize_linear(x, M: int, ldx: int, row_index, qflags: int, w: Weights, w_up, out, ldo: int, out_dtype: int,
                         lflags: int, workspace, workspace_bytes: int, stream=None):
    """Quantizer and linear as one call (fp16 rows in, fp16/bf16 rows out); see include/sqap.h."""
    _check(lib().sqap_quantize_linear(_ptr(x), M, ldx, _ptr(row_index), qflags, w.handle,
                                      w_up.handle if w_up else None, _ptr(out), ldo, out_dtype, lflags,
                                      _ptr(workspace), workspace_bytes, _stream(stream)), "sqap_quantize_linear")


def sqap_w4a4_linear_static(q_packed, act_scales, M: int, w: Weights, w_up, out, ldo: int, out_dtype: int, flags: int,
                            stream=None):
    """The linear without a caller workspace, for callers that cannot allocate device memory: the scratch
    is a fixed array inside the library (see include/sqap.h for its size limit and sharing rules)."""
    _check(lib().sqap_w4a4_linear_static(_ptr(q_packed), _ptr(act_scales), M, w.handle,
                                         w_up.handle if w_up else None, _ptr(out), ldo, out_dtype, flags,
                                         _stream(stream)), "sqap_w4a4_linear_static")


def sqap_prune_tokens(params: dict, scores, ring_center, x, ldx: int, K: int, x_out, ldo: int, out_rows: int,
                      kept_idx, n_kept, stream=None):
    p = PruneParams(**{k: int(v) for k, v in params.items()})
    _check(lib().sqap_prune_tokens(ctypes.byref(p), _ptr(scores), _ptr(ring_center), _ptr(x), ldx, K, _ptr(x_out),
                                   ldo, out_rows, _ptr(kept_idx), _ptr(n_kept), _stream(stream)),
           "sqap_prune_tokens")


def sqap_prune_select(params: dict, scores, ring_center, out_rows: int, kept_idx, n_kept, row_index, stream=None):
    """The criterion without the row copy: kept indices plus the flat source-row list for a quantizer's row_index."""
    p = PruneParams(**{k: int(v) for k, v in params.items()})
    _check(lib().sqap_prune_select(ctypes.byref(p), _ptr(scores), _ptr(ring_center), out_rows, _ptr(kept_idx),
                                   _ptr(n_kept), _ptr(row_index), _stream(stream)), "sqap_prune_select")


def sqap_attention_scores(qkv, ldq: int, batch: int, rows: int, query_row: int, visual_start: int, n_visual: int,
                          n_heads: int, head_dim: int, q_col0: int, k_col0: int, scores_out, stream=None):
    _check(lib().sqap_attention_scores(_ptr(qkv), ldq, batch, rows, query_row, visual_start, n_visual, n_heads, head_dim,
                                       q_col0, k_col0, _ptr(scores_out), _stream(stream)), "sqap_attention_scores")


def sqap_project_center(Kmat, Rt, xyz, patch_w: float, patch_h: float):
    k = (ctypes.c_double * 9)(*[float(v) for v in Kmat])
    r = (ctypes.c_double * 12)(*[float(v) for v in Rt])
    p = (ctypes.c_double * 3)(*[float(v) for v in xyz])
    out = (ctypes.c_int32 * 2)()
    front = ctypes.c_int()
    _check(lib().sqap_project_center(k, r, p, patch_w, patch_h, out, ctypes.byref(front)), "sqap_project_center")
    return (out[0], out[1]), bool(front.value)


def sqap_device_status(stream=None) -> int:
    return int(lib().sqap_device_status(_stream(stream)))


def sqap_selftest_bounded_wait(limit_clocks: int, stream=None):
    _check(lib().sqap_selftest_bounded_wait(limit_clocks, _stream(stream)), "sqap_selftest_bounded_wait")


def sqap_kernel_launch_count() -> int:
    return int(lib().sqap_kernel_launch_count())
