"""CPU oracle of the SQAP-VLA hot path: numpy-facing wrappers around ``sqap_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the bench's
cpu_baseline / reference arm. The CUDA library never imports it and it never imports the
CUDA library. All arithmetic lives in the C file; this module only marshals numpy arrays.

Parity with the authors' implementation is unpinned for the quantizer conventions, the
Hadamard stage order and the pruning hyper-parameters / tie rules (the paper prints none);
everything else is pinned by the CPU tests.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sqap_oracle.c")
_LIB = os.path.join(_HERE, "libsqap_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FMA contraction, OpenMP over independent rows)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-o", _LIB + ".tmp", _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


class PruneParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("batch", "rows", "visual_start", "n_visual", "grid_w", "grid_h",
                                            "score_rows", "k_attn", "keep_total", "ring_radius")] + \
               [("flags", ctypes.c_uint32)]


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_hadamard_norm.restype = ctypes.c_float
        _lib.oracle_dot_i32.restype = ctypes.c_int32
        _lib.oracle_exp2_neg.restype = ctypes.c_float
        _lib.oracle_exp2_neg.argtypes = [ctypes.c_float]
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def half_to_float(h_bits):
    h = _c(h_bits, np.uint16)
    out = np.empty(h.shape, np.float32)
    lib().oracle_half_to_float(_p(h), ctypes.c_int64(h.size), _p(out))
    return out


def float_to_half(f):
    f = _c(f, np.float32)
    out = np.empty(f.shape, np.uint16)
    lib().oracle_float_to_half(_p(f), ctypes.c_int64(f.size), _p(out))
    return out


def float_to_bf16(f):
    f = _c(f, np.float32)
    out = np.empty(f.shape, np.uint16)
    lib().oracle_float_to_bf16(_p(f), ctypes.c_int64(f.size), _p(out))
    return out


def fwht_f32(v):
    v = np.array(v, dtype=np.float32, copy=True)
    lib().oracle_fwht_f32(_p(v), ctypes.c_int(v.size))
    return v


def fwht_f64(v):
    v = np.array(v, dtype=np.float64, copy=True)
    lib().oracle_fwht_f64(_p(v), ctypes.c_int(v.size))
    return v


def hadamard_norm(K: int) -> np.float32:
    return np.float32(lib().oracle_hadamard_norm(ctypes.c_int(K)))


def rotate_rows(x_bits, rotate=True):
    x = _c(x_bits, np.uint16)
    M, K = x.shape
    out = np.empty((M, K), np.float32)
    lib().oracle_rotate_rows(_p(x), M, K, ctypes.c_int64(K), int(rotate), _p(out))
    return out


def exp2_neg(t: float) -> np.float32:
    return np.float32(lib().oracle_exp2_neg(ctypes.c_float(float(t))))


def attention_scores(qkv_bits, batch, rows, query_row, visual_start, n_visual, n_heads, head_dim, q_col0, k_col0):
    """qkv_bits: uint16 view of fp16 [batch*rows, ldq]. Returns fp16 bits u16 [batch, n_heads, n_visual]."""
    x = _c(qkv_bits, np.uint16)
    out = np.empty((batch, n_heads, n_visual), np.uint16)
    rc = lib().oracle_attention_scores(_p(x), ctypes.c_int64(x.shape[1]), batch, rows, query_row, visual_start, n_visual,
                                       n_heads, head_dim, q_col0, k_col0, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_attention_scores: {rc}")
    return out


def quantize_weights(w_bits, rotate=False, ch_mul=None):
    """w_bits: uint16 view of fp16 [N, K]; ch_mul: fp32 [K] or None. Returns (codes i8 [N,K], scales fp16 bits u16 [N])."""
    w = _c(w_bits, np.uint16)
    N, K = w.shape
    codes = np.empty((N, K), np.int8)
    scales = np.empty((N,), np.uint16)
    cm = _c(ch_mul, np.float32) if ch_mul is not None else None
    rc = lib().oracle_quantize_weights(_p(w), N, K, ctypes.c_int64(K), int(rotate), _p(cm), _p(codes), _p(scales))
    if rc != 0:
        raise ValueError(f"oracle_quantize_weights: {rc}")
    return codes, scales


def quantize_act(x_bits, rotate=False, row_index=None, ldx=None, K=None, per_tensor=False, ch_mul=None):
    """x_bits: uint16 view of fp16 [rows, ldx]. Returns (packed u8 [M,K/2], scales f32 [M], codes i8 [M,K]).
    per_tensor: one scale over all rows; ch_mul: fp32 [K] channel multiplier applied first."""
    x = _c(x_bits, np.uint16)
    if ldx is None:
        ldx = x.shape[1]
    if K is None:
        K = x.shape[1]
    if row_index is not None:
        row_index = _c(row_index, np.int32)
        M = row_index.size
    else:
        M = x.shape[0]
    packed = np.empty((M, K // 2), np.uint8)
    scales = np.empty((M,), np.float32)
    codes = np.empty((M, K), np.int8)
    cm = _c(ch_mul, np.float32) if ch_mul is not None else None
    if per_tensor or cm is not None:
        rc = lib().oracle_quantize_act_ex(_p(x), M, K, ctypes.c_int64(ldx), _p(row_index), int(rotate), int(per_tensor),
                                          _p(cm), _p(packed), _p(scales), _p(codes))
    else:
        rc = lib().oracle_quantize_act(_p(x), M, K, ctypes.c_int64(ldx), _p(row_index), int(rotate), _p(packed),
                                       _p(scales), _p(codes))
    if rc != 0:
        raise ValueError(f"oracle_quantize_act: bad arguments ({rc})")
    return packed, scales, codes


def unpack_nibbles(packed):
    p = _c(packed, np.uint8)
    codes = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), np.int8)
    lib().oracle_unpack_nibbles(_p(p), ctypes.c_int64(codes.size), _p(codes))
    return codes


def pack_nibbles(codes):
    c = _c(codes, np.int8)
    packed = np.empty(c.shape[:-1] + (c.shape[-1] // 2,), np.uint8)
    lib().oracle_pack_nibbles(_p(c), ctypes.c_int64(c.size), _p(packed))
    return packed


def check_weights(codes, scales_bits) -> int:
    c = _c(codes, np.int8)
    s = _c(scales_bits, np.uint16)
    return int(lib().oracle_check_weights(_p(c), _p(s), c.shape[0], c.shape[1]))


def gemm_i32(qx, qw):
    qx = _c(qx, np.int8)
    qw = _c(qw, np.int8)
    M, K = qx.shape
    N, K2 = qw.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    lib().oracle_gemm_i32(_p(qx), _p(qw), M, N, K, _p(acc))
    return acc


def dot_i32(a, b) -> int:
    a = _c(a, np.int8)
    b = _c(b, np.int8)
    assert a.size == b.size
    return int(lib().oracle_dot_i32(_p(a), _p(b), a.size))


def epilogue(acc, sx, sw_bits, bf16=False):
    acc = _c(acc, np.int32)
    sx = _c(sx, np.float32)
    sw = _c(sw_bits, np.uint16)
    M, N = acc.shape
    out = np.empty((M, N), np.uint16)
    lib().oracle_epilogue(_p(acc), _p(sx), _p(sw), M, N, int(bf16), _p(out))
    return out


def epilogue_swiglu(acc_g, acc_u, sx, swg_bits, swu_bits, bf16=False):
    acc_g = _c(acc_g, np.int32)
    acc_u = _c(acc_u, np.int32)
    sx = _c(sx, np.float32)
    M, N = acc_g.shape
    out = np.empty((M, N), np.uint16)
    lib().oracle_epilogue_swiglu(_p(acc_g), _p(acc_u), _p(sx), _p(_c(swg_bits, np.uint16)),
                                 _p(_c(swu_bits, np.uint16)), M, N, int(bf16), _p(out))
    return out


def project_center(Kmat, Rt, xyz, patch_w, patch_h):
    Kmat = _c(Kmat, np.float64).reshape(9)
    Rt = _c(Rt, np.float64).reshape(12)
    xyz = _c(xyz, np.float64).reshape(3)
    out = np.zeros(2, np.int32)
    front = ctypes.c_int(0)
    lib().oracle_project_center(_p(Kmat), _p(Rt), _p(xyz), ctypes.c_double(patch_w), ctypes.c_double(patch_h),
                                _p(out), ctypes.byref(front))
    return (int(out[0]), int(out[1])), bool(front.value)


def score_sum(A_bits):
    A = _c(A_bits, np.uint16)
    R, nv = A.shape
    a = np.empty(nv, np.float32)
    lib().oracle_score_sum(_p(A), R, nv, _p(a))
    return a


def topk_mask(a, k):
    a = _c(a, np.float32)
    mask = np.zeros(a.size, np.uint8)
    lib().oracle_topk_mask(_p(a), a.size, int(k), _p(mask))
    return mask.astype(bool)


def ring_mask(grid_w, grid_h, c_u, c_v, radius):
    mask = np.zeros(grid_w * grid_h, np.uint8)
    lib().oracle_ring_mask(grid_w, grid_h, int(c_u), int(c_v), int(radius), _p(mask))
    return mask.astype(bool)


def fps_mask(grid_w, grid_h, remain, m):
    remain = _c(remain, np.uint8)
    picked = np.zeros(grid_w * grid_h, np.uint8)
    lib().oracle_fps_mask(grid_w, grid_h, _p(remain), int(m), _p(picked))
    return picked.astype(bool)


def prune_tokens(params: dict, scores, ring_center=None, want_masks=False):
    """params: dict with the PruneParams fields. scores: uint16 (fp16 bits) [B,R,nv] or float32 [B,nv]."""
    p = PruneParams(**{k: int(v) for k, v in params.items()})
    if p.score_rows > 0:
        scores = _c(scores, np.uint16)
    else:
        scores = _c(scores, np.float32)
    rc_arr = _c(ring_center, np.int32) if ring_center is not None else None
    kept = np.empty((p.batch, p.rows), np.int32)
    n_kept = np.empty((p.batch,), np.int32)
    masks = np.zeros((p.batch, 3, p.n_visual), np.uint8) if want_masks else None
    rc = lib().oracle_prune_tokens(ctypes.byref(p), _p(scores), _p(rc_arr), _p(kept), _p(n_kept), _p(masks))
    if rc != 0:
        raise ValueError("oracle_prune_tokens: bad arguments")
    if want_masks:
        return kept, n_kept, masks.astype(bool)
    return kept, n_kept


def gather_rows(x_bits, kept_idx, n_kept, out_rows, K=None):
    """x_bits: uint16 [B, rows, ldx]; returns uint16 [B, out_rows, K] (rows past n_kept are zero)."""
    x = _c(x_bits, np.uint16)
    B, rows, ldx = x.shape
    if K is None:
        K = ldx
    kept_idx = _c(kept_idx, np.int32)
    n_kept = _c(n_kept, np.int32)
    out = np.zeros((B, out_rows, K), np.uint16)
    lib().oracle_gather_rows(_p(x), B, rows, K, ctypes.c_int64(ldx), _p(kept_idx), _p(n_kept), int(out_rows),
                             ctypes.c_int64(K), _p(out))
    return out
