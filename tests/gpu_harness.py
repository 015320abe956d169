"""Helpers for the GPU parity tests: move numpy inputs to the device, call the C ABI through the
binding, bring results back as numpy. No arithmetic of the method happens here."""
from __future__ import annotations

import numpy as np
import torch

from paper_2509_09090_b200 import binding as B

DEV = "cuda:0"


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def pack(codes: np.ndarray, scales_f16: np.ndarray, flags: int = 0, on_device: bool = False) -> B.Weights:
    N, K = codes.shape
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    scales = np.ascontiguousarray(scales_f16, dtype=np.float16)
    if on_device:
        c, s = to_dev(codes), to_dev(scales)
        w = B.sqap_pack_weights(c, s, N, K, flags)
        torch.cuda.synchronize()
        return w
    return B.sqap_pack_weights(codes, scales, N, K, flags)


def quantize(x_f16: np.ndarray, rotate: bool = False, row_index=None, K=None, col_offset: int = 0):
    """x_f16: fp16 [rows, ld]. Quantizes columns [col_offset, col_offset + K). Returns (packed, scales)."""
    xd = to_dev(np.ascontiguousarray(x_f16, dtype=np.float16))
    rows, ld = x_f16.shape
    if K is None:
        K = ld - col_offset
    ri = to_dev(np.asarray(row_index, np.int32)) if row_index is not None else None
    M = len(row_index) if row_index is not None else rows
    q = torch.full((max(M, 1), K // 2), 0x5A, dtype=torch.uint8, device=DEV)
    s = torch.full((max(M, 1),), -1.0, dtype=torch.float32, device=DEV)
    xp = xd.data_ptr() + 2 * col_offset
    B.sqap_quantize_act(xp, M, K, ld, ri, B.SQAP_Q_ROTATE if rotate else 0, q, s)
    torch.cuda.synchronize()
    return q.cpu().numpy()[:M], s.cpu().numpy()[:M]


def linear(packed: np.ndarray, scales: np.ndarray, w: B.Weights, w_up=None, out_dtype=B.SQAP_FP16, flags=0,
           ldo=None, canary: bool = True):
    """Returns the [M, N] output as numpy: uint16 bit patterns for fp16/bf16, int32 for SQAP_I32."""
    M = packed.shape[0]
    N = w.N
    ldo = ldo or (N + 7) // 8 * 8          # row pitch must be a multiple of 16 bytes
    qd, sd = to_dev(packed), to_dev(scales)
    tdt = torch.int32 if out_dtype == B.SQAP_I32 else torch.int16
    fill = 0x7B7B7B7B if out_dtype == B.SQAP_I32 else 0x7B7B
    out = torch.full((M + 1, ldo), fill, dtype=tdt, device=DEV)      # one canary row past the end
    nbytes = B.sqap_workspace_bytes(M, N, w.K, flags)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=DEV)
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    B.sqap_w4a4_linear(qd, sd, M, w, w_up, out, ldo, out_dtype, flags, ws_ptr, nbytes)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    o = out.cpu().numpy()
    if canary:
        assert (o[M] == (fill if out_dtype == B.SQAP_I32 else np.int16(fill))).all(), "wrote past the last row"
        if ldo > N:
            assert (o[:M, N:] == o[M, 0]).all(), "wrote past the row end"
    o = o[:M, :N]
    return o if out_dtype == B.SQAP_I32 else o.view(np.uint16)


def quantize_linear(x_f16: np.ndarray, w: B.Weights, w_up=None, rotate: bool = False, row_index=None,
                    out_dtype=B.SQAP_FP16, flags=0, col_offset: int = 0):
    """The fused call on the columns [col_offset, col_offset + K) of x_f16; output as in linear()."""
    xd = to_dev(np.ascontiguousarray(x_f16, dtype=np.float16))
    rows, ld = x_f16.shape
    ri = to_dev(np.asarray(row_index, np.int32)) if row_index is not None else None
    M = len(row_index) if row_index is not None else rows
    N = w.N
    ldo = (N + 7) // 8 * 8
    tdt = torch.int32 if out_dtype == B.SQAP_I32 else torch.int16
    fill = 0x7B7B7B7B if out_dtype == B.SQAP_I32 else 0x7B7B
    out = torch.full((M + 1, ldo), fill, dtype=tdt, device=DEV)
    nbytes = B.sqap_quantize_linear_workspace_bytes(M, N, w.K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=DEV)
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    B.sqap_quantize_linear(xd.data_ptr() + 2 * col_offset, M, ld, ri, B.SQAP_Q_ROTATE if rotate else 0, w, w_up, out,
                           ldo, out_dtype, flags, ws_ptr, nbytes)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    o = out.cpu().numpy()
    assert (o[M] == (fill if out_dtype == B.SQAP_I32 else np.int16(fill))).all(), "wrote past the last row"
    if ldo > N:
        assert (o[:M, N:] == o[M, 0]).all(), "wrote past the row end"
    o = o[:M, :N]
    return o if out_dtype == B.SQAP_I32 else o.view(np.uint16)


def prune(params: dict, scores: np.ndarray, centers=None, x_f16=None, out_rows: int = 0, K=None):
    """Returns (kept_idx [B, rows], n_kept [B], x_out [B, out_rows, K] bits or None)."""
    Bn, rows = params["batch"], params["rows"]
    sd = to_dev(np.ascontiguousarray(scores)) if scores is not None else None
    cd = to_dev(np.asarray(centers, np.int32)) if centers is not None else None
    kept = torch.full((max(Bn, 1), max(rows, 1)), -7, dtype=torch.int32, device=DEV)
    nk = torch.full((max(Bn, 1),), -7, dtype=torch.int32, device=DEV)
    xo = None
    if x_f16 is not None:
        xd = to_dev(np.ascontiguousarray(x_f16, dtype=np.float16))
        ld = x_f16.shape[-1]
        K = K or ld
        xo = torch.full((Bn * out_rows + 1, K), 0x7B7B, dtype=torch.int16, device=DEV)
        B.sqap_prune_tokens(params, sd, cd, xd, ld, K, xo, K, out_rows, kept, nk)
    else:
        B.sqap_prune_tokens(params, sd, cd, None, 0, 0, None, 0, 0, kept, nk)
    torch.cuda.synchronize()
    xo_np = None
    if xo is not None:
        o = xo.cpu().numpy()
        assert (o[Bn * out_rows] == 0x7B7B).all()
        xo_np = o[:Bn * out_rows].reshape(Bn, out_rows, K).view(np.uint16)
    return kept.cpu().numpy()[:Bn, :rows], nk.cpu().numpy()[:Bn], xo_np


def within_tolerance(got_bits: np.ndarray, ref_bits: np.ndarray, bf16: bool = False):
    """|got - ref| <= max(1 ulp of the 16-bit type at ref, 2e-3 * |ref|), elementwise."""
    if bf16:
        g = (got_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        r = (ref_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        # one unit in the last place of bf16 (8 significant bits) at ref: 2^(floor(log2 |ref|) - 7)
        ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(r), 2.0 ** -126))) - 7.0)
    else:
        g = got_bits.view(np.float16).astype(np.float64)
        r = ref_bits.view(np.float16).astype(np.float64)
        ulp = np.spacing(np.abs(ref_bits.view(np.float16))).astype(np.float64)
    assert np.isfinite(r).all(), "oracle output overflowed: workload error"
    return np.abs(g - r) <= np.maximum(ulp, 2e-3 * np.abs(r))
