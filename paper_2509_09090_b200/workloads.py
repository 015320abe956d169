"""Seeded synthetic inputs shaped like the paper's workload (Llama-2-7B linears, 256 visual +
32 text tokens, a few fixed outlier channels far larger than the rest).

This module serves both the CPU oracle and the CUDA path and therefore holds none of the
method's arithmetic: no quantizer, no GEMM, no pruning rule. Every tensor is a pure function
of (seed, tensor id, element index) through a counter-based splitmix64 stream, so any slice
can be regenerated anywhere without state.
"""
from __future__ import annotations

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLD + np.uint64(0x1234567)], dtype=np.uint64))
        k = _mix(k + np.uint64(tensor_id) * _M2 + _GOLD)
    return k[0]


def raw_u64(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """count 64-bit words of stream (seed, tensor_id), beginning at element index start."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _mix(_key(seed, tensor_id) + (idx + np.uint64(1)) * _GOLD)


def uniform01(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """Doubles in (0, 1): top 53 bits, offset by half an ulp so 0 never occurs."""
    r = raw_u64(seed, tensor_id, start, count)
    return ((r >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, tensor_id: int, count: int) -> np.ndarray:
    """Standard normals (fp64) by Box-Muller from two sub-streams."""
    u1 = uniform01(seed, tensor_id * 2 + 1_000_003, count)
    u2 = uniform01(seed, tensor_id * 2 + 1_000_004, count)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def int4_codes(seed: int, tensor_id: int, count: int) -> np.ndarray:
    """Uniform integers in [-8, 7] as int8, 16 per 64-bit word."""
    nwords = (count + 15) // 16
    r = raw_u64(seed, tensor_id, 0, nwords)
    out = np.empty((nwords, 16), dtype=np.int8)
    for i in range(16):
        out[:, i] = ((r >> np.uint64(4 * i)) & np.uint64(15)).astype(np.int8)
    out -= 8
    return out.reshape(-1)[:count]


# ----------------------------------------------------------------------------- tensors

def activations(seed: int, tensor_id: int, M: int, K: int, n_outlier: int, outlier_scale: float) -> np.ndarray:
    """fp16 [M, K] ~ N(0,1) with n_outlier fixed channels (columns) multiplied by outlier_scale."""
    x = normal(seed, tensor_id, M * K).reshape(M, K)
    if n_outlier > 0:
        order = np.argsort(uniform01(seed, tensor_id * 2 + 2_000_003, K), kind="stable")
        x[:, order[:n_outlier]] *= outlier_scale
    return x.astype(np.float16)


def outlier_channels(seed: int, tensor_id: int, K: int, n_outlier: int) -> np.ndarray:
    order = np.argsort(uniform01(seed, tensor_id * 2 + 2_000_003, K), kind="stable")
    return np.sort(order[:n_outlier])


def weight_codes(seed: int, tensor_id: int, N: int, K: int) -> np.ndarray:
    return int4_codes(seed, tensor_id, N * K).reshape(N, K)


def weight_scales(seed: int, tensor_id: int, N: int, lo: float = 0.005, hi: float = 0.02,
                  mult: float = 1.0) -> np.ndarray:
    u = uniform01(seed, tensor_id * 2 + 3_000_003, N)
    return ((lo + (hi - lo) * u) * mult).astype(np.float16)


def scores_normal(seed: int, tensor_id: int, batch: int, n_visual: int) -> np.ndarray:
    """fp32 [batch, n_visual] ~ N(0,1): one score per visual token."""
    return normal(seed, tensor_id, batch * n_visual).reshape(batch, n_visual).astype(np.float32)


def scores_softmax_rows(seed: int, tensor_id: int, batch: int, R: int, n_visual: int) -> np.ndarray:
    """fp16 [batch, R, n_visual]: each row a softmax (fp32) over N(0,1) logits, rounded once to fp16."""
    z = normal(seed, tensor_id, batch * R * n_visual).reshape(batch, R, n_visual).astype(np.float32)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z, dtype=np.float32)
    return (e / e.sum(axis=-1, keepdims=True, dtype=np.float32)).astype(np.float16)


def ring_centers(seed: int, tensor_id: int, batch: int, grid_w: int, grid_h: int) -> np.ndarray:
    """int32 [batch, 2] token coordinates (t_u, t_v) of a stand-in end-effector, on the grid."""
    u = uniform01(seed, tensor_id * 2 + 4_000_003, batch * 2).reshape(batch, 2)
    c = np.empty((batch, 2), np.int32)
    c[:, 0] = np.minimum((u[:, 0] * grid_w).astype(np.int32), grid_w - 1)
    c[:, 1] = np.minimum((u[:, 1] * grid_h).astype(np.int32), grid_h - 1)
    return c


# ----------------------------------------------------------------------------- the five configurations

# Llama-2-7B geometry.
HIDDEN = 4096
FFN = 11008
QKV = 3 * HIDDEN
N_LAYERS = 32
ROWS = 288           # 1 leading text row + 256 visual + 31 text rows
N_VISUAL = 256
VISUAL_START = 1
GRID = 16

# tensor ids
T_X, T_W, T_S, T_SCORE, T_X2, T_CENTER = 1, 2, 3, 4, 5, 6


def prune_params(batch, rows, visual_start, n_visual, grid_w, grid_h, score_rows, k_attn, keep_total,
                 ring_radius=-1, flags=0) -> dict:
    return dict(batch=batch, rows=rows, visual_start=visual_start, n_visual=n_visual, grid_w=grid_w,
                grid_h=grid_h, score_rows=score_rows, k_attn=k_attn, keep_total=keep_total,
                ring_radius=ring_radius, flags=flags)


def config0(seed: int = 0) -> dict:
    """64 tokens x 512, 4 outlier channels x20; W 512x512; rows 0-47 visual (8 wide x 6 high), 48-63 text."""
    return dict(
        x=activations(seed, T_X, 64, 512, 4, 20.0),
        w_codes=weight_codes(seed, T_W, 512, 512),
        w_scales=weight_scales(seed, T_S, 512),
        scores=scores_normal(seed, T_SCORE, 1, 48),
        prune=prune_params(1, 64, 0, 48, 8, 6, 0, 24, 24),
    )


def config1(seed: int = 1) -> dict:
    """Attention projections of one layer at M = 288: fused QKV (N = 12288) and O (N = 4096)."""
    return dict(
        x=activations(seed, T_X, ROWS, HIDDEN, 41, 30.0),
        x_o=activations(seed, T_X2, ROWS, HIDDEN, 41, 30.0),
        wqkv_codes=weight_codes(seed, T_W, QKV, HIDDEN),
        wqkv_scales=weight_scales(seed, T_S, QKV),
        wo_codes=weight_codes(seed, T_W + 10, HIDDEN, HIDDEN),
        wo_scales=weight_scales(seed, T_S + 10, HIDDEN),
    )


def config2(seed: int = 2) -> dict:
    """MLP after pruning 288 -> 160 rows: gate/up (SwiGLU fused) and down."""
    return dict(
        x=activations(seed, T_X, ROWS, HIDDEN, 41, 30.0),
        scores=scores_softmax_rows(seed, T_SCORE, 1, 32, N_VISUAL),
        prune=prune_params(1, ROWS, VISUAL_START, N_VISUAL, GRID, GRID, 32, 128, 128),
        wg_codes=weight_codes(seed, T_W, FFN, HIDDEN),
        wg_scales=weight_scales(seed, T_S, FFN),
        wu_codes=weight_codes(seed, T_W + 10, FFN, HIDDEN),
        wu_scales=weight_scales(seed, T_S + 10, FFN),
        wd_codes=weight_codes(seed, T_W + 20, HIDDEN, FFN),
        wd_scales=weight_scales(seed, T_S + 20, HIDDEN),
    )


LAYER_LINEARS = (("qkv", QKV, HIDDEN), ("o", HIDDEN, HIDDEN), ("gate", FFN, HIDDEN), ("up", FFN, HIDDEN),
                 ("down", HIDDEN, FFN))


def config3_layer(layer: int, seed: int = 3) -> dict:
    """Codes and scales of the five linears of one layer of the 32-layer stack. Scales carry a
    16/sqrt(K) factor so that a chain of linears keeps fp16 activations finite."""
    out = {}
    for i, (name, N, K) in enumerate(LAYER_LINEARS):
        tid = 100 + layer * 10 + i
        out[name + "_codes"] = weight_codes(seed, tid, N, K)
        out[name + "_scales"] = weight_scales(seed, tid, N, mult=16.0 / np.sqrt(K))
    return out


def config3_inputs(seed: int = 3) -> dict:
    return dict(
        x=activations(seed, T_X, ROWS, HIDDEN, 41, 30.0),
        x_decode=activations(seed, T_X2, 7, HIDDEN, 41, 30.0),
        scores=scores_softmax_rows(seed, T_SCORE, 1, 32, N_VISUAL),
        prune=prune_params(1, ROWS, VISUAL_START, N_VISUAL, GRID, GRID, 32, 128, 128),
    )


def config4_inputs(seed: int = 4, batch: int = 16) -> dict:
    """16 observations x 288 rows; every observation has its own stream; shared outlier channels."""
    xs = []
    for b in range(batch):
        xb = normal(seed, 1000 + b, ROWS * HIDDEN).reshape(ROWS, HIDDEN)
        xs.append(xb)
    x = np.stack(xs)
    ch = outlier_channels(seed, T_X, HIDDEN, 41)
    x[:, :, ch] *= 30.0
    return dict(
        x=x.astype(np.float16),
        scores=scores_softmax_rows(seed, T_SCORE, batch, 32, N_VISUAL),
        centers=ring_centers(seed, T_CENTER, batch, GRID, GRID),
    )


def config4_weights(seed: int = 4) -> dict:
    out = {}
    for i, (name, N, K) in enumerate(LAYER_LINEARS):
        out[name + "_codes"] = weight_codes(seed, 200 + i, N, K)
        out[name + "_scales"] = weight_scales(seed, 200 + i, N, mult=16.0 / np.sqrt(K))
    return out
