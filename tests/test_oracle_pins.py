"""Pins for the CPU oracle: each oracle function is checked against something other than
itself — a closed form, an invariant, brute force on tiny inputs, exact rational arithmetic,
or a library routine that the case reduces to. No GPU is needed.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.linalg
import scipy.special

import oracle
from paper_2509_09090_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f16(a):
    return np.asarray(a, dtype=np.float16)


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float16).view(np.uint16)


# ------------------------------------------------------------------ fp16 / bf16 conversions

def test_half_conversion_exhaustive_against_numpy():
    allbits = np.arange(65536, dtype=np.uint16)
    f = oracle.half_to_float(allbits)
    ref = allbits.view(np.float16).astype(np.float32)
    finite = np.isfinite(ref)
    assert np.array_equal(f[finite], ref[finite])
    assert np.array_equal(np.isnan(f), np.isnan(ref))
    # round trip and RNE on the fp32 side: midpoints between adjacent halves, and random floats
    back = oracle.float_to_half(ref[finite])
    assert np.array_equal(back, allbits[finite])
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(200000).astype(np.float32) * s for s in (1e-7, 1e-4, 1.0, 300.0, 7e4)])
    with np.errstate(over="ignore"):
        assert np.array_equal(oracle.float_to_half(x), x.astype(np.float16).view(np.uint16))
    pos = allbits[(allbits < 0x7BFF)].astype(np.uint16)
    lo = pos.view(np.float16).astype(np.float64)
    hi = (pos + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)  # exactly representable in fp32
    assert np.array_equal(oracle.float_to_half(mid), mid.astype(np.float16).view(np.uint16))


def test_bf16_conversion_against_truncation_rule():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(100000).astype(np.float32) * np.float32(37.0)
    got = oracle.float_to_bf16(x).astype(np.uint32) << 16
    val = got.view(np.float32).astype(np.float64)
    xb = x.view(np.uint32)
    lo = (xb & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    hi = ((xb & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    xd = x.astype(np.float64)
    # nearest of the two neighbours; ties to the one with an even last kept bit
    dlo, dhi = np.abs(xd - lo), np.abs(xd - hi)
    expect = np.where(dlo < dhi, lo, hi)
    tie = dlo == dhi
    even_lo = ((xb >> 16) & 1) == 0
    expect = np.where(tie, np.where(even_lo, lo, hi), expect)
    assert np.array_equal(val, expect)


# ------------------------------------------------------------------ Hadamard rotation (Eq. 6)

@pytest.mark.parametrize("K", [2, 8, 64, 512])
def test_fwht_equals_dense_sylvester_matrix(K):
    H = scipy.linalg.hadamard(K).astype(np.float64)
    rng = np.random.default_rng(K)
    v = rng.standard_normal(K)
    assert np.allclose(oracle.fwht_f64(v), H @ v, rtol=1e-12, atol=1e-12)
    v32 = v.astype(np.float32)
    assert np.allclose(oracle.fwht_f32(v32), H @ v32.astype(np.float64), rtol=1e-5, atol=1e-4)
    # small integers: every partial sum is exact in fp32, so the fp32 transform must be exact
    vi = rng.integers(-8, 8, K).astype(np.float32)
    assert np.array_equal(oracle.fwht_f32(vi), (H @ vi.astype(np.float64)).astype(np.float32))


def test_fwht_delta_gives_matrix_column_and_involution():
    K = 64
    H = scipy.linalg.hadamard(K)
    for i in (0, 1, 5, 63):
        e = np.zeros(K, np.float32)
        e[i] = 1.0
        assert np.array_equal(oracle.fwht_f32(e), H[:, i].astype(np.float32))
    rng = np.random.default_rng(3)
    v = rng.standard_normal(K)
    assert np.allclose(oracle.fwht_f64(oracle.fwht_f64(v)) / K, v, rtol=1e-12)


def test_hadamard_norm_values():
    assert oracle.hadamard_norm(4096) == np.float32(2.0 ** -6)
    assert oracle.hadamard_norm(512) == np.float32(1.0 / math.sqrt(512.0))
    assert oracle.hadamard_norm(512).view(np.uint32) == np.float32(float.fromhex("0x1.6a09e6p-5")).view(np.uint32)


def test_rotation_preserves_norm_and_inner_products_eq6():
    # (W^T H^T)(H X) = W^T X for orthonormal H: check in fp64 on rotated rows
    K = 512
    rng = np.random.default_rng(4)
    w = rng.standard_normal((5, K))
    x = rng.standard_normal((7, K))
    c = 1.0 / math.sqrt(K)
    wr = np.stack([oracle.fwht_f64(r) * c for r in w])
    xr = np.stack([oracle.fwht_f64(r) * c for r in x])
    assert np.allclose(wr @ xr.T, w @ x.T, rtol=1e-11, atol=1e-11)
    assert np.allclose(np.linalg.norm(xr, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    # the fp32 rows the quantizer sees agree with the fp64 rotation
    xh = f16(x)
    got = oracle.rotate_rows(bits(xh), rotate=True)
    ref = np.stack([oracle.fwht_f64(r.astype(np.float64)) * c for r in xh])
    assert np.allclose(got, ref, rtol=1e-5, atol=1e-5)


def test_rotation_spreads_outlier_energy():
    # the effect the paper attributes to H: outlier channels stop dominating the row maximum
    c1x = wl.activations(1, wl.T_X, 8, 4096, 41, 30.0)
    plain = oracle.rotate_rows(bits(c1x), rotate=False)
    rot = oracle.rotate_rows(bits(c1x), rotate=True)
    crest = lambda v: np.abs(v).max(axis=1) / np.sqrt((v.astype(np.float64) ** 2).mean(axis=1))
    assert (crest(rot) < 0.6 * crest(plain)).all()
    _, _, cp = oracle.quantize_act(bits(c1x), rotate=False)
    _, _, cr = oracle.quantize_act(bits(c1x), rotate=True)
    assert (cr != 0).sum() > 2 * (cp != 0).sum()


# ------------------------------------------------------------------ activation quantizer

def _exact_codes(v_row):
    """Nearest-even of v*7/amax in exact rational arithmetic; None where the real value is
    so close to a half-integer that fp32 rounding of inv and of the product may decide."""
    fr = [Fraction(float(t)) for t in v_row]
    amax = max(abs(t) for t in fr)
    out = []
    for t in fr:
        if amax == 0:
            out.append(0)
            continue
        r = t * 7 / amax
        fl = math.floor(r)
        frac = r - fl
        if abs(frac - Fraction(1, 2)) < Fraction(1, 2 ** 19):
            out.append(None)
            continue
        out.append(fl + (1 if frac > Fraction(1, 2) else 0))
    return out


@pytest.mark.parametrize("rotate", [False, True])
def test_quantizer_error_bound_codes_and_exact_rounding(rotate):
    c0 = wl.config0()
    x = c0["x"]
    packed, s, codes = oracle.quantize_act(bits(x), rotate=rotate)
    v = oracle.rotate_rows(bits(x), rotate=rotate).astype(np.float64)
    assert codes.min() >= -7 and codes.max() <= 7            # -8 only via the clamp, never reached
    err = np.abs(v - s[:, None].astype(np.float64) * codes)
    assert (err <= s[:, None] / 2 * (1 + 2.0 ** -20)).all()  # dequantised error <= scale/2
    amax = np.abs(v).max(axis=1)
    assert np.array_equal(s, (amax.astype(np.float32) / np.float32(7.0)))
    am = np.abs(v).argmax(axis=1)
    assert (np.abs(codes[np.arange(len(am)), am]) == 7).all()
    undecided = 0
    for m in range(0, 64, 7):
        ex = _exact_codes(v[m])
        for k, e in enumerate(ex):
            if e is None:
                undecided += 1
            else:
                assert codes[m, k] == e, (m, k)
    assert undecided < 10
    assert np.array_equal(oracle.unpack_nibbles(packed), codes)


def test_quantizer_ties_round_to_even_and_zero_row():
    # amax = 7 -> inv = 1 exactly, so halves are exact ties
    row = np.array([7, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, -3.5, 6.5, -6.5, 0, 0.25, -0.75, 4.5, 5.5], np.float16)
    x = np.stack([row, np.zeros(16, np.float16)])
    packed, s, codes = oracle.quantize_act(bits(x))
    assert codes[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 4, -4, 6, -6, 0, 0, -1, 4, 6]
    assert s[0] == np.float32(1.0)
    assert s[1] == np.float32(1.0) and not codes[1].any()
    # nibble layout: even index low, two's complement
    assert packed[0, 0] == ((7 & 0xF) | (0 << 4))
    assert packed[0, 2] == ((0 & 0xF) | ((-2 & 0xF) << 4))


def test_quantizer_power_of_two_scaling_invariance():
    x = wl.activations(7, 1, 16, 256, 3, 20.0)
    p1, s1, c1 = oracle.quantize_act(bits(x))
    p2, s2, c2 = oracle.quantize_act(bits((x.astype(np.float32) * 8).astype(np.float16)))
    assert np.array_equal(c1, c2)
    assert np.array_equal(s2, s1 * np.float32(8))


def test_quantizer_row_index_and_stride():
    x = wl.activations(8, 1, 10, 128, 2, 20.0)
    idx = np.array([9, 0, 3, 3], np.int32)
    p, s, c = oracle.quantize_act(bits(x), row_index=idx)
    p2, s2, c2 = oracle.quantize_act(bits(x[idx]))
    assert np.array_equal(p, p2) and np.array_equal(s, s2)
    # strided view: only the last 64 columns, row stride 128
    xs = np.ascontiguousarray(x[:, 64:])
    p3, s3, _ = oracle.quantize_act(bits(xs))
    flat = bits(x).reshape(-1)[64:]
    flat = np.concatenate([flat, np.zeros(64, np.uint16)]).reshape(10, 128)
    p4, s4, _ = oracle.quantize_act(flat, ldx=128, K=64)
    assert np.array_equal(p3, p4) and np.array_equal(s3, s4)


def test_per_tensor_and_channel_multiplier_granularities():
    """Per-tensor: every row carries numpy's global amax / 7, the error bound holds with that one scale, and a
    one-row tensor gives the per-token result. Channel multiplier: with powers of two it equals quantizing the
    pre-multiplied fp16 tensor (the products are exact), all ones changes nothing, and dividing the outlier
    channels down before quantizing (the factor moved into the weights) lowers the error of the W4A4 product."""
    x = wl.activations(51, 3, 12, 256, 4, 30.0)
    for rot in (False, True):
        packed, s, codes = oracle.quantize_act(bits(x), rotate=rot, per_tensor=True)
        v = oracle.rotate_rows(bits(x), rotate=rot)
        g = np.abs(v).max()
        assert (s == np.float32(g) / np.float32(7.0)).all()
        assert (np.abs(v.astype(np.float64) - s[:, None].astype(np.float64) * codes) <= s[0] / 2 * (1 + 2.0 ** -20)).all()
        assert np.array_equal(oracle.unpack_nibbles(packed), codes)
        p1, s1, c1 = oracle.quantize_act(bits(x[3:4]), rotate=rot, per_tensor=True)
        p0, s0, c0 = oracle.quantize_act(bits(x[3:4]), rotate=rot)
        assert np.array_equal(c1, c0) and np.array_equal(s1, s0)
    m = np.exp2(np.arange(256) % 5 - 2).astype(np.float32)                       # 1/4 .. 4
    pre = (x.astype(np.float32) * m).astype(np.float16)
    assert np.array_equal(pre.astype(np.float32), x.astype(np.float32) * m)      # exact in fp16
    for rot in (False, True):
        a = oracle.quantize_act(bits(x), rotate=rot, ch_mul=m)
        b = oracle.quantize_act(bits(pre), rotate=rot)
        assert np.array_equal(a[2], b[2]) and np.array_equal(a[1], b[1])
        c = oracle.quantize_act(bits(x), rotate=rot, ch_mul=np.ones(256, np.float32))
        d = oracle.quantize_act(bits(x), rotate=rot)
        assert np.array_equal(c[0], d[0]) and np.array_equal(c[1], d[1])
    # smoothing: divide each channel by its typical magnitude, multiply the weights' columns by it
    N, K, M = 32, 256, 12
    w = _fp16_weights(52, N, K)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    d = np.maximum(np.abs(x.astype(np.float32)).max(axis=0), np.float32(1e-3))
    d = np.exp2(np.round(0.5 * np.log2(d))).astype(np.float32)                   # half the outlier scale moves into the
                                                                                 # weights; powers of two: 1/d exact
    errs = []
    for mul_x, mul_w in ((None, None), (1.0 / d, d)):
        wc, ws = oracle.quantize_weights(bits(w), ch_mul=mul_w)
        _, sx, xc = oracle.quantize_act(bits(x), ch_mul=None if mul_x is None else mul_x.astype(np.float32))
        y = oracle.gemm_i32(xc, wc).astype(np.float64) * sx[:, None] * ws.view(np.float16).astype(np.float64)[None, :]
        errs.append(np.sqrt(np.mean((y - ref) ** 2)) / np.sqrt(np.mean(ref ** 2)))
    assert errs[1] < 0.7 * errs[0], errs


# ------------------------------------------------------------------ offline weight quantizer

def _fp16_weights(seed, N, K, outlier_cols=0):
    w = (wl.activations(seed, 9, N, K, outlier_cols, 25.0).astype(np.float32) * np.float32(0.02)).astype(np.float16)
    return w


@pytest.mark.parametrize("rotate", [False, True])
def test_weight_quantizer_scale_error_bound_and_exact_rounding(rotate):
    """Per-channel RTN: the scale is numpy's own fp16 rounding of amax/7, every code is the nearest integer of
    v / scale (exact rational arithmetic away from ties), and the dequantised error is at most half a scale."""
    N, K = 24, 256
    w = _fp16_weights(31, N, K, outlier_cols=3)
    w[5] = 0
    codes, s_bits = oracle.quantize_weights(bits(w), rotate=rotate)
    v = oracle.rotate_rows(bits(w), rotate=rotate)                      # the fp32 rows the quantizer sees
    amax = np.abs(v).max(axis=1)
    s_np = (amax / np.float32(7.0)).astype(np.float16)                  # independent fp16 rounding
    s_np[amax == 0] = np.float16(1.0)
    assert np.array_equal(s_bits.view(np.float16), s_np)
    sf = s_bits.view(np.float16).astype(np.float64)
    assert codes.min() >= -7 and codes.max() <= 7                       # fp16 rounding moves v/s by < 2^-10: no clamp
    err = np.abs(v.astype(np.float64) - sf[:, None] * codes)
    assert (err <= sf[:, None] / 2 * (1 + 2.0 ** -20)).all()
    assert not codes[5].any()
    undecided = 0
    for n in range(0, N, 5):
        if amax[n] == 0:
            continue
        sfr = Fraction(float(sf[n]))
        for k in range(K):
            r = Fraction(float(v[n, k])) / sfr
            fl = math.floor(r)
            frac = r - fl
            if abs(frac - Fraction(1, 2)) < Fraction(1, 2 ** 19):
                undecided += 1
                continue
            assert codes[n, k] == fl + (1 if frac > Fraction(1, 2) else 0), (n, k)
    assert undecided < 10


def test_weight_quantizer_ties_scaling_and_tiny_rows():
    row = np.array([7, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, -3.5, 6.5, -6.5, 0, 0.25, -0.75, 4.5, 5.5], np.float16)
    codes, s = oracle.quantize_weights(bits(np.stack([row, row * np.float16(4)])))
    assert codes[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 4, -4, 6, -6, 0, 0, -1, 4, 6]    # scale exactly 1: ties to even
    assert s.view(np.float16).tolist() == [1.0, 4.0] and np.array_equal(codes[0], codes[1])  # power-of-two invariance
    tiny = np.zeros((1, 32), np.float16)
    tiny[0, 3] = np.float16(2.0 ** -24)                                  # amax/7 underflows fp16: smallest scale used
    codes, s = oracle.quantize_weights(bits(tiny))
    assert s[0] == 1 and codes[0, 3] == 1 and np.count_nonzero(codes) == 1


def test_eq6_rotated_w4a4_product_approximates_the_fp_product():
    """Eq. 6 end to end on the oracle: quantizing W H^T and H x and multiplying the codes approximates W x, the
    rotation changes nothing in exact arithmetic (checked in fp64 on the unquantized rows), and with outlier
    channels the rotated product is the more accurate one (the reason the paper rotates)."""
    N, K, M = 32, 512, 16
    w = _fp16_weights(33, N, K)
    x = wl.activations(34, 2, M, K, 6, 30.0)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    # exactness of the rotation itself
    hw = oracle.rotate_rows(bits(w), rotate=True).astype(np.float64)
    hx = oracle.rotate_rows(bits(x), rotate=True).astype(np.float64)
    assert np.allclose(hx @ hw.T, ref, rtol=0, atol=1e-3 * np.abs(ref).max())
    errs = {}
    for rot in (False, True):
        wc, ws = oracle.quantize_weights(bits(w), rotate=rot)
        _, sx, xc = oracle.quantize_act(bits(x), rotate=rot)
        acc = oracle.gemm_i32(xc, wc).astype(np.float64)
        y = acc * sx[:, None].astype(np.float64) * ws.view(np.float16).astype(np.float64)[None, :]
        errs[rot] = np.sqrt(np.mean((y - ref) ** 2)) / np.sqrt(np.mean(ref ** 2))
    assert errs[True] < 0.25 and errs[True] < 0.6 * errs[False], errs


def test_pack_unpack_round_trip_all_pairs():
    a, b = np.meshgrid(np.arange(-8, 8), np.arange(-8, 8))
    codes = np.stack([a.ravel(), b.ravel()], axis=1).astype(np.int8)
    packed = oracle.pack_nibbles(codes)
    assert packed.shape == (256, 1)
    assert sorted(packed.ravel().tolist()) == list(range(256))
    assert np.array_equal(oracle.unpack_nibbles(packed), codes)
    assert packed[(codes[:, 0] == -8) & (codes[:, 1] == 7)][0, 0] == 0x78


def test_check_weights():
    c0 = wl.config0()
    assert oracle.check_weights(c0["w_codes"], bits(c0["w_scales"])) == 0
    bad = c0["w_codes"].copy()
    bad[3, 5] = 8
    assert oracle.check_weights(bad, bits(c0["w_scales"])) == 1
    sc = c0["w_scales"].copy()
    sc[0] = 0
    assert oracle.check_weights(c0["w_codes"], bits(sc)) == 2
    assert c0["w_codes"].min() == -8 and c0["w_codes"].max() == 7
    assert 0.005 <= float(c0["w_scales"].min()) and float(c0["w_scales"].max()) <= 0.02


# ------------------------------------------------------------------ GEMM and epilogue

def test_gemm_equals_wide_integer_matmul_and_special_cases():
    rng = np.random.default_rng(5)
    qx = rng.integers(-8, 8, (37, 352)).astype(np.int8)
    qw = rng.integers(-8, 8, (53, 352)).astype(np.int8)
    acc = oracle.gemm_i32(qx, qw)
    assert np.array_equal(acc, qx.astype(np.int64) @ qw.astype(np.int64).T)
    # not symmetric in its operands: a transposed-operand mistake changes the shape / values
    assert acc.shape == (37, 53)
    eye = np.eye(352, dtype=np.int8)
    assert np.array_equal(oracle.gemm_i32(qx, eye), qx.astype(np.int32))
    ones = np.ones((4, 352), np.int8)
    assert (oracle.gemm_i32(ones, ones) == 352).all()
    qw7 = np.clip(qw, -7, 7)
    assert np.array_equal(oracle.gemm_i32(qx, -qw7), -oracle.gemm_i32(qx, qw7))
    assert np.array_equal(oracle.gemm_i32(qx[:1], qw), acc[:1])
    assert oracle.dot_i32(qx[3], qw[11]) == acc[3, 11]
    # extreme magnitude stays exact: 64 * K
    m8 = np.full((1, 11008), -8, np.int8)
    assert oracle.gemm_i32(m8, m8)[0, 0] == 64 * 11008


def test_epilogue_against_numpy_float32():
    rng = np.random.default_rng(6)
    acc = rng.integers(-60000, 60000, (9, 33)).astype(np.int32)
    sx = rng.uniform(0.01, 4.0, 9).astype(np.float32)
    sw = f16(rng.uniform(0.005, 0.02, 33))
    ref = ((acc.astype(np.float32) * sx[:, None]) * sw.astype(np.float32)[None, :])
    with np.errstate(over="ignore"):
        assert np.array_equal(oracle.epilogue(acc, sx, bits(sw)), ref.astype(np.float16).view(np.uint16))
    got_bf = (oracle.epilogue(acc, sx, bits(sw), bf16=True).astype(np.uint32) << 16).view(np.float32)
    assert np.allclose(got_bf, ref, rtol=2.0 ** -8)
    assert np.array_equal(oracle.epilogue(acc, sx, bits(sw), bf16=True), oracle.float_to_bf16(ref))
    # row scale belongs to rows, channel scale to columns
    one = np.ones((2, 3), np.int32)
    out = oracle.epilogue(one, np.array([1, 2], np.float32), bits(f16([1, 4, 16]))).view(np.float16)
    assert out.tolist() == [[1, 4, 16], [2, 8, 32]]


def test_swiglu_epilogue_against_scipy():
    rng = np.random.default_rng(7)
    ag = rng.integers(-3000, 3000, (6, 40)).astype(np.int32)
    au = rng.integers(-3000, 3000, (6, 40)).astype(np.int32)
    sx = rng.uniform(0.05, 1.0, 6).astype(np.float32)
    swg = f16(rng.uniform(0.005, 0.02, 40))
    swu = f16(rng.uniform(0.005, 0.02, 40))
    g = ((ag.astype(np.float32) * sx[:, None]) * swg.astype(np.float32)).astype(np.float64)
    u = ((au.astype(np.float32) * sx[:, None]) * swu.astype(np.float32)).astype(np.float64)
    ref = (g * scipy.special.expit(g) * u)
    got = oracle.epilogue_swiglu(ag, au, sx, bits(swg), bits(swu)).view(np.float16).astype(np.float64)
    assert np.allclose(got, ref, rtol=2.0 ** -10, atol=1e-7)
    # gate and up are not interchangeable
    got_sw = oracle.epilogue_swiglu(au, ag, sx, bits(swu), bits(swg)).view(np.float16).astype(np.float64)
    assert not np.allclose(got_sw, ref, rtol=1e-2)
    # silu(0) * u = 0 ; large positive gate passes g*u through
    z = oracle.epilogue_swiglu(np.zeros((1, 1), np.int32), np.ones((1, 1), np.int32), np.ones(1, np.float32),
                               bits(f16([1])), bits(f16([1]))).view(np.float16)
    assert z[0, 0] == 0
    big = oracle.epilogue_swiglu(np.full((1, 1), 30, np.int32), np.full((1, 1), 2, np.int32),
                                 np.ones(1, np.float32), bits(f16([1])), bits(f16([1]))).view(np.float16)
    assert big[0, 0] == np.float16(60.0)


# ------------------------------------------------------------------ pruning criterion

def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                rows.append([float(t) for t in line.split()])
    return rows


def test_projection_pinhole_cases():
    # tests/golden/projection_cases.txt: hand-computed from Eq. 2-3
    for row in _read_golden("projection_cases.txt"):
        Kmat, Rt, xyz = row[0:9], row[9:21], row[21:24]
        pw, ph, tu, tv, front = row[24], row[25], int(row[26]), int(row[27]), int(row[28])
        (gu, gv), gf = oracle.project_center(Kmat, Rt, xyz, pw, ph)
        assert gf == bool(front)
        if front:
            assert (gu, gv) == (tu, tv)


def test_exp2_polynomial_against_numpy():
    ts = np.concatenate([-np.linspace(0, 30, 4001), -np.array([0.0, 1.0, 2.0, 0.5, 125.9, 126.0, 127.0, 500.0])]).astype(np.float32)
    got = np.array([oracle.exp2_neg(t) for t in ts], np.float64)
    ref = np.exp2(ts.astype(np.float64))
    ok = ts >= -126
    assert (np.abs(got[ok] - ref[ok]) <= 4e-7 * ref[ok]).all()
    assert (got[~ok] == 0).all()
    assert oracle.exp2_neg(0.0) == 1.0 and oracle.exp2_neg(-1.0) == 0.5 and oracle.exp2_neg(-7.0) == 2.0 ** -7   # exact


def test_attention_scores_against_float64_softmax_and_closed_forms():
    """The query token's attention over the visual tokens: against a float64 softmax(q.k / sqrt D) per head, rows
    summing to one, uniform keys giving exactly fp16(1/n), and a dominant key taking all the mass."""
    B_, rows, vs, nv, H, D = 2, 40, 3, 24, 4, 32
    ld = 3 * H * D
    rng = np.random.default_rng(5)
    qkv = (rng.standard_normal((B_ * rows, ld)) * 1.5).astype(np.float16)
    a = oracle.attention_scores(bits(qkv), B_, rows, rows - 1, vs, nv, H, D, 0, H * D).view(np.float16)
    x = qkv.astype(np.float64).reshape(B_, rows, ld)
    for b in range(B_):
        for h in range(H):
            q = x[b, rows - 1, h * D:(h + 1) * D]
            k = x[b, vs:vs + nv, H * D + h * D:H * D + (h + 1) * D]
            l = k @ q / math.sqrt(D)
            p = np.exp(l - l.max())
            p /= p.sum()
            assert (np.abs(a[b, h].astype(np.float64) - p) <= p * 2.0 ** -10 + 1e-7).all()
            assert abs(a[b, h].astype(np.float64).sum() - 1.0) < nv * 2.0 ** -11
    # all keys equal: every e_j = 1, the sum n is exact, a_j = fp16(1/n)
    qkv2 = qkv.copy().reshape(B_, rows, ld)
    qkv2[:, vs:vs + nv, H * D:2 * H * D] = qkv2[:, vs:vs + 1, H * D:2 * H * D]
    a2 = oracle.attention_scores(bits(qkv2.reshape(B_ * rows, ld)), B_, rows, rows - 1, vs, nv, H, D, 0, H * D).view(np.float16)
    assert (a2 == np.float16(np.float32(1.0) / np.float32(nv))).all()
    # one key aligned with a large query: it takes everything
    qkv3 = np.zeros((rows, ld), np.float16)
    qkv3[rows - 1, :D] = 8.0
    qkv3[vs + 5, H * D:H * D + D] = 8.0
    a3 = oracle.attention_scores(bits(qkv3), 1, rows, rows - 1, vs, nv, H, D, 0, H * D).view(np.float16)
    assert a3[0, 0, 5] == 1.0 and a3[0, 0].astype(np.float32).sum() == 1.0
    assert (a3[0, 1] == np.float16(np.float32(1.0) / np.float32(nv))).all()        # other heads: all logits zero


def test_score_sum_is_left_to_right_fp32():
    rng = np.random.default_rng(8)
    A = f16(rng.uniform(0, 1, (32, 40)))
    ref = np.zeros(40, np.float32)
    for r in range(32):
        ref = (ref + A[r].astype(np.float32)).astype(np.float32) if r else A[0].astype(np.float32)
    assert np.array_equal(oracle.score_sum(bits(A)), ref)
    # 2049 + 1 + 1 in fp16->fp32 is exact; pick a case where order matters in fp32
    B = f16([[2048.0], [1.0]])
    assert oracle.score_sum(bits(B))[0] == np.float32(2049.0)


def test_topk_equals_stable_full_sort():
    rng = np.random.default_rng(9)
    for n, k in [(48, 24), (256, 128), (256, 0), (256, 256), (17, 5)]:
        a = rng.standard_normal(n).astype(np.float32)
        a[rng.integers(0, n, n // 3)] = a[0]          # many exact ties
        order = np.argsort(-a.astype(np.float64), kind="stable")
        expect = np.zeros(n, bool)
        expect[order[:k]] = True
        assert np.array_equal(oracle.topk_mask(a, k), expect)
    # ties go to the lower index; +0 and -0 tie
    a = np.array([1.0, 3.0, 3.0, -0.0, 0.0, 3.0], np.float32)
    assert oracle.topk_mask(a, 2).nonzero()[0].tolist() == [1, 2]
    assert oracle.topk_mask(a, 5).nonzero()[0].tolist() == [0, 1, 2, 3, 5]


def test_ring_closed_forms():
    for (w, h, cu, cv, r) in [(16, 16, 8, 8, 1), (16, 16, 0, 0, 2), (16, 16, 15, 3, 3), (8, 6, 2, 5, 1),
                              (16, 16, -3, 4, 2), (16, 16, 20, 20, 2), (16, 16, 5, 5, 0), (16, 16, 5, 5, -1)]:
        m = oracle.ring_mask(w, h, cu, cv, r)
        nu = max(0, min(w - 1, cu + r) - max(0, cu - r) + 1) if r >= 0 else 0
        nvv = max(0, min(h - 1, cv + r) - max(0, cv - r) + 1) if r >= 0 else 0
        assert m.sum() == nu * nvv
        for j in m.nonzero()[0]:
            assert max(abs(j % w - cu), abs(j // w - cv)) <= r
    m = oracle.ring_mask(16, 16, 8, 8, 1)
    assert m.sum() == 9 and m[8 * 16 + 8] and m[7 * 16 + 7] and m[9 * 16 + 9] and not m[8 * 16 + 10]
    # u is the column (fast) coordinate: a centre at (t_u, t_v) = (15, 0) is the top-right corner
    assert oracle.ring_mask(16, 16, 15, 0, 0).nonzero()[0].tolist() == [15]


def _fps_brute(w, h, remain, m):
    """From-scratch FPS: recompute the distance to the picked set for every candidate each step."""
    cand = [j for j in range(w * h) if remain[j]]
    picked = []
    for _ in range(min(m, len(cand))):
        best, best_d = None, None
        for j in cand:
            if j in picked:
                continue
            if picked:
                d = min((j % w - p % w) ** 2 + (j // w - p // w) ** 2 for p in picked)
            else:
                d = float("inf")
            if best is None or d > best_d:
                best, best_d = j, d
        picked.append(best)
    return picked


def test_fps_against_brute_force_small_grids():
    rng = np.random.default_rng(10)
    for trial in range(40):
        w, h = int(rng.integers(1, 7)), int(rng.integers(1, 7))
        remain = rng.uniform(size=w * h) < 0.7
        m = int(rng.integers(0, w * h + 1))
        got = oracle.fps_mask(w, h, remain, m)
        exp = _fps_brute(w, h, remain, m)
        assert sorted(got.nonzero()[0].tolist()) == sorted(exp)
        assert not (got & ~remain).any()
        assert got.sum() == min(m, remain.sum())


def test_fps_worked_example_16x16():
    # tests/golden/fps_16x16_empty_union.txt: first picks on an empty union, derived from Eq. 5
    # with the tie rule "lowest index"
    expect = [int(v) for v in _read_golden("fps_16x16_empty_union.txt")[0]]
    assert expect == _fps_brute(16, 16, np.ones(256, bool), len(expect))
    for m in range(1, len(expect) + 1):
        got = oracle.fps_mask(16, 16, np.ones(256, bool), m)
        assert sorted(got.nonzero()[0].tolist()) == sorted(expect[:m])
    allm = oracle.fps_mask(16, 16, np.ones(256, bool), 256)
    assert allm.all()


def test_prune_union_quota_and_order():
    B = 3
    scores = wl.scores_softmax_rows(11, 1, B, 32, 256)
    centers = np.array([[8, 8], [0, 15], [30, 30]], np.int32)
    p = wl.prune_params(B, 288, 1, 256, 16, 16, 32, 40, 154, ring_radius=1)
    kept, n_kept, masks = oracle.prune_tokens(p, bits(scores), centers, want_masks=True)
    for b in range(B):
        attn, ring, fps = masks[b]
        a = oracle.score_sum(bits(scores[b]))
        assert np.array_equal(attn, oracle.topk_mask(a, 40))
        assert np.array_equal(ring, oracle.ring_mask(16, 16, centers[b, 0], centers[b, 1], 1))
        union = attn | ring
        assert not (fps & union).any()
        assert fps.sum() == 154 - union.sum()
        assert n_kept[b] == 32 + 154
        k = kept[b, :n_kept[b]]
        assert (np.diff(k) > 0).all()
        assert (kept[b, n_kept[b]:] == -1).all()
        vis = k[(k >= 1) & (k < 257)] - 1
        assert np.array_equal(np.sort(vis), (union | fps).nonzero()[0])
        text = k[(k < 1) | (k >= 257)]
        assert text.tolist() == [0] + list(range(257, 288))
    assert [masks[b, 1].sum() for b in range(B)] == [9, 4, 0]


def test_prune_pure_topk_and_quota_exceeded_and_degenerate():
    c0 = wl.config0()
    kept, n_kept = oracle.prune_tokens(c0["prune"], c0["scores"])
    assert n_kept[0] == 40
    order = np.argsort(-c0["scores"][0].astype(np.float64), kind="stable")[:24]
    assert kept[0, :40].tolist() == sorted(order.tolist()) + list(range(48, 64))
    # quota exceeded: union larger than keep_total -> keep the union, no FPS
    p = wl.prune_params(1, 64, 0, 48, 8, 6, 0, 20, 10, ring_radius=1)
    kept, n_kept, masks = oracle.prune_tokens(p, c0["scores"], np.array([[3, 3]], np.int32), want_masks=True)
    assert masks[0, 2].sum() == 0 and n_kept[0] == 16 + (masks[0, 0] | masks[0, 1]).sum()
    # k = 0, no ring: everything comes from FPS; keep_total = n_visual keeps all
    p = wl.prune_params(1, 64, 0, 48, 8, 6, 0, 0, 48)
    kept, n_kept = oracle.prune_tokens(p, c0["scores"])
    assert n_kept[0] == 64 and kept[0].tolist() == list(range(64))
    p = wl.prune_params(1, 64, 0, 48, 8, 6, 0, 0, 0)
    kept, n_kept = oracle.prune_tokens(p, c0["scores"])
    assert n_kept[0] == 16 and kept[0, :16].tolist() == list(range(48, 64))


def test_gather_is_a_bit_copy_in_order():
    rng = np.random.default_rng(12)
    x = rng.integers(0, 65536, (2, 10, 24)).astype(np.uint16)   # arbitrary bit patterns incl. NaNs
    kept = np.array([[1, 4, 9, -1, -1, -1, -1, -1, -1, -1], [0, 2, 3, 5, -1, -1, -1, -1, -1, -1]], np.int32)
    n_kept = np.array([3, 4], np.int32)
    out = oracle.gather_rows(x, kept, n_kept, 4, K=16)
    assert np.array_equal(out[0, :3], x[0, [1, 4, 9], :16]) and not out[0, 3].any()
    assert np.array_equal(out[1], x[1, [0, 2, 3, 5], :16])


# ------------------------------------------------------------------ generators (structure only)

def test_workload_structure():
    c0 = wl.config0()
    assert c0["x"].shape == (64, 512) and c0["x"].dtype == np.float16
    col_rms = np.sqrt((c0["x"].astype(np.float64) ** 2).mean(axis=0))
    assert (col_rms > 10).sum() == 4
    x1 = wl.activations(1, wl.T_X, 32, 4096, 41, 30.0)
    assert (np.sqrt((x1.astype(np.float64) ** 2).mean(axis=0)) > 12).sum() == 41
    s = wl.scores_softmax_rows(2, wl.T_SCORE, 2, 32, 256).astype(np.float64)
    assert np.allclose(s.sum(axis=-1), 1.0, atol=2e-3) and (s >= 0).all()
    codes = wl.int4_codes(5, 9, 100000)
    assert np.bincount(codes + 8, minlength=16).min() > 5500
    assert np.array_equal(wl.config0()["x"], c0["x"])            # deterministic
