"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bar: INT4 codes, activation scales, int32 accumulators and kept-token indices bit-exact; fp16 /
bf16 outputs within max(1 ulp, 2e-3 relative) of the oracle's.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2509_09090_b200 import workloads as wl

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    from paper_2509_09090_b200 import binding as B
    import gpu_harness as G


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float16).view(np.uint16)


KERNELS = [("simt", 1), ("auto", 0)]


def _linear_flags():
    return [0, B.SQAP_L_FORCE_SIMT]


def check_linear(x_f16, w_codes, w_scales, rotate=False, row_index=None, up=None, flags_list=None, bf16=False):
    """Quantize + linear on the GPU vs the oracle; returns the oracle's fp16 output bits."""
    packed_o, s_o, codes_o = oracle.quantize_act(bits(x_f16), rotate=rotate, row_index=row_index)
    packed_g, s_g = G.quantize(x_f16, rotate=rotate, row_index=row_index)
    assert np.array_equal(packed_g, packed_o)
    assert np.array_equal(s_g, s_o)
    acc_o = oracle.gemm_i32(codes_o, w_codes)
    w = G.pack(w_codes, w_scales)
    if up is None:
        ref = oracle.epilogue(acc_o, s_o, bits(w_scales), bf16=bf16)
        wu = None
    else:
        acc_u = oracle.gemm_i32(codes_o, up[0])
        ref = oracle.epilogue_swiglu(acc_o, acc_u, s_o, bits(w_scales), bits(up[1]), bf16=bf16)
        wu = G.pack(up[0], up[1])
    for flags in (flags_list if flags_list is not None else _linear_flags()):
        if up is None:
            acc_g = G.linear(packed_g, s_g, w, out_dtype=B.SQAP_I32, flags=flags)
            assert np.array_equal(acc_g, acc_o), f"int32 accumulators differ (flags={flags})"
        out = G.linear(packed_g, s_g, w, w_up=wu, out_dtype=B.SQAP_BF16 if bf16 else B.SQAP_FP16, flags=flags)
        ok = G.within_tolerance(out, ref, bf16=bf16)
        assert ok.all(), f"{(~ok).sum()} outputs outside tolerance (flags={flags})"
        # the fused quantize + linear call: same accumulators, and the same output bits as the two-call route
        if up is None:
            acc_f = G.quantize_linear(x_f16, w, rotate=rotate, row_index=row_index, out_dtype=B.SQAP_I32, flags=flags)
            assert np.array_equal(acc_f, acc_o), f"fused call: int32 accumulators differ (flags={flags})"
        out_f = G.quantize_linear(x_f16, w, w_up=wu, rotate=rotate, row_index=row_index,
                                  out_dtype=B.SQAP_BF16 if bf16 else B.SQAP_FP16, flags=flags)
        assert np.array_equal(out_f, out), f"fused call differs from quantize_act + w4a4_linear (flags={flags})"
    w.close()
    if wu:
        wu.close()
    return ref


# ------------------------------------------------------------------ quantizer

@pytest.mark.parametrize("M,K", [(1, 32), (2, 64), (7, 512), (64, 512), (33, 4096), (5, 11008), (3, 16384),
                                 (2, 20480), (9, 128), (9, 256)])
@pytest.mark.parametrize("rotate", [False, True])
def test_quantizer_bit_exact(M, K, rotate):
    if rotate and ((K & (K - 1)) or K < 64):
        pytest.skip("rotation needs a power of two >= 64")
    x = wl.activations(100 + M, K, M, K, max(1, K // 100), 30.0)
    x[M // 2] = 0                                              # an all-zero row
    po, so, _ = oracle.quantize_act(bits(x), rotate=rotate)
    pg, sg = G.quantize(x, rotate=rotate)
    assert np.array_equal(pg, po)
    assert np.array_equal(sg, so)


@pytest.mark.parametrize("K,rotate", [(512, False), (4096, False), (11008, False)])
def test_quantizer_products_that_round_onto_a_tie(K, rotate):
    """v = amax/2 gives v * fl(7/amax) = 3.5 * (1 + d), |d| <= 2^-24: for many amax the fp32 product rounds to
    exactly 3.5 and the tie goes to 4, while a multiply fused with the next operation sees 3.5 - tiny and gives
    3. The rows where that happens are found here in fp64; they catch a kernel that does not round the product."""
    M = 64
    x = (wl.activations(77, K, M, K, 0, 1.0) * np.float16(0.01)).astype(np.float16)
    amax = (np.arange(M, dtype=np.float32) * 0.71875 + 40.0).astype(np.float16)
    for r in range(M):
        x[r, 5], x[r, K // 2 + 1], x[r, K - 2] = amax[r], amax[r] / np.float16(2), -amax[r] / np.float16(2)
    po, so, codes = oracle.quantize_act(bits(x), rotate=rotate)
    inv = np.float32(7.0) / amax.astype(np.float32)
    exact = amax.astype(np.float64) / 2 * inv.astype(np.float64)          # 11 x 24 bits: exact in fp64
    onto_tie_from_below = (exact.astype(np.float32) == np.float32(3.5)) & (exact < 3.5)
    assert onto_tie_from_below.sum() >= 16
    assert (codes[onto_tie_from_below, K // 2 + 1] == 4).all() and (codes[onto_tie_from_below, K - 2] == -4).all()
    pg, sg = G.quantize(x, rotate=rotate)
    assert np.array_equal(pg, po) and np.array_equal(sg, so)
    wc, ws = wl.weight_codes(77, K, 8, K), wl.weight_scales(77, K, 8)
    w = G.pack(wc, ws)
    acc = G.quantize_linear(x, w, rotate=rotate, out_dtype=B.SQAP_I32)
    assert np.array_equal(acc, oracle.gemm_i32(codes, wc))
    w.close()


def test_quantizer_row_index_stride_and_empty():
    x = wl.activations(5, 5, 40, 1024, 10, 30.0)
    idx = np.array([39, 0, 7, 7, 12], np.int32)
    po, so, _ = oracle.quantize_act(bits(x), row_index=idx)
    pg, sg = G.quantize(x, row_index=idx)
    assert np.array_equal(pg, po) and np.array_equal(sg, so)
    # a column slice of a wider matrix (the V third of a fused QKV output): ldx = 1024, K = 256 at offset 512
    sub = np.ascontiguousarray(x[:, 512:768])
    po, so, _ = oracle.quantize_act(bits(sub), rotate=True)
    pg, sg = G.quantize(x, rotate=True, K=256, col_offset=512)
    assert np.array_equal(pg, po) and np.array_equal(sg, so)
    # M = 0 is a no-op
    B.sqap_quantize_act(None, 0, 64, 64, None, 0, None, None)


def test_quantizer_rejects_bad_arguments():
    t = torch.zeros(64 * 64, dtype=torch.float16, device="cuda")
    q = torch.zeros(64 * 32, dtype=torch.uint8, device="cuda")
    s = torch.zeros(64, dtype=torch.float32, device="cuda")
    L = B.lib()
    st = lambda *a: L.sqap_quantize_act(*a, None)
    assert st(t.data_ptr(), -1, 64, 64, None, 0, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID
    assert st(t.data_ptr(), 4, 48, 48, None, 0, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_ALIGN
    assert st(t.data_ptr() + 2, 4, 64, 64, None, 0, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_ALIGN
    assert st(t.data_ptr(), 4, 96, 96, None, B.SQAP_Q_ROTATE, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_UNSUPPORTED
    assert st(t.data_ptr(), 4, 64, 32, None, 0, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID
    assert st(None, 4, 64, 64, None, 0, q.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID


# ------------------------------------------------------------------ weights

@pytest.mark.parametrize("N,K", [(8, 32), (128, 512), (40, 96), (512, 4096), (16, 11008)])
@pytest.mark.parametrize("on_device", [False, True])
def test_pack_unpack_round_trip(N, K, on_device):
    codes = wl.weight_codes(9, N + K, N, K)
    scales = wl.weight_scales(9, N + K, N)
    w = G.pack(codes, scales, on_device=on_device)
    c2, s2 = B.sqap_unpack_weights(w)
    assert np.array_equal(c2, codes) and np.array_equal(s2.view(np.uint16), scales.view(np.uint16))
    assert B.sqap_weights_info(w) == (N, K, 0)
    w.close()


def test_pack_rejects_bad_codes_and_scales():
    codes = wl.weight_codes(9, 1, 16, 64)
    scales = wl.weight_scales(9, 1, 16)
    bad = codes.copy()
    bad[3, 7] = 8
    with pytest.raises(B.SqapError) as e:
        G.pack(bad, scales)
    assert e.value.status == B.SQAP_ERR_RANGE
    sc = scales.copy()
    sc[2] = np.float16(0)
    with pytest.raises(B.SqapError) as e:
        G.pack(codes, sc)
    assert e.value.status == B.SQAP_ERR_RANGE
    sc[2] = np.float16(np.inf)
    with pytest.raises(B.SqapError) as e:
        G.pack(codes, sc)
    assert e.value.status == B.SQAP_ERR_RANGE
    with pytest.raises(B.SqapError) as e:
        B.sqap_pack_weights(codes, scales, 16, 48)
    assert e.value.status == B.SQAP_ERR_ALIGN


@pytest.mark.parametrize("N,K,rotate", [(24, 256, False), (24, 256, True), (130, 4096, True), (9, 11008, False),
                                        (3, 64, True), (5, 16384, True), (40, 96, False)])
def test_weight_quantizer_bit_exact_and_feeds_the_linear(N, K, rotate):
    """sqap_quantize_weights against the oracle (codes and fp16 scale bits), then the quantized weights through
    pack + linear against the oracle's integer GEMM on the same codes."""
    w = (wl.activations(41, N + K, N, K, max(1, K // 100), 25.0).astype(np.float32) * np.float32(0.02)).astype(np.float16)
    w[N // 2] = 0
    wd = G.to_dev(w)
    codes = torch.empty(N, K, dtype=torch.int8, device="cuda")
    scales = torch.empty(N, dtype=torch.float16, device="cuda")
    B.sqap_quantize_weights(wd, N, K, K, B.SQAP_Q_ROTATE if rotate else 0, None, codes, scales)
    torch.cuda.synchronize()
    co, so = oracle.quantize_weights(bits(w), rotate=rotate)
    assert np.array_equal(codes.cpu().numpy(), co)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), so)
    if rotate or K % 32 == 0:
        x = wl.activations(42, K, 20, K, max(1, K // 100), 30.0)
        handle = B.sqap_pack_weights(codes, scales, N, K, B.SQAP_W_ROTATED if rotate else 0)   # device pointers
        torch.cuda.synchronize()
        _, sx, xc = oracle.quantize_act(bits(x), rotate=rotate)
        acc = G.quantize_linear(x, handle, rotate=rotate, out_dtype=B.SQAP_I32)
        assert np.array_equal(acc, oracle.gemm_i32(xc, co))
        out = G.quantize_linear(x, handle, rotate=rotate)
        ref = oracle.epilogue(oracle.gemm_i32(xc, co), sx, so)
        assert G.within_tolerance(out, ref).all()
        handle.close()


@pytest.mark.parametrize("M,K,rotate", [(12, 256, False), (12, 256, True), (37, 4096, True), (5, 11008, False),
                                        (300, 512, True), (9, 64, True), (9, 128, True), (33, 4096, False),
                                        (6, 20480, False), (1300, 4096, True), (3, 16384, True)])
def test_quantizer_per_tensor_and_channel_multiplier(M, K, rotate):
    """sqap_quantize_act_ex in its two extra granularities (and both at once) against the oracle, with a row index
    list; then a smoothed linear end to end: activations times 1/d, weights times d, codes through the GEMM."""
    x = wl.activations(61, K + M, M + 3, K, max(1, K // 100), 30.0)
    x[1] = 0
    idx = [(5 * i + 2) % (M + 3) for i in range(M)]
    mul = np.exp2((np.arange(K) % 7) - 3).astype(np.float32) * np.float32(1.25)
    xd, md, ri = G.to_dev(x), G.to_dev(mul), G.to_dev(np.asarray(idx, np.int32))
    for per_tensor, use_mul in ((True, False), (False, True), (True, True)):
        q = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device="cuda")
        s = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
        fl = (B.SQAP_Q_ROTATE if rotate else 0) | (B.SQAP_Q_PER_TENSOR if per_tensor else 0)
        B.sqap_quantize_act_ex(xd, M, K, K, ri, fl, md if use_mul else None, q, s)
        torch.cuda.synchronize()
        po, so, _ = oracle.quantize_act(bits(x), rotate=rotate, row_index=idx, per_tensor=per_tensor,
                                        ch_mul=mul if use_mul else None)
        assert np.array_equal(q.cpu().numpy(), po), (per_tensor, use_mul)
        assert np.array_equal(s.cpu().numpy(), so), (per_tensor, use_mul)
    # smoothed W4A4 linear: x * (1/d) against W * d
    N = 40
    w = (wl.activations(62, N + K, N, K, 0, 1.0).astype(np.float32) * np.float32(0.02)).astype(np.float16)
    d = np.exp2(np.round(0.5 * np.log2(np.maximum(np.abs(x.astype(np.float32)).max(axis=0), 1e-3)))).astype(np.float32)
    inv_d = (np.float32(1.0) / d).astype(np.float32)
    codes = torch.empty(N, K, dtype=torch.int8, device="cuda")
    scales = torch.empty(N, dtype=torch.float16, device="cuda")
    B.sqap_quantize_weights(G.to_dev(w), N, K, K, B.SQAP_Q_ROTATE if rotate else 0, G.to_dev(d), codes, scales)
    co, so_w = oracle.quantize_weights(bits(w), rotate=rotate, ch_mul=d)
    assert np.array_equal(codes.cpu().numpy(), co) and np.array_equal(scales.cpu().numpy().view(np.uint16), so_w)
    q = torch.empty(M, K // 2, dtype=torch.uint8, device="cuda")
    s = torch.empty(M, dtype=torch.float32, device="cuda")
    B.sqap_quantize_act_ex(xd, M, K, K, ri, B.SQAP_Q_ROTATE if rotate else 0, G.to_dev(inv_d), q, s)
    handle = B.sqap_pack_weights(codes, scales, N, K)
    torch.cuda.synchronize()
    _, sx, xc = oracle.quantize_act(bits(x), rotate=rotate, row_index=idx, ch_mul=inv_d)
    out = G.linear(q.cpu().numpy(), s.cpu().numpy(), handle)
    ref = oracle.epilogue(oracle.gemm_i32(xc, co), sx, so_w)
    assert G.within_tolerance(out, ref).all()
    handle.close()


def test_per_tensor_quantizer_calls_in_flight_on_two_streams():
    """The tensor's max-abs travels between the two launches of a per-tensor call in a word of a pool owned by the
    library; calls on different streams must not see each other's word. Two streams, different tensors (one with a
    far larger max-abs), many calls each, issued alternately without synchronising in between."""
    M, K = 96, 1024
    xa = wl.activations(63, 1, M, K, 4, 30.0)
    xb = (wl.activations(63, 2, M, K, 4, 30.0).astype(np.float32) * np.float32(0.01)).astype(np.float16)
    ref = [oracle.quantize_act(bits(v), per_tensor=True) for v in (xa, xb)]
    dev = [G.to_dev(v) for v in (xa, xb)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    reps = 12
    q = [[torch.empty(M, K // 2, dtype=torch.uint8, device="cuda") for _ in range(reps)] for _ in range(2)]
    s = [[torch.empty(M, dtype=torch.float32, device="cuda") for _ in range(reps)] for _ in range(2)]
    torch.cuda.synchronize()
    for r in range(reps):
        for i in range(2):
            B.sqap_quantize_act_ex(dev[i], M, K, K, None, B.SQAP_Q_PER_TENSOR, None, q[i][r], s[i][r], stream=streams[i])
    torch.cuda.synchronize()
    for i in range(2):
        for r in range(reps):
            assert np.array_equal(q[i][r].cpu().numpy(), ref[i][0]), (i, r)
            assert np.array_equal(s[i][r].cpu().numpy(), ref[i][1]), (i, r)


def test_weight_quantizer_rejects_bad_arguments():
    w = torch.zeros(8 * 96, dtype=torch.float16, device="cuda")
    c = torch.zeros(8 * 96, dtype=torch.int8, device="cuda")
    s = torch.zeros(8, dtype=torch.float16, device="cuda")
    L = B.lib()
    st = lambda *a: L.sqap_quantize_weights(*a, None)
    assert st(w.data_ptr(), -1, 96, 96, 0, None, c.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID
    assert st(w.data_ptr(), 8, 96, 64, 0, None, c.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID
    assert st(w.data_ptr(), 8, 48, 48, 0, None, c.data_ptr(), s.data_ptr()) == B.SQAP_ERR_ALIGN
    assert st(w.data_ptr(), 8, 96, 96, B.SQAP_Q_ROTATE, None, c.data_ptr(), s.data_ptr()) == B.SQAP_ERR_UNSUPPORTED
    assert st(None, 8, 96, 96, 0, None, c.data_ptr(), s.data_ptr()) == B.SQAP_ERR_INVALID
    assert st(w.data_ptr(), 0, 96, 96, 0, None, None, None) == B.SQAP_OK


# ------------------------------------------------------------------ linear: small and ragged shapes

@pytest.mark.parametrize("M,N,K", [(1, 8, 32), (2, 128, 64), (7, 8, 512), (64, 512, 512), (65, 130, 96),
                                   (9, 72, 11008), (130, 264, 1024), (300, 520, 256), (1, 200, 11008), (1, 3000, 4224),
                                   (1, 72, 16384), (1, 40, 20480)])
def test_linear_small_shapes(M, N, K):
    x = wl.activations(20, M * 7 + K, M, K, max(1, K // 100), 20.0)
    wc = wl.weight_codes(20, N * 3 + K, N, K)
    ws = wl.weight_scales(20, N * 3 + K, N)
    check_linear(x, wc, ws)
    if M <= 8:
        check_linear(x, wc, ws, flags_list=[B.SQAP_L_FORCE_GEMV])


def _random_linear_shapes(n, seed):
    """Seeded shapes across every regime of the dispatcher (single rows, a handful, mid-size, many tiles; short and
    long rows; K % 128 == 0 or not), small enough for the oracle."""
    rng = np.random.default_rng(seed)
    ms = [1, 1, 1, 2, 3, 5, 8, 9, 16, 17, 31, 32, 33, 63, 64, 100, 143, 144, 200, 320, 321, 511, 512, 600]
    ks = [32, 64, 96, 128, 256, 384, 1024, 2048, 4096, 4224, 8192, 11008, 12288, 16384]
    out = []
    while len(out) < n:
        M, K = int(rng.choice(ms)), int(rng.choice(ks))
        N = 8 * int(rng.integers(1, 400))
        if M * N * K > 4e8:
            continue
        out.append((M, N, K, bool(rng.integers(0, 2)), bool(rng.integers(0, 2)) and (K & (K - 1)) == 0 and K >= 64))
    return out


@pytest.mark.parametrize("M,N,K,swiglu,rotate", _random_linear_shapes(40, 2509))
def test_linear_random_shapes_through_the_dispatcher(M, N, K, swiglu, rotate):
    """Whatever kernel the dispatcher picks for a shape: int32 accumulators bit-exact, outputs within tolerance, the
    fused call identical to the two-call route."""
    x = wl.activations(27, M + N + K, M, K, max(1, K // 100), 20.0)
    g = (wl.weight_codes(27, N + K, N, K), wl.weight_scales(27, N + K, N, mult=0.5))
    u = (wl.weight_codes(27, N + K + 1, N, K), wl.weight_scales(27, N + K + 1, N, mult=0.5)) if swiglu else None
    check_linear(x, g[0], g[1], rotate=rotate, up=u, flags_list=[0])


@pytest.mark.parametrize("M,N,K,swiglu", [(16, 128, 128, False), (9, 8, 256, False), (257, 130, 384, False),
                                          (144, 320, 1024, False), (700, 200, 512, False), (40, 192, 512, True),
                                          (300, 64, 256, True), (513, 448, 1152, True), (17, 1088, 11008, False),
                                          (384, 256, 2304, False), (200, 128, 2048, True)])
def test_linear_tcgen05_forced(M, N, K, swiglu):
    """The tensor-core kernel on shapes with ragged token tiles, partial weight tiles and the fused gate; the last
    two walk rings of odd depth (3 and 5 stages) several times around within one tile."""
    x = wl.activations(25, M + K, M, K, max(1, K // 100), 20.0)
    g = (wl.weight_codes(25, N + K, N, K), wl.weight_scales(25, N + K, N, mult=0.5))
    u = (wl.weight_codes(25, N + K + 1, N, K), wl.weight_scales(25, N + K + 1, N, mult=0.5)) if swiglu else None
    kernels = [B.SQAP_L_FORCE_TCGEN05, B.SQAP_L_FORCE_TCGEN05_TS, B.SQAP_L_FORCE_TCGEN05_PAIR, B.SQAP_L_FORCE_TCGEN05_SPLITK]
    check_linear(x, g[0], g[1], up=u, flags_list=kernels)
    check_linear(x, g[0], g[1], up=u, flags_list=kernels, bf16=True)


@pytest.mark.parametrize("M,N,K,swiglu", [(1300, 3500, 384, False), (1000, 2368, 256, True)])
def test_linear_tcgen05_many_tiles(M, N, K, swiglu):
    """More tiles than SMs: every CTA walks several tiles, so both accumulator buffers and every ring wrap
    around; ragged last token tile and a partial last weight tile."""
    x = wl.activations(26, M + K, M, K, max(1, K // 100), 20.0)
    g = (wl.weight_codes(26, N + K, N, K), wl.weight_scales(26, N + K, N, mult=0.5))
    u = (wl.weight_codes(26, N + K + 1, N, K), wl.weight_scales(26, N + K + 1, N, mult=0.5)) if swiglu else None
    check_linear(x, g[0], g[1], up=u, flags_list=[B.SQAP_L_FORCE_TCGEN05, B.SQAP_L_FORCE_TCGEN05_TS, B.SQAP_L_FORCE_TCGEN05_PAIR,
                                                  B.SQAP_L_FORCE_TCGEN05_SPLITK])


@pytest.mark.parametrize("M,N,K,swiglu,split", [
    (160, 384, 4096, False, 4), (160, 264, 11008, False, 4), (288, 384, 4096, False, 2), (150, 320, 768, True, 3),
    (17, 130, 1024, False, 4), (192, 256, 1280, True, 2), (100, 200, 2048, False, 3), (511, 136, 512, False, 2),
    (33, 72, 256, False, 1), (160, 1024, 4096, True, 3), (176, 640, 2816, False, 0), (64, 4096, 1024, False, 0)])
def test_linear_cluster_split_k(M, N, K, swiglu, split):
    """The kernel that splits K over the CTAs of a cluster and adds the partial accumulators through distributed
    shared memory: every cluster size, stage counts that do not divide evenly among the CTAs (43 over 4, 5 over 2,
    8 over 3), one stage per CTA, two token tiles, chunk counts that leave some CTAs of the cluster one chunk
    short, partial weight tiles, the fused gate, all three output types; split = 0 lets the library choose."""
    x = wl.activations(35, M + K, M, K, max(1, K // 100), 20.0)
    g = (wl.weight_codes(35, N + K, N, K), wl.weight_scales(35, N + K, N, mult=0.5))
    u = (wl.weight_codes(35, N + K + 1, N, K), wl.weight_scales(35, N + K + 1, N, mult=0.5)) if swiglu else None
    fl = [B.SQAP_L_FORCE_TCGEN05_SPLITK | B.SQAP_L_KSPLIT(split)]
    check_linear(x, g[0], g[1], up=u, flags_list=fl)
    check_linear(x, g[0], g[1], up=u, flags_list=fl, bf16=True)


def test_linear_cluster_split_k_rejects_more_slices_than_stages():
    K, N, M = 512, 128, 32         # two stages of 256 codes
    w = G.pack(wl.weight_codes(36, 1, N, K), wl.weight_scales(36, 1, N))
    q = torch.zeros(M * K // 2, dtype=torch.uint8, device="cuda")
    s = torch.ones(M, dtype=torch.float32, device="cuda")
    out = torch.zeros(M * N, dtype=torch.float16, device="cuda")
    nb = B.sqap_workspace_bytes(M, N, K)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    L = B.lib()
    call = lambda fl: L.sqap_w4a4_linear(q.data_ptr(), s.data_ptr(), M, w.handle, None, out.data_ptr(), N, B.SQAP_FP16, fl,
                                         ws.data_ptr(), nb, None)
    assert call(B.SQAP_L_FORCE_TCGEN05_SPLITK | B.SQAP_L_KSPLIT(3)) == B.SQAP_ERR_UNSUPPORTED
    assert call(B.SQAP_L_FORCE_TCGEN05_SPLITK | B.SQAP_L_KSPLIT(5)) == B.SQAP_ERR_INVALID
    assert call(B.SQAP_L_KSPLIT(2)) == B.SQAP_ERR_INVALID            # a cluster size without the kernel it belongs to
    assert call(B.SQAP_L_FORCE_TCGEN05_SPLITK | B.SQAP_L_KSPLIT(2)) == B.SQAP_OK
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    w.close()


@pytest.mark.parametrize("K", [64, 128, 256, 512, 4096])
def test_fused_quantize_linear_rotated_rows_and_row_index(K):
    """The fused call with the Hadamard rotation at every supported row length class, reading its rows
    through an index list (repeated and out-of-order rows), against the oracle."""
    M, N = 37, 72
    x = wl.activations(27, K, 50, K, max(1, K // 100), 30.0)
    x[11] = 0
    idx = [(7 * i + 3) % 50 for i in range(M - 1)] + [11]
    wc = wl.weight_codes(27, N + K, N, K)
    ws = wl.weight_scales(27, N + K, N)
    check_linear(x, wc, ws, rotate=True, row_index=idx)
    check_linear(x, wc, ws, rotate=False, row_index=idx)


@pytest.mark.parametrize("M", [1, 2, 3, 5, 8])
def test_gemv_rows_and_swiglu(M):
    K, N = 4096, 264
    x = wl.activations(21, M, M, K, 41, 30.0)
    g = (wl.weight_codes(21, 1, N, K), wl.weight_scales(21, 1, N, mult=0.25))
    u = (wl.weight_codes(21, 2, N, K), wl.weight_scales(21, 2, N, mult=0.25))
    check_linear(x, g[0], g[1], flags_list=[B.SQAP_L_FORCE_GEMV, B.SQAP_L_FORCE_SIMT, 0])
    check_linear(x, g[0], g[1], up=u, flags_list=[B.SQAP_L_FORCE_GEMV, B.SQAP_L_FORCE_SIMT, 0])


@pytest.mark.parametrize("M,N,K,swiglu", [(1, 16, 128, False), (3, 264, 4096, False), (8, 40, 384, True),
                                          (9, 130, 1152, False), (16, 1088, 11008, False), (17, 72, 256, True),
                                          (24, 264, 4096, True), (25, 48, 2048, False), (32, 200, 1024, True)])
def test_linear_register_mma_streamer(M, N, K, swiglu):
    """The weight-streaming register-MMA kernel for a handful of tokens: every token-group count (1-4), token
    counts that leave a group partly empty, channel counts that are not multiples of 16, K blocks that do not
    divide among the warps evenly, fp16 / bf16 / int32 outputs, with and without the fused gate."""
    x = wl.activations(28, M + K, M, K, max(1, K // 100), 25.0)
    g = (wl.weight_codes(28, N + K, N, K), wl.weight_scales(28, N + K, N, mult=0.5))
    u = (wl.weight_codes(28, N + K + 1, N, K), wl.weight_scales(28, N + K + 1, N, mult=0.5)) if swiglu else None
    check_linear(x, g[0], g[1], up=u, flags_list=[B.SQAP_L_FORCE_MMA, 0])
    check_linear(x, g[0], g[1], up=u, flags_list=[B.SQAP_L_FORCE_MMA], bf16=True)


@pytest.mark.parametrize("M,N,K,swiglu", [(1, 136, 4224, False), (16, 8192, 256, False), (17, 8192, 256, False),
                                          (32, 264, 384, True), (33, 264, 384, True), (143, 8192, 128, False),
                                          (144, 8192, 128, False), (150, 4096, 256, True), (63, 384, 8192, False),
                                          (64, 384, 8192, False), (100, 384, 7936, False), (320, 384, 8192, False), (321, 384, 8192, False)])
def test_linear_dispatch_boundaries(M, N, K, swiglu):
    """The kernel the dispatcher picks by itself on either side of each of its thresholds (one row longer than 4096
    codes; 16 | 17 rows with many weight tiles; 32 | 33 rows with few; 143 | 144 rows with many tiles, plain and
    gated; few weight tiles with K below | from 8192 and 63 | 64 and 320 | 321 rows: the cluster split-K kernel), against the
    oracle and against the plain CUDA-core kernel."""
    x = wl.activations(29, M + K, M, K, max(1, K // 100), 25.0)
    g = (wl.weight_codes(29, N + K, N, K), wl.weight_scales(29, N + K, N, mult=0.5))
    u = (wl.weight_codes(29, N + K + 1, N, K), wl.weight_scales(29, N + K + 1, N, mult=0.5)) if swiglu else None
    check_linear(x, g[0], g[1], up=u, flags_list=[0, B.SQAP_L_FORCE_SIMT])


@pytest.mark.parametrize("M,K,rotate", [(1, 4096, False), (1, 4096, True), (1, 11008, False), (1, 384, False),
                                        (5, 4096, False), (40, 4096, False)])
def test_fused_call_leaves_the_expanded_activations_for_reuse(M, K, rotate):
    """After sqap_quantize_linear the workspace holds the expanded codes, the row sums and (behind them) the
    scales of those activations: a second weight matrix applied with SQAP_L_REUSE_EXPANDED must give exactly what
    the full call gives. M = 1 without rotation is the case where the streamers quantize the row themselves (the
    dp4a one up to 4096 codes, the register-MMA one beyond)."""
    N = 264
    x = wl.activations(30, M + 7, M, K, max(1, K // 100), 30.0)
    w1 = G.pack(wl.weight_codes(30, 1, N, K), wl.weight_scales(30, 1, N, mult=0.25))
    w2 = G.pack(wl.weight_codes(30, 2, N, K), wl.weight_scales(30, 2, N, mult=0.25))
    ref2 = G.quantize_linear(x, w2, rotate=rotate)
    xd = torch.from_numpy(np.ascontiguousarray(x)).to("cuda")
    nb = B.sqap_quantize_linear_workspace_bytes(M, N, K)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    out1 = torch.empty(M, N, dtype=torch.float16, device="cuda")
    out2 = torch.empty(M, N, dtype=torch.float16, device="cuda")
    B.sqap_quantize_linear(xd, M, K, None, B.SQAP_Q_ROTATE if rotate else 0, w1, None, out1, N, B.SQAP_FP16, 0, ws, nb)
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    scales_ptr = ws.data_ptr() + B.sqap_workspace_bytes(M, N, K)
    B.sqap_w4a4_linear(dummy, scales_ptr, M, w2, None, out2, N, B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED, ws, nb)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    assert np.array_equal(out2.cpu().numpy().view(np.uint16), ref2)
    w1.close()
    w2.close()


def test_linear_special_operands():
    K = N = 256
    x = wl.activations(22, 1, 16, K, 3, 20.0)
    _, s, codes = oracle.quantize_act(bits(x))
    pg, sg = G.quantize(x)
    one = np.float16(1.0)
    eye = G.pack(np.eye(K, dtype=np.int8), np.full(N, one))
    for f in _linear_flags():
        assert np.array_equal(G.linear(pg, sg, eye, out_dtype=B.SQAP_I32, flags=f), codes.astype(np.int32))
    m8 = G.pack(np.full((N, K), -8, np.int8), np.full(N, one))
    allm8 = oracle.pack_nibbles(np.full((4, K), -8, np.int8))
    for f in _linear_flags():
        assert (G.linear(allm8, np.ones(4, np.float32), m8, out_dtype=B.SQAP_I32, flags=f) == 64 * K).all()
    p7 = G.pack(np.full((N, K), 7, np.int8), np.full(N, one))
    for f in _linear_flags():
        assert (G.linear(allm8, np.ones(4, np.float32), p7, out_dtype=B.SQAP_I32, flags=f) == -56 * K).all()


def test_linear_bf16_output_and_padded_rows():
    M, N, K = 37, 200, 512
    x = wl.activations(23, 1, M, K, 5, 20.0)
    wc, ws = wl.weight_codes(23, 2, N, K), wl.weight_scales(23, 2, N)
    ref = check_linear(x, wc, ws, bf16=True)
    assert ref.shape == (M, N)
    pg, sg = G.quantize(x)
    w = G.pack(wc, ws)
    a = G.linear(pg, sg, w, ldo=N)
    b = G.linear(pg, sg, w, ldo=N + 56)
    assert np.array_equal(a, b)
    w.close()


def test_linear_rejects_bad_arguments():
    wc, ws = wl.weight_codes(24, 2, 64, 128), wl.weight_scales(24, 2, 64)
    w = G.pack(wc, ws)
    w2 = G.pack(wl.weight_codes(24, 3, 32, 128), wl.weight_scales(24, 3, 32))
    q = torch.zeros(16 * 64, dtype=torch.uint8, device="cuda")
    s = torch.ones(16, dtype=torch.float32, device="cuda")
    out = torch.zeros(16 * 64, dtype=torch.float16, device="cuda")
    ws_t = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    L = B.lib()

    def call(M=16, w_=w, up=None, o=out.data_ptr(), ldo=64, dt=B.SQAP_FP16, fl=0, wsp=ws_t.data_ptr(), wsb=1 << 16):
        return L.sqap_w4a4_linear(q.data_ptr(), s.data_ptr(), M, w_.handle, up.handle if up else None, o, ldo, dt, fl,
                                  wsp, wsb, None)

    assert call() == B.SQAP_OK
    assert call(M=-1) == B.SQAP_ERR_INVALID
    assert call(ldo=32) == B.SQAP_ERR_INVALID
    assert call(up=w2) == B.SQAP_ERR_INVALID
    assert call(dt=7) == B.SQAP_ERR_INVALID
    assert call(up=w, dt=B.SQAP_I32) == B.SQAP_ERR_INVALID
    assert call(o=out.data_ptr() + 2) == B.SQAP_ERR_ALIGN
    assert call(ldo=68) == B.SQAP_ERR_ALIGN
    assert call(wsb=128) == B.SQAP_ERR_NOMEM
    assert call(fl=B.SQAP_L_FORCE_GEMV) == B.SQAP_ERR_UNSUPPORTED
    # the register-MMA streamer stops at 32 rows (buffers sized for the 40 rows asked for)
    q40 = torch.zeros(40 * 64, dtype=torch.uint8, device="cuda")
    s40 = torch.ones(40, dtype=torch.float32, device="cuda")
    out40 = torch.zeros(40 * 64, dtype=torch.float16, device="cuda")
    assert L.sqap_w4a4_linear(q40.data_ptr(), s40.data_ptr(), 40, w.handle, None, out40.data_ptr(), 64, B.SQAP_FP16,
                              B.SQAP_L_FORCE_MMA, ws_t.data_ptr(), 1 << 16, None) == B.SQAP_ERR_UNSUPPORTED
    assert call(fl=3) == B.SQAP_ERR_INVALID
    assert call(M=0) == B.SQAP_OK
    torch.cuda.synchronize()
    w.close()
    w2.close()


def test_decode_chain_back_to_back_on_one_workspace():
    """A decode layer issued eagerly with no host synchronisation in between, every call on the same workspace, as a
    layer runs it: quantize+linear with the row quantized inside the streamer, two more weight matrices on the
    expanded codes it left (SQAP_L_REUSE_EXPANDED), the next fused call overwriting the workspace, a rotated call
    (separate quantizer kernel launched as a programmatic dependent), twice around. Kernels of such a chain may
    overlap their predecessor up to their dependency wait; every output must still equal the oracle's."""
    K, N = 4096, 264
    x = wl.activations(33, 1, 3, K, 41, 30.0)
    ws_ = [(wl.weight_codes(33, 10 + i, N, K), wl.weight_scales(33, 10 + i, N, mult=0.25)) for i in range(4)]
    w = [G.pack(c, s) for c, s in ws_]
    xd = G.to_dev(x)
    nb = B.sqap_quantize_linear_workspace_bytes(1, N, K)
    wsp = torch.empty(nb, dtype=torch.uint8, device="cuda")
    sc_ptr = wsp.data_ptr() + B.sqap_workspace_bytes(1, N, K)
    outs = torch.full((2, 6, N), 0x7B7B, dtype=torch.int16, device="cuda")
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    row = lambda r: xd.data_ptr() + 2 * K * r
    for rep in range(2):
        o = outs[rep]
        B.sqap_quantize_linear(row(0), 1, K, None, 0, w[0], None, o[0], N, B.SQAP_FP16, 0, wsp, nb)
        B.sqap_w4a4_linear(dummy, sc_ptr, 1, w[1], None, o[1], N, B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED, wsp, nb)
        B.sqap_w4a4_linear(dummy, sc_ptr, 1, w[2], w[3], o[2], N, B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED, wsp, nb)
        B.sqap_quantize_linear(row(1), 1, K, None, 0, w[2], w[3], o[3], N, B.SQAP_FP16, 0, wsp, nb)
        B.sqap_quantize_linear(row(2), 1, K, None, B.SQAP_Q_ROTATE, w[1], None, o[4], N, B.SQAP_FP16, 0, wsp, nb)
        B.sqap_w4a4_linear(dummy, sc_ptr, 1, w[0], None, o[5], N, B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED, wsp, nb)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    got = outs.cpu().numpy().view(np.uint16)

    def ref(r, rotate, g, u=None):
        _, s, codes = oracle.quantize_act(bits(x[r:r + 1]), rotate=rotate)
        acc = oracle.gemm_i32(codes, ws_[g][0])
        if u is None:
            return oracle.epilogue(acc, s, bits(ws_[g][1]))
        return oracle.epilogue_swiglu(acc, oracle.gemm_i32(codes, ws_[u][0]), s, bits(ws_[g][1]), bits(ws_[u][1]))

    want = [ref(0, False, 0), ref(0, False, 1), ref(0, False, 2, 3), ref(1, False, 2, 3), ref(2, True, 1), ref(2, True, 0)]
    for rep in range(2):
        for i, r in enumerate(want):
            assert G.within_tolerance(got[rep, i][None], r).all(), (rep, i)
    for h in w:
        h.close()


def test_bounded_wait_runs_out_and_reports_timeout():
    """The failure-detection path: a wait that nothing satisfies gives up after its limit, the status word reports
    SQAP_ERR_TIMEOUT exactly once, and the device keeps working (a linear right after matches the oracle)."""
    assert B.sqap_device_status() == B.SQAP_OK
    L = B.lib()
    assert L.sqap_selftest_bounded_wait(10, None) == B.SQAP_ERR_INVALID
    assert L.sqap_selftest_bounded_wait(10 ** 10, None) == B.SQAP_ERR_INVALID
    B.sqap_selftest_bounded_wait(2_000_000)          # about a millisecond
    assert B.sqap_device_status() == B.SQAP_ERR_TIMEOUT
    assert B.sqap_device_status() == B.SQAP_OK
    M, N, K = 150, 256, 512
    x = wl.activations(34, 1, M, K, 5, 20.0)
    check_linear(x, wl.weight_codes(34, 2, N, K), wl.weight_scales(34, 2, N),
                 flags_list=[B.SQAP_L_FORCE_TCGEN05_TS, B.SQAP_L_FORCE_TCGEN05_PAIR])


# ------------------------------------------------------------------ pruning

def check_prune(params, scores, centers=None, x=None, out_rows=0):
    sc = bits(scores) if params["score_rows"] > 0 else scores
    kept_o, nk_o = oracle.prune_tokens(params, sc, centers)
    kept_g, nk_g, xo = G.prune(params, scores, centers, x, out_rows)
    assert np.array_equal(nk_g, nk_o)
    assert np.array_equal(kept_g, kept_o)
    if x is not None:
        xb = bits(x).reshape(params["batch"], params["rows"], -1)
        ref = oracle.gather_rows(xb, kept_o, nk_o, out_rows)
        for b in range(params["batch"]):
            n = min(nk_o[b], out_rows)
            assert np.array_equal(xo[b, :n], ref[b, :n])
            assert (xo[b, n:] == 0x7B7B).all()         # rows past n_kept are never written
    return kept_o, nk_o


@pytest.mark.parametrize("k_attn,keep,radius", [(24, 24, -1), (0, 0, -1), (48, 48, -1), (10, 30, 1), (0, 20, 0),
                                                (5, 48, 2), (60, 10, 1), (0, 100, -1)])
def test_prune_small_grid(k_attn, keep, radius):
    c0 = wl.config0()
    p = wl.prune_params(1, 64, 0, 48, 8, 6, 0, k_attn, keep, ring_radius=radius)
    check_prune(p, c0["scores"], np.array([[6, 1]], np.int32), c0["x"], 64)


def test_prune_batched_full_criterion_and_offgrid_centres():
    Bn = 16
    scores = wl.scores_softmax_rows(30, 1, Bn, 32, 256)
    centers = wl.ring_centers(30, 2, Bn, 16, 16)
    centers[3] = (-1, 7)
    centers[4] = (40, 40)
    centers[5] = (15, 15)
    x = wl.activations(30, 3, Bn * 288, 512, 5, 30.0)
    for keep, k_attn, radius in [(64, 32, 1), (128, 64, 1), (192, 96, 2), (154, 40, 1), (128, 128, -1)]:
        p = wl.prune_params(Bn, 288, 1, 256, 16, 16, 32, k_attn, keep, ring_radius=radius)
        kept, nk = check_prune(p, scores, centers, x, 32 + keep)
        assert (nk == 32 + keep).all()


def test_prune_ties_large_grid_and_ragged_rows():
    # many tied scores, a 32x32 grid (the largest supported), rows not a multiple of the block size
    rng = np.random.default_rng(31)
    s = rng.integers(0, 6, (2, 1024)).astype(np.float32)
    p = wl.prune_params(2, 1024 + 77, 50, 1024, 32, 32, 0, 100, 400, ring_radius=3)
    check_prune(p, s, np.array([[0, 0], [31, 16]], np.int32))
    s = rng.integers(0, 3, (3, 30)).astype(np.float32)
    p = wl.prune_params(3, 41, 11, 30, 5, 6, 0, 7, 19, ring_radius=0)
    check_prune(p, s, np.array([[2, 2], [4, 5], [9, 9]], np.int32))
    # no visual tokens at all
    p = wl.prune_params(2, 10, 0, 0, 0, 0, 0, 0, 0)
    kept, nk, _ = G.prune(p, np.zeros((2, 1), np.float32))
    assert (nk == 10).all() and (kept == np.arange(10)).all()


@pytest.mark.parametrize("grid_w,grid_h", [(1, 40), (40, 1), (1, 1), (2, 33), (1, 1024)])
def test_prune_fps_on_one_token_wide_and_high_grids(grid_w, grid_h):
    """Grids that are a single column or a single row of tokens, with farthest-point sampling active (and a ring,
    and some top-k): the picked token's coordinates must come out right when grid_w = 1."""
    nv = grid_w * grid_h
    rng = np.random.default_rng(grid_w * 1000 + grid_h)
    s = rng.integers(0, 4, (2, nv)).astype(np.float32)
    for k_attn, keep, radius in [(0, nv // 2 + 1, -1), (min(3, nv), min(nv, 17), 1), (0, nv, -1)]:
        p = wl.prune_params(2, nv + 9, 4, nv, grid_w, grid_h, 0, k_attn, keep, ring_radius=radius)
        check_prune(p, s, np.array([[0, grid_h // 2], [grid_w - 1, 0]], np.int32))


def test_prune_select_row_list_feeds_the_quantizer():
    """sqap_prune_select: the same kept set as sqap_prune_tokens, and the flat source-row list b*rows + kept row (the
    observation's last kept row repeated where fewer rows were kept than asked for); a quantize + linear that reads
    x through that list equals one that reads the oracle's gathered copy."""
    Bn, rows, K = 3, 70, 256
    scores = wl.scores_normal(38, 1, Bn, 48)
    centers = np.array([[2, 2], [7, 5], [30, 30]], np.int32)
    x = wl.activations(38, 2, Bn * rows, K, 3, 20.0)
    for keep, k_attn, radius, out_rows in [(24, 10, 1, 46), (24, 10, 1, 50), (0, 0, -1, 30)]:
        p = wl.prune_params(Bn, rows, 5, 48, 8, 6, 0, k_attn, keep, ring_radius=radius)
        kept_o, nk_o = oracle.prune_tokens(p, scores, centers)
        kept = torch.full((Bn, rows), -7, dtype=torch.int32, device="cuda")
        nk = torch.full((Bn,), -7, dtype=torch.int32, device="cuda")
        ri = torch.full((Bn * out_rows + 1,), -7, dtype=torch.int32, device="cuda")
        B.sqap_prune_select(p, G.to_dev(scores), G.to_dev(centers), out_rows, kept, nk, ri)
        torch.cuda.synchronize()
        assert np.array_equal(kept.cpu().numpy(), kept_o) and np.array_equal(nk.cpu().numpy(), nk_o)
        want = np.empty((Bn, out_rows), np.int64)
        for b in range(Bn):
            n = min(int(nk_o[b]), out_rows)
            want[b, :n] = b * rows + kept_o[b, :n]
            want[b, n:] = b * rows + (kept_o[b, nk_o[b] - 1] if nk_o[b] > 0 else 0)
        got = ri.cpu().numpy()
        assert got[-1] == -7 and np.array_equal(got[:-1].reshape(Bn, out_rows), want)
        wc, ws = wl.weight_codes(38, 3, 72, K), wl.weight_scales(38, 3, 72)
        check_linear(x, wc, ws, rotate=True, row_index=want.reshape(-1).astype(np.int32), flags_list=[0])
        w = G.pack(wc, ws)
        a = G.quantize_linear(x, w, rotate=True, row_index=got[:-1])
        b_ = G.quantize_linear(np.ascontiguousarray(x[want.reshape(-1)]), w, rotate=True)
        assert np.array_equal(a, b_)
        w.close()


def test_prune_fps_worked_example():
    p = wl.prune_params(1, 256, 0, 256, 16, 16, 0, 0, 5)
    kept, nk, _ = G.prune(p, np.zeros((1, 256), np.float32))
    assert kept[0, :5].tolist() == [0, 15, 119, 240, 255]


@pytest.mark.parametrize("batch,rows,vs,nv,H,D", [(2, 40, 3, 24, 4, 32), (3, 288, 1, 256, 32, 128), (1, 70, 0, 64, 2, 8),
                                                  (1, 620, 4, 600, 2, 256),      # three key tiles, the longest head
                                                  (16, 300, 2, 288, 32, 32),     # 512 CTAs: half-size tiles, ragged
                                                  (15, 80, 0, 64, 32, 64)])
def test_attention_scores_bit_exact_and_feed_the_criterion(batch, rows, vs, nv, H, D):
    """sqap_attention_scores against the oracle (fp16 bits), then scores -> criterion on the device against the
    oracle's kept rows: quantizer output -> attention -> pruning without leaving the GPU."""
    ld = 3 * H * D
    qkv = (wl.activations(71, rows + D, batch * rows, ld, 0, 1.0).astype(np.float32) * np.float32(1.2)).astype(np.float16)
    qd = G.to_dev(qkv)
    sc = torch.empty(batch, H, nv, dtype=torch.float16, device="cuda")
    B.sqap_attention_scores(qd, ld, batch, rows, rows - 1, vs, nv, H, D, 0, H * D, sc)
    torch.cuda.synchronize()
    so = oracle.attention_scores(bits(qkv), batch, rows, rows - 1, vs, nv, H, D, 0, H * D)
    assert np.array_equal(sc.cpu().numpy().view(np.uint16), so)
    gw = int(round(math.sqrt(nv))) if int(round(math.sqrt(nv))) ** 2 == nv else nv
    p = wl.prune_params(batch, rows, vs, nv, gw, nv // gw, H, nv // 4, nv // 2, ring_radius=-1)
    kept = torch.empty(batch, rows, dtype=torch.int32, device="cuda")
    nk = torch.empty(batch, dtype=torch.int32, device="cuda")
    B.sqap_prune_tokens(p, sc, None, None, 0, 0, None, 0, 0, kept, nk)
    torch.cuda.synchronize()
    ko, no = oracle.prune_tokens(p, so, None)
    assert np.array_equal(nk.cpu().numpy(), no)
    for b in range(batch):
        assert np.array_equal(kept.cpu().numpy()[b, :no[b]], ko[b, :no[b]])


def test_prune_rejects_bad_arguments():
    L = B.lib()
    k = torch.zeros(64, dtype=torch.int32, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    s = torch.zeros(48, dtype=torch.float32, device="cuda")

    def call(**kw):
        d = wl.prune_params(1, 64, 0, 48, 8, 6, 0, 24, 24)
        d.update(kw)
        p = B.PruneParams(**d)
        import ctypes
        return L.sqap_prune_tokens(ctypes.byref(p), s.data_ptr(), None, None, 0, 0, None, 0, 0, k.data_ptr(),
                                   n.data_ptr(), None)

    assert call() == B.SQAP_OK
    assert call(grid_w=7) == B.SQAP_ERR_INVALID
    assert call(visual_start=20) == B.SQAP_ERR_INVALID
    assert call(k_attn=-1) == B.SQAP_ERR_INVALID
    assert call(n_visual=2048, rows=4096, grid_w=64, grid_h=32) == B.SQAP_ERR_UNSUPPORTED
    torch.cuda.synchronize()


# ------------------------------------------------------------------ the five configurations

def test_config0_prune_then_linear():
    c0 = wl.config0()
    kept, nk = check_prune(c0["prune"], c0["scores"], None, c0["x"], 40)
    assert nk[0] == 40
    idx = kept[0, :40]
    for rotate in (False, True):
        check_linear(c0["x"], c0["w_codes"], c0["w_scales"], rotate=rotate, row_index=idx)
        check_linear(c0["x"], c0["w_codes"], c0["w_scales"], rotate=rotate)


def test_config1_attention_projections():
    c1 = wl.config1()
    check_linear(c1["x"], c1["wqkv_codes"], c1["wqkv_scales"], rotate=True, flags_list=[0])
    check_linear(c1["x"], c1["wqkv_codes"], c1["wqkv_scales"], rotate=False, flags_list=[0])
    check_linear(c1["x_o"], c1["wo_codes"], c1["wo_scales"], flags_list=[0, B.SQAP_L_FORCE_SIMT])


def test_config2_pruned_mlp():
    c2 = wl.config2()
    kept, nk = check_prune(c2["prune"], c2["scores"], None, c2["x"], 160)
    assert nk[0] == 160
    xg = oracle.gather_rows(bits(c2["x"])[None], kept, nk, 160)[0].view(np.float16)
    # gate/up with the SiLU-gated product fused; the oracle's H then feeds the down projection on both sides
    h_bits = check_linear(xg, c2["wg_codes"], c2["wg_scales"], up=(c2["wu_codes"], c2["wu_scales"]), flags_list=[0])
    h = h_bits.view(np.float16)
    assert np.isfinite(h.astype(np.float32)).all()
    check_linear(h, c2["wd_codes"], c2["wd_scales"], flags_list=[0])


@pytest.mark.parametrize("layer,M", [(0, 288), (31, 160)])
def test_config3_one_layer_of_the_stack(layer, M):
    inp = wl.config3_inputs()
    lw = wl.config3_layer(layer)
    x = inp["x"]
    if M == 160:
        kept, nk = check_prune(inp["prune"], inp["scores"], None, x, 160)
        x = oracle.gather_rows(bits(x)[None], kept, nk, 160)[0].view(np.float16)
    qkv = check_linear(x, lw["qkv_codes"], lw["qkv_scales"], rotate=True, flags_list=[0]).view(np.float16)
    v = np.ascontiguousarray(qkv[:, 8192:])
    o = check_linear(v, lw["o_codes"], lw["o_scales"], flags_list=[0]).view(np.float16)
    h = check_linear(o, lw["gate_codes"], lw["gate_scales"], up=(lw["up_codes"], lw["up_scales"]),
                     flags_list=[0]).view(np.float16)
    d = check_linear(h, lw["down_codes"], lw["down_scales"], flags_list=[0]).view(np.float16)
    assert np.isfinite(d.astype(np.float32)).all() and np.abs(d.astype(np.float32)).max() > 0


def test_config3_decode_step_gemv():
    inp = wl.config3_inputs()
    lw = wl.config3_layer(1)
    x = inp["x_decode"][:1]
    qkv = check_linear(x, lw["qkv_codes"], lw["qkv_scales"], rotate=True, flags_list=[0]).view(np.float16)
    o = check_linear(np.ascontiguousarray(qkv[:, 8192:]), lw["o_codes"], lw["o_scales"], flags_list=[0]).view(np.float16)
    h = check_linear(o, lw["gate_codes"], lw["gate_scales"], up=(lw["up_codes"], lw["up_scales"]),
                     flags_list=[0]).view(np.float16)
    check_linear(h, lw["down_codes"], lw["down_scales"], flags_list=[0])


def _check_sampled(acc, out, codes, so, wc, ws, rng, M, N):
    """Whole sampled rows and columns and 512 single entries of a full-size GEMM against the oracle; returns the
    sampled row numbers and their oracle accumulators."""
    rows = np.unique(np.concatenate([[0, M - 1, 255, 256], rng.integers(0, M, 4)]))
    ref_rows = oracle.gemm_i32(codes[rows], wc)
    assert np.array_equal(acc[rows], ref_rows)
    assert G.within_tolerance(out[rows], oracle.epilogue(ref_rows, so[rows], bits(ws))).all()
    cols = np.unique(np.concatenate([[0, N - 1, 127, 128], rng.integers(0, N, 4)]))
    ref_cols = oracle.gemm_i32(codes, wc[cols])
    assert np.array_equal(acc[:, cols], ref_cols)
    for _ in range(512):
        m, n = int(rng.integers(0, M)), int(rng.integers(0, N))
        assert acc[m, n] == oracle.dot_i32(codes[m], wc[n])
    return rows, ref_rows


@pytest.mark.parametrize("keep", [64, 128, 192, 256])
def test_config4_batched_sampled(keep):
    """Full-size GEMMs (M = 1536, 2560, 3584, 4608; every shape of the layer, the down projection with its 11008
    codes per row included): accumulators checked on sampled entries and on whole sampled rows and columns."""
    Bn = 16
    inp = wl.config4_inputs()
    wts = wl.config4_weights()
    x = inp["x"].reshape(Bn * 288, 4096)
    if keep < 256:
        p = wl.prune_params(Bn, 288, 1, 256, 16, 16, 32, keep // 2, keep, ring_radius=1)
        kept, nk = check_prune(p, inp["scores"], inp["centers"], x, 32 + keep)
        xg = oracle.gather_rows(bits(inp["x"]), kept, nk, 32 + keep).reshape(Bn * (32 + keep), 4096).view(np.float16)
    else:
        xg = x
    M = xg.shape[0]
    po, so, codes = oracle.quantize_act(bits(xg), rotate=True)
    pg, sg = G.quantize(xg, rotate=True)
    assert np.array_equal(pg, po) and np.array_equal(sg, so)
    rng = np.random.default_rng(keep)
    for name in ("qkv", "gate", "o"):
        wc, ws = wts[name + "_codes"], wts[name + "_scales"]
        N = wc.shape[0]
        w = G.pack(wc, ws)
        acc = G.linear(pg, sg, w, out_dtype=B.SQAP_I32)
        out = G.linear(pg, sg, w)
        rows, ref_rows = _check_sampled(acc, out, codes, so, wc, ws, rng, M, N)
        if name == "gate":
            wu = G.pack(wts["up_codes"], wts["up_scales"])
            hs = G.linear(pg, sg, w, w_up=wu)
            ref_u = oracle.gemm_i32(codes[rows], wts["up_codes"])
            ref_h = oracle.epilogue_swiglu(ref_rows, ref_u, so[rows], bits(ws), bits(wts["up_scales"]))
            assert G.within_tolerance(hs[rows], ref_h).all()
            wu.close()
        w.close()
    # the down projection: rows of 11008 codes (43 pipeline stages of 256), fed by a stand-in for the gated MLP output
    del codes, po, pg
    xh = wl.activations(4, 900 + keep, M, wl.FFN, 110, 30.0)
    po, so, codes = oracle.quantize_act(bits(xh))
    pg, sg = G.quantize(xh)
    assert np.array_equal(pg, po) and np.array_equal(sg, so)
    wc, ws = wts["down_codes"], wts["down_scales"]
    w = G.pack(wc, ws)
    acc = G.linear(pg, sg, w, out_dtype=B.SQAP_I32)
    out = G.linear(pg, sg, w)
    _check_sampled(acc, out, codes, so, wc, ws, rng, M, wl.HIDDEN)
    assert np.array_equal(G.quantize_linear(xh, w), out)       # the one-call route the layer uses
    w.close()
