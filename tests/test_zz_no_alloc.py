"""The allocation-free linear (`sqap_w4a4_linear_static`) against the ordinary entry point.

Some callers of this library cannot allocate device memory at the moment they need a linear — they
sit inside a control loop with a hard deadline, have given all device memory to another component's
pool, or were handed a fixed memory budget by their host runtime — so they cannot provide the
workspace `sqap_w4a4_linear` wants.
For them the library carries its own fixed scratch array. This test calls that entry point through
the C ABI twice in a row (the second call finds the first call's leftovers in the scratch) and
requires the same bits as the ordinary entry point gives with a caller workspace.

Collected last on purpose: if it fails under `-x`, every other test has already run.
"""
import numpy as np
import pytest

import oracle
from paper_2509_09090_b200 import workloads as wl

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    from paper_2509_09090_b200 import binding as B
    import gpu_harness as G


def _run_static(pg, sg, w, w_up, out_dtype, flags=0):
    M, N = pg.shape[0], w.N
    qd, sd = G.to_dev(pg), G.to_dev(sg)
    tdt = torch.int32 if out_dtype == B.SQAP_I32 else torch.int16
    out = torch.zeros((M, N), dtype=tdt, device=G.DEV)
    B.sqap_w4a4_linear_static(qd, sd, M, w, w_up, out, N, out_dtype, flags)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    o = out.cpu().numpy()
    return o if out_dtype == B.SQAP_I32 else o.view(np.uint16)


def test_static_scratch_linear_matches_workspace_linear_twice_in_a_row():
    cases = [
        # (M, N, K, fused gate, output type): a tensor-core shape first, then a different shape that
        # reuses the scratch while it still holds the first call's data, then the few-row kernel.
        (288, 512, 4096, False, "i32"),
        (160, 384, 1024, True, "f16"),
        (1, 256, 11008, False, "f16"),
        (288, 512, 4096, False, "f16"),
    ]
    for M, N, K, fused, kind in cases:
        x = wl.activations(77, M + K, M, K, max(1, K // 100), 20.0)
        pg, sg = G.quantize(x)
        w = G.pack(wl.weight_codes(77, N + K, N, K), wl.weight_scales(77, N + K, N, mult=0.5))
        wu = G.pack(wl.weight_codes(77, N + K + 1, N, K), wl.weight_scales(77, N + K + 1, N, mult=0.5)) if fused else None
        dt = B.SQAP_I32 if kind == "i32" else B.SQAP_FP16
        want = G.linear(pg, sg, w, w_up=wu, out_dtype=dt)
        first = _run_static(pg, sg, w, wu, dt)
        second = _run_static(pg, sg, w, wu, dt)
        # same kernels, same inputs: the tolerance of the other tests (exact integers, fp16 within one ulp /
        # 2e-3) is met with room to spare — the bits are identical
        assert np.array_equal(first, want)
        assert np.array_equal(second, want)
        # and against the CPU oracle, so that a defect shared by both entry points cannot pass: exact integers,
        # fp16 within max(1 ulp, 2e-3 relative)
        _, so, codes = oracle.quantize_act(np.ascontiguousarray(x).view(np.uint16))
        wc, sw = wl.weight_codes(77, N + K, N, K), wl.weight_scales(77, N + K, N, mult=0.5).view(np.uint16)
        acc = oracle.gemm_i32(codes, wc)
        if kind == "i32":
            assert np.array_equal(second, acc)
        elif fused:
            acc_u = oracle.gemm_i32(codes, wl.weight_codes(77, N + K + 1, N, K))
            su = wl.weight_scales(77, N + K + 1, N, mult=0.5).view(np.uint16)
            assert G.within_tolerance(second, oracle.epilogue_swiglu(acc, acc_u, so, sw, su)).all()
        else:
            assert G.within_tolerance(second, oracle.epilogue(acc, so, sw)).all()
        w.close()
        if wu:
            wu.close()


def test_static_scratch_linear_rejects_what_does_not_fit():
    K, N = 4096, 128
    w = G.pack(wl.weight_codes(78, 1, N, K), wl.weight_scales(78, 1, N))
    L = B.lib()
    M_big = B.SQAP_STATIC_WORKSPACE_BYTES // K + 8
    assert B.sqap_workspace_bytes(M_big, N, K) > B.SQAP_STATIC_WORKSPACE_BYTES
    q = torch.zeros(M_big * K // 2, dtype=torch.uint8, device=G.DEV)
    s = torch.ones(M_big, dtype=torch.float32, device=G.DEV)
    out = torch.zeros(M_big * N, dtype=torch.float16, device=G.DEV)
    before = B.sqap_kernel_launch_count()
    st = L.sqap_w4a4_linear_static(q.data_ptr(), s.data_ptr(), M_big, w.handle, None, out.data_ptr(), N, B.SQAP_FP16,
                                   0, None)
    assert st == B.SQAP_ERR_TOO_LARGE
    assert B.sqap_kernel_launch_count() == before
    st = L.sqap_w4a4_linear_static(q.data_ptr(), s.data_ptr(), 16, w.handle, None, out.data_ptr(), N, B.SQAP_FP16,
                                   B.SQAP_L_REUSE_EXPANDED, None)
    assert st == B.SQAP_ERR_INVALID
    w.close()
