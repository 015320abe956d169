"""The whole 32-layer stack of the fourth workload configuration, run the way the bench times it (every launch of
the prefill and of the seven decode steps captured into one CUDA graph and replayed), against the CPU oracle.

Every linear of every layer is checked on the input it actually received: the oracle is applied to the device's own
input of that stage (for the first linear of a layer the token matrix, afterwards the device's previous output), so
a one-ulp difference in one stage cannot hide or fake a difference in the next. Kept indices and gathered rows are
bit-exact; fp16 outputs within max(1 ulp, 2e-3 relative).
"""
import numpy as np
import pytest

import oracle
from paper_2509_09090_b200 import workloads as wl

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if torch.cuda.is_available():
    from paper_2509_09090_b200 import binding as B
    from paper_2509_09090_b200.stack import Stack
    import gpu_harness as G


def bits(a):
    return np.ascontiguousarray(a).view(np.uint16)


def _oracle_linear(x_bits, lw, name, rotate=False, up=None):
    _, s, codes = oracle.quantize_act(np.ascontiguousarray(x_bits), rotate=rotate)
    acc = oracle.gemm_i32(codes, lw[name + "_codes"])
    sw = bits(lw[name + "_scales"])
    if up is None:
        return oracle.epilogue(acc, s, sw)
    acc_u = oracle.gemm_i32(codes, lw[up + "_codes"])
    return oracle.epilogue_swiglu(acc, acc_u, s, sw, bits(lw[up + "_scales"]))


def _check_layer(lw, x_bits, qkv, o, h, d, where):
    """qkv, o, h, d: the device's outputs (uint16 bits) for the rows of x_bits."""
    H = wl.HIDDEN
    for name, got, ref in (
            ("qkv", qkv, _oracle_linear(x_bits, lw, "qkv", rotate=True)),
            ("o", o, _oracle_linear(qkv[:, 2 * H:], lw, "o")),
            ("gate/up", h, _oracle_linear(o, lw, "gate", up="up")),
            ("down", d, _oracle_linear(h, lw, "down"))):
        ok = G.within_tolerance(got, ref)
        assert ok.all(), f"{where}, {name}: {(~ok).sum()} of {ok.size} outputs outside tolerance"


def test_config3_whole_stack_prefill_prune_decode_replayed_from_one_graph():
    import psutil
    n_layers, n_dec = wl.N_LAYERS, 7
    keep, k_attn, radius = 128, 64, 1
    inp = wl.config3_inputs()
    keep_host = psutil.virtual_memory().available > 24 * 2 ** 30     # 6.5 GB of codes; else regenerate per layer
    layers, host = [], []
    for li in range(n_layers):
        lw = wl.config3_layer(li)
        layers.append({name: G.pack(lw[name + "_codes"], lw[name + "_scales"]) for name, _, _ in wl.LAYER_LINEARS})
        host.append(lw if keep_host else None)
        del lw
    st = Stack(torch, B, G.DEV, layers, keep=keep, k_attn=k_attn, ring_radius=radius, n_decode=n_dec,
               keep_intermediates=True)
    x, scores = G.to_dev(inp["x"]), G.to_dev(inp["scores"])
    centers_np = np.array([[5, 9]], np.int32)
    centers = G.to_dev(centers_np)
    xdec = G.to_dev(inp["x_decode"])

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        st.prefill(x, scores, centers)      # eager once (first-call set-up happens outside the capture)
        st.decode(xdec)
        side.synchronize()
        for buf in (st.qkv, st.o, st.h, st.d, st.qkv_dec, st.o_dec, st.h_dec, st.d_dec):
            buf.view(torch.int16).fill_(0x7B7B)              # only what the replay writes may pass the check
        st.kept.fill_(-9)
        st.row_index.fill_(-9)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            st.prefill(x, scores, centers)
            st.decode(xdec)
        graph.replay()
        side.synchronize()
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK

    # the pruning criterion and the compaction
    p = st.prune_params
    kept_o, nk_o = oracle.prune_tokens(p, bits(inp["scores"]), centers_np)
    assert int(st.nkept.cpu()[0]) == int(nk_o[0]) == st.rows_kept
    assert np.array_equal(st.kept.cpu().numpy(), kept_o)
    # the pruned layers read the kept rows of x in place: the row list must name exactly the oracle's kept rows
    assert np.array_equal(st.row_index.cpu().numpy(), kept_o[0, :st.rows_kept])
    x1_o = oracle.gather_rows(bits(inp["x"])[None], kept_o, nk_o, st.rows_kept)[0]

    xd_bits = bits(inp["x_decode"])
    for li in range(n_layers):
        lw = host[li] if keep_host else wl.config3_layer(li)
        M = wl.ROWS if li < st.prune_after else st.rows_kept
        xin = bits(inp["x"]) if li < st.prune_after else x1_o
        get = lambda t: bits(t[li, :M].cpu().numpy())
        _check_layer(lw, xin, get(st.qkv), get(st.o), get(st.h), get(st.d), f"prefill layer {li} (M={M})")
        # the seven decode tokens of this layer, as seven rows (rows are independent)
        idx = torch.arange(n_dec, device=G.DEV) * n_layers + li
        dec = lambda t: bits(t[idx, 0].cpu().numpy())
        _check_layer(lw, xd_bits, dec(st.qkv_dec), dec(st.o_dec), dec(st.h_dec),
                     bits(st.d_dec[:, li, 0].cpu().numpy()), f"decode, layer {li}")
        host[li] = None
    for L in layers:
        for w in L.values():
            w.close()
