#!/usr/bin/env python
"""Bench of the SQAP-VLA hot path on B200: W4A4 linears of a Llama-2-7B-style layer on a batch of
observations, with the quantization-aware visual-token pruning between two layers.

One step (per rank, 16 observations x 288 token rows = 4608 rows, configuration 4 of the workload):
  layer A at M = 4608 : quantize(+Hadamard) -> QKV -> quantize -> O -> quantize -> gate/up (SwiGLU) -> quantize -> down
  prune               : scores -> top-k U ring U FPS -> compaction (256 -> 128 visual tokens); the kept rows leave
                        as a source-row list, so the gather is folded into layer B's first quantizer
  layer B at M = 2560 : the same four linears on the surviving rows (distinct weights)
  decode              : one new token per observation (M = 16) through layer B's linears
`value` = algorithmic tera-ops (2*M*N*K of every linear) per second of whole-step time, all ranks.

Usage: python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_09090_b200 import workloads as wl  # noqa: E402
from paper_2509_09090_b200 import dist_utils as du  # noqa: E402

N_OBS = 16
KEEP = 128
K_ATTN = 64
RING_RADIUS = 1
M_FULL = N_OBS * wl.ROWS
ROWS_KEPT = 32 + KEEP
M_PRUNED = N_OBS * ROWS_KEPT
METRIC = "W4A4 linear TOPS (whole pruned-prefill step); tokens/s beside it"
WORKLOAD = ("configs[4]: 16 observations x 288 tokens (4608 rows), Llama-2-7B QKV/O/gate-up/down W4A4, "
            "prune 256->128 visual tokens (top-k 64 U ring R_t=1 U FPS), pruned layer at 2560 rows, decode at 16 rows")


def layer_ops(M: int) -> float:
    H, F = wl.HIDDEN, wl.FFN
    return 2.0 * M * (H * 3 * H + H * H + 2 * H * F + F * H)


STEP_OPS = layer_ops(M_FULL) + layer_ops(M_PRUNED) + layer_ops(N_OBS)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return dict(hbm_gbs=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(np.max(mx)), reasons=sorted(reasons),
                    samples=len(sm))


# ----------------------------------------------------------------------------------------- our arm

class Layer:
    def __init__(self, B, G_pack, weights: dict):
        self.w = {}
        for name, N, K in wl.LAYER_LINEARS:
            self.w[name] = G_pack(weights[name + "_codes"], weights[name + "_scales"], N, K)


class Path:
    """Device state of one rank and the step function (all work goes through the C ABI)."""

    def __init__(self, torch, B, device, seed: int, keep_host_weights: bool = False):
        self.torch, self.B, self.dev = torch, B, device
        t = torch
        inp = wl.config4_inputs(seed=seed, batch=N_OBS)
        self.inputs_host = inp
        self.x_host = t.from_numpy(inp["x"].reshape(M_FULL, wl.HIDDEN)).pin_memory()
        self.scores_host = t.from_numpy(inp["scores"]).pin_memory()
        self.centers_host = t.from_numpy(inp["centers"]).pin_memory()
        self.xdec_host = t.from_numpy(wl.activations(seed, wl.T_X2, N_OBS, wl.HIDDEN, 41, 30.0)).pin_memory()
        on_dev = lambda h: t.empty(h.shape, dtype=h.dtype, device=device)
        self.x, self.scores = on_dev(self.x_host), on_dev(self.scores_host)
        self.centers, self.xdec = on_dev(self.centers_host), on_dev(self.xdec_host)

        def pack(codes, scales, N, K):
            return B.sqap_pack_weights(np.ascontiguousarray(codes), np.ascontiguousarray(scales), N, K)

        self.layers = []
        self.host_weights_b = None      # layer B's codes and scales stay on the host for the untimed oracle check
        for li in range(2):
            wts = wl.config4_weights(seed=seed + 100 * li)
            self.layers.append(Layer(B, pack, wts))
            if li == 1 and keep_host_weights:
                self.host_weights_b = wts
            del wts
        M = M_FULL
        f16, u8, f32, i32 = t.float16, t.uint8, t.float32, t.int32
        self.q = t.empty(M * wl.FFN // 2, dtype=u8, device=device)
        self.sx = t.empty(M, dtype=f32, device=device)
        self.qkv = t.empty(M, wl.QKV, dtype=f16, device=device)
        self.o = t.empty(M, wl.HIDDEN, dtype=f16, device=device)
        self.h = t.empty(M, wl.FFN, dtype=f16, device=device)
        self.d = t.empty(M, wl.HIDDEN, dtype=f16, device=device)
        self.x1 = t.empty(M_PRUNED, wl.HIDDEN, dtype=f16, device=device)   # only for timing the gather kernel alone
        self.d1 = t.empty(M_PRUNED, wl.HIDDEN, dtype=f16, device=device)
        self.ddec = t.empty(N_OBS, wl.HIDDEN, dtype=f16, device=device)
        self.kept = t.empty(N_OBS, wl.ROWS, dtype=i32, device=device)
        self.row_index = t.empty(M_PRUNED, dtype=i32, device=device)
        self.nkept = t.empty(N_OBS, dtype=i32, device=device)
        self.ws_bytes = B.sqap_quantize_linear_workspace_bytes(M, wl.QKV, wl.FFN)
        self.ws = t.empty(self.ws_bytes, dtype=u8, device=device)
        assert self.ws.data_ptr() % 256 == 0
        self.prune_params = wl.prune_params(N_OBS, wl.ROWS, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32,
                                            K_ATTN, KEEP, ring_radius=RING_RADIUS)
        self.d1_host = t.empty(M_PRUNED, wl.HIDDEN, dtype=f16).pin_memory()
        self.ddec_host = t.empty(N_OBS, wl.HIDDEN, dtype=f16).pin_memory()
        self.kept_host = t.empty(N_OBS, wl.ROWS, dtype=i32).pin_memory()
        self.h2d_bytes = sum(v.numel() * v.element_size() for v in
                             (self.x_host, self.scores_host, self.centers_host, self.xdec_host))
        self.d2h_bytes = sum(v.numel() * v.element_size() for v in (self.d1_host, self.ddec_host, self.kept_host))
        self.gemm_events = []
        self.overlap_prune = True
        self.side = t.cuda.Stream(device=device)
        self.ev_fork, self.ev_join = t.cuda.Event(), t.cuda.Event()
        # second set of input / output device buffers: the end-to-end loop uploads step i+1 and downloads step i-1
        # while step i computes (intermediate buffers are shared: the compute stream runs the steps in order)
        self.io = [dict(x=self.x, scores=self.scores, centers=self.centers, xdec=self.xdec, d1=self.d1, ddec=self.ddec,
                        kept=self.kept)]
        self.io.append({k: t.empty_like(v) for k, v in self.io[0].items()})

    def linear(self, x_ptr, M, K, ldx, w, w_up, out, rotate=False, flags=0, row_index=None):
        B = self.B
        B.sqap_quantize_linear(x_ptr, M, ldx, row_index, B.SQAP_Q_ROTATE if rotate else 0, w, w_up, out, out.shape[1],
                               B.SQAP_FP16, flags, self.ws, self.ws_bytes)

    def layer(self, x, M, L: Layer, d_out, row_index=None):
        H = wl.HIDDEN
        self.linear(x.data_ptr(), M, H, H, L.w["qkv"], None, self.qkv, rotate=True, row_index=row_index)
        self.linear(self.qkv.data_ptr() + 2 * 2 * H, M, H, wl.QKV, L.w["o"], None, self.o)   # V third of QKV
        self.linear(self.o.data_ptr(), M, H, H, L.w["gate"], L.w["up"], self.h)
        self.linear(self.h.data_ptr(), M, wl.FFN, wl.FFN, L.w["down"], None, d_out)

    def step(self, k: int = 0):
        B, io, t = self.B, self.io[k], self.torch
        H, L = wl.HIDDEN, self.layers[0]
        # Layer A. The pruning criterion needs only the attention scores, which a model has once the layer's attention
        # is done, so it does not have to wait for the layer's last linears: it is issued on a second stream after the
        # gate / up projection and runs (16 small CTAs, latency-bound) beside the down projection's quantizer; layer B
        # waits for both. It writes the kept rows as a source-row list, which layer B's first quantizer reads in place.
        self.linear(io["x"].data_ptr(), M_FULL, H, H, L.w["qkv"], None, self.qkv, rotate=True)
        self.linear(self.qkv.data_ptr() + 2 * 2 * H, M_FULL, H, wl.QKV, L.w["o"], None, self.o)   # V third of QKV
        self.linear(self.o.data_ptr(), M_FULL, H, H, L.w["gate"], L.w["up"], self.h)
        main = t.cuda.current_stream()
        if self.overlap_prune:
            self.ev_fork.record(main)
            self.side.wait_event(self.ev_fork)
            with t.cuda.stream(self.side):
                B.sqap_prune_select(self.prune_params, io["scores"], io["centers"], ROWS_KEPT, io["kept"], self.nkept,
                                    self.row_index)
                self.ev_join.record(self.side)
        self.linear(self.h.data_ptr(), M_FULL, wl.FFN, wl.FFN, L.w["down"], None, self.d)
        if self.overlap_prune:
            main.wait_event(self.ev_join)
        else:
            B.sqap_prune_select(self.prune_params, io["scores"], io["centers"], ROWS_KEPT, io["kept"], self.nkept,
                                self.row_index)
        self.layer(io["x"], M_PRUNED, self.layers[1], io["d1"], row_index=self.row_index)
        self.layer(io["xdec"], N_OBS, self.layers[1], io["ddec"])

    def upload(self, k: int = 0):
        io = self.io[k]
        io["x"].copy_(self.x_host, non_blocking=True)
        io["scores"].copy_(self.scores_host, non_blocking=True)
        io["centers"].copy_(self.centers_host, non_blocking=True)
        io["xdec"].copy_(self.xdec_host, non_blocking=True)

    def download(self, k: int = 0):
        io = self.io[k]
        self.d1_host.copy_(io["d1"], non_blocking=True)
        self.ddec_host.copy_(io["ddec"], non_blocking=True)
        self.kept_host.copy_(io["kept"], non_blocking=True)


def time_region(torch, fn, steps: int, world: int):
    du.barrier(world)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    du.barrier(world)
    ms = e0.elapsed_time(e1)
    return du.max_over_ranks(ms, world, device="cuda")


def _within_tolerance(got_bits, ref_bits):
    """fp16: |got - ref| <= max(1 ulp at ref, 2e-3 |ref|), elementwise."""
    g = got_bits.view(np.float16).astype(np.float64)
    r = ref_bits.view(np.float16).astype(np.float64)
    ulp = np.spacing(np.abs(ref_bits.view(np.float16))).astype(np.float64)
    return np.isfinite(r) & (np.abs(g - r) <= np.maximum(ulp, 2e-3 * np.abs(r)))


def check_step_against_oracle(torch, path: Path, step_fn):
    """Untimed. Replays the timed step once more and compares what it left on the device with the CPU oracle:
    the kept-token indices of every observation and their source-row list (bit-exact), and, for sampled token
    rows of the pruned layer and of the decode step, every linear of the chain on the input it actually received
    (the oracle applied to the device's own input of that stage), fp16 within max(1 ulp, 2e-3)."""
    import oracle
    oracle.build()
    t = torch
    step_fn()
    t.cuda.synchronize()
    inp, wts = path.inputs_host, path.host_weights_b
    bits = lambda a: np.ascontiguousarray(a).view(np.uint16)
    kept = path.io[0]["kept"].cpu().numpy()
    kept_o, nk_o = oracle.prune_tokens(path.prune_params, bits(inp["scores"]), inp["centers"])
    if not (np.array_equal(kept, kept_o) and np.array_equal(path.nkept.cpu().numpy(), nk_o)):
        return False, "kept indices differ from the oracle"
    want_rows = (np.arange(N_OBS)[:, None] * wl.ROWS + kept_o[:, :ROWS_KEPT]).reshape(-1)
    if not ((nk_o == ROWS_KEPT).all() and np.array_equal(path.row_index.cpu().numpy(), want_rows)):
        return False, "the kept rows' source-row list differs from the oracle"
    x1_o = oracle.gather_rows(bits(inp["x"]), kept_o, nk_o, ROWS_KEPT).reshape(M_PRUNED, wl.HIDDEN)

    def lin(x_bits, name, rotate=False, up=None):
        _, s, codes = oracle.quantize_act(np.ascontiguousarray(x_bits), rotate=rotate)
        acc = oracle.gemm_i32(codes, wts[name + "_codes"])
        sw = bits(wts[name + "_scales"])
        if up is None:
            return oracle.epilogue(acc, s, sw)
        return oracle.epilogue_swiglu(acc, oracle.gemm_i32(codes, wts[up + "_codes"]), s, sw, bits(wts[up + "_scales"]))

    H = wl.HIDDEN
    rng = np.random.default_rng(7)
    # rows 0..15 of the shared qkv / o / h buffers hold the decode step (it ran last), the rest the pruned layer
    rows_b = np.unique(np.concatenate([[N_OBS, M_PRUNED - 1], rng.integers(N_OBS, M_PRUNED, 4)]))
    rows_d = np.arange(0, N_OBS, 5)
    for rows, x_in, d_out, what in ((rows_b, x1_o, path.io[0]["d1"], "pruned layer"),
                                    (rows_d, bits(path.xdec_host.numpy()), path.io[0]["ddec"], "decode")):
        idx = t.from_numpy(rows).to(path.dev)
        get = lambda buf: bits(buf[idx].cpu().numpy())
        qkv, o, h, d = get(path.qkv), get(path.o), get(path.h), get(d_out)
        for name, got, ref in (("qkv", qkv, lin(x_in[rows], "qkv", rotate=True)), ("o", o, lin(qkv[:, 2 * H:], "o")),
                               ("gate/up", h, lin(o, "gate", up="up")), ("down", d, lin(h, "down"))):
            ok = _within_tolerance(got, ref)
            if not ok.all():
                return False, f"{what}, {name}: {int((~ok).sum())} of {ok.size} sampled outputs outside tolerance"
    return True, (f"kept indices and source-row list of {N_OBS} observations bit-exact; {len(rows_b)} rows of the pruned layer and "
                  f"{len(rows_d)} decode rows through all four linears within max(1 ulp, 2e-3) of the oracle")


def dominant_gemm_roofline(torch, B, path: Path, steps: int, peaks: dict):
    """The QKV GEMM at M = 4608 (largest single launch), timed alone with CUDA events on its stream.
    The expand pass is skipped (SQAP_L_REUSE_EXPANDED), so the events bracket GEMM launches only."""
    L0, L1 = path.layers
    M, N, K = M_FULL, wl.QKV, wl.HIDDEN
    B.sqap_quantize_act(path.x, M, K, K, None, B.SQAP_Q_ROTATE, path.q, path.sx)
    B.sqap_w4a4_linear(path.q, path.sx, M, L0.w["qkv"], None, path.qkv, N, B.SQAP_FP16, 0, path.ws, path.ws_bytes)
    ws = [L0.w["qkv"], L1.w["qkv"]]
    for i in range(3):
        B.sqap_w4a4_linear(path.q, path.sx, M, ws[i % 2], None, path.qkv, N, B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED,
                           path.ws, path.ws_bytes)
    torch.cuda.synchronize()
    # `reps` launches back to back on one stream (captured once, replayed), CUDA events around the run on that
    # stream: the average duration of a launch without the host's submission gaps between eager launches
    reps = max(8, min(steps, 32))
    ms = graph_time_us(torch, lambda i: B.sqap_w4a4_linear(path.q, path.sx, M, ws[i % 2], None, path.qkv, N, B.SQAP_FP16,
                                                           B.SQAP_L_REUSE_EXPANDED, path.ws, path.ws_bytes),
                       reps=reps) * 1e-3
    ops = 2.0 * M * N * K
    achieved = ops / (ms * 1e-3) / 1e12
    peak = 2.0 * peaks["bf16"]       # int8 dense = 2 x bf16 dense (nominal ratio) x the measured bf16 burst figure
    traffic, traffic_src = profile_traffic("w4a4_tc_pair_kernel_qkv_m4608.md")
    return dict(bound="tensor", kernel="w4a4_tc_pair_kernel: W4A4 linear GEMM, M=4608 N=12288 K=4096 (int8 MMA on CTA "
                                       "pairs, int32 accumulate in tensor memory)",
                achieved=achieved, peak=peak, unit="TOP/s", frac=achieved / peak, traffic=traffic,
                traffic_source=traffic_src, algorithmic_bytes=N * K // 2 + M * K + 2 * M * N,
                peak_source=f"2 x bf16 cuBLAS burst ({peaks['source']}); a power-capped library run, not a ceiling",
                frac_of_nominal_int8=achieved / NOMINAL_INT8_TOPS, nominal_int8_tops=NOMINAL_INT8_TOPS,
                ms_per_launch=ms)


NOMINAL_INT8_TOPS = 4500.0      # B200 dense int8, nominal
INT8_MAC_PER_CLK_SM = 8192      # what one SM's tensor pipe retires (measured: 128 cycles per 128x256x32 MMA)


def pipe_peak_tops(sm_mhz, sms=148):
    """int8 tensor-pipe ceiling at a given SM clock: 8192 MAC per clock and SM."""
    return 2.0 * INT8_MAC_PER_CLK_SM * sms * sm_mhz * 1e6 / 1e12


def profile_traffic(name):
    """dram__bytes_read.sum + dram__bytes_write.sum of launch 0 from an ncu summary under profiles/ (bytes), or
    (None, reason) when the file or the counters are missing."""
    import re
    path = os.path.join(ROOT, "profiles", name)
    try:
        text = open(path).read()
    except OSError:
        return None, "no ncu summary for this kernel"
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    tot = 0.0
    for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(r"`" + re.escape(key) + r"`\)\s*\|\s*([0-9.]+)\s*([KMG]?byte)", text)
        if not m:
            return None, "counters not found in profiles/" + name
        tot += float(m.group(1)) * unit[m.group(2)]
    return tot, "profiles/" + name + " (launch 0)"


def hbm_kernel_rooflines(torch, B, path: Path, peaks: dict):
    """The HBM-bound kernels of the step, each timed alone (CUDA-graph replays over buffers rotating through more
    than the L2 capacity): algorithmic bytes / time / measured HBM copy bandwidth."""
    t, dev = torch, path.dev
    H = wl.HIDDEN
    hbm = peaks["hbm_gbs"]
    out = []
    gen = t.Generator(device=dev)
    gen.manual_seed(99)

    def add(kernel, nbytes, us):
        ach = nbytes / (us * 1e-6) / 1e9
        out.append(dict(kernel=kernel, bound="hbm", bytes=nbytes, us=us, achieved=ach, peak=hbm, unit="GB/s", frac=ach / hbm))

    n = 5                                               # 5 x 37.7 MB of activations > L2
    xs = [t.randn(M_FULL, H, device=dev, generator=gen).to(t.float16) for _ in range(n)]
    for rot in (False, True):
        fl = B.SQAP_Q_ROTATE if rot else 0
        us = graph_time_us(t, lambda i: B.sqap_quantize_act(xs[i % n], M_FULL, H, H, None, fl, path.q, path.sx), reps=10)
        add("quantize_act" + (" + Hadamard" if rot else "") + f", M={M_FULL} K={H}", M_FULL * H * 2.5 + 4 * M_FULL, us)
    p = path.prune_params
    io = path.io[0]
    us_sel = graph_time_us(t, lambda i: B.sqap_prune_tokens(p, io["scores"], io["centers"], None, 0, 0, None, 0, 0,
                                                            io["kept"], path.nkept), reps=8)
    us_all = graph_time_us(t, lambda i: B.sqap_prune_tokens(p, io["scores"], io["centers"], xs[i % n], H, H, path.x1, H,
                                                            ROWS_KEPT, io["kept"], path.nkept), reps=10)
    add(f"gather_rows, {N_OBS} x {ROWS_KEPT} rows x {H} (prune call minus its selection kernel)", 2 * M_PRUNED * H * 2,
        max(us_all - us_sel, 1e-3))
    out.append(dict(kernel="prune_select (top-k U ring U FPS, compaction)", bound="latency", us=us_sel,
                    note="serial farthest-point steps; no bandwidth fraction applies"))
    del xs
    # the M = 16 weight streamer on the QKV shape, over more weight matrices than the L2 holds
    codes = t.randint(-8, 8, (wl.QKV, H), dtype=t.int8, device=dev, generator=gen)
    scales = (t.rand(wl.QKV, device=dev, generator=gen) * 0.015 + 0.005).to(t.float16)
    ws = [B.sqap_pack_weights(codes, scales, wl.QKV, H) for _ in range(7)]
    t.cuda.synchronize()
    del codes
    sc_ptr = path.ws.data_ptr() + B.sqap_workspace_bytes(N_OBS, wl.QKV, H)
    B.sqap_quantize_linear(path.xdec, N_OBS, H, None, 0, ws[0], None, path.qkv, wl.QKV, B.SQAP_FP16, 0, path.ws, path.ws_bytes)
    us = graph_time_us(t, lambda i: B.sqap_w4a4_linear(path.ws, sc_ptr, N_OBS, ws[i % 7], None, path.qkv, wl.QKV, B.SQAP_FP16,
                                                       B.SQAP_L_REUSE_EXPANDED, path.ws, path.ws_bytes), reps=14)
    add(f"w4a4_mma_kernel (weight streamer), M={N_OBS} N={wl.QKV} K={H}", wl.QKV * H // 2 + N_OBS * H + 2 * N_OBS * wl.QKV, us)
    for w in ws:
        w.close()
    return out


def cpu_baseline(seconds_budget: float = 15.0):
    """The oracle, as it stands, on the host cores: a bounded sample of the same step (whole observations through
    layer A's four linears plus the pruning criterion of those observations), sized to about seconds_budget."""
    import oracle
    oracle.build()
    wts = wl.config4_weights(seed=4)
    x = wl.config4_inputs(seed=4, batch=N_OBS)
    t0 = time.perf_counter()
    probe = 96    # enough rows to occupy every host thread, as the sample itself does
    _oracle_layer(oracle, x["x"][0, :probe], wts)
    per_row = (time.perf_counter() - t0) / probe
    n_obs = int(max(1, min(N_OBS, seconds_budget / max(per_row * wl.ROWS, 1e-3))))
    rows = n_obs * wl.ROWS
    xs = x["x"][:n_obs].reshape(rows, wl.HIDDEN)
    p = wl.prune_params(n_obs, wl.ROWS, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32, K_ATTN, KEEP,
                        ring_radius=RING_RADIUS)
    t0 = time.perf_counter()
    _oracle_layer(oracle, xs, wts)
    oracle.prune_tokens(p, x["scores"][:n_obs].view(np.uint16), x["centers"][:n_obs])
    dt = time.perf_counter() - t0
    ops = layer_ops(rows)
    return dict(value=ops / dt / 1e12, unit="TOPS", cores=oracle.num_threads(), kind="oracle",
                sample=f"{n_obs} observations ({rows} token rows) through one layer's four W4A4 linears + the pruning "
                       f"criterion of those observations ({dt:.1f} s)", tokens_per_s=rows / dt)


def _oracle_layer(oracle, x_f16, wts):
    def lin(xin, name, rotate=False, up=None):
        _, s, codes = oracle.quantize_act(np.ascontiguousarray(xin).view(np.uint16), rotate=rotate)
        acc = oracle.gemm_i32(codes, wts[name + "_codes"])
        sw = wts[name + "_scales"].view(np.uint16)
        if up is None:
            return oracle.epilogue(acc, s, sw).view(np.float16)
        acc_u = oracle.gemm_i32(codes, wts[up + "_codes"])
        return oracle.epilogue_swiglu(acc, acc_u, s, sw, wts[up + "_scales"].view(np.uint16)).view(np.float16)

    qkv = lin(x_f16, "qkv", rotate=True)
    o = lin(qkv[:, 2 * wl.HIDDEN:], "o")
    h = lin(o, "gate", up="up")
    return lin(h, "down")


def run_ours(args):
    import torch
    from paper_2509_09090_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product path has no CPU fallback")
    rank, local_rank, world = du.init("nccl") if args.gpus > 1 else (0, 0, 1)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    B.lib()
    peaks = measured_peaks()
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    path = Path(torch, B, device, seed=4 + 1000 * rank, keep_host_weights=(rank == 0 and not args.no_parity_check))
    path.overlap_prune = not args.serial_prune
    path.upload()
    torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        path.step()
    torch.cuda.synchronize()
    if B.sqap_device_status() != B.SQAP_OK:
        raise SystemExit("bench.py: a kernel reported an expired bounded wait")

    # The step's launches are recorded once into a CUDA graph and replayed: the same kernels, arguments and
    # order as the eager calls above, without a host round trip per launch (--no-graph times the eager calls).
    l0 = B.sqap_kernel_launch_count()
    if args.no_graph:
        step_fn = path.step
        path.step()
    else:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            path.step()
        step_fn = graph.replay
    launches_per_step = B.sqap_kernel_launch_count() - l0
    for _ in range(3):
        step_fn()
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms = time_region(torch, step_fn, args.steps, world)
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if rank == 0 else None

    # End to end: every step uploads its inputs from pinned host memory and downloads its results; the copies run on
    # their own streams, double-buffered, so step i+1's upload and step i-1's download overlap step i's kernels.
    if args.no_graph:
        step_k = [lambda: path.step(0), lambda: path.step(1)]
    else:
        graph1 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph1):
            path.step(1)
        step_k = [graph.replay, graph1.replay]
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ev_up = [torch.cuda.Event(), torch.cuda.Event()]
    ev_cmp = [torch.cuda.Event(), torch.cuda.Event()]
    ev_down = [torch.cuda.Event(), torch.cuda.Event()]
    e2e_i = [0]

    def e2e_step():
        k = e2e_i[0] & 1
        e2e_i[0] += 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_cmp[k])      # the step that last read this input set is done
            path.upload(k)
            ev_up[k].record(s_in)
        s_cmp.wait_event(ev_up[k])
        s_cmp.wait_event(ev_down[k])        # the download that last read this output set is done
        step_k[k]()
        ev_cmp[k].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[k])
            path.download(k)
            ev_down[k].record(s_out)

    def e2e_region():
        for _ in range(args.steps):
            e2e_step()
        s_cmp.wait_stream(s_in)
        s_cmp.wait_stream(s_out)            # the timed region ends when the last download has landed

    for _ in range(4):
        e2e_step()
    torch.cuda.synchronize()
    ms_e2e = time_region(torch, e2e_region, 1, world)
    # A second, long timed region of the same replayed step: what the step does over seconds, under the power cap
    # (the regime the sustained library figure describes). It does not change `value`.
    sus_steps = int(min(max(np.ceil(args.sustain_s * 1e3 / (ms / args.steps)), 1), 20000)) if args.sustain_s > 0 else 0
    sus = None
    if sus_steps:
        sampler2 = ClockSampler(local_rank)
        if rank == 0:
            sampler2.start()
        ms_sus = time_region(torch, step_fn, sus_steps, world)
        clocks_sus = sampler2.stop() if rank == 0 else None
        sus = (ms_sus, sus_steps, clocks_sus)
    roof = dominant_gemm_roofline(torch, B, path, max(args.steps, 10), peaks) if rank == 0 else None
    roof_hbm = hbm_kernel_rooflines(torch, B, path, peaks) if rank == 0 else None
    if B.sqap_device_status() != B.SQAP_OK:
        raise SystemExit("bench.py: a kernel reported an expired bounded wait")
    parity = None
    if rank == 0 and not args.no_parity_check:
        ok, what = check_step_against_oracle(torch, path, step_fn)
        if not ok:
            raise SystemExit("bench.py: the timed step does not match the CPU oracle: " + what)
        parity = what

    ms_step = ms / args.steps
    tops = world * STEP_OPS / (ms_step * 1e-3) / 1e12
    tops_e2e = world * STEP_OPS / (ms_e2e / args.steps * 1e-3) / 1e12
    if rank == 0:
        cpu = cpu_baseline() if world == 1 and not args.no_cpu_baseline else None
        line = {
            "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x int8 -> int32 (INT4 codes), fp32 epilogue, fp16 out",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "observations_per_gpu": N_OBS, "rows_per_observation": wl.ROWS,
                       "keep_visual": KEEP, "l2": "inputs larger than L2 (202 MB packed weights, 38 MB activations, "
                                                  "113 MB QKV output per step)"},
            "tokens_per_s": world * M_FULL / (ms_step * 1e-3),
            "e2e": {"value": tops_e2e, "unit": "TOPS", "h2d_bytes_per_step": path.h2d_bytes,
                    "d2h_bytes_per_step": path.d2h_bytes, "tokens_per_s": world * M_FULL / (ms_e2e / args.steps * 1e-3),
                    "copies": "every step's H2D and D2H run inside the timed region, on their own streams, double-"
                              "buffered against the kernels of the neighbouring steps"},
            "gpu_launches": int(launches), "launch_mode": "eager" if args.no_graph else "cuda_graph replay",
            "clocks": clocks,
            "roofline": roof,
            "roofline_hbm": roof_hbm,
            "cpu_baseline": cpu,
            "parity_checked": parity is not None, "parity": parity,
        }
        mhz = clocks.get("sm_mhz") if clocks else None
        if mhz:
            # the tensor pipe itself, at the clock the timed region ran at (8192 int8 MAC per clock and SM)
            line["ms_x_mhz"] = ms_step * mhz
            line["roofline"]["pipe_peak_at_sampled_clock"] = pipe_peak_tops(mhz, sm_count)
            line["roofline"]["frac_of_pipe"] = roof["achieved"] / pipe_peak_tops(mhz, sm_count)
            line["value_frac_of_pipe"] = tops / world / pipe_peak_tops(mhz, sm_count)
        if sus:
            ms_sus, sus_steps, clocks_sus = sus
            ms_s = ms_sus / sus_steps
            tops_s = world * STEP_OPS / (ms_s * 1e-3) / 1e12
            line["sustained"] = {"seconds": ms_sus * 1e-3, "steps": sus_steps, "ms_per_step": ms_s, "value": tops_s,
                                 "unit": "TOPS", "clocks": clocks_sus,
                                 "frac_sustained": tops_s / world / (2.0 * peaks["bf16_sustained"]),
                                 "peak_sustained": 2.0 * peaks["bf16_sustained"],
                                 "peak_source": f"2 x bf16 cuBLAS sustained ({peaks['source']})"}
            if clocks_sus and clocks_sus.get("sm_mhz"):
                line["sustained"]["ms_x_mhz"] = ms_s * clocks_sus["sm_mhz"]
                line["sustained"]["frac_of_pipe"] = tops_s / world / pipe_peak_tops(clocks_sus["sm_mhz"], sm_count)
        print(json.dumps(line))
    du.finish(world)


def run_reference(args):
    """The reference arm is the CPU oracle, timed on the host cores (rank 0 only)."""
    rank, _, world = du.world_from_env()
    if rank != 0:
        return
    import oracle
    oracle.build()
    wts = wl.config4_weights(seed=4)
    x = wl.config4_inputs(seed=4, batch=1)
    p = wl.prune_params(1, wl.ROWS, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32, K_ATTN, KEEP,
                        ring_radius=RING_RADIUS)
    t0 = time.perf_counter()
    _oracle_layer(oracle, x["x"][0, :4], wts)
    per_row = (time.perf_counter() - t0) / 4
    total = args.steps + args.warmup
    rows = int(max(1, min(wl.ROWS, 150.0 / max(total, 1) / max(per_row, 1e-4))))

    def step():
        _oracle_layer(oracle, x["x"][0, :rows], wts)
        oracle.prune_tokens(p, x["scores"].view(np.uint16), x["centers"])

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    tops = layer_ops(rows) / dt / 1e12
    sample = (f"{rows} token rows of one observation through one layer's four W4A4 linears + the pruning criterion "
              f"of that observation, per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32 exact / fp32 (CPU oracle)", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "tokens_per_s": rows / dt,
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def graph_time_us(torch, launch, reps: int, replays: int = 5) -> float:
    """Average device time of one `launch(i)`: `reps` launches (i = 0 .. reps-1, rotating buffers) captured
    into one CUDA graph, replayed, timed with events on the replay stream; best of `replays`."""
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        for i in range(min(reps, 3)):
            launch(i)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for i in range(reps):
                launch(i)
        g.replay()
        st.synchronize()
        best = float("inf")
        for _ in range(replays):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            g.replay()
            b.record(st)
            st.synchronize()
            best = min(best, a.elapsed_time(b))
    return best * 1e3 / reps


def kernel_table(torch, B, peaks, device):
    """Every kernel of the path timed alone at the workload's shapes, against the roofline that bounds it.
    Buffers rotate through more than the L2 capacity, so the HBM figures are DRAM figures. Weights for this
    table are random codes generated on the device (timing does not depend on their values)."""
    t = torch
    H, F, Q = wl.HIDDEN, wl.FFN, wl.QKV
    hbm = peaks["hbm_gbs"]
    tpk = 2.0 * peaks["bf16"]
    rows = []
    L2 = 160e6   # rotate through at least this many bytes

    def ncopies(nbytes):
        return max(2, int(np.ceil(L2 / max(nbytes, 1))))

    # what a kernel that does nothing costs as a node of such a graph chain (a one-element torch add): the floor
    # under every time below; HBM rows shorter than 20 us also get their fraction with the floor taken out
    tiny = t.zeros(1, device=device)
    floor_us = graph_time_us(t, lambda i: tiny.add_(1.0), reps=64)
    rows.append(dict(kernel="empty kernel (graph node floor)", shape="-", bound="latency", us=round(floor_us, 2), note=""))

    def add(name, shape, bound, work, us, note=""):
        if bound == "hbm":
            ach = work / (us * 1e-6) / 1e9
            row = dict(kernel=name, shape=shape, bound="hbm", bytes=work, us=round(us, 2), achieved_gbs=round(ach, 1),
                       frac=round(ach / hbm, 3), note=note)
            if us < 20.0 and us > floor_us:
                row["frac_above_floor"] = round(work / ((us - floor_us) * 1e-6) / 1e9 / hbm, 3)
            rows.append(row)
        elif bound == "tensor":
            ach = work / (us * 1e-6) / 1e12
            rows.append(dict(kernel=name, shape=shape, bound="tensor", ops=work, us=round(us, 2), achieved_tops=round(ach, 1),
                             frac=round(ach / tpk, 3), note=note))
        else:
            rows.append(dict(kernel=name, shape=shape, bound=bound, us=round(us, 2), note=note))

    gen = t.Generator(device=device)
    gen.manual_seed(1234)

    def rand_x(M, K):
        return (t.randn(M, K, device=device, generator=gen) * 1.0).to(t.float16)

    def rand_w(N, K):
        codes = t.randint(-8, 8, (N, K), dtype=t.int8, device=device, generator=gen)
        scales = (t.rand(N, device=device, generator=gen) * 0.015 + 0.005).to(t.float16)
        w = B.sqap_pack_weights(codes, scales, N, K)
        t.cuda.synchronize()
        return w

    # ---- quantizer (public nibble output) and the fused form (expanded output is timed inside the linears)
    for (M, K, rot) in ((4608, H, True), (4608, H, False), (4608, F, False), (2560, H, True), (288, H, True),
                        (160, F, False), (16, H, False)):
        nb = M * K * 2.5 + 4 * M
        n = ncopies(M * K * 2)
        xs = [rand_x(M, K) for _ in range(n)]
        q = t.empty(M * K // 2, dtype=t.uint8, device=device)
        sx = t.empty(M, dtype=t.float32, device=device)
        fl = B.SQAP_Q_ROTATE if rot else 0
        us = graph_time_us(t, lambda i: B.sqap_quantize_act(xs[i % n], M, K, K, None, fl, q, sx), reps=max(n, 8))
        add("quantize_act" + ("+hadamard" if rot else ""), f"M={M} K={K}", "hbm", nb, us)
        if M == M_FULL and K == H:
            # the other granularities (sqap_quantize_act_ex); the tensor-wise form reads x twice (two launches), its
            # algorithmic bytes stay those of one pass
            mul = (t.rand(K, device=device, generator=gen) + 0.5).float()
            for nm, f2, cm in (("channel-wise", fl, mul), ("tensor-wise", fl | B.SQAP_Q_PER_TENSOR, None)):
                us = graph_time_us(t, lambda i: B.sqap_quantize_act_ex(xs[i % n], M, K, K, None, f2, cm, q, sx), reps=max(n, 8))
                add("quantize_act_ex " + nm + ("+hadamard" if rot else ""), f"M={M} K={K}", "hbm", nb, us,
                    note="two launches, x read twice" if cm is None else "")
        del xs

    # ---- gather (prune compaction) and the criterion
    inp = wl.config4_inputs(seed=4, batch=N_OBS)
    sc, ce = t.from_numpy(inp["scores"]).to(device), t.from_numpy(inp["centers"]).to(device)
    n = ncopies(M_FULL * H * 2)
    xs = [rand_x(M_FULL, H) for _ in range(n)]
    x1 = t.empty(M_PRUNED, H, dtype=t.float16, device=device)
    kept = t.empty(N_OBS, wl.ROWS, dtype=t.int32, device=device)
    nk = t.empty(N_OBS, dtype=t.int32, device=device)
    p = wl.prune_params(N_OBS, wl.ROWS, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32, K_ATTN, KEEP,
                        ring_radius=RING_RADIUS)
    us_sel = graph_time_us(t, lambda i: B.sqap_prune_tokens(p, sc, ce, None, 0, 0, None, 0, 0, kept, nk), reps=8)
    us_all = graph_time_us(t, lambda i: B.sqap_prune_tokens(p, sc, ce, xs[i % n], H, H, x1, H, ROWS_KEPT, kept, nk),
                           reps=max(n, 8))
    add("prune_select (top-k U ring U FPS, compaction)", f"16 obs x 256 visual -> {KEEP}", "latency", 0, us_sel,
        note=f"{KEEP - K_ATTN} or fewer dependent FPS steps per observation")
    add("gather_rows", f"16 x {ROWS_KEPT} rows x {H}", "hbm", 2 * M_PRUNED * H * 2, max(us_all - us_sel, 1e-3),
        note="prune call minus the selection kernel")
    del xs

    # ---- linears: fused quantize + GEMM is what a layer runs; the GEMM alone via REUSE_EXPANDED
    shapes = (("qkv", Q, H, False), ("o", H, H, False), ("gate_up_swiglu", F, H, True), ("down", H, F, False))
    for (nm, N, K, sw) in shapes:
        wbytes = N * K // 2 * (2 if sw else 1)
        n = ncopies(wbytes)
        ws = [(rand_w(N, K), rand_w(N, K) if sw else None) for _ in range(n)]
        for M in (4608, 2560, 288, 160, 16, 1):
            x = rand_x(M, K)
            out = t.empty(M, N, dtype=t.float16, device=device)
            nb = B.sqap_quantize_linear_workspace_bytes(M, N, K)
            wsp = t.empty(nb, dtype=t.uint8, device=device)
            sc_ptr = wsp.data_ptr() + B.sqap_workspace_bytes(M, N, K)
            B.sqap_quantize_linear(x, M, K, None, 0, ws[0][0], ws[0][1], out, N, B.SQAP_FP16, 0, wsp, nb)
            us = graph_time_us(t, lambda i: B.sqap_w4a4_linear(wsp, sc_ptr, M, ws[i % n][0], ws[i % n][1], out, N,
                                                               B.SQAP_FP16, B.SQAP_L_REUSE_EXPANDED, wsp, nb),
                               reps=max(n, 8))
            ops = 2.0 * M * N * K * (2 if sw else 1)
            byts = wbytes + M * K + 2 * M * N
            if M >= 512:
                add("w4a4_linear GEMM " + nm, f"M={M} N={N} K={K}", "tensor", ops, us)
            else:
                add("w4a4_linear GEMM " + nm, f"M={M} N={N} K={K}", "hbm", byts, us,
                    note=f"{ops / (us * 1e-6) / 1e12:.0f} TOP/s = {ops / (us * 1e-6) / 1e12 / tpk:.2f} of tensor peak")
            del x, out, wsp
        for a, b in ws:
            a.close()
            if b:
                b.close()
    return rows


def run_detail(args):
    import torch
    from paper_2509_09090_b200 import binding as B
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    rows = kernel_table(torch, B, peaks, dev)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    print(json.dumps({"kernels": rows, "peaks": {"hbm_gbs": peaks["hbm_gbs"], "int8_tops": 2 * peaks["bf16"],
                                                  "source": peaks["source"]}}))


def run_stack(args):
    """configs[3]: the 32-layer Llama-2-7B linear stack for one observation: a prefill of 288 token rows (pruned to
    160 after two layers with the full criterion), then 7 single-token decode steps, all launches replayed from one
    CUDA graph. Random weights generated on the device (3.2 GB packed; timing does not depend on their values).
    Prints its own JSON line (not the bench line): times, tokens/s and the weight-streaming fraction of HBM."""
    import torch
    from paper_2509_09090_b200 import binding as B
    t = torch
    t.cuda.set_device(0)
    dev = t.device("cuda", 0)
    peaks = measured_peaks()
    gen = t.Generator(device=dev)
    gen.manual_seed(3)
    H, F, Q = wl.HIDDEN, wl.FFN, wl.QKV

    def rand_w(N, K):
        codes = t.randint(-8, 8, (N, K), dtype=t.int8, device=dev, generator=gen)
        scales = ((t.rand(N, device=dev, generator=gen) * 0.015 + 0.005) * (16.0 / np.sqrt(K))).to(t.float16)
        w = B.sqap_pack_weights(codes, scales, N, K)
        t.cuda.synchronize()
        return w

    from paper_2509_09090_b200.stack import Stack
    n_layers = wl.N_LAYERS
    layers = [dict(qkv=rand_w(Q, H), o=rand_w(H, H), gate=rand_w(F, H), up=rand_w(F, H), down=rand_w(H, F))
              for _ in range(n_layers)]
    inp = wl.config4_inputs(seed=3, batch=1)
    x = t.from_numpy(inp["x"].reshape(wl.ROWS, H)).to(dev)
    sc, ce = t.from_numpy(inp["scores"]).to(dev), t.from_numpy(inp["centers"]).to(dev)
    xdec = t.from_numpy(wl.activations(3, wl.T_X2, 7, H, 41, 30.0)).to(dev)
    keep = 128
    rows_kept = 32 + keep
    M = wl.ROWS
    st = Stack(t, B, dev, layers, keep=keep, k_attn=keep // 2, ring_radius=1, n_decode=7)
    prefill = lambda: st.prefill(x, sc, ce)
    decode = lambda: st.decode(xdec)

    def timed(fn, reps):
        fn()
        t.cuda.synchronize()
        l0 = B.sqap_kernel_launch_count()
        g = t.cuda.CUDAGraph()
        with t.cuda.graph(g):
            fn()
        launches = B.sqap_kernel_launch_count() - l0
        g.replay()
        t.cuda.synchronize()
        a, b = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        t.cuda.synchronize()
        return a.elapsed_time(b) / reps, launches

    ms_pre, l_pre = timed(prefill, max(3, args.steps // 10))
    ms_dec, l_dec = timed(decode, max(3, args.steps // 10))
    assert B.sqap_device_status() == B.SQAP_OK
    wbytes = n_layers * (Q * H + H * H + 2 * F * H + H * F) // 2
    ops_pre = sum(layer_ops(M if li < 2 else rows_kept) for li in range(n_layers))
    print(json.dumps({
        "workload": "configs[3]: 32-layer Llama-2-7B W4A4 linear stack, one observation: prefill of 288 rows (pruned to 160 "
                    "after two layers), then 7 single-token decode steps; CUDA-graph replay; random device weights",
        "prefill_ms": ms_pre, "prefill_tops": ops_pre / (ms_pre * 1e-3) / 1e12, "prefill_launches": l_pre,
        "prefill_weight_stream_gbs": wbytes / (ms_pre * 1e-3) / 1e9,
        "decode_ms_per_token": ms_dec / 7, "decode_launches": l_dec,
        "decode_weight_stream_gbs": 7 * wbytes / (ms_dec * 1e-3) / 1e9,
        "decode_frac_of_hbm": 7 * wbytes / (ms_dec * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "total_ms": ms_pre + ms_dec, "packed_weight_bytes": wbytes,
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]}}))


def run_single_kernel(args):
    """Profiling aid: a few launches of one kernel of the path on a small, larger-than-L2 case
    (what `ncu -k ... -c 3` captures). Prints nothing that counts as a bench value."""
    import torch
    from paper_2509_09090_b200 import binding as B
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    M, H = M_FULL, wl.HIDDEN
    x = torch.from_numpy(wl.config4_inputs(seed=4, batch=N_OBS)["x"].reshape(M, H)).to(dev)
    q = torch.empty(M * wl.FFN // 2, dtype=torch.uint8, device=dev)
    sx = torch.empty(M, dtype=torch.float32, device=dev)
    if args.kernel == "quantize":
        for i in range(args.steps):
            B.sqap_quantize_act(x, M, H, H, None, B.SQAP_Q_ROTATE if i % 2 == 0 else 0, q, sx)
    elif args.kernel in ("gemm", "gemv", "gemvpair", "gemvlong", "stream", "midm", "downm", "swiglu"):
        names = {"gemm": ("qkv",), "gemv": ("qkv",), "gemvpair": ("gate", "up"), "gemvlong": ("down",), "stream": ("qkv",),
                 "midm": ("o",), "downm": ("down",), "swiglu": ("gate", "up")}[args.kernel]
        wts = wl.config4_weights(seed=4)
        ws = [B.sqap_pack_weights(np.ascontiguousarray(wts[n + "_codes"]), np.ascontiguousarray(wts[n + "_scales"]),
                                  wts[n + "_codes"].shape[0], wts[n + "_codes"].shape[1]) for n in names]
        # stream: one decode token per observation; midm / downm: one observation pruned to 160 rows (O projection on
        # the one-CTA-per-tile kernel; down projection, 11008 codes per row, on the cluster split-K kernel)
        # gemv / gemvpair / gemvlong: the single row of a decode step (QKV; gate + up; down with 11008 codes per row)
        Mk = {"gemv": 1, "gemvpair": 1, "gemvlong": 1, "stream": N_OBS, "midm": 160, "downm": 160}.get(args.kernel, M)
        N = ws[0].N
        Kk = ws[0].K
        if Kk != H:
            x = torch.from_numpy(wl.activations(4, 77, Mk, Kk, 110, 30.0)).to(dev)
        H_ = H
        H = Kk
        out = torch.empty(Mk, N, dtype=torch.float16, device=dev)
        nb = B.sqap_workspace_bytes(Mk, N, H)
        wsp = torch.empty(nb, dtype=torch.uint8, device=dev)
        B.sqap_quantize_act(x, Mk, H, H, None, B.SQAP_Q_ROTATE if Kk == H_ else 0, q, sx)
        for i in range(args.steps):
            B.sqap_w4a4_linear(q, sx, Mk, ws[0], ws[1] if len(ws) > 1 else None, out, N, B.SQAP_FP16,
                               B.SQAP_L_REUSE_EXPANDED if i else 0, wsp, nb)
    elif args.kernel == "prune":
        inp = wl.config4_inputs(seed=4, batch=N_OBS)
        sc, ce = torch.from_numpy(inp["scores"]).to(dev), torch.from_numpy(inp["centers"]).to(dev)
        x1 = torch.empty(M_PRUNED, H, dtype=torch.float16, device=dev)
        kept = torch.empty(N_OBS, wl.ROWS, dtype=torch.int32, device=dev)
        nk = torch.empty(N_OBS, dtype=torch.int32, device=dev)
        p = wl.prune_params(N_OBS, wl.ROWS, wl.VISUAL_START, wl.N_VISUAL, wl.GRID, wl.GRID, 32, K_ATTN, KEEP,
                            ring_radius=RING_RADIUS)
        for i in range(args.steps):
            B.sqap_prune_tokens(p, sc, ce, x, H, H, x1, H, ROWS_KEPT, kept, nk)
    torch.cuda.synchronize()
    assert B.sqap_device_status() == B.SQAP_OK
    print(json.dumps({"profiling_run": args.kernel, "launches": B.sqap_kernel_launch_count()}))


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one process per GPU, rendezvous on
    127.0.0.1), pass rank 0's output through and return the worst exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for pr in procs:
        rc = max(rc, abs(pr.wait()))
    return rc


def run_stub(args):
    """The multi-rank plumbing of run_ours around a CPU stand-in for the step (no GPU, no kernels): process-group
    start-up from the environment, barrier-bracketed timing, maximum over ranks, one JSON line from rank 0."""
    rank, _, world = du.init(args.stub_backend)
    first, cnt = du.shard_observations(N_OBS * world, world, rank)
    du.barrier(world)
    t0 = time.perf_counter()
    acc = 0
    for _ in range(args.steps):
        acc += sum(range(1000 * (rank + 1)))
    ms = du.max_over_ranks((time.perf_counter() - t0) * 1e3, world)
    total = du.sum_over_ranks(cnt, world)
    du.barrier(world)
    if rank == 0:
        print(json.dumps({"stub": True, "n_gpus": world, "steps": args.steps, "ms_per_step": ms / max(args.steps, 1),
                          "observations": int(total), "scaling": "weak"}))
    du.finish(world)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity-check", action="store_true", help="skip the untimed oracle check of the replayed step")
    ap.add_argument("--sustain-s", type=float, default=2.0,
                    help="length in seconds of the second, sustained timed region (0: none)")
    ap.add_argument("--stub-backend", default=None, choices=["gloo"],
                    help="plumbing test: run the rank start-up, barriers and max-over-ranks timing around a CPU stub step")
    ap.add_argument("--serial-prune", action="store_true",
                    help="issue the pruning criterion on the main stream after layer A instead of beside its last quantizer")
    ap.add_argument("--no-graph", action="store_true", help="issue the step's launches eagerly instead of replaying a CUDA graph")
    ap.add_argument("--detail", action="store_true",
                    help="time every kernel of the path alone at the workload's shapes (one JSON table, no bench line)")
    ap.add_argument("--stack", action="store_true",
                    help="time configs[3] (32-layer stack: prefill + 7 decode tokens for one observation); own JSON line")
    ap.add_argument("--kernel", default=None, choices=["gemm", "swiglu", "gemv", "gemvpair", "gemvlong", "stream", "midm", "downm", "quantize", "prune"],
                    help="profiling aid: launch only this kernel --steps times (no bench line)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.stub_backend:
        run_stub(args)
    elif args.stack:
        run_stack(args)
    elif args.detail:
        run_detail(args)
    elif args.kernel:
        run_single_kernel(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
