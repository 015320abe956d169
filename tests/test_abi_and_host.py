"""CPU-only checks of the boundary: the C-ABI library loads, exports every symbol that
include/sqap.h declares, and its host-side logic (argument validation, the projection helper,
workspace sizing) behaves; plus the multi-rank host plumbing over gloo. No kernel is launched."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2509_09090_b200 import binding as B
from paper_2509_09090_b200 import dist_utils as du

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sqap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sqap_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = B.lib()
    syms = declared_symbols()
    assert set(syms) == set(B.EXPORTS), (syms, B.EXPORTS)
    for s in syms:
        assert hasattr(L, s)


def test_status_strings_and_counters():
    L = B.lib()
    seen = {L.sqap_status_string(i).decode() for i in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert L.sqap_status_string(99).decode() == "unknown status"
    assert L.sqap_kernel_launch_count() >= 0


def test_host_side_validation_without_a_gpu():
    L = B.lib()
    assert L.sqap_quantize_act(None, -1, 64, 64, None, 0, None, None, None) == B.SQAP_ERR_INVALID
    assert L.sqap_quantize_act(None, 0, 64, 64, None, 0, None, None, None) == B.SQAP_OK
    assert L.sqap_quantize_act(None, 4, 64, 64, None, 0, None, None, None) == B.SQAP_ERR_INVALID
    assert L.sqap_quantize_act(16, 4, 64, 64, None, 2, 16, 16, None) == B.SQAP_ERR_INVALID
    assert L.sqap_quantize_act(16, 4, 40, 40, None, 0, 16, 16, None) == B.SQAP_ERR_ALIGN
    assert L.sqap_quantize_act(16, 4, 96, 96, None, B.SQAP_Q_ROTATE, 16, 16, None) == B.SQAP_ERR_UNSUPPORTED
    out = ctypes.c_void_p()
    assert L.sqap_pack_weights(None, None, 4, 64, 0, None, ctypes.byref(out)) == B.SQAP_ERR_INVALID
    assert L.sqap_pack_weights(16, 16, 4, 40, 0, None, ctypes.byref(out)) == B.SQAP_ERR_ALIGN
    assert L.sqap_pack_weights(16, 16, 0, 64, 0, None, ctypes.byref(out)) == B.SQAP_ERR_INVALID
    assert L.sqap_w4a4_linear(None, None, 4, None, None, None, 0, 0, 0, None, 0, None) == B.SQAP_ERR_INVALID
    assert L.sqap_free_weights(None) == B.SQAP_OK
    assert L.sqap_prune_tokens(None, None, None, None, 0, 0, None, 0, 0, None, None, None) == B.SQAP_ERR_INVALID
    p = B.PruneParams(batch=1, rows=10, visual_start=4, n_visual=8, grid_w=4, grid_h=2, score_rows=0, k_attn=1,
                      keep_total=2, ring_radius=-1, flags=0)
    assert L.sqap_prune_tokens(ctypes.byref(p), None, None, None, 0, 0, None, 0, 0, None, None, None) == B.SQAP_ERR_INVALID
    p.batch = 0
    p.visual_start = 0
    assert L.sqap_prune_tokens(ctypes.byref(p), None, None, None, 0, 0, None, 0, 0, None, None, None) == B.SQAP_OK


def test_workspace_bytes():
    assert B.sqap_workspace_bytes(0, 1, 1) == 256
    for M, K in [(1, 32), (288, 4096), (4608, 11008), (7, 96)]:
        n = B.sqap_workspace_bytes(M, 123, K)
        assert n % 256 == 0 and n >= M * K + 4 * M and n <= M * K + 4 * M + 512


def test_project_center_matches_golden_cases_and_oracle():
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", "projection_cases.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                rows.append([float(t) for t in line.split()])
    assert len(rows) >= 7
    for r in rows:
        (tu, tv), front = B.sqap_project_center(r[0:9], r[9:21], r[21:24], r[24], r[25])
        assert front == bool(int(r[28]))
        if front:
            assert (tu, tv) == (int(r[26]), int(r[27]))
    rng = np.random.default_rng(0)
    for _ in range(200):
        Kmat = np.array([[rng.uniform(50, 400), rng.uniform(-5, 5), rng.uniform(50, 300)],
                         [0, rng.uniform(50, 400), rng.uniform(50, 300)], [0, 0, 1]])
        Rt = np.concatenate([np.linalg.qr(rng.standard_normal((3, 3)))[0], rng.uniform(-1, 1, (3, 1))], axis=1)
        xyz = rng.uniform(-2, 2, 3)
        a = B.sqap_project_center(Kmat.ravel(), Rt.ravel(), xyz, 14.0, 14.0)
        b = oracle.project_center(Kmat, Rt, xyz, 14.0, 14.0)
        assert a == b
    L = B.lib()
    assert L.sqap_project_center(None, None, None, 14.0, 14.0, None, None) == B.SQAP_ERR_INVALID


def test_shard_observations():
    for n, w in [(16, 1), (16, 2), (16, 3), (5, 8), (0, 2)]:
        parts = [du.shard_observations(n, w, r) for r in range(w)]
        assert sum(c for _, c in parts) == n
        pos = 0
        for first, cnt in parts:
            assert first == pos
            pos += cnt
        assert max(c for _, c in parts) - min(c for _, c in parts) <= 1
    with pytest.raises(ValueError):
        du.shard_observations(4, 2, 2)


_GLOO_CHILD = r"""
import os, sys
sys.path.insert(0, {root!r})
from paper_2509_09090_b200 import dist_utils as du
rank, local, world = du.init("gloo")
assert world == 2
du.barrier(world)
first, cnt = du.shard_observations(33, world, rank)
mx = du.max_over_ranks(10.0 + rank, world)
tot = du.sum_over_ranks(cnt, world)
assert mx == 11.0 and tot == 33.0, (mx, tot)
du.barrier(world)
du.finish(world)
print("rank", rank, "ok", first, cnt)
"""


def test_two_rank_plumbing_over_gloo(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(_GLOO_CHILD.format(root=ROOT))
    port = 29600 + os.getpid() % 300
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
    assert "ok 0 17" in outs[0] and "ok 17 16" in outs[1]


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment must start two ranks itself; here around
    the CPU stub step over gloo. Rank 0 prints one line that counts both ranks."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "3", "--stub-backend", "gloo"],
                         env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["observations"] == 32 and line["stub"] is True
