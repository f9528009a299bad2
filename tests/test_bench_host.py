"""Host-side logic of bench.py: cost model, rank reduction (gloo, 2 processes), reference arm."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2403_03507_b200 import workloads as wl  # noqa: E402


def test_algorithmic_cost_matches_hand_computation():
    # 4096 x 11008 bf16, r = 1024, 8-bit states: G + 2 W + 4 bytes per state element + absmax + P
    w = wl.WORKLOADS["llama_7b_q8"]
    by, fl = bench.algorithmic_cost(w, 4096, 11008)
    nel = 1024 * 11008
    assert by == 4096 * 11008 * 2 * 3 + 4 * nel + 16 * (nel // 2048) + 4096 * 1024 * 2
    assert fl == 4 * 4096 * 11008 * 1024
    # whole layer sets: parameters as listed for the workloads
    assert w.params == 6_476_005_376 and w.matrices == 224
    assert wl.WORKLOADS["llama_1b_q8"].params == 1_207_910_400
    assert wl.WORKLOADS["llama_130m"].params == 84_934_656
    total_flops = sum(bench.algorithmic_cost(w, m, n)[1] * c for m, n, c in w.shapes)
    assert abs(total_flops / 26.53e12 - 1) < 1e-3
    total_bytes = sum(bench.algorithmic_cost(w, m, n)[0] * c for m, n, c in w.shapes)
    assert abs(total_bytes / 47.22e9 - 1) < 5e-3


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        got = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
        out[rank] = got
    finally:
        dist.destroy_process_group()


def test_timing_is_the_maximum_over_ranks_gloo_world_size_2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(2, 29533, out), nprocs=2, join=True)
    assert out[0] == 15.0 and out[1] == 15.0
    assert bench.max_over_ranks(3.5, None, None) == 3.5


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "single_60m_mlp",
           "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "params/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_clock_sampler_tolerates_a_missing_nvidia_smi():
    s = bench.ClockSampler(0)
    s.start()
    res = s.stop()
    assert set(res) >= {"sm_mhz", "sm_max_mhz", "reasons"}
