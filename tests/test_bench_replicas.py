"""Host logic of the multi-GPU bench path (independent replicas), on CPU with gloo, world size 2."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r's timed region took (10 + 5 r) ms, its end-to-end loop (1 + r) s
    total_ms, e2e_s = bench.max_over_ranks([10.0 + 5.0 * rank, 1.0 + rank], torch.device("cpu"), True)
    q.put((rank, total_ms, e2e_s, bench.aggregate_value(8, 100, world, total_ms * 1e-3)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_gloo():
    world, port = 2, 29731
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total_ms, e2e_s, value in got:
        assert total_ms == 15.0 and e2e_s == 2.0           # the slowest rank sets the time
        assert abs(value - 2 * 8 * 100 / 0.015) < 1e-6     # every rank's tokens count


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_roofline_bound_selection():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2501_19309_b200 import inputs as I
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    r3 = bench.roofline_of(I.CONFIGS[3], peaks, 0.7, False, "measured")
    assert r3["bound"] == "hbm" and r3["algorithmic_bytes"] == 128256 * 16384 * 2 + 26 * 16384 * 2
    assert abs(r3["frac"] - r3["achieved"] / 6500.0) < 1e-12
    r4 = bench.roofline_of(I.CONFIGS[4], peaks, 2.0, False, "measured")
    assert r4["bound"] == "tensor" and abs(r4["achieved"] - 2 * 1088 * 128256 * 8192 / 2e-3 / 1e12) < 1e-6
    line = json.dumps(r4)
    assert "traffic" in line


def test_workload_tokens_of_the_bench():
    """An id, then f = FP8 head, g / k = greedy / top-5 rule, n = RMSNorm; anything else is no workload."""
    sys.path.insert(0, ROOT)
    import bench
    wl, o = bench.parse_workload_token("3")
    assert wl.name == "cfg3-405B-head" and wl.dtype == "bf16" and o == bench.NO_OPTIONS
    wl, o = bench.parse_workload_token("4f")
    assert wl.name == "cfg4-batched-fp8" and wl.dtype == "fp8" and o["rule"] == "sampling" and o["rms_eps"] is None
    wl, o = bench.parse_workload_token("2gn")
    assert wl.name == "cfg2-70B-head-greedy-rmsnorm" and (o["rule"], o["top_k"]) == ("topk", 1) and o["rms_eps"] > 0
    wl, o = bench.parse_workload_token("1fk")
    assert wl.dtype == "fp8" and (o["rule"], o["top_k"]) == ("topk", 5) and (wl.B, wl.M, wl.d) == (1, 8, 4096)
    for bad in ("", "9", "3x", "g3", "3gk", "3nf"):
        assert bench.parse_workload_token(bad) == (None, None)
    cfg = bench.config_of(*bench.parse_workload_token("4g")[:1], 1, bench.parse_workload_token("4g")[1])
    assert cfg["rule"] == "top-1" and cfg["norm"] == "none" and cfg["workload"] == "cfg4-batched-greedy"
