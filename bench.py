#!/usr/bin/env python
"""Benchmark of the fused verification step (jd_verify) on synthetic Llama-3.1-shaped heads.

One step = one verification call (LM head -> softmax -> tests -> prefix -> next token) over one
synthetic draft block.  Prints ONE JSON line:

  value     verified tokens/s (B*M per call), inputs resident in device memory, CUDA-event time
  e2e       the same through jd_verify_host: pinned host inputs copied in, outputs copied back
  roofline  achieved (W bytes + H bytes) / kernel time against the measured HBM copy bandwidth
            (or 2*R*V*d flop / time against the measured bf16 peak when that bound is larger)
  cpu_baseline  the float64 CPU checker timed on a bounded sample of the same workload

`--impl reference` times the CPU checker alone (rank 0 only).
With --gpus N > 1 (launched under torchrun) every rank runs an independent replica: the path has
no exchange step, so the aggregate is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2501_19309_b200 import inputs as I  # noqa: E402

METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (read + write) per verification call from the ncu captures summarised under profiles/
# (dominant kernels of each workload); set an entry to None when its kernel changes.
NCU_TRAFFIC_BYTES = {"cfg1-8B-head": 1.0593e9, "cfg2-70B-head": 2.1576e9, "cfg3-405B-head": 4.2244e9,
                     "cfg3-405B-head-fp8": 2.1230e9,
                     "cfg4-batched": 2.1495e9 + 2.1448e9,          # GEMM pass + second pass
                     "cfg4-batched-fp8": 1.0666e9 + 1.0905e9}
VARIANT_NAMES = {1: "simt", 2: "fused", 3: "batched"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.rows = []
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            try:
                pw.append(float(f[6]))
            except (IndexError, ValueError):
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "power_w": statistics.median(pw) if pw else None}


def max_over_ranks(values, device, dist_on: bool):
    """Element-wise maximum of a few floats over all ranks (the slowest rank sets the time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist_on:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_value(units_per_rank_step: int, steps: int, world: int, max_seconds: float) -> float:
    """Whole-job throughput of independent replicas: all ranks' units over the slowest rank's time."""
    return world * units_per_rank_step * steps / max_seconds


NOMINAL_HBM_GBS = 8000.0      # the "~8 TB/s" the metric's definition quotes
NOMINAL_BF16_TFLOPS = 2250.0  # dense


def roofline_of(wl: I.Workload, peaks: dict, kernel_ms: float, sustained: bool, which: str,
                stream_gbs: float = None) -> dict:
    if wl.dtype == "fp8":   # one byte per weight + a float per vocabulary row; H read as bf16 once
        bytes_alg = wl.V * wl.d + wl.V * 4 + wl.R * wl.d * 2
    else:
        bytes_alg = wl.V * wl.d * 2 + wl.R * wl.d * 2        # W once + H once
    # everything the call must move: + the draft logits once for their statistics and one row per sequence
    # again for the residual, tokens in, results out (the metric's own byte count leaves these out)
    bytes_all = bytes_alg + wl.B * wl.M * wl.V * 4 + wl.B * wl.V * 4 + wl.B * wl.M * 4 + wl.B * (8 + 8 * wl.M)
    flops = 2.0 * wl.R * wl.V * wl.d
    tf_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    tf_sustained = peaks["bf16_tflops_sustained"]
    if wl.dtype == "fp8":   # no measured FP8 figure: the measured bf16 peak x the nominal 2:1 ratio of the two kinds
        tf_peak, tf_sustained = 2 * tf_peak, 2 * tf_sustained
    t_bytes = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_flops = flops / (tf_peak * 1e12)
    traffic = NCU_TRAFFIC_BYTES.get(wl.name)
    if t_bytes >= t_flops:
        ach = bytes_alg / (kernel_ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "peak_source": which,
                "frac_of_nominal_peak": ach / NOMINAL_HBM_GBS,
                "read_stream_gbs": stream_gbs, "frac_of_read_stream": ach / stream_gbs if stream_gbs else None,
                "algorithmic_bytes": bytes_alg, "all_bytes": bytes_all,
                "frac_all_bytes": bytes_all / (kernel_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "kernel_ms": kernel_ms}
    ach = flops / (kernel_ms * 1e-3) / 1e12
    return {"bound": "tensor", "achieved": ach, "peak": tf_peak, "unit": "TFLOP/s", "frac": ach / tf_peak,
            "frac_of_sustained_peak": ach / tf_sustained,
            "frac_of_nominal_peak": ach / (NOMINAL_BF16_TFLOPS * (2 if wl.dtype == "fp8" else 1)),
            "traffic": traffic, "peak_source": which, "algorithmic_flops": flops, "all_bytes": bytes_all,
            "kernel_ms": kernel_ms}


def oracle_step(inp: I.Inputs, seed: int, sequences):
    from oracle import jd_oracle as O
    return O.jd_oracle_verify(inp.W, inp.w_judge, inp.b_judge, inp.H, inp.draft_tokens, inp.draft_logits,
                              inp.tau, seed, "judge_or_standard", sequences=sequences, w_scale=inp.w_scale)


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(inp: I.Inputs, steps: int, budget_s: float = 25.0) -> dict:
    """The checker as it stands on a bounded sample: whole sequences b = 0, 1, ... of the workload."""
    wl = inp.wl
    t0 = time.perf_counter()
    oracle_step(inp, 0, [0])
    one = time.perf_counter() - t0
    nseq = int(max(1, min(wl.B, budget_s / max(one, 1e-3) / max(steps, 1))))
    seqs = list(range(nseq))
    t0 = time.perf_counter()
    for s in range(steps):
        oracle_step(inp, s, seqs)
    dt = time.perf_counter() - t0
    return {"value": nseq * wl.M * steps / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": "%d step(s) x %d of %d sequences (%d rows x V=%d x d=%d each), float64 numpy" %
                      (steps, nseq, wl.B, wl.M + 1, wl.V, wl.d),
            "seconds": dt}


def run_reference(args, wl) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = I.make_inputs(wl, 0)
    steps = max(1, min(args.steps, 3))
    for _ in range(min(args.warmup, 1)):
        oracle_step(inp, 0, [0])
    r = time_oracle(inp, steps, budget_s=60.0)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": r["seconds"] / steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": wl.name, "B": wl.B, "M": wl.M, "d": wl.d, "V": wl.V},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def measure_workload(wl, args, torch, jd, device, data_seed, sample_clocks):
    """Times K device-resident calls and K_e2e host-buffer calls of one workload on this rank."""
    inp = I.make_inputs(wl, data_seed)
    fp8 = wl.dtype == "fp8"
    W = torch.from_numpy(inp.W).to(device) if fp8 else torch.from_numpy(inp.W).view(torch.bfloat16).to(device)
    w_scale = torch.from_numpy(inp.w_scale).to(device) if fp8 else None
    H = torch.from_numpy(inp.H).view(torch.bfloat16).to(device)
    w = torch.from_numpy(inp.w_judge).view(torch.bfloat16).to(device)
    x = torch.from_numpy(inp.draft_tokens).to(device)
    dl = torch.from_numpy(inp.draft_logits).to(device)
    ver = jd.Verifier(wl.B, wl.M, wl.d, wl.V, "fp8" if fp8 else "bf16", device.index)
    ver.set_head(W, w, inp.b_judge, w_scale=w_scale)
    out = ver.alloc_outputs(wl.B, wl.M)
    a_args = [ver.make_args(H, x, dl, inp.tau, s, "judge_or_standard", out=out)[0] for s in range(8)]
    stream = torch.cuda.current_stream(device)

    def step(i):
        st = jd.jd_verify(ver.h, a_args[i % 8], stream.cuda_stream)
        if st != jd.JD_OK:
            raise jd.JdError(st, "jd_verify")

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize(device)
    assert ver.device_status() == jd.JD_OK
    variant, launches = ver.launch_info()

    sampler = ClockSampler(device.index) if sample_clocks else None
    if sampler:
        time.sleep(0.6)          # let the sampler start
    if args.dist:
        torch.distributed.barrier()
    torch.cuda.synchronize(device)
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(K):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize(device)
    if args.dist:
        torch.distributed.barrier()
    total_ms = e0.elapsed_time(e1)
    # per-call distribution on a short second pass (events between calls)
    Kp = min(K, 200)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(Kp + 1)]
    evs[0].record(stream)
    for i in range(Kp):
        step(i)
        evs[i + 1].record(stream)
    torch.cuda.synchronize(device)
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(Kp)]
    # the same calls replayed from a CUDA graph (eight calls, one per verify seed, per replay)
    graph_ms = None
    if not args.no_graph:
        cap = torch.cuda.Stream(device)
        cap.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            cs = torch.cuda.current_stream(device).cuda_stream
            for i in range(8):
                st = jd.jd_verify(ver.h, a_args[i], cs)
                if st != jd.JD_OK:
                    raise jd.JdError(st, "jd_verify (capture)")
        reps = max(2, K // 8)
        for _ in range(2):
            g.replay()
        torch.cuda.synchronize(device)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(reps):
            g.replay()
        g1.record(stream)
        torch.cuda.synchronize(device)
        graph_ms = g0.elapsed_time(g1) / (8 * reps)
        del g
    clocks = sampler.stop() if sampler else None
    assert ver.device_status() == jd.JD_OK
    # tokens a call emits (accepted prefix + the drawn token), averaged over the verify seeds in use
    accepted = []
    for i in range(8):
        step(i)
        accepted.append(out["accept_len"].cpu().numpy().astype(np.float64))
    accepted = np.stack(accepted)

    # read-only streaming ceiling of this device: the library's probe over the same W
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    w_bytes = W.numel() * W.element_size()
    pevs = [torch.cuda.Event(enable_timing=True) for _ in range(8)]
    pevs[0].record(stream)
    for i in range(7):
        jd.jd_stream_read_probe(W.data_ptr(), w_bytes, sink.data_ptr(), stream.cuda_stream)
        pevs[i + 1].record(stream)
    torch.cuda.synchronize(device)
    stream_gbs = w_bytes / (statistics.median(pevs[i].elapsed_time(pevs[i + 1]) for i in range(2, 7)) * 1e-3) / 1e9

    # end to end: pinned host buffers in, outputs back, every step
    hH = torch.from_numpy(inp.H).view(torch.bfloat16).pin_memory()
    hx = torch.from_numpy(inp.draft_tokens).pin_memory()
    hdl = torch.from_numpy(inp.draft_logits).pin_memory()
    hout = ver.alloc_outputs(wl.B, wl.M, host=True)
    h_args = [ver.make_args(hH, hx, hdl, inp.tau, s, "judge_or_standard", out=hout, host=True)[0] for s in range(8)]
    Ke = max(3, min(K, args.e2e_steps))
    for i in range(3):
        jd.jd_verify_host(ver.h, h_args[i % 8], stream.cuda_stream)
    torch.cuda.synchronize(device)
    if args.dist:
        torch.distributed.barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        st = jd.jd_verify_host(ver.h, h_args[i % 8], stream.cuda_stream)
        if st != jd.JD_OK:
            raise jd.JdError(st, "jd_verify_host")
    torch.cuda.synchronize(device)
    e2e_s = time.perf_counter() - t0
    h2d = hH.numel() * 2 + hx.numel() * 4 + hdl.numel() * 4
    d2h = sum(hout[k].numel() * hout[k].element_size() for k in hout)
    ver.close()
    res = dict(total_ms=total_ms, median_ms=statistics.median(per), min_ms=min(per), mean_ms=total_ms / K,
               variant=variant, launches=launches, clocks=clocks, e2e_s=e2e_s, e2e_steps=Ke, h2d=h2d, d2h=d2h,
               mean_accept=float(accepted.mean()), emitted_per_call=float((accepted + 1).sum(axis=1).mean()),
               stream_gbs=stream_gbs, graph_ms=graph_ms, inp=inp)
    del W, H, dl
    torch.cuda.empty_cache()
    return res


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="workload id of the headline line (1..4)")
    ap.add_argument("--others", default="2,3,4,3f,4f", help="comma list of further workloads summarised in the same "
                    "line; a trailing f = the same shape with an FP8 E4M3 head")
    ap.add_argument("--fp8", action="store_true", help="headline workload with an FP8 E4M3 head")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = I.CONFIGS[args.config]
    if args.fp8:
        wl = wl.scaled(wl.name + "-fp8", dtype="fp8")

    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    from paper_2501_19309_b200 import jd
    jd.load()   # raises if the CUDA library is missing: there is no other path

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    args.dist = world > 1
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if args.dist:
        torch.distributed.init_process_group("nccl", device_id=device)

    peaks, which = load_peaks()
    res = measure_workload(wl, args, torch, jd, device, data_seed=rank, sample_clocks=True)

    # max over ranks of the timed region, sum of the units
    total_ms, e2e_s = max_over_ranks([res["total_ms"], res["e2e_s"]], device, args.dist)
    K = args.steps
    tokens_per_step = wl.B * wl.M
    value = aggregate_value(tokens_per_step, K, world, total_ms * 1e-3)
    e2e_value = aggregate_value(tokens_per_step, res["e2e_steps"], world, e2e_s)

    others = {}
    if rank == 0 and args.others:
        small = argparse.Namespace(**vars(args))
        small.dist = False
        for tok in [c.strip() for c in args.others.split(",") if c.strip()]:
            as_fp8 = tok.endswith("f")
            cid = int(tok.rstrip("f"))
            if (cid == args.config and not as_fp8) or cid not in I.CONFIGS:
                continue
            owl = I.CONFIGS[cid]
            if as_fp8:
                owl = owl.scaled(owl.name + "-fp8", dtype="fp8")
            small.steps = max(50, min(args.steps, 300))
            small.e2e_steps = 10
            r = measure_workload(owl, small, torch, jd, device, data_seed=0, sample_clocks=True)
            others[owl.name] = {
                "B": owl.B, "M": owl.M, "d": owl.d, "V": owl.V, "ms_per_step": r["mean_ms"],
                "median_ms": r["median_ms"], "value": owl.B * owl.M / (r["mean_ms"] * 1e-3), "unit": UNIT,
                "variant": VARIANT_NAMES.get(r["variant"], "?"), "kernel_launches_per_step": r["launches"],
                "steps": small.steps, "mean_accept_len": r["mean_accept"], "best_ms": r["min_ms"],
                "clocks": r["clocks"],
                "graph_replay_ms_per_step": r["graph_ms"],
                "emitted_tokens_per_s": r["emitted_per_call"] / (r["mean_ms"] * 1e-3),
                "e2e_value": owl.B * owl.M * r["e2e_steps"] / r["e2e_s"],
                "roofline": roofline_of(owl, peaks, r["mean_ms"], sustained=r["mean_ms"] * small.steps > 1000, which=which,
                                        stream_gbs=r["stream_gbs"])}

    if rank == 0:
        cpu = None
        if not args.no_cpu_baseline:
            c = time_oracle(res["inp"], 1)
            cpu = {k: c[k] for k in ("value", "unit", "cores", "kind", "sample")}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8" if wl.dtype == "fp8" else "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "M": wl.M, "d": wl.d, "V": wl.V, "mode": "judge_or_standard",
                       "variant": VARIANT_NAMES.get(res["variant"], "?"),
                       "l2": "inputs larger than L2: W (%.2f GB) streams from HBM every call" % (wl.V * wl.d * 2 / 1e9),
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "mean_accept_len": res["mean_accept"]},
            "calls_per_s": world * K / (total_ms * 1e-3),
            "median_ms_per_step": res["median_ms"],
            "best_ms_per_step": res["min_ms"],
            "graph_replay_ms_per_step": res["graph_ms"],
            "emitted_tokens_per_s": world * res["emitted_per_call"] * K / (total_ms * 1e-3),
            "clocks": res["clocks"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": res["h2d"],
                    "d2h_bytes_per_step": res["d2h"], "steps": res["e2e_steps"]},
            "gpu_launches": res["launches"] * K,
            "roofline": roofline_of(wl, peaks, res["mean_ms"], sustained=total_ms > 1000, which=which,
                                    stream_gbs=res["stream_gbs"]),
            "cpu_baseline": cpu,
            "other_workloads": others,
        }
        print(json.dumps(line), flush=True)
    if args.dist:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
