#!/usr/bin/env python
"""Benchmark of the fused verification step (jd_verify) on synthetic Llama-3.1-shaped heads.

One step = one verification call (LM head -> softmax -> tests -> prefix -> next token) over one
synthetic draft block.  Prints ONE JSON line:

  value     verified tokens/s (B*M per call), inputs resident in device memory, CUDA-event time
  e2e       the same through jd_verify_host: pinned host inputs copied in, outputs copied back
  roofline  achieved (W bytes + H bytes) / kernel time against the measured HBM copy bandwidth
            (or 2*R*V*d flop / time against the measured bf16 peak when that bound is larger)
  cpu_baseline  the float64 CPU checker timed on a bounded sample of the same workload
  parity    the device results of the timed workload compared with that checker run (same inputs,
            verify seed 0, same sequences) under the rules of the parity tests

The headline workload is the 405B-shaped head (largest single-GPU configuration); the other
configurations are timed in the same run and summarised under `other_workloads`.
`--record-traffic CSV...` does not measure anything: it reads ncu raw-page CSV exports and rewrites
profiles/ncu_traffic.json (DRAM bytes per launch of the dominant kernels, with the hash of the
kernel sources they were taken on).

`--impl reference` times the CPU checker alone (rank 0 only).
With --gpus N > 1 (launched under torchrun) every rank runs an independent replica: the path has
no exchange step, so the aggregate is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2501_19309_b200 import inputs as I  # noqa: E402

T_START = time.perf_counter()
METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

VARIANT_NAMES = {1: "simt", 2: "fused", 3: "batched"}
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")
KERNEL_SOURCES = ["jd_fused_sm100.cu", "jd_batched_sm100.cu", "jd_sm100_ptx.cuh", "jd_common.cuh"]


def kernel_source_hash() -> str:
    """sha256 over the sources of the tensor-core kernels: the DRAM counters are only quoted while
    the kernels are the ones they were captured on."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2501_19309_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic_bytes(workload: str):
    """DRAM bytes (read + write) per verification call from the ncu captures summarised under
    profiles/, or None when there is no capture of the present kernels."""
    try:
        with open(TRAFFIC_FILE) as f:
            t = json.load(f)
    except (OSError, ValueError):
        return None
    if t.get("kernel_source_sha256_16") != kernel_source_hash():
        return None
    e = t.get("workloads", {}).get(workload)
    return None if e is None else float(e["dram_bytes_per_call"])


def record_traffic(csv_specs) -> None:
    """csv_specs: 'workload=path[,path...]' items; every CSV is an `ncu --page raw --csv` export with
    dram__bytes_read.sum / dram__bytes_write.sum columns. The bytes of the first captured launch of
    each file are added up per workload (a workload whose call runs two kernels gives two files)."""
    import csv
    import re
    out = {"kernel_source_sha256_16": kernel_source_hash(), "workloads": {},
           "note": "dram__bytes_read.sum + dram__bytes_write.sum of one launch of each dominant kernel"}
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    for spec in csv_specs:
        name, paths = spec.split("=", 1)
        total, kernels = 0.0, []
        for path in paths.split(","):
            with open(path, newline="") as f:
                rows = [r for r in csv.reader(f) if r]
            hdr = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
            cols, units, first = rows[hdr], rows[hdr + 1], rows[hdr + 2]
            kname = first[cols.index("Kernel Name")]
            m = re.search(r"(\w+<[^>]*>)", kname)
            kernels.append(m.group(1) if m else kname.split("(")[0])
            for m in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                i = cols.index(m)
                total += float(first[i].replace(",", "")) * scale[units[i]]
        out["workloads"][name] = {"dram_bytes_per_call": total, "kernels": kernels}
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")


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
    traffic = ncu_traffic_bytes(wl.name)
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


RMS_EPS = 1e-5          # the epsilon of the RMSNorm option where a workload token asks for it
NO_OPTIONS = {"rule": "sampling", "top_k": 1, "rms_eps": None}


def parse_workload_token(tok: str):
    """'<id>[f][g|k][n]': workload id, then f = FP8 E4M3 head, g = greedy rule (top-K with K = 1),
    k = top-5 rule, n = final RMSNorm ahead of the LM head. Returns (workload or None, options)."""
    m = re.fullmatch(r"(\d+)(f?)([gk]?)(n?)", tok)
    if not m or int(m.group(1)) not in I.CONFIGS:
        return None, None
    wl = I.CONFIGS[int(m.group(1))]
    name = wl.name + ("-fp8" if m.group(2) else "")
    opts = dict(NO_OPTIONS)
    if m.group(3):
        opts.update(rule="topk", top_k=1 if m.group(3) == "g" else 5)
        name += "-greedy" if m.group(3) == "g" else "-top5"
    if m.group(4):
        opts["rms_eps"] = RMS_EPS
        name += "-rmsnorm"
    if name != wl.name:
        wl = wl.scaled(name, dtype="fp8" if m.group(2) else wl.dtype)
    return wl, opts


def oracle_step(inp: I.Inputs, seed: int, sequences, opts=None):
    from oracle import jd_oracle as O
    o = opts or NO_OPTIONS
    return O.jd_oracle_verify(inp.W, inp.w_judge, inp.b_judge, inp.H, inp.draft_tokens, inp.draft_logits,
                              inp.tau, seed, "judge_or_standard", sequences=sequences, w_scale=inp.w_scale,
                              rule=o["rule"], top_k=o["top_k"], rms_eps=o["rms_eps"])


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(inp: I.Inputs, steps: int, budget_s: float = 25.0, extra_warmup: int = 0, opts=None) -> dict:
    """The checker as it stands on a bounded sample: whole sequences b = 0, 1, ... of the workload.
    Step s uses verify seed s; "first" is the result of step 0 (kept for the parity check)."""
    wl = inp.wl
    t0 = time.perf_counter()
    oracle_step(inp, 0, [0], opts)
    one = time.perf_counter() - t0
    for _ in range(extra_warmup):          # untimed, on top of the sizing call above
        oracle_step(inp, 0, [0], opts)
    nseq = int(max(1, min(wl.B, budget_s / max(one, 1e-3) / max(steps, 1))))
    seqs = list(range(nseq))
    first = None
    t0 = time.perf_counter()
    for s in range(steps):
        r = oracle_step(inp, s, seqs, opts)
        first = first or r
    dt = time.perf_counter() - t0
    return {"value": nseq * wl.M * steps / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": "%d step(s) x %d of %d sequences (%d rows x V=%d x d=%d each), float64 numpy" %
                      (steps, nseq, wl.B, wl.M + 1, wl.V, wl.d),
            "seconds": dt, "first": first}


def parity_of(wl: I.Workload, got: dict, ref, rule: str = "sampling") -> dict:
    """Device outputs of verify seed 0 against the checker's result for the same inputs, under the
    rules of the parity tests (tests/jd_testlib.py: tolerances, margin exemptions, CDF intervals)."""
    tests_dir = os.path.join(ROOT, "tests")
    if tests_dir not in sys.path:
        sys.path.insert(0, tests_dir)
    import jd_testlib as T
    rep = T.Report()
    try:
        T.compare(got, ref, "judge_or_standard", wl.M, rep, rule=rule)
        ok, why = True, None
    except AssertionError as e:
        ok, why = False, str(e)[:200]
    out = {"sequences": rep.sequences, "ok": ok, "exempt": rep.exempt_accept + rep.exempt_judge,
           "exempt_len": rep.exempt_len, "token_exact": rep.token_exact, "token_in_margin": rep.token_in_margin,
           "max_rel_p": rep.max_rel_p, "max_rel_lse": rep.max_rel_lse, "max_abs_judge": rep.max_abs_judge}
    if why:
        out["failure"] = why
    return out


def config_of(wl: I.Workload, world: int, opts=None) -> dict:
    """The `config` object, identical in both arms."""
    o = opts or NO_OPTIONS
    return {"workload": wl.name, "B": wl.B, "M": wl.M, "d": wl.d, "V": wl.V, "mode": "judge_or_standard",
            "rule": o["rule"] if o["rule"] == "sampling" else "top-%d" % o["top_k"],
            "norm": "rms" if o["rms_eps"] else "none",
            "l2": "not flushed between calls: inputs larger than L2 (W is %.2f GB, L2 126 MB)" %
                  (wl.V * wl.d * (1 if wl.dtype == "fp8" else 2) / 1e9),
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def run_reference(args, wl, opts) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = I.make_inputs(wl, 0)
    # K timed steps after W warm-up steps, as asked, each step a bounded sample (whole sequences) of
    # the workload; only when K steps of even one sequence would run for more than ~5 minutes are
    # they cut down, and the line says so
    t0 = time.perf_counter()
    oracle_step(inp, 0, [0], opts)
    one = time.perf_counter() - t0
    steps = int(max(1, min(args.steps, 300.0 / max(one, 1e-3))))
    warmup = int(max(2, min(args.warmup, 60.0 / max(one, 1e-3))))   # the call above + time_oracle's sizing call + ...
    r = time_oracle(inp, steps, budget_s=max(60.0, one * steps), extra_warmup=warmup - 2, opts=opts)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": r["seconds"] / steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(wl, 1, opts),
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def log(msg: str) -> None:
    """Progress on stderr (the JSON line is the only thing on stdout)."""
    sys.stderr.write("[bench %7.1f s] %s\n" % (time.perf_counter() - T_START, msg))
    sys.stderr.flush()


def measure_workload(wl, args, torch, jd, device, data_seed, sample_clocks, opts=None):
    """Times K device-resident calls and K_e2e host-buffer calls of one workload on this rank."""
    o = dict(opts or NO_OPTIONS)
    log("%s: drawing inputs" % wl.name)
    inp = I.make_inputs(wl, data_seed)
    log("%s: inputs drawn" % wl.name)
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
    a_args = [ver.make_args(H, x, dl, inp.tau, s, "judge_or_standard", out=out, **o)[0] for s in range(8)]
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
    step(0)                                   # verify seed 0 once more: the outputs the parity check reads
    torch.cuda.synchronize(device)
    out0 = {k: v.detach().cpu().numpy().copy() for k, v in out.items()}

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
    h_args = [ver.make_args(hH, hx, hdl, inp.tau, s, "judge_or_standard", out=hout, host=True, **o)[0] for s in range(8)]
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
    log("%s: measured" % wl.name)
    res = dict(total_ms=total_ms, median_ms=statistics.median(per), min_ms=min(per), mean_ms=total_ms / K,
               variant=variant, launches=launches, clocks=clocks, e2e_s=e2e_s, e2e_steps=Ke, h2d=h2d, d2h=d2h,
               mean_accept=float(accepted.mean()), emitted_per_call=float((accepted + 1).sum(axis=1).mean()),
               stream_gbs=stream_gbs, graph_ms=graph_ms, inp=inp, out0=out0)
    del W, H, dl
    torch.cuda.empty_cache()
    return res


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="3", help="workload of the headline line: an id 1..4, optionally followed by "
                    "the option letters of --others; default: the 405B-shaped head, the largest single-GPU configuration")
    ap.add_argument("--others", default="2,1,4,3f,4f", help="comma list of further workloads summarised in the same "
                    "line: an id, then f = FP8 E4M3 head, g / k = greedy / top-5 rule, n = RMSNorm ahead of the head")
    ap.add_argument("--record-traffic", nargs="+", metavar="WORKLOAD=CSV[,CSV]", help="rewrite profiles/ncu_traffic.json "
                    "from ncu raw-page CSV exports and exit")
    ap.add_argument("--fp8", action="store_true", help="headline workload with an FP8 E4M3 head")
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay timing")
    args = ap.parse_args()
    if args.record_traffic:
        record_traffic(args.record_traffic)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    tok = args.config.strip()
    if args.fp8 and "f" not in tok:
        tok = re.sub(r"^(\d+)", r"\1f", tok)
    wl, opts = parse_workload_token(tok)
    if wl is None:
        ap.error("--config %s: not a workload" % args.config)

    if args.impl == "reference":
        run_reference(args, wl, opts)
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
    res = measure_workload(wl, args, torch, jd, device, data_seed=rank, sample_clocks=True, opts=opts)

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
            owl, oopts = parse_workload_token(tok)
            if owl is None or owl.name == wl.name:
                continue
            small.steps = max(50, min(args.steps, 300))
            small.e2e_steps = 10
            r = measure_workload(owl, small, torch, jd, device, data_seed=0, sample_clocks=True, opts=oopts)
            oparity = None
            if not args.no_cpu_baseline:      # the checker on the first sequence of this workload
                oparity = parity_of(owl, r["out0"], oracle_step(r["inp"], 0, [0], oopts), rule=oopts["rule"])
            e2e_note = None
            if owl.B * owl.M * owl.V * 4 > 100e6:
                e2e_note = ("%.0f MB of fp32 draft logits cross PCIe per host-buffer call" % (owl.B * owl.M * owl.V * 4 / 1e6))
            others[owl.name] = {
                "B": owl.B, "M": owl.M, "d": owl.d, "V": owl.V, "ms_per_step": r["mean_ms"],
                "median_ms": r["median_ms"], "value": owl.B * owl.M / (r["mean_ms"] * 1e-3), "unit": UNIT,
                "variant": VARIANT_NAMES.get(r["variant"], "?"), "kernel_launches_per_step": r["launches"],
                "rule": oopts["rule"] if oopts["rule"] == "sampling" else "top-%d" % oopts["top_k"],
                "norm": "rms" if oopts["rms_eps"] else "none", "steps": small.steps, "mean_accept_len": r["mean_accept"], "best_ms": r["min_ms"],
                "clocks": r["clocks"],
                "graph_replay_ms_per_step": r["graph_ms"],
                "emitted_tokens_per_s": r["emitted_per_call"] / (r["mean_ms"] * 1e-3),
                "e2e": {"value": owl.B * owl.M * r["e2e_steps"] / r["e2e_s"], "unit": UNIT,
                        "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"], "steps": r["e2e_steps"],
                        "note": e2e_note},
                "parity": oparity,
                "roofline": roofline_of(owl, peaks, r["mean_ms"], sustained=r["mean_ms"] * small.steps > 1000, which=which,
                                        stream_gbs=r["stream_gbs"])}

    if rank == 0:
        cpu, parity = None, None
        log("workloads done; CPU baseline")
        if not args.no_cpu_baseline:
            c = time_oracle(res["inp"], 1, opts=opts)
            cpu = {k: c[k] for k in ("value", "unit", "cores", "kind", "sample")}
            parity = parity_of(wl, res["out0"], c["first"], rule=opts["rule"])
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8" if wl.dtype == "fp8" else "bf16", "data": "synthetic",
            "config": config_of(wl, world, opts),
            "variant": VARIANT_NAMES.get(res["variant"], "?"), "mean_accept_len": res["mean_accept"],
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
            "parity": parity,
            "other_workloads": others,
        }
        print(json.dumps(line), flush=True)
    if args.dist:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
