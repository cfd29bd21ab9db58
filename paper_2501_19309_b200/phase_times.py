"""Where a fused verification call spends its time: per-phase global-timer stamps of the fused kernel.

Needs the phase-stamp build of the library (``python -m paper_2501_19309_b200.build --stamps``), in which
thread 0 of every CTA records the GPU's global timer at the phase boundaries of the call, and a B200.

Usage: ``python -m paper_2501_19309_b200.phase_times [workloads, default 1,2,3; a trailing f = FP8 head]``

For every workload (the synthetic shapes of ``inputs.CONFIGS``) it runs batches of back-to-back calls,
reads the stamps of the last call of each batch (of a batched-variant call: those of its second pass) and prints, per phase, the minimum / median / maximum over
the CTAs of the median over batches, in microseconds from the first CTA's start, then the distance between
one call's last stamp and the next call's first, and the time per call of a longer back-to-back loop.
"""
from __future__ import annotations

import ctypes
import os
import sys

import numpy as np

PKG = os.path.dirname(os.path.abspath(__file__))
os.environ.setdefault("JD_LIBRARY", os.path.join(PKG, "libjd_b200_stamps.so"))

from . import inputs as I  # noqa: E402
from . import jd  # noqa: E402

CTAS, SLOTS = 256, 16
PHASES = [(0, "start of the epilogue"), (1, "draft statistics + judge dots done"), (12, "early sweep complete"),
          (14, "early tiles' statistics done"), (2, "W stream complete"), (3, "row statistics done"), (4, "barrier 1 passed"), (5, "fold done"),
          (6, "barrier 2 passed"), (7, "decisions done"), (8, "sampling masses done"), (9, "barrier 3 passed"),
          (10, "owner found"), (11, "end of the epilogue")]


def read_stamps() -> np.ndarray:
    buf = np.zeros(CTAS * SLOTS, dtype=np.uint64)
    st = jd.jd_debug_phase_stamps(buf.ctypes.data_as(ctypes.c_void_p).value, buf.size)
    if st != jd.JD_OK:
        raise jd.JdError(st, "jd_debug_phase_stamps (is this the --stamps build?)")
    return buf.reshape(CTAS, SLOTS).astype(np.int64)


def main() -> None:
    import torch
    jd.load()
    dev = torch.device("cuda", 0)
    for tok in (sys.argv[1] if len(sys.argv) > 1 else "1,2,3").split(","):
        fp8 = tok.endswith("f")
        wl = I.CONFIGS[int(tok.rstrip("f"))]
        if fp8:
            wl = wl.scaled(wl.name + "-fp8", dtype="fp8")
        inp = I.make_inputs(wl, 0)
        W = torch.from_numpy(inp.W).to(dev) if fp8 else torch.from_numpy(inp.W).view(torch.bfloat16).to(dev)
        ws = torch.from_numpy(inp.w_scale).to(dev) if fp8 else None
        H = torch.from_numpy(inp.H).view(torch.bfloat16).to(dev)
        w = torch.from_numpy(inp.w_judge).view(torch.bfloat16).to(dev)
        x = torch.from_numpy(inp.draft_tokens).to(dev)
        dl = torch.from_numpy(inp.draft_logits).to(dev)
        ver = jd.Verifier(wl.B, wl.M, wl.d, wl.V, "fp8" if fp8 else "bf16", 0)
        ver.set_head(W, w, inp.b_judge, w_scale=ws)
        out = ver.alloc_outputs(wl.B, wl.M)
        # more than 96 rows: the batched variant, whose second pass is the fused kernel in its sample-only mode
        variant = "fused" if wl.B * (wl.M + 1) <= 96 else "auto"
        args = [ver.make_args(H, x, dl, inp.tau, s, "judge_or_standard", out=out, variant=variant)[0] for s in range(8)]
        stream = torch.cuda.current_stream(dev)

        def run(n):
            for i in range(n):
                st = jd.jd_verify(ver.h, args[i % 8], stream.cuda_stream)
                if st != jd.JD_OK:
                    raise jd.JdError(st, "jd_verify")

        run(30)
        torch.cuda.synchronize()
        n_ctas = torch.cuda.get_device_properties(dev).multi_processor_count
        rel, gaps = [], []
        for _ in range(9):
            run(20)
            torch.cuda.synchronize()
            s = read_stamps()[:n_ctas]
            t0 = s[:, 0].min()
            rel.append((s - t0) / 1000.0)
            gaps.append((t0 - s[:, 13].max()) / 1000.0)
        r = np.median(np.stack(rel), axis=0)
        print("== %s: us from the first CTA's start (min / median / max over %d CTAs)" % (wl.name, n_ctas))
        for k, name in PHASES:
            col = r[:, k]
            if (col <= 0).all():      # a phase this call does not have (its slot still holds an older or no stamp)
                continue
            print("  %-38s %8.1f %8.1f %8.1f" % (name, col.min(), np.median(col), col.max()))
        print("  %-38s %8.1f" % ("next call's first stamp after the last", float(np.median(gaps))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run(200)
        e1.record(stream)
        torch.cuda.synchronize()
        print("  %-38s %8.1f" % ("per call, 200 back to back", e0.elapsed_time(e1) / 200 * 1e3), flush=True)
        assert ver.device_status() == jd.JD_OK
        ver.close()
        del W, H, dl
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
