"""jd_verify_static: the handle-free, allocation-free form of the verification call.

Who needs it: hosts that cannot allocate device memory when they verify a draft block, for
example a server whose own memory pool already owns the whole GPU, or a decode loop that must
not pay the synchronisation an allocation implies.  The entry point keeps the fused kernel's
scratch in a fixed array inside the library, so the test checks two things through the C ABI:
that it gives exactly what jd_verify (fused variant, handle-owned scratch) gives, and that a
second call right after the first, on a different and smaller block, is not disturbed by what
the first call left in the shared array.  Both calls are also compared with the CPU checker, so
the test does not rest on the handle path alone, and the device's free memory is read before
and after them: it must not move.  Floating-point outputs are compared with the tolerance
the other GPU tests use (relative 2e-3; judge scores 2e-5), integer outputs must be equal.
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

import jd_testlib as T
from paper_2501_19309_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _same(a: dict, b: dict):
    for k in ("accept_len", "next_token", "masks"):
        assert np.array_equal(a[k], b[k]), k
    for k in ("p_draft", "q_draft", "row_max", "row_lse"):
        assert np.allclose(a[k], b[k], rtol=T.REL_TOL, atol=0), k
    assert np.allclose(a["judge_scores"], b["judge_scores"], rtol=0, atol=T.JUDGE_ABS_TOL)


def test_static_entry_point_matches_handle_path_on_two_calls_in_a_row():
    import torch
    from paper_2501_19309_b200 import jd

    big = I.CONFIGS[2].scaled("static-big", B=4, M=16, d=256, V=128256)     # 68 rows, overflow tiles
    small = I.CONFIGS[1].scaled("static-small", B=1, M=8, d=256, V=50000)   # 9 rows, other vocabulary
    calls = []
    for wl, seed in ((big, 3), (small, 4)):
        inp = I.make_inputs(wl, 1)
        dev = T.upload(inp)
        ver = T.make_verifier(inp, dev)
        want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], inp.tau, seed, "judge_or_standard",
                                     variant="fused"))
        assert ver.device_status() == jd.JD_OK
        calls.append((wl, inp, dev, ver, seed, want))

    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    # output buffers first, then one warm-up call (the first call on a device looks up the scratch
    # address and loads the kernels); from here on the free memory of the device must stay put
    prepared = [ver.make_args(dev["H"], dev["x"], dev["dl"], inp.tau, seed, "judge_or_standard")
                for wl, inp, dev, ver, seed, want in calls]
    wl, inp, dev, ver, seed, _ = calls[1]
    assert jd.jd_verify_static(wl.d, wl.V, dev["W"].data_ptr(), dev["w"].data_ptr(), inp.b_judge, prepared[1][0],
                               status.data_ptr(), stream) == jd.JD_OK
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    outs = []
    for (wl, inp, dev, ver, seed, want), (args, out) in zip(calls, prepared):   # back to back, no sync in between
        st = jd.jd_verify_static(wl.d, wl.V, dev["W"].data_ptr(), dev["w"].data_ptr(), inp.b_judge, args,
                                 status.data_ptr(), stream)
        assert st == jd.JD_OK, jd.jd_status_string(st)
        outs.append(out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before         # nothing was allocated on the device
    assert int(status.item()) == jd.JD_OK
    for (wl, inp, dev, ver, seed, want), out in zip(calls, outs):
        got = T.to_numpy(out)
        _same(got, want)
        T.compare(got, T.run_oracle(inp, "judge_or_standard", seed=seed), "judge_or_standard", wl.M)

    # a draft token outside the vocabulary is clamped and reported in the caller's status word
    wl, inp, dev, ver, seed, _ = calls[1]
    x_bad = dev["x"].clone()
    x_bad[0, 2] = wl.V + 9
    args, _ = ver.make_args(dev["H"], x_bad, dev["dl"], inp.tau, seed)
    assert jd.jd_verify_static(wl.d, wl.V, dev["W"].data_ptr(), dev["w"].data_ptr(), inp.b_judge, args,
                               status.data_ptr(), stream) == jd.JD_OK
    torch.cuda.synchronize()
    assert int(status.item()) == jd.JD_ERR_BAD_TOKEN

    # sizes beyond the fixed scratch are refused with a clear status, nothing is launched
    wl, inp, dev, ver, seed, _ = calls[0]
    args, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], inp.tau, seed)
    args.B, args.M = 7, 16                                      # 119 rows > 96
    assert jd.jd_verify_static(wl.d, wl.V, dev["W"].data_ptr(), dev["w"].data_ptr(), inp.b_judge, args, 0,
                               stream) == jd.JD_ERR_UNSUPPORTED
    args.B, args.M = 4, 16
    assert jd.jd_verify_static(100, wl.V, dev["W"].data_ptr(), dev["w"].data_ptr(), inp.b_judge, args, 0,
                               stream) == jd.JD_ERR_UNSUPPORTED  # d not a multiple of 64
    for c in calls:
        c[3].close()
