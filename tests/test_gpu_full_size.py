"""Parity at the published workload sizes, in the launch configuration the benchmark times
(variant chosen automatically): every listed configuration, mode, seed and threshold against the
CPU checker, which recomputes whole sequences.  Every case adds its counts (margin exemptions,
exactly equal next tokens, largest deviations) to the session's parity table."""
import numpy as np
import pytest

import jd_testlib as T
from paper_2501_19309_b200 import inputs as I

pytestmark = pytest.mark.gpu

ALL_MODES = ("standard", "judge", "judge_or_standard")


def full_case(cfg, data_seed, cases, sequences=None, expect_variant=None, rule="sampling", top_k=1, fp8=False,
              check_logits=False, label=None):
    """cases: list of (mode, tau or None). Returns (report, inputs, outputs of the last case)."""
    import torch
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[cfg]
    if fp8:
        wl = wl.scaled(wl.name + "-fp8", dtype="fp8")
    inp = I.make_inputs(wl, data_seed)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    rep = T.Report()
    got = None
    for mode, tau in cases:
        tau = inp.tau if tau is None else tau
        out = ver.alloc_outputs(wl.B, wl.M, debug_logits=check_logits)
        ver.verify(dev["H"], dev["x"], dev["dl"], tau, inp.seed, mode, rule=rule, top_k=top_k, out=out)
        assert ver.device_status() == jd.JD_OK
        if expect_variant:
            assert ver.launch_info()[0] == jd.VARIANTS[expect_variant]
        got = T.to_numpy(out)
        ref = T.run_oracle(inp, mode, tau=tau, sequences=sequences, rule=rule, top_k=top_k, keep_logits=check_logits)
        T.compare(got, ref, mode, wl.M, rep, rule=rule)
        if check_logits:
            T.compare_logits(got["logits_debug"], ref, rep)
    assert ver.damaged_guards() == 0
    if fp8:
        assert T.fp8_row_code_mismatches(inp, dev) == 0
    ver.close()
    del dev
    torch.cuda.empty_cache()
    T.record(label or (wl.name + ("" if rule == "sampling" else "-top%d" % top_k)), rep)
    return rep, inp, got


@pytest.mark.parametrize("data_seed", range(10))
def test_cfg1_8b_head_every_seed_and_threshold(data_seed):
    """Seeds 0..9 (data seed = verify seed), the threshold sweep on each; the two single-test modes on
    seed 0, together with the element-wise logits of the tensor-core kernel."""
    cases = [("judge_or_standard", 0.3), ("judge_or_standard", 0.5), ("judge_or_standard", 0.7)]
    if data_seed == 0:
        cases += [("standard", None), ("judge", None)]
    rep, _, _ = full_case(1, data_seed, cases, expect_variant="fused", check_logits=(data_seed == 0))
    assert rep.sequences == len(cases)
    if data_seed == 0:
        assert 0 < rep.max_rel_logit <= T.REL_TOL


def test_cfg2_70b_head_every_sequence():
    rep, _, _ = full_case(2, 0, [("judge_or_standard", None)], expect_variant="fused")
    assert rep.sequences == 4


def test_cfg3_405b_head_all_modes_forced_rejection():
    wl = I.CONFIGS[3]
    for mode in ALL_MODES:
        rep, inp, got = full_case(3, 0, [(mode, None)], expect_variant="fused")
        assert rep.sequences == 1
        assert got["accept_len"][0] <= wl.forced_reject_at           # rejection forced at slot 12
        assert got["masks"][0, wl.forced_reject_at] == 0


def test_cfg3_masks_independent_of_mode():
    wl = I.CONFIGS[3].scaled("cfg3-narrow", d=1024)
    inp = I.make_inputs(wl, 0)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    masks = [T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], inp.tau, 0, m))["masks"] for m in ALL_MODES]
    assert np.array_equal(masks[0], masks[1]) and np.array_equal(masks[0], masks[2])
    for mode in ("standard", "judge"):
        got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], inp.tau, 0, mode))
        T.compare(got, T.run_oracle(inp, mode, seed=0), mode, wl.M)
    ver.close()


def test_cfg4_batched_every_sequence_against_cuda_core_variant_and_sixteen_against_checker():
    """Seed 0: every one of the 64 sequences against the CUDA-core variant on the device at full d and
    V, and every fourth sequence against the CPU checker."""
    import torch
    rep, inp, got = full_case(4, 0, [("judge_or_standard", None)], sequences=list(range(0, 64, 4)),
                              expect_variant="batched")
    assert rep.sequences == 16
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    ref = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], inp.tau, inp.seed, "judge_or_standard", variant="simt"))
    assert np.array_equal(got["accept_len"], ref["accept_len"])
    assert np.array_equal(got["masks"], ref["masks"])
    assert np.allclose(got["row_lse"], ref["row_lse"], rtol=0, atol=2e-4)
    assert np.allclose(got["p_draft"], ref["p_draft"], rtol=2e-4)
    assert np.allclose(got["judge_scores"], ref["judge_scores"], rtol=0, atol=T.JUDGE_ABS_TOL)
    ver.close()
    del dev
    torch.cuda.empty_cache()


@pytest.mark.parametrize("data_seed", [1, 2, 3, 4])
def test_cfg4_remaining_seeds_eight_sequences_each(data_seed):
    seqs = [(7 * data_seed + 8 * i) % 64 for i in range(8)]
    rep, _, _ = full_case(4, data_seed, [("judge_or_standard", None)], sequences=seqs, expect_variant="batched")
    assert rep.sequences == 8


def test_cfg1_greedy_and_top5_rules():
    full_case(1, 0, [("standard", None), ("judge_or_standard", None)], expect_variant="fused", rule="topk", top_k=1)
    full_case(1, 0, [("standard", None)], expect_variant="fused", rule="topk", top_k=5)


def test_cfg4_greedy_rule_sampled_sequences():
    rep, _, _ = full_case(4, 0, [("judge_or_standard", None)], sequences=[5, 21, 40, 60], expect_variant="batched",
                          rule="topk", top_k=1)
    assert rep.sequences == 4


def test_cfg3_fp8_head_full_size():
    rep, _, _ = full_case(3, 0, [("judge_or_standard", None)], expect_variant="fused", fp8=True)
    assert rep.sequences == 1


def test_cfg4_fp8_head_sampled_sequences():
    rep, _, _ = full_case(4, 0, [("judge_or_standard", None)], sequences=list(range(0, 64, 8)),
                          expect_variant="batched", fp8=True)
    assert rep.sequences == 8
