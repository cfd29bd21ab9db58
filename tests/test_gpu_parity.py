"""GPU parity: the library, called through its C ABI, against the CPU checker on the same
seeded inputs.  Every test here needs a B200."""
import numpy as np
import pytest

import jd_testlib as T
from oracle import jd_oracle as O
from paper_2501_19309_b200 import inputs as I

pytestmark = pytest.mark.gpu

MODES = ("standard", "judge", "judge_or_standard")


def run_case(wl, data_seed, modes=MODES, variant="auto", seeds=None, tau=None, check_logits=False,
             sequences=None, expect_variant=None, rule="sampling", top_k=1, rms_eps=None, record_as=None):
    from paper_2501_19309_b200 import jd
    inp = I.make_inputs(wl, data_seed)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    rep = T.Report()
    for mode in modes:
        for seed in (seeds or [inp.seed]):
            out = ver.alloc_outputs(wl.B, wl.M, debug_logits=check_logits)
            ver.verify(dev["H"], dev["x"], dev["dl"], inp.tau if tau is None else tau, seed, mode,
                       variant=variant, out=out, rule=rule, top_k=top_k, rms_eps=rms_eps)
            assert ver.device_status() == jd.JD_OK
            if expect_variant is not None:
                assert ver.launch_info()[0] == jd.VARIANTS[expect_variant]
            got = T.to_numpy(out)
            ref = T.run_oracle(inp, mode, seed=seed, tau=tau, sequences=sequences, keep_logits=check_logits,
                               rule=rule, top_k=top_k, rms_eps=rms_eps)
            T.compare(got, ref, mode, wl.M, rep, rule=rule)
            if check_logits:
                T.compare_logits(got["logits_debug"], ref, rep)
    assert ver.damaged_guards() == 0          # no kernel wrote past the end of a workspace region
    if wl.dtype == "fp8":
        assert T.fp8_row_code_mismatches(inp, dev) == 0
    ver.close()
    if record_as:
        T.record(record_as, rep, bound=False)
    return rep


def test_philox_bit_equality_with_checker():
    import torch
    from paper_2501_19309_b200 import jd
    n = 60000
    rng = np.random.default_rng(0)
    b = rng.integers(0, 1 << 20, n).astype(np.int32)
    slot = rng.integers(0, 64, n).astype(np.int32)
    stream = rng.integers(0, 2, n).astype(np.int32)
    b[:4] = [0, 1, 2 ** 31 - 1, 5]
    for seed in (0, 1, (0xDEADBEEF << 32) | 0x12345678):
        tb, ts, tst = (torch.from_numpy(a).cuda() for a in (b, slot, stream))
        out = torch.empty(n, dtype=torch.float32, device="cuda")
        assert jd.jd_philox_uniforms(seed, tb.data_ptr(), ts.data_ptr(), tst.data_ptr(), n, out.data_ptr()) == 0
        got = out.cpu().numpy().astype(np.float64)
        m = n if seed == 0 else 3000
        want = np.array([O.uniform24(seed, int(b[i]), int(slot[i]), int(stream[i])) for i in range(m)])
        assert np.array_equal(got[:m], want)


def test_cfg0_tiny_fp32_all_modes_with_logits():
    rep = run_case(I.CONFIGS[0], 0, check_logits=True, expect_variant="simt")
    assert rep.sequences == 3 and rep.max_rel_logit < 1e-4


@pytest.mark.parametrize("B,M,d,V", [(1, 1, 64, 130), (2, 5, 192, 1037), (3, 33, 100, 515), (5, 8, 256, 4096 + 77)])
def test_simt_bf16_ragged_shapes(B, M, d, V):
    wl = I.CONFIGS[2].scaled("ragged", B=B, M=M, d=d, V=V)
    rep = run_case(wl, 1, variant="simt", seeds=[0, 1, 2], check_logits=True)
    assert rep.sequences == 9 * B


def test_simt_fp32_ragged():
    wl = I.CONFIGS[0].scaled("ragged32", B=2, M=3, d=77, V=333)
    run_case(wl, 2, variant="simt", seeds=[0, 1], check_logits=True)


def test_tau_extremes_and_literal_resampling():
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[1].scaled("small", d=256, V=2048, B=3, M=6)
    inp = I.make_inputs(wl, 5)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    res = {}
    for tau in (0.0, 1.0):
        for mode in MODES:
            out = ver.verify(dev["H"], dev["x"], dev["dl"], tau, 3, mode)
            got = T.to_numpy(out)
            ref = T.run_oracle(inp, mode, seed=3, tau=tau)
            T.compare(got, ref, mode, wl.M)
            res[(tau, mode)] = got
    # tau = 1: the judge never accepts, so the OR mode is the standard test (Sec. 4.1)
    assert np.array_equal(res[(1.0, "judge_or_standard")]["accept_len"], res[(1.0, "standard")]["accept_len"])
    assert np.array_equal(res[(1.0, "judge_or_standard")]["next_token"], res[(1.0, "standard")]["next_token"])
    assert (res[(1.0, "judge")]["accept_len"] == 0).all()
    assert (res[(0.0, "judge")]["accept_len"] == wl.M).all()          # sigmoid > 0 always
    out = ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 3, "standard", resample="target_p")
    ref = O.jd_oracle_verify(inp.W, inp.w_judge, inp.b_judge, inp.H, inp.draft_tokens, inp.draft_logits, 0.5, 3,
                             "standard", "target_p")
    T.compare(T.to_numpy(out), ref, "standard", wl.M)
    ver.close()


def test_or_mode_monotone_on_device():
    wl = I.CONFIGS[2].scaled("small", d=128, V=1500, B=8, M=12)
    inp = I.make_inputs(wl, 9)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    for seed in range(4):
        a = {m: T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, m))["accept_len"] for m in MODES}
        assert (a["judge_or_standard"] >= np.maximum(a["standard"], a["judge"])).all()
        assert (a["judge_or_standard"] <= wl.M).all() and (a["standard"] >= 0).all()
    ver.close()


def test_q_equals_p_accepts_everything():
    import torch
    wl = I.CONFIGS[1].scaled("small", d=128, V=1000, B=2, M=7)
    inp = I.make_inputs(wl, 4)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    out = ver.alloc_outputs(wl.B, wl.M, debug_logits=True)
    ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "standard", variant="simt", out=out)
    dl = out["logits_debug"][:, :wl.M, :].contiguous()          # the device's own logits as draft logits
    for seed in range(5):
        got = T.to_numpy(ver.verify(dev["H"], dev["x"], dl, 0.5, seed, "standard", variant="simt"))
        assert (got["accept_len"] == wl.M).all()
        assert np.allclose(got["p_draft"], got["q_draft"], rtol=1e-5)
    ver.close()


def test_zero_draft_probability_and_bad_token_status():
    import torch
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[1].scaled("small", d=64, V=600, B=1, M=3)
    inp = I.make_inputs(wl, 6)
    inp.draft_logits[0, 0, inp.draft_tokens[0, 0]] = -np.inf
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "standard"))
    ref = T.run_oracle(inp, "standard", seed=0)
    T.compare(got, ref, "standard", wl.M)
    assert got["q_draft"][0, 0] == 0.0 and got["masks"][0, 0] & 1
    x_bad = dev["x"].clone()
    x_bad[0, 1] = wl.V + 5
    ver.verify(dev["H"], x_bad, dev["dl"], 0.5, 0, "standard")
    assert ver.device_status() == jd.JD_ERR_BAD_TOKEN
    ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "standard")
    assert ver.device_status() == jd.JD_OK                   # the status word is per call
    ver.close()


def test_argument_validation_returns_codes():
    import torch
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[1].scaled("small", d=64, V=600, B=2, M=3)
    inp = I.make_inputs(wl, 7)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    a, out = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0)
    assert jd.jd_verify(ver.h, a) == jd.JD_OK
    for field, value in (("B", 0), ("B", 3), ("M", 0), ("M", 4), ("tau", 1.5), ("tau", -0.1), ("mode", 3),
                         ("resample", 2), ("variant", 9), ("H", None), ("draft_tokens", None),
                         ("accept_len", None), ("p_draft", None)):
        a2, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, out=out)
        setattr(a2, field, value)
        assert jd.jd_verify(ver.h, a2) == jd.JD_ERR_INVALID_ARG, field
    a3, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, out=out)
    a3.H = dev["H"].data_ptr() + 2                           # misaligned
    assert jd.jd_verify(ver.h, a3) == jd.JD_ERR_INVALID_ARG
    for field in ("draft_logits", "draft_tokens", "accept_len", "judge_scores", "q_draft", "row_lse"):
        a5, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, out=out)
        setattr(a5, field, getattr(a5, field) + 2)           # a float / int32 array off its 4-byte boundary
        assert jd.jd_verify(ver.h, a5) == jd.JD_ERR_INVALID_ARG, field
    v2 = jd.Verifier(2, 3, wl.d, wl.V, "bf16")
    a4, _ = v2.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, out=out)
    assert jd.jd_verify(v2.h, a4) == jd.JD_ERR_INVALID_ARG   # no head registered yet
    v2.close()
    with pytest.raises(jd.JdError):
        jd.jd_create(jd.jd_config_t(1, 1, 64, 600, 5, 0))
    ver.close()


@pytest.mark.parametrize("variant,B,M,d,V", [("fused", 2, 5, 128, 40000), ("simt", 2, 5, 96, 4000),
                                             ("batched", 12, 9, 128, 20000)])
def test_draft_logits_view_that_is_only_4_byte_aligned(variant, B, M, d, V):
    """A slice of a larger buffer: the draft logits start one float past a 16-byte boundary although
    V % 4 == 0. The kernels must take their 4-byte loads (never a misaligned 16-byte one) and give
    the same results as for an aligned copy."""
    import torch
    wl = I.CONFIGS[2].scaled("dlview-" + variant, B=B, M=M, d=d, V=V)
    inp = I.make_inputs(wl, 21)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    big = torch.empty(dev["dl"].numel() + 8, dtype=torch.float32, device="cuda")
    assert big.data_ptr() % 16 == 0
    view = big[1:1 + dev["dl"].numel()].view(B, M, V)
    view.copy_(dev["dl"])
    assert view.data_ptr() % 16 == 4 and view.is_contiguous()
    for seed in (0, 1):
        want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant=variant))
        got = T.to_numpy(ver.verify(dev["H"], dev["x"], view, 0.5, seed, "judge_or_standard", variant=variant))
        from paper_2501_19309_b200 import jd
        assert ver.device_status() == jd.JD_OK
        T.compare(got, T.run_oracle(inp, "judge_or_standard", seed=seed), "judge_or_standard", M)
        for k in ("accept_len", "masks", "next_token"):
            assert np.array_equal(want[k], got[k]), k
        assert np.allclose(want["q_draft"], got["q_draft"], rtol=1e-5)
    ver.close()


def test_host_buffer_entry_point_matches_device_call_and_is_repeatable():
    import torch
    wl = I.CONFIGS[2].scaled("small", d=256, V=3000, B=4, M=9)
    inp = I.make_inputs(wl, 8)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    d1 = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 11, "judge_or_standard"))
    d2 = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 11, "judge_or_standard"))
    hostH = torch.from_numpy(inp.H).view(torch.bfloat16).pin_memory()
    hx = torch.from_numpy(inp.draft_tokens).pin_memory()
    hdl = torch.from_numpy(inp.draft_logits).pin_memory()
    h1 = {k: v.numpy().copy() for k, v in ver.verify_host(hostH, hx, hdl, 0.5, 11, "judge_or_standard").items()}
    for k in d1:
        assert np.array_equal(d1[k], d2[k]), k              # run-to-run determinism
        assert np.array_equal(d1[k], h1[k]), k
    ver.close()


# ------------------------------------------------------------------ fused tensor-core variant
FUSED_SHAPES = [
    (1, 1, 64, 130),          # two vocabulary tiles, ragged tail, n_pad 16
    (2, 3, 64, 1000),         # only 8 of the CTAs own a tile
    (1, 8, 256, 128256),      # 8B-head rows: n_pad 16, seven tiles per CTA
    (1, 25, 192, 50000),      # n_pad 32, ragged last tile
    (3, 20, 128, 40000),      # n_pad 64
    (4, 16, 128, 128256),     # 70B-head rows: n_pad 80, one tile per CTA overflows to shared memory
    (5, 15, 128, 128256 + 77),  # same with a ragged last tile
    (6, 15, 64, 128256),      # n_pad 96, two overflow tiles
    (1, 8, 2048, 40000),      # n_pad 16 with 32 k-slices: early sweep + late sweep on pairs of k-slices
    (2, 12, 320, 60000),      # odd number of k-slices (5): one slice per ring slot, no paired late sweep
]


@pytest.mark.parametrize("B,M,d,V", FUSED_SHAPES)
def test_fused_variant_parity(B, M, d, V):
    wl = I.CONFIGS[2].scaled("fused-%d-%d-%d-%d" % (B, M, d, V), B=B, M=M, d=d, V=V)
    rep = run_case(wl, 3, variant="fused", seeds=[0, 1], expect_variant="fused", check_logits=True,
                   record_as="small-shapes-fused")
    assert rep.sequences == 6 * B and 0 < rep.max_rel_logit <= T.REL_TOL


def test_fused_matches_simt_variant_on_device():
    wl = I.CONFIGS[2].scaled("x", B=4, M=16, d=256, V=128256)
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    for seed in range(3):
        a = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant="fused"))
        b = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant="simt"))
        a2 = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant="fused"))
        for k in a:
            assert np.array_equal(a[k], a2[k]), k                     # repeatable bit for bit
        assert np.array_equal(a["accept_len"], b["accept_len"])
        assert np.array_equal(a["masks"], b["masks"])
        assert np.allclose(a["row_lse"], b["row_lse"], rtol=0, atol=1e-4)
        assert np.allclose(a["p_draft"], b["p_draft"], rtol=1e-4)
    ver.close()


def test_fused_unsupported_shapes_are_refused_not_faked():
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[2].scaled("x", B=8, M=16, d=128, V=2000)           # 136 rows > 96
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    a, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, variant="fused")
    assert jd.jd_verify(ver.h, a) == jd.JD_ERR_UNSUPPORTED
    ver.close()


# ------------------------------------------------------------------ batched tensor-core variant
BATCHED_SHAPES = [
    (8, 16, 128, 128256),       # 136 rows: two row blocks, the second mostly padding
    (3, 50, 128, 5000 + 77),    # 153 rows, ragged last vocabulary block
    (64, 16, 64, 128256),       # the serving shape's rows (1088) at a narrow d
    (2, 3, 64, 700),            # fewer tiles than CTAs
    (40, 2, 128, 33000),        # many short sequences
    (130, 3, 64, 9000),         # more sequences than one second-pass launch takes: 64 + 64 + 2
    (100, 1, 128, 128256),      # 64 + 36 at the full vocabulary
]


@pytest.mark.parametrize("B,M,d,V", BATCHED_SHAPES)
def test_batched_variant_parity(B, M, d, V):
    wl = I.CONFIGS[4].scaled("batched-%d-%d-%d-%d" % (B, M, d, V), B=B, M=M, d=d, V=V)
    seqs = None if B <= 8 else sorted({0, 1, B // 2, B - 1})
    rep = run_case(wl, 5, variant="batched", modes=("judge_or_standard", "standard"), seeds=[0, 1],
                   sequences=seqs, expect_variant="batched", check_logits=True, record_as="small-shapes-batched")
    assert rep.sequences == 4 * (B if seqs is None else len(seqs)) and 0 < rep.max_rel_logit <= T.REL_TOL


@pytest.mark.parametrize("B,M", [(48, 7), (150, 3)])
def test_batched_matches_simt_on_every_sequence(B, M):
    wl = I.CONFIGS[4].scaled("x", B=B, M=M, d=128, V=20000)
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    for seed in range(2):
        a = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant="batched"))
        b = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, seed, "judge_or_standard", variant="simt"))
        assert np.array_equal(a["accept_len"], b["accept_len"])
        assert np.array_equal(a["masks"], b["masks"])
        assert np.mean(a["next_token"] == b["next_token"]) > 0.9      # CDF-edge cases may differ by a token
        assert np.allclose(a["row_lse"], b["row_lse"], rtol=0, atol=1e-4)
        assert np.allclose(a["p_draft"], b["p_draft"], rtol=1e-4)
    # greedy / top-K rule: the batched variant ranks each row in its one GEMM pass against a logit
    # computed ahead of it; the CUDA-core variant ranks against its own logits in a second pass
    for k in (1, 3, 50):
        a = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard", variant="batched",
                                  rule="topk", top_k=k))
        b = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard", variant="simt",
                                  rule="topk", top_k=k))
        assert ver.device_status() == 0
        assert np.mean(a["masks"] == b["masks"]) > 0.995              # a near tie at the K-th rank may differ
        same = a["accept_len"] == b["accept_len"]
        assert same.mean() > 0.97
        assert np.array_equal(a["next_token"][same], b["next_token"][same])   # argmax of the same row
    ver.close()


# ------------------------------------------------------------------ greedy / top-K rule (all variants)
TOPK_CASES = [
    ("simt", 2, 5, 100, 515, [1, 3, 515]),
    ("simt", 3, 4, 64, 1300, [1, 40]),
    ("fused", 1, 8, 128, 128256, [1, 5]),
    ("fused", 4, 16, 128, 128256, [1, 2, 1000]),
    ("fused", 2, 3, 64, 1000, [1, 1000]),
    ("fused", 6, 15, 64, 40000 + 77, [1, 10]),        # overflow tiles + ragged last tile
    ("batched", 8, 16, 128, 128256, [1, 4]),
    ("batched", 3, 50, 128, 5000 + 77, [1, 100, 5077]),
    ("batched", 20, 12, 192, 33000 + 5, [1, 2]),      # three row blocks, three k-steps, ragged vocabulary
]


@pytest.mark.parametrize("variant,B,M,d,V,ks", TOPK_CASES)
def test_topk_rule_parity(variant, B, M, d, V, ks):
    wl = I.CONFIGS[2].scaled("topk-%s-%d-%d-%d-%d" % (variant, B, M, d, V), B=B, M=M, d=d, V=V)
    for k in ks:
        rep = run_case(wl, 7, variant=variant, modes=("standard", "judge_or_standard"), seeds=[0],
                       expect_variant=variant, rule="topk", top_k=k)
        assert rep.sequences == 2 * B


def test_greedy_accepts_the_targets_own_tokens_and_topk_all_accepts_everything():
    import torch
    wl = I.CONFIGS[1].scaled("greedy", B=3, M=6, d=128, V=30000)
    inp = I.make_inputs(wl, 3)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    out = ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "standard", rule="topk", top_k=wl.V)
    assert (T.to_numpy(out)["accept_len"] == wl.M).all()                 # K = V: the draft alone decides
    # planted tokens are the target's greedy tokens here (alpha = 4): greedy verification accepts them
    got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "standard", rule="greedy"))
    ref = T.run_oracle(inp, "standard", seed=0, rule="greedy")
    T.compare(got, ref, "standard", wl.M, rule="topk")
    assert (got["accept_len"] == ref.accept_len).all() and got["accept_len"].min() >= 1
    # a wrong token at slot 2 is rejected and corrected to the target's token
    x2 = dev["x"].clone()
    x2[:, 2] = (x2[:, 2] + 1) % wl.V
    got2 = T.to_numpy(ver.verify(dev["H"], x2, dev["dl"], 0.5, 0, "standard", rule="greedy"))
    full = got["accept_len"] == wl.M
    assert (got2["accept_len"][full] == 2).all()
    assert (got2["next_token"][full] == inp.draft_tokens[full, 2]).all()
    ver.close()


# ------------------------------------------------------------------ final RMS normalisation (all variants)
NORM_CASES = [
    ("simt", 2, 5, 100, 515, "f32"),
    ("simt", 3, 4, 192, 1300, "bf16"),
    ("fused", 1, 8, 256, 128256, "bf16"),
    ("fused", 4, 16, 128, 40000 + 77, "bf16"),
    ("fused", 6, 15, 64, 128256, "bf16"),            # overflow tiles
    ("batched", 8, 16, 128, 128256, "bf16"),
    ("batched", 40, 2, 128, 33000, "bf16"),
]


@pytest.mark.parametrize("variant,B,M,d,V,dtype", NORM_CASES)
def test_rms_normalised_head_parity(variant, B, M, d, V, dtype):
    wl = I.CONFIGS[2].scaled("norm-%s-%d-%d-%d-%d" % (variant, B, M, d, V), B=B, M=M, d=d, V=V, dtype=dtype,
                             alpha_range=(2.0, 9.0))           # rows of clearly different norms
    seqs = None if B <= 8 else [0, B // 2, B - 1]
    rep = run_case(wl, 11, variant=variant, modes=("judge_or_standard", "standard"), seeds=[0, 1],
                   sequences=seqs, expect_variant=variant, rms_eps=1e-5, check_logits=True)
    assert rep.sequences == 4 * (B if seqs is None else len(seqs))
    if variant == "fused":
        rep = run_case(wl, 11, variant=variant, modes=("standard",), seeds=[0], rule="greedy", rms_eps=1e-5)


def test_rms_norm_makes_target_side_scale_invariant_on_device():
    import torch
    wl = I.CONFIGS[1].scaled("inv", B=2, M=6, d=256, V=20000)
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    a = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 4, "standard", rms_eps=0.0))
    H4 = (dev["H"].float() * 4.0).to(torch.bfloat16)            # exact in bf16: a power of two
    b = T.to_numpy(ver.verify(H4, dev["x"], dev["dl"], 0.5, 4, "standard", rms_eps=0.0))
    assert np.allclose(a["row_lse"], b["row_lse"], rtol=0, atol=1e-4)
    assert np.array_equal(a["accept_len"], b["accept_len"]) and np.array_equal(a["masks"] & 1, b["masks"] & 1)
    assert not np.allclose(a["judge_scores"], b["judge_scores"])     # the judge reads the raw rows
    ver.close()


# ------------------------------------------------------------------ FP8 E4M3 head
FP8_CASES = [
    ("simt", 2, 5, 100, 515),
    ("simt", 3, 4, 256, 1300),
    ("fused", 1, 8, 256, 128256),
    ("fused", 4, 16, 128, 40000 + 77),
    ("fused", 1, 25, 512, 128256),
    ("fused", 6, 15, 128, 128256),            # overflow tiles
    ("fused", 4, 16, 256, 128256),            # 80 padded rows, two k-slices of codes: early sweep + paired late sweep
    ("batched", 8, 16, 128, 128256),          # two row blocks of the FP8 GEMM, the second mostly padding
    ("batched", 3, 50, 256, 5000 + 77),       # ragged last vocabulary block, two k-steps
    ("batched", 64, 16, 128, 20000),          # the serving shape's rows
    ("batched", 100, 2, 128, 9000),           # two second-pass launches (64 + 36 sequences)
]


@pytest.mark.parametrize("variant,B,M,d,V", FP8_CASES)
def test_fp8_head_parity(variant, B, M, d, V):
    wl = I.CONFIGS[2].scaled("fp8-%s-%d-%d-%d-%d" % (variant, B, M, d, V), B=B, M=M, d=d, V=V, dtype="fp8")
    rep = run_case(wl, 13, variant=variant, modes=("judge_or_standard", "standard"), seeds=[0, 1],
                   expect_variant=variant, check_logits=True, record_as="small-shapes-fp8-" + variant)
    assert rep.sequences == 4 * B and 0 < rep.max_rel_logit <= T.REL_TOL
    if variant != "simt":
        run_case(wl, 13, variant=variant, modes=("standard",), seeds=[0], rule="greedy", rms_eps=1e-5)
        run_case(wl, 13, variant=variant, modes=("judge_or_standard",), seeds=[0], rule="topk", top_k=7)


def test_fp8_fused_matches_fp8_simt_and_row_codes_match_checker():
    from oracle import jd_oracle as O
    wl = I.CONFIGS[2].scaled("fp8x", B=4, M=16, d=256, V=128256, dtype="fp8")
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    a = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 1, "judge_or_standard", variant="fused"))
    b = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 1, "judge_or_standard", variant="simt"))
    assert np.array_equal(a["accept_len"], b["accept_len"]) and np.array_equal(a["masks"], b["masks"])
    assert np.allclose(a["row_lse"], b["row_lse"], rtol=0, atol=1e-4)
    c = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 1, "judge_or_standard", variant="batched"))
    assert np.array_equal(a["accept_len"], c["accept_len"]) and np.array_equal(a["masks"], c["masks"])
    assert np.allclose(a["row_lse"], c["row_lse"], rtol=0, atol=1e-4)
    assert np.allclose(a["p_draft"], c["p_draft"], rtol=1e-4)
    # an FP8 handle refuses the bf16 registration call
    from paper_2501_19309_b200 import jd
    assert jd.jd_set_head(ver.h, dev["W"].data_ptr(), dev["w"].data_ptr(), 0.0) == jd.JD_ERR_INVALID_ARG
    ver.close()
    # the tensor-core variants need whole 128-byte k-steps of codes: d = 192 is refused, not faked
    wl = I.CONFIGS[2].scaled("fp8y", B=2, M=3, d=192, V=1000, dtype="fp8")
    inp = I.make_inputs(wl, 2)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    for variant in ("fused", "batched"):
        args, _ = ver.make_args(dev["H"], dev["x"], dev["dl"], 0.5, 0, variant=variant)
        assert jd.jd_verify(ver.h, args) == jd.JD_ERR_UNSUPPORTED
    ver.close()


# ------------------------------------------------------------------ failure path and edge shapes
def test_bounded_wait_reports_timeout_and_handle_stays_usable():
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[1].scaled("small", d=128, V=3000, B=2, M=4)
    inp = I.make_inputs(wl, 1)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    assert jd.jd_selftest_timeout(ver.h, 2000) == jd.JD_OK        # a wait nothing can satisfy, ~0.1 ms
    assert ver.device_status() == jd.JD_ERR_TIMEOUT
    assert jd.jd_selftest_timeout(ver.h, 0) == jd.JD_ERR_INVALID_ARG
    got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard"))
    assert ver.device_status() == jd.JD_OK                        # the next call starts clean
    T.compare(got, T.run_oracle(inp, "judge_or_standard", seed=0), "judge_or_standard", wl.M)
    ver.close()


@pytest.mark.parametrize("B,M,d,V", [(1, 8, 256, 128256), (4, 16, 128, 128256), (6, 15, 64, 128256)])
def test_fused_calls_stop_after_an_uncleared_timeout_and_recover_once_it_was_read(B, M, d, V):
    """Back-to-back fused calls share no memset: the kernel keeps its barrier counters clean and tags its
    status writes. A call that gave up leaves the counters unknown, so every later call must give up at once
    (device status JD_ERR_TIMEOUT, no wait runs its full limit) until the host has read the status; the call
    after that starts from a cleared block and is correct again."""
    import time
    import torch
    from paper_2501_19309_b200 import jd
    wl = I.CONFIGS[2].scaled("stale-%d-%d-%d-%d" % (B, M, d, V), B=B, M=M, d=d, V=V)
    inp = I.make_inputs(wl, 3)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    ref = T.run_oracle(inp, "judge_or_standard", seed=0)
    for _ in range(3):                                            # launches 0, 1, 2: both counter sets in use
        got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard", variant="fused"))
    assert ver.device_status() == jd.JD_OK
    T.compare(got, ref, "judge_or_standard", M)
    assert jd.jd_selftest_stale_timeout(ver.h, torch.cuda.current_stream().cuda_stream) == jd.JD_OK
    t0 = time.perf_counter()
    for _ in range(2):                                            # both give up at once
        ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard", variant="fused")
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0                         # nowhere near a wait's full limit
    assert ver.device_status() == jd.JD_ERR_TIMEOUT               # read: the next call clears the block
    for _ in range(2):
        got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 0, "judge_or_standard", variant="fused"))
        assert ver.device_status() == jd.JD_OK
        T.compare(got, ref, "judge_or_standard", M)
    assert ver.damaged_guards() == 0
    ver.close()


@pytest.mark.parametrize("B,M,d,V", [(1, 95, 64, 2000), (48, 1, 64, 5000), (1, 1, 64, 2), (2, 2, 64, 129)])
def test_extreme_shapes(B, M, d, V):
    wl = I.CONFIGS[2].scaled("edge-%d-%d-%d-%d" % (B, M, d, V), B=B, M=M, d=d, V=V)
    seqs = None if B <= 4 else [0, B - 1]
    for variant in ("fused", "simt"):
        run_case(wl, 17, variant=variant, modes=("judge_or_standard",), seeds=[0], sequences=seqs,
                 expect_variant=variant)


def test_boundary_tokens_and_forced_outcomes():
    import torch
    wl = I.CONFIGS[1].scaled("bt", B=3, M=5, d=128, V=128 * 9)
    inp = I.make_inputs(wl, 19)
    inp.draft_tokens[0, :] = [0, wl.V - 1, 127, 128, wl.V - 129]           # tile edges and vocabulary ends
    inp.draft_tokens[1, :] = inp.draft_tokens[1, 0]                         # the same token in every slot
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    for variant in ("fused", "simt"):
        for tau, mode in ((0.0, "judge"), (1.0, "judge"), (0.5, "standard")):   # all accepted / all rejected / mixed
            got = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], tau, 2, mode, variant=variant))
            T.compare(got, T.run_oracle(inp, mode, seed=2, tau=tau), mode, wl.M)
            if mode == "judge":
                assert (got["accept_len"] == (wl.M if tau == 0.0 else 0)).all()
    ver.close()


def test_host_entry_point_with_batched_and_fp8_handles():
    import torch
    for dtype, B, M in (("bf16", 8, 16), ("fp8", 2, 6)):
        wl = I.CONFIGS[2].scaled("host-" + dtype, B=B, M=M, d=128, V=30000, dtype=dtype)
        inp = I.make_inputs(wl, 23)
        dev = T.upload(inp)
        ver = T.make_verifier(inp, dev)
        want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 5, "judge_or_standard"))
        hH = torch.from_numpy(inp.H).view(torch.bfloat16).pin_memory()
        hx = torch.from_numpy(inp.draft_tokens).pin_memory()
        hdl = torch.from_numpy(inp.draft_logits).pin_memory()
        got = {k: v.numpy().copy() for k, v in ver.verify_host(hH, hx, hdl, 0.5, 5, "judge_or_standard").items()}
        for k in want:
            assert np.array_equal(want[k], got[k]), (dtype, k)
        ver.close()


def test_stream_read_probe_reads_every_word_once():
    import torch
    from paper_2501_19309_b200 import jd
    rng = np.random.default_rng(5)
    for nwords in (4, 4 * 2048 * 4 * 148 + 4 * 37, 12345 * 4 + 3):     # one 16-byte word; ragged groups; 3 words ignored
        host = rng.integers(0, 2 ** 32, size=nwords, dtype=np.uint32)
        dev = torch.from_numpy(host.view(np.int32)).cuda()
        sink = torch.zeros(1, dtype=torch.int32, device="cuda")
        assert jd.jd_stream_read_probe(dev.data_ptr(), nwords * 4, sink.data_ptr()) == jd.JD_OK
        torch.cuda.synchronize()
        want = np.bitwise_xor.reduce(host[: nwords // 4 * 4])
        assert np.uint32(sink.cpu().numpy().view(np.uint32)[0]) == want
    assert jd.jd_stream_read_probe(0, 64, sink.data_ptr()) == jd.JD_ERR_INVALID_ARG
    assert jd.jd_stream_read_probe(dev.data_ptr() + 4, 64, sink.data_ptr()) == jd.JD_ERR_INVALID_ARG


# ------------------------------------------------------------------ streams and graphs
@pytest.mark.parametrize("variant,B,M,d,V", [("fused", 3, 7, 128, 40000), ("batched", 24, 5, 128, 30000),
                                             ("simt", 2, 4, 96, 3000)])
def test_call_can_be_captured_in_a_cuda_graph_and_replayed(variant, B, M, d, V):
    import torch
    wl = I.CONFIGS[2].scaled("graph-" + variant, B=B, M=M, d=d, V=V)
    inp = I.make_inputs(wl, 31)
    dev = T.upload(inp)
    ver = T.make_verifier(inp, dev)
    want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 3, "judge_or_standard", variant=variant))
    out = ver.alloc_outputs(B, M)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 3, "judge_or_standard", variant=variant, out=out,
                   stream=torch.cuda.current_stream())
    for _ in range(3):
        for v in out.values():
            v.zero_()
        g.replay()
        got = T.to_numpy(out)
        for k in want:
            assert np.array_equal(want[k], got[k]), (variant, k)
    del g
    ver.close()


def test_two_handles_on_two_streams_do_not_disturb_each_other():
    import torch
    cases = []
    for i, (B, M, V) in enumerate([(4, 16, 50000), (2, 9, 128256)]):
        wl = I.CONFIGS[2].scaled("two-%d" % i, B=B, M=M, d=128, V=V)
        inp = I.make_inputs(wl, 40 + i)
        dev = T.upload(inp)
        ver = T.make_verifier(inp, dev)
        want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 9, "judge_or_standard"))
        cases.append((inp, dev, ver, want, torch.cuda.Stream(), ver.alloc_outputs(B, M)))
    torch.cuda.synchronize()
    for _ in range(5):                      # interleaved, nothing synchronises between the two streams
        for inp, dev, ver, want, st, out in cases:
            ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, 9, "judge_or_standard", out=out, stream=st)
    torch.cuda.synchronize()
    for inp, dev, ver, want, st, out in cases:
        got = T.to_numpy(out)
        for k in want:
            assert np.array_equal(want[k], got[k]), k
        ver.close()


@pytest.mark.parametrize("variant,B,M,d,V,dtype,pinned", [
    ("simt", 3, 5, 100, 4000, "bf16", True),       # the copy of the draft logits is waited for by an event
    ("fused", 2, 12, 128, 128256, "bf16", True),   # ... by the kernel itself, on a flag the copy's stream sets
    ("fused", 2, 12, 128, 128256, "bf16", False),  # pageable buffers: the copy is staged, nothing overlaps
    ("batched", 20, 6, 128, 60000, "bf16", True),  # ... by stream order on the side stream
    ("batched", 100, 2, 128, 9000, "fp8", True),
])
def test_host_call_with_draft_logits_in_flight(variant, B, M, d, V, dtype, pinned):
    """jd_verify_host copies the draft logits on a second stream while the verification starts; every
    variant must wait for them where it first reads them, call after call, with changing inputs."""
    import torch
    wl = I.CONFIGS[2].scaled("inflight-" + variant, B=B, M=M, d=d, V=V, dtype=dtype)
    ver = None
    for data_seed in (50, 51, 52):
        inp = I.make_inputs(wl, data_seed)
        dev = T.upload(inp)
        if ver is None:
            ver = T.make_verifier(inp, dev)
        else:
            ver.set_head(dev["W"], dev["w"], inp.b_judge, w_scale=dev.get("w_scale"))
        want = T.to_numpy(ver.verify(dev["H"], dev["x"], dev["dl"], 0.5, data_seed, "judge_or_standard", variant=variant))
        hH = torch.from_numpy(inp.H).view(torch.bfloat16)
        hx = torch.from_numpy(inp.draft_tokens)
        hdl = torch.from_numpy(inp.draft_logits)
        if pinned:
            hH, hx, hdl = hH.pin_memory(), hx.pin_memory(), hdl.pin_memory()
        got = ver.verify_host(hH, hx, hdl, 0.5, data_seed, "judge_or_standard", variant=variant)
        got = {k: v.numpy().copy() for k, v in got.items()}
        from paper_2501_19309_b200 import jd
        assert ver.device_status() == jd.JD_OK
        for k in want:
            assert np.array_equal(want[k], got[k]), (variant, data_seed, k)
    ver.close()


# ------------------------------------------------------------------ the C ABI from C
def test_plain_c_program_calls_the_library():
    """tests/c_abi/jd_c_caller.c (C99, gcc, no Python or torch in the process) runs one host-buffer
    verification through the C ABI; its outputs are checked against the CPU checker like any other."""
    import os
    import shutil
    import struct
    import subprocess
    import tempfile
    from paper_2501_19309_b200 import jd
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cuda = "/usr/local/cuda"
    if shutil.which("gcc") is None or not os.path.exists(cuda + "/lib64/libcudart.so"):
        pytest.skip("gcc or libcudart is not installed")
    wl = I.CONFIGS[2].scaled("c-caller", B=3, M=7, d=128, V=40000)
    inp = I.make_inputs(wl, 61)
    mode = "judge_or_standard"
    libdir = os.path.dirname(jd.library_path())
    with tempfile.TemporaryDirectory() as tmp:
        exe, prob, res = (os.path.join(tmp, n) for n in ("caller", "problem.bin", "result.bin"))
        build = ["gcc", "-std=c99", "-O1", "-I", os.path.join(root, "include"), "-I", cuda + "/include",
                 os.path.join(root, "tests", "c_abi", "jd_c_caller.c"), "-o", exe, "-L", libdir, "-ljd_b200",
                 "-L", cuda + "/lib64", "-lcudart", "-Wl,-rpath," + libdir, "-Wl,-rpath," + cuda + "/lib64"]
        proc = subprocess.run(build, capture_output=True, text=True)
        assert proc.returncode == 0, proc.stderr
        with open(prob, "wb") as f:
            f.write(struct.pack("<5i2fQ", wl.B, wl.M, wl.d, wl.V, jd.MODES[mode], inp.tau, inp.b_judge, inp.seed))
            for a in (inp.W, inp.w_judge, inp.H, inp.draft_tokens, inp.draft_logits):
                f.write(np.ascontiguousarray(a).tobytes())
        proc = subprocess.run([exe, prob, res], capture_output=True, text=True, timeout=300)
        assert proc.returncode == 0, proc.stderr
        raw = open(res, "rb").read()
    B, M, R = wl.B, wl.M, wl.B * (wl.M + 1)
    off = 0

    def take(dtype, n):
        nonlocal off
        a = np.frombuffer(raw, dtype=dtype, count=n, offset=off)
        off += a.nbytes
        return a
    status, variant, launches = take(np.int32, 3)
    assert status == jd.JD_OK and variant == jd.JD_VARIANT_FUSED and launches >= 1
    got = dict(accept_len=take(np.int32, B), next_token=take(np.int32, B),
               judge_scores=take(np.float32, B * M).reshape(B, M), p_draft=take(np.float32, B * M).reshape(B, M),
               q_draft=take(np.float32, B * M).reshape(B, M), masks=take(np.uint8, B * M).reshape(B, M),
               row_max=take(np.float32, R).reshape(B, M + 1), row_lse=take(np.float32, R).reshape(B, M + 1))
    assert off == len(raw)
    ref = T.run_oracle(inp, mode)
    rep = T.compare(got, ref, mode, M)
    assert rep.sequences == B
