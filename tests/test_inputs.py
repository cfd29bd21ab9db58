"""The seeded generators: shapes, determinism, storage format, and the statistics the
recipe promises (checked through the CPU checker's projection on a reduced vocabulary)."""
import numpy as np

from oracle import jd_oracle as O
from paper_2501_19309_b200 import inputs as I


def small(cfg, **kw):
    wl = I.CONFIGS[cfg]
    return wl.scaled(wl.name + "-small", **kw)


def test_published_shapes():
    c = I.CONFIGS
    assert (c[0].B, c[0].M, c[0].d, c[0].V, c[0].dtype) == (1, 4, 256, 1024, "f32")
    assert (c[1].B, c[1].M, c[1].d, c[1].V) == (1, 8, 4096, 128256)
    assert (c[2].B, c[2].M, c[2].d, c[2].V) == (4, 16, 8192, 128256)
    assert (c[3].B, c[3].M, c[3].d, c[3].V, c[3].forced_reject_at) == (1, 25, 16384, 128256, 12)
    assert (c[4].B, c[4].M, c[4].d, c[4].V, c[4].R) == (64, 16, 8192, 128256, 1088)


def test_bf16_round_trip_and_rounding():
    a = np.array([1.0, 1.00390625, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 0.0], dtype=np.float32)
    bits = I.f32_to_bf16_bits(a)
    back = I.bf16_bits_to_f32(bits)
    # ties to even: 1 + 2^-8 -> 1.0 ; 1 + 3*2^-8 -> 1 + 2^-6
    assert back.tolist() == [1.0, 1.0, 1.0, 1.015625, -2.5, 0.0]


def test_determinism_and_block_independence():
    wl = small(1, V=5000, d=64)
    a = I.make_inputs(wl, 3)
    b = I.make_inputs(wl, 3)
    for f in ("W", "H", "w_judge", "draft_tokens", "draft_logits"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert not np.array_equal(a.W, I.make_inputs(wl, 4).W)
    part = I.make_W_rows(wl, 3, 2000, 4100)
    assert np.array_equal(part, a.W[2000:4100])
    assert a.W.dtype == np.uint16 and a.H.shape == (1, 9, 64) and a.draft_logits.dtype == np.float32
    assert I.make_inputs(I.CONFIGS[0]).W.dtype == np.float32


def test_recipe_statistics():
    wl = small(1, V=20000, d=1024)
    inp = I.make_inputs(wl, 0)
    L = O.project_logits(inp.W, inp.H[0])
    x = inp.planted_tokens[0]
    planted = L[np.arange(wl.M + 1), x]
    assert np.all(np.abs(planted - wl.alpha) < 4 * wl.sigma + 0.2)
    mask = np.ones_like(L, dtype=bool)
    mask[np.arange(wl.M + 1), x] = False
    std = L[mask].std()
    assert abs(std - np.sqrt(wl.sigma ** 2 + wl.alpha ** 2 / wl.d)) < 0.02
    dl = inp.draft_logits[0]
    assert abs(dl.std() - wl.dl_std) < 0.02


def test_forced_rejection_rejects_in_every_mode():
    wl = small(3, V=4096, d=512, M=14)
    inp = I.make_inputs(wl, 0)
    k = wl.forced_reject_at
    for mode in ("standard", "judge", "judge_or_standard"):
        for seed in range(5):
            r = O.jd_oracle_verify(inp.W, inp.w_judge, inp.b_judge, inp.H, inp.draft_tokens,
                                   inp.draft_logits, inp.tau, seed, mode)
            assert r.accept_len[0] <= k
            assert r.masks[0, k] == 0
    assert abs(np.log(1 / r.judge_scores[0, k] - 1) - 4.0) < 0.05     # judge logit = -4


def test_per_sequence_and_per_row_alpha():
    wl2 = small(2, V=3000, d=256)
    wl4 = small(4, V=3000, d=256, B=6)
    for wl in (wl2, wl4):
        inp = I.make_inputs(wl, 1)
        assert inp.H.shape == (wl.B, wl.M + 1, wl.d)
        assert inp.draft_tokens.min() >= 0 and inp.draft_tokens.max() < wl.V
    assert I.make_inputs(wl2, 1).b_judge != 0.0
