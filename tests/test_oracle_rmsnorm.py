"""Pins for the checker's final RMS normalisation (the judge reads the embedding before it,
the LM head after it; Sec. 4.1 "Model design and training")."""
import math

import numpy as np

from oracle import jd_oracle as O


def problem(rng, B=2, M=3, d=6, V=7):
    W = rng.standard_normal((V, d))
    H = rng.standard_normal((B, M + 1, d)) * 3.0
    w = rng.standard_normal(d)
    x = rng.integers(0, V, size=(B, M)).astype(np.int32)
    dl = rng.standard_normal((B, M, V))
    return W, H, w, x, dl


def test_logits_follow_the_definition_by_hand_loops():
    rng = np.random.default_rng(0)
    W, H, w, x, dl = problem(rng)
    eps = 1e-3
    r = O.jd_oracle_verify(W, w, 0.1, H, x, dl, 0.5, 0, rms_eps=eps, keep_logits=True)
    for b in range(2):
        for j in range(4):
            ms = sum(float(H[b, j, k]) ** 2 for k in range(6)) / 6
            for v in range(7):
                want = sum(float(W[v, k]) * float(H[b, j, k]) for k in range(6)) / math.sqrt(ms + eps)
                assert math.isclose(r.logits[b][j, v], want, rel_tol=1e-12, abs_tol=1e-13)


def test_scale_invariance_of_the_target_side_and_not_of_the_judge():
    rng = np.random.default_rng(1)
    W, H, w, x, dl = problem(rng)
    a = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 3, rms_eps=0.0)
    c = np.array([0.5, 2.0, 7.0, 0.1])[None, :, None]              # a different positive factor per row
    b = O.jd_oracle_verify(W, w, 0.0, H * c, x, dl, 0.5, 3, rms_eps=0.0)
    assert np.allclose(a.row_lse, b.row_lse, rtol=1e-12) and np.allclose(a.p_draft, b.p_draft, rtol=1e-10)
    assert (a.masks & 1 == b.masks & 1).all()
    assert not np.allclose(a.judge_scores, b.judge_scores)          # the judge sees the raw embedding
    raw = O.jd_oracle_verify(W, w, 0.0, H * c, x, dl, 0.5, 3)
    assert np.allclose(b.judge_scores, raw.judge_scores, rtol=1e-15)


def test_rows_of_unit_rms_are_left_alone():
    rng = np.random.default_rng(2)
    W, H, w, x, dl = problem(rng)
    H = np.sign(H)                                                   # every entry +-1: rms = 1
    a = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, rms_eps=0.0, keep_logits=True)
    b = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, keep_logits=True)
    for k in a.logits:
        assert np.allclose(a.logits[k], b.logits[k], rtol=1e-15)
    assert (a.accept_len == b.accept_len).all() and (a.next_token == b.next_token).all()
