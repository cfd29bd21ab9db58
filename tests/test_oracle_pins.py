"""Pins for the CPU checker: closed forms, invariants, special cases, brute force.

Each test pins the checker to something other than itself: integer arithmetic done by
hand loops, the closed-form acceptance law of speculative sampling, exact rational
arithmetic, or a separately written textbook routine.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import jd_oracle as O


# ---------------------------------------------------------------- helpers (test-side, independent)
def softmax_py(row):
    m = max(row)
    e = [math.exp(v - m) for v in row]
    s = math.fsum(e)
    return [v / s for v in e]


def tiny_problem(rng, B, M, d, V, scale=1.0):
    W = rng.standard_normal((V, d)) * scale
    H = rng.standard_normal((B, M + 1, d))
    w = rng.standard_normal(d)
    x = rng.integers(0, V, size=(B, M)).astype(np.int32)
    dl = rng.standard_normal((B, M, V)) * 1.5
    return W, H, w, x, dl


# ---------------------------------------------------------------- projection + softmax
def test_projection_matches_integer_hand_loops():
    # integer-valued inputs: every dot product is an exact integer; a transposed operand or
    # a wrong index cannot survive non-square shapes and asymmetric data
    rng = np.random.default_rng(1)
    V, d, rows = 7, 5, 3
    W = rng.integers(-9, 10, size=(V, d)).astype(np.float32)
    Hb = rng.integers(-9, 10, size=(rows, d)).astype(np.float32)
    L = O.project_logits(W, Hb, vocab_chunk=3)      # chunk smaller than V: ragged slabs
    for j in range(rows):
        for v in range(V):
            acc = 0
            for k in range(d):
                acc += int(Hb[j, k]) * int(W[v, k])
            assert L[j, v] == acc


def test_projection_widens_bf16_bit_patterns_exactly():
    # 0x3F80 = 1.0, 0xC000 = -2.0, 0x3F00 = 0.5 in bfloat16
    W = np.array([[0x3F80, 0xC000], [0x3F00, 0x3F80]], dtype=np.uint16)
    Hb = np.array([[0x3F80, 0x3F80]], dtype=np.uint16)
    L = O.project_logits(W, Hb)
    assert L.tolist() == [[-1.0, 1.5]]


def test_softmax_normalises_and_matches_independent_formula():
    rng = np.random.default_rng(2)
    W, H, w, x, dl = tiny_problem(rng, 1, 3, 6, 11, scale=2.0)
    res = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed=3, keep_logits=True)
    L = res.logits[0]
    for j in range(4):
        p = np.exp(L[j] - res.row_lse[0, j])
        assert abs(p.sum() - 1.0) < 1e-12
        ref = softmax_py([float(np.dot(H[0, j], W[v])) for v in range(11)])
        assert np.allclose(p, ref, rtol=1e-12, atol=0)
        assert res.row_max[0, j] == L[j].max()
    for j in range(3):
        assert math.isclose(res.p_draft[0, j], softmax_py(list(L[j]))[x[0, j]], rel_tol=1e-12)
        assert math.isclose(res.q_draft[0, j], softmax_py(list(dl[0, j]))[x[0, j]], rel_tol=1e-12)


def test_first_distribution_depends_on_context_row_only():
    # p_1 is a function of the context alone (Sec. 3.1): changing draft rows must not move it
    rng = np.random.default_rng(3)
    W, H, w, x, dl = tiny_problem(rng, 1, 3, 6, 9)
    r1 = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed=0)
    H2 = H.copy()
    H2[0, 1:] += 1.0
    r2 = O.jd_oracle_verify(W, w, 0.0, H2, x, dl, 0.5, seed=0)
    assert r1.row_lse[0, 0] == r2.row_lse[0, 0] and r1.p_draft[0, 0] == r2.p_draft[0, 0]
    assert r1.row_lse[0, 1] != r2.row_lse[0, 1]


# ---------------------------------------------------------------- acceptance law (closed form)
def test_accept_length_law_by_enumeration():
    """P(accept_len = k | x) = prod_{j<k} beta_j * (1 - beta_k), beta = min(1, p/q) (Eq. 4)."""
    rng = np.random.default_rng(4)
    V, M, d, G = 3, 2, 4, 32
    W, H, w, _, dl = tiny_problem(rng, 1, M, d, V)
    grid = (np.arange(G) + 0.5) / G
    for xs in itertools.product(range(V), repeat=M):
        x = np.array([xs], dtype=np.int32)
        beta = []
        for j in range(M):
            p = softmax_py([float(np.dot(H[0, j], W[v])) for v in range(V)])
            q = softmax_py(list(dl[0, j]))
            beta.append(min(1.0, p[xs[j]] / q[xs[j]]))
        n_acc = [int(np.sum(grid < bj)) for bj in beta]       # grid points that accept slot j
        expect = {0: (G - n_acc[0]) * G, 1: n_acc[0] * (G - n_acc[1]), 2: n_acc[0] * n_acc[1]}
        got = {0: 0, 1: 0, 2: 0}
        for u0 in grid:
            for u1 in grid:
                r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed=0, mode="standard",
                                       u_accept=np.array([[u0, u1]]), u_sample=np.array([0.5]))
                got[int(r.accept_len[0])] += 1
        assert got == expect, (xs, beta)


def test_emitted_token_law_is_target_distribution():
    """With x ~ q: q(t) min(1,p/q) + (1 - beta_total) r(t)/sum(r) = p(t): integrate the checker's
    decisions over dyadic grids of both uniforms and over x weighted by q."""
    rng = np.random.default_rng(5)
    V, d, G, G2 = 4, 4, 64, 256
    W, H, w, _, dl = tiny_problem(rng, 1, 1, d, V, scale=1.5)
    p = softmax_py([float(np.dot(H[0, 0], W[v])) for v in range(V)])
    q = softmax_py(list(dl[0, 0]))
    gu = (np.arange(G) + 0.5) / G
    gs = (np.arange(G2) + 0.5) / G2
    emitted = np.zeros(V)
    for xt in range(V):
        x = np.array([[xt]], dtype=np.int32)
        # accept decisions do not depend on u_sample and vice versa: two 1-D sweeps
        acc = [int(O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, "standard",
                                      u_accept=np.array([[u]]), u_sample=np.array([0.5])).accept_len[0])
               for u in gu]
        n_acc = sum(acc)
        emitted[xt] += q[xt] * n_acc / G
        if n_acc < G:
            u_rej = gu[acc.index(0)]
            cnt = np.zeros(V)
            for us in gs:
                r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, "standard",
                                       u_accept=np.array([[u_rej]]), u_sample=np.array([us]))
                assert r.accept_len[0] == 0
                cnt[int(r.next_token[0])] += 1
            # the residual never returns a token with p <= q
            for t in range(V):
                if p[t] <= q[t]:
                    assert cnt[t] == 0
            emitted += q[xt] * (1 - n_acc / G) * cnt / G2
    assert abs(emitted.sum() - 1.0) < 1e-12
    assert np.max(np.abs(emitted - np.array(p))) < 1.0 / G + 1.0 / G2 + 1e-9


def test_q_equals_p_accepts_every_token_in_standard_mode():
    rng = np.random.default_rng(6)
    B, M, d, V = 3, 5, 8, 33
    W, H, w, x, _ = tiny_problem(rng, B, M, d, V)
    dl = np.einsum("bjk,vk->bjv", H[:, :M], W)       # draft logits = target logits -> q = p
    for seed in range(20):
        r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed, mode="standard")
        assert (r.accept_len == M).all()
        assert (r.masks & 1).all()


def test_zero_draft_probability_accepts_iff_target_positive():
    rng = np.random.default_rng(7)
    W, H, w, x, dl = tiny_problem(rng, 1, 2, 4, 5)
    dl = dl.copy()
    dl[0, 0, x[0, 0]] = -np.inf                      # q(x_0) = 0, p(x_0) > 0 -> accept
    r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 1, mode="standard")
    assert r.q_draft[0, 0] == 0.0 and (r.masks[0, 0] & 1) == 1


# ---------------------------------------------------------------- judge
def test_judge_special_cases_pin_row_and_formula():
    rng = np.random.default_rng(8)
    B, M, d, V = 2, 4, 6, 7
    W, H, w, x, dl = tiny_problem(rng, B, M, d, V)
    b0 = 0.3
    r = O.jd_oracle_verify(W, np.zeros(d), b0, H, x, dl, 0.5, 0)
    assert np.allclose(r.judge_scores, 1 / (1 + math.exp(-b0)), rtol=1e-15)
    for k in (0, 3):
        e = np.zeros(d)
        e[k] = 1.0
        r = O.jd_oracle_verify(W, e, b0, H, x, dl, 0.5, 0)
        for b in range(B):
            for j in range(M):
                # the judge for draft token j reads the embedding produced by feeding it: row j+1
                assert math.isclose(r.judge_scores[b, j], 1 / (1 + math.exp(-(H[b, j + 1, k] + b0))),
                                    rel_tol=1e-14)
    # d + 1 parameters: a scalar logit per token (Sec. 4.1 "Model design")
    assert r.judge_scores.shape == (B, M)


def test_judge_threshold_is_strict_and_tau_one_never_accepts():
    rng = np.random.default_rng(9)
    W, H, w, x, dl = tiny_problem(rng, 2, 3, 4, 5)
    r = O.jd_oracle_verify(W, np.zeros(4), 0.0, H, x, dl, 0.5, 0, mode="judge")   # s = 0.5 exactly
    assert (r.judge_scores == 0.5).all() and (r.masks >> 1 == 0).all() and (r.accept_len == 0).all()
    r = O.jd_oracle_verify(W, w * 50, 0.0, H, x, dl, 1.0, 0, mode="judge")       # saturating scores
    assert (r.masks >> 1 == 0).all()


def test_prefix_rule_exhaustive_helper():
    for M in range(1, 11):
        for m in range(1 << M):
            z = [(m >> j) & 1 for j in range(M)]
            first_zero = ((~m) & (m + 1)).bit_length() - 1     # lowest clear bit
            assert O.accepted_prefix_length(z) == min(first_zero, M)


def test_prefix_rule_through_the_whole_checker():
    # judge mode with w = e_0 and H[b, j+1, 0] = +-10 realises any mask bit pattern
    rng = np.random.default_rng(10)
    M, d, V = 6, 4, 5
    W, H, _, x, dl = tiny_problem(rng, 1, M, d, V)
    e0 = np.zeros(d)
    e0[0] = 1.0
    for m in range(1 << M):
        Hm = H.copy()
        for j in range(M):
            Hm[0, j + 1, 0] = 10.0 if (m >> j) & 1 else -10.0
        r = O.jd_oracle_verify(W, e0, 0.0, Hm, x, dl, 0.5, 0, mode="judge")
        want = next((j for j in range(M) if not (m >> j) & 1), M)
        assert r.accept_len[0] == want
        assert [int(v) >> 1 for v in r.masks[0]] == [(m >> j) & 1 for j in range(M)]


def test_or_mode_is_monotone_and_consistent():
    rng = np.random.default_rng(11)
    for trial in range(30):
        B, M, d, V = 2, int(rng.integers(1, 7)), 5, int(rng.integers(2, 12))
        W, H, w, x, dl = tiny_problem(rng, B, M, d, V)
        rs = {m: O.jd_oracle_verify(W, w, 0.1, H, x, dl, 0.5, trial, mode=m)
              for m in ("standard", "judge", "judge_or_standard")}
        a_or = rs["judge_or_standard"].accept_len
        assert (a_or >= np.maximum(rs["standard"].accept_len, rs["judge"].accept_len)).all()
        assert ((0 <= a_or) & (a_or <= M)).all()
        # the individual tests do not depend on the mode
        assert (rs["standard"].masks == rs["judge"].masks).all()
        assert (rs["standard"].masks == rs["judge_or_standard"].masks).all()
        for b in range(B):
            z = [(int(v) & 1) | (int(v) >> 1) for v in rs["judge_or_standard"].masks[b]]
            assert a_or[b] == next((j for j, zj in enumerate(z) if not zj), M)


# ---------------------------------------------------------------- judge off == textbook routine
def textbook_speculative_sampling(p_rows, q_rows, x, u, u2):
    """Standard speculative sampling of one sequence, written independently of the checker:
    accept while u < p/q; at the first rejection draw from norm(max(0, p - q)); after a full
    block draw from the extra row."""
    M = len(x)
    a = M
    for j in range(M):
        pj, qj = p_rows[j][x[j]], q_rows[j][x[j]]
        ok = (pj > 0) if qj == 0 else (u[j] < min(1.0, pj / qj))
        if not ok:
            a = j
            break
    if a < M:
        r = [max(0.0, pv - qv) for pv, qv in zip(p_rows[a], q_rows[a])]
        if sum(r) == 0:
            r = list(p_rows[a])
    else:
        r = list(p_rows[M])
    T = u2 * sum(r)
    acc = 0.0
    tok = None
    for t, rv in enumerate(r):
        acc += rv
        if acc > T:
            tok = t
            break
    if tok is None:
        tok = max(t for t, rv in enumerate(r) if rv > 0)
    return a, tok


def test_judge_off_reduces_to_textbook_speculative_sampling():
    rng = np.random.default_rng(12)
    for trial in range(40):
        B, M, d, V = 1, int(rng.integers(1, 6)), 6, int(rng.integers(2, 20))
        W, H, w, x, dl = tiny_problem(rng, B, M, d, V)
        u = rng.integers(0, 1 << 24, size=(B, M)) / 2.0 ** 24
        u2 = rng.integers(0, 1 << 24, size=B) / 2.0 ** 24
        p_rows = [softmax_py([float(np.dot(H[0, j], W[v])) for v in range(V)]) for j in range(M + 1)]
        q_rows = [softmax_py(list(dl[0, j])) for j in range(M)]
        a, tok = textbook_speculative_sampling(p_rows, q_rows, list(x[0]), list(u[0]), float(u2[0]))
        r_std = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, "standard", u_accept=u, u_sample=u2)
        r_tau1 = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 1.0, 0, "judge_or_standard", u_accept=u, u_sample=u2)
        assert (int(r_std.accept_len[0]), int(r_std.next_token[0])) == (a, tok)
        assert (int(r_tau1.accept_len[0]), int(r_tau1.next_token[0])) == (a, tok)   # delta = 1 reduces to SD


def test_philox_path_equals_explicit_uniform_path():
    rng = np.random.default_rng(13)
    B, M, d, V = 3, 4, 5, 9
    W, H, w, x, dl = tiny_problem(rng, B, M, d, V)
    seed = 77
    r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed, "judge_or_standard")
    u = np.array([[O.uniform24(seed, b, j, O.STREAM_ACCEPT) for j in range(M)] for b in range(B)])
    u2 = np.array([O.uniform24(seed, b, int(r.accept_len[b]), O.STREAM_SAMPLE) for b in range(B)])
    r2 = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, seed, "judge_or_standard", u_accept=u, u_sample=u2)
    assert (r.accept_len == r2.accept_len).all() and (r.next_token == r2.next_token).all()
    assert (r.u_accept == u).all() and (r.u_sample == u2).all()


# ---------------------------------------------------------------- sampler
def test_inverse_cdf_exact_rational_brute_force():
    # dyadic weights: float64 prefix sums are exact, so the checker must agree with exact
    # rational arithmetic everywhere, including on and next to every CDF boundary
    rng = np.random.default_rng(14)
    for V in range(1, 9):
        r = rng.integers(0, 6, size=V).astype(np.float64) / 8.0
        if r.sum() == 0:
            r[rng.integers(0, V)] = 0.25
        total = Fraction(float(r.sum()))
        cum = np.cumsum(r)
        us = set()
        for c in cum:
            k = int(Fraction(float(c)) / total * (1 << 24))
            for dk in (-1, 0, 1):
                if 0 <= k + dk < (1 << 24):
                    us.add(k + dk)
        us |= {0, (1 << 24) - 1}
        for k in sorted(us):
            u = k / 2.0 ** 24
            T = Fraction(k, 1 << 24) * total
            acc = Fraction(0)
            want = None
            for t in range(V):
                acc += Fraction(float(r[t]))
                if acc > T:
                    want = t
                    break
            got, _, _ = O.inverse_cdf(r, u)
            assert got == want, (V, r, k)
            assert r[got] > 0                         # zero-mass tokens are never chosen


def test_one_hot_weights_always_return_that_token():
    for V in (1, 5, 64):
        for hot in (0, V // 2, V - 1):
            r = np.zeros(V)
            r[hot] = 0.37
            for u in (0.0, 0.5, 1 - 2.0 ** -24):
                assert O.inverse_cdf(r, u)[0] == hot


def test_residual_fallback_and_literal_reading():
    rng = np.random.default_rng(15)
    M, d, V = 2, 4, 6
    W, H, w, x, _ = tiny_problem(rng, 1, M, d, V)
    e0 = np.zeros(d)
    e0[0] = 1.0
    Hm = H.copy()
    Hm[0, 1, 0] = -10.0                               # judge rejects slot 0
    # bit-identical logits on both sides (taken from a first pass), so that p - q == 0 exactly
    L = O.jd_oracle_verify(W, e0, 0.0, Hm, x, np.zeros((1, M, V)), 0.5, 0, keep_logits=True).logits[0]
    dl = L[None, :M, :].copy()
    u2 = np.array([0.6])
    r = O.jd_oracle_verify(W, e0, 0.0, Hm, x, dl, 0.5, 0, "judge", u_sample=u2)
    assert r.accept_len[0] == 0
    p0 = np.array(softmax_py([float(np.dot(Hm[0, 0], W[v])) for v in range(V)]))
    want = int(np.searchsorted(np.cumsum(p0), 0.6 * np.cumsum(p0)[-1], side="right"))
    assert r.next_token[0] == want
    # resample="target_p" draws from p at the rejected slot even when a residual exists
    dl2 = rng.standard_normal((1, M, V))
    r2 = O.jd_oracle_verify(W, e0, 0.0, Hm, x, dl2, 0.5, 0, "judge", resample="target_p", u_sample=u2)
    assert r2.accept_len[0] == 0 and r2.next_token[0] == want


# ---------------------------------------------------------------- distribution (chi-square)
def _chi2_sf_bound(stat, dof):
    # Wilson-Hilferty normal approximation of the chi-square survival function
    zz = ((stat / dof) ** (1 / 3) - (1 - 2 / (9 * dof))) / math.sqrt(2 / (9 * dof))
    return 0.5 * math.erfc(zz / math.sqrt(2))


@pytest.mark.parametrize("V", [8, 32])
def test_chi_square_emitted_token_follows_p(V):
    """Standard mode, x ~ q drawn by the harness: the token emitted at slot 0 (the draft token
    if accepted, the corrected one otherwise) is distributed as p (lossless speculative sampling)."""
    rng = np.random.default_rng(100 + V)
    d, n = 6, 30000
    W = rng.standard_normal((V, d))
    h = rng.standard_normal((1, 2, d))
    dlrow = rng.standard_normal(V) * 1.5
    p = np.array(softmax_py([float(np.dot(h[0, 0], W[v])) for v in range(V)]))
    q = np.array(softmax_py(list(dlrow)))
    xs = rng.choice(V, size=n, p=q).astype(np.int32)
    H = np.repeat(h, n, axis=0)
    dl = np.repeat(dlrow[None, None, :], n, axis=0)
    r = O.jd_oracle_verify(W, np.zeros(d), 0.0, H, xs.reshape(n, 1), dl, 0.5, seed=2024, mode="standard")
    emitted = np.where(r.accept_len == 1, xs, r.next_token)
    counts = np.bincount(emitted, minlength=V)
    stat = float(np.sum((counts - n * p) ** 2 / (n * p)))
    assert _chi2_sf_bound(stat, V - 1) > 1e-3, (stat, V)
    # and the acceptance rate is sum_t min(p, q)
    assert abs((r.accept_len == 1).mean() - np.minimum(p, q).sum()) < 4 * 0.5 / math.sqrt(n)


def test_chi_square_bonus_token_follows_last_row():
    rng = np.random.default_rng(200)
    V, d, n = 16, 6, 30000
    W = rng.standard_normal((V, d))
    h = rng.standard_normal((1, 2, d))
    H = np.repeat(h, n, axis=0)
    dl = np.repeat((h[0, 0] @ W.T)[None, None, :], n, axis=0)     # q = p -> always accepted
    xs = rng.integers(0, V, size=(n, 1)).astype(np.int32)
    r = O.jd_oracle_verify(W, np.zeros(d), 0.0, H, xs, dl, 0.5, seed=99, mode="standard")
    assert (r.accept_len == 1).all()
    pM = np.array(softmax_py([float(np.dot(h[0, 1], W[v])) for v in range(V)]))
    counts = np.bincount(r.next_token, minlength=V)
    stat = float(np.sum((counts - n * pM) ** 2 / (n * pM)))
    assert _chi2_sf_bound(stat, V - 1) > 1e-3


def test_margins_are_reported():
    rng = np.random.default_rng(16)
    W, H, w, x, dl = tiny_problem(rng, 2, 3, 4, 7)
    r = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 5)
    for b in range(2):
        for j in range(3):
            ratio = min(1.0, r.p_draft[b, j] / r.q_draft[b, j])
            assert math.isclose(r.margin_accept[b, j], abs(r.u_accept[b, j] - ratio), abs_tol=1e-15)
            assert math.isclose(r.margin_judge[b, j], abs(r.judge_scores[b, j] - 0.5), abs_tol=1e-15)
        lo, hi = r.token_interval(b, int(r.next_token[b]))
        assert lo <= r.sample_T[b] < hi
        assert math.isclose(r.margin_cdf[b], min(r.sample_T[b] - lo, hi - r.sample_T[b]) / r.sample_mass[b],
                            rel_tol=1e-12, abs_tol=1e-18)
