"""Pins for the checker's deterministic rules: greedy and top-K verification (Sec. 3.2; Sec. 5.1
"Training-free baseline")."""
import itertools

import numpy as np

from oracle import jd_oracle as O


def problem(rng, B, M, d, V):
    W = rng.standard_normal((V, d))
    H = rng.standard_normal((B, M + 1, d))
    w = rng.standard_normal(d)
    x = rng.integers(0, V, size=(B, M)).astype(np.int32)
    dl = rng.standard_normal((B, M, V))
    return W, H, w, x, dl


def run(W, H, w, x, dl, **kw):
    return O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 0, **kw)


def test_rank_helper_brute_force_with_ties():
    row = np.array([1.0, 3.0, 3.0, -2.0, 3.0, 1.0])
    order = sorted(range(6), key=lambda v: (-row[v], v))          # highest first, ties by token id
    for x in range(6):
        assert O.rank_in_row(row, x) == order.index(x)


def test_topk_is_membership_in_the_k_largest():
    rng = np.random.default_rng(0)
    B, M, d, V = 2, 4, 5, 9
    W, H, w, x, dl = problem(rng, B, M, d, V)
    L = np.einsum("bjk,vk->bjv", H, W)
    for K in range(1, V + 1):
        r = run(W, H, w, x, dl, mode="standard", rule="topk", top_k=K)
        for b in range(B):
            for j in range(M):
                topk = set(np.argsort(-L[b, j], kind="stable")[:K].tolist())
                assert (int(r.masks[b, j]) & 1) == int(int(x[b, j]) in topk)
            z = [int(v) & 1 for v in r.masks[b]]
            a = next((j for j, zj in enumerate(z) if not zj), M)
            assert r.accept_len[b] == a
            assert r.next_token[b] == int(np.argmax(L[b, a]))      # greedy target token, also the bonus


def test_k_equals_vocabulary_accepts_everything_and_k_one_is_greedy():
    rng = np.random.default_rng(1)
    B, M, d, V = 3, 5, 4, 7
    W, H, w, x, dl = problem(rng, B, M, d, V)
    r = run(W, H, w, x, dl, mode="standard", rule="topk", top_k=V)      # K = V: the draft alone decides
    assert (r.accept_len == M).all()
    L = np.einsum("bjk,vk->bjv", H, W)
    xg = np.argmax(L[:, :M], axis=2).astype(np.int32)                    # draft = target's greedy tokens
    r = run(W, H, w, xg, dl, mode="standard", rule="greedy")
    assert (r.accept_len == M).all()
    xb = xg.copy()
    xb[:, 2] = (xb[:, 2] + 1) % V                                        # one wrong token at slot 2
    r = run(W, H, w, xb, dl, mode="standard", rule="greedy")
    assert (r.accept_len == 2).all() and (r.next_token == xg[:, 2]).all()  # corrected to the target's token


def test_topk_monotone_in_k_and_independent_of_draft_logits_and_seed():
    rng = np.random.default_rng(2)
    W, H, w, x, dl = problem(rng, 2, 6, 4, 11)
    prev = None
    for K in (1, 2, 3, 5, 11):
        r = run(W, H, w, x, dl, mode="standard", rule="topk", top_k=K)
        if prev is not None:
            assert (r.accept_len >= prev).all()
        prev = r.accept_len.copy()
    a = O.jd_oracle_verify(W, w, 0.0, H, x, dl, 0.5, 1, "standard", rule="topk", top_k=2)
    b = O.jd_oracle_verify(W, w, 0.0, H, x, dl * 3 + 1, 0.5, 99, "standard", rule="topk", top_k=2)
    assert (a.accept_len == b.accept_len).all() and (a.next_token == b.next_token).all()


def test_ties_are_ordered_by_token_id():
    # two identical rows of W give equal logits: the lower id wins the argmax and the rank
    W = np.array([[1.0, 0.0], [2.0, 1.0], [2.0, 1.0], [0.0, 0.5]])
    H = np.array([[[1.0, 1.0], [1.0, 0.0]]])
    dl = np.zeros((1, 1, 4))
    for xt, want in ((1, 1), (2, 0)):
        r = O.jd_oracle_verify(W, np.zeros(2), 0.0, H, np.array([[xt]], np.int32), dl, 0.5, 0, "standard",
                               rule="greedy")
        assert r.accept_len[0] == want
    r = O.jd_oracle_verify(W, np.zeros(2), 0.0, H, np.array([[2]], np.int32), dl, 0.5, 0, "standard", rule="topk", top_k=2)
    assert r.accept_len[0] == 1 and r.next_token[0] == 1


def test_or_with_judge_and_margins():
    rng = np.random.default_rng(3)
    W, H, w, x, dl = problem(rng, 2, 5, 4, 8)
    rs = {m: run(W, H, w, x, dl, mode=m, rule="greedy") for m in ("standard", "judge", "judge_or_standard")}
    assert (rs["judge_or_standard"].accept_len >= np.maximum(rs["standard"].accept_len, rs["judge"].accept_len)).all()
    samp = run(W, H, w, x, dl, mode="judge")
    assert (rs["judge"].accept_len == samp.accept_len).all()             # the judge test does not depend on the rule
    r = rs["standard"]
    assert (r.margin_accept >= 0).all() and (r.margin_cdf > 0).all()
    L = np.einsum("bjk,vk->bjv", H, W)
    for b, j in itertools.product(range(2), range(5)):
        srt = np.sort(L[b, j])[::-1]
        scale = max(abs(srt[0]), np.sqrt(np.mean(L[b, j] ** 2)))
        want = (srt[0] - srt[1]) / scale if x[b, j] == np.argmax(L[b, j]) else (srt[0] - L[b, j, x[b, j]]) / scale
        assert abs(r.margin_accept[b, j] - want) < 1e-12
