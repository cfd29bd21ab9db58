"""CPU checker for the verification step of judge decoding (arXiv 2501.19309).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 restatement of what
one verification call computes, written from the paper so that a reader can
check it by eye.  Nothing in the product may import it: only the tests, the
smoke check and the CPU-baseline leg of the benchmark do.  It shares no code
with the CUDA library and never sees a value the CUDA library produced.

What one call computes (paper Sec. 3.1 "Speculative decoding", Eq. 2-4, and
Sec. 4.1 "Inference"; 0-indexed here, the paper is 1-indexed):

  for every sequence b and every row j = 0..M of its embeddings H[b]:
      L[j, :] = W @ H[b, j]                      LM head (Eq. 2)
      p_j     = softmax(L[j, :])                 target distribution of slot j
  for every draft slot j = 0..M-1 with drafted token x_j:
      q_j     = softmax(draft_logits[b, j, :])   draft distribution (Eq. 3)
      z_std[j]   = u_j * q_j[x_j] < p_j[x_j]     standard test (Eq. 4)
      s[j]       = sigmoid(w . H[b, j+1] + b0)   judge score of x_j's own embedding
      z_judge[j] = s[j] > tau                    (Sec. 4.1 "Inference")
      z[j]       = z_std[j] or z_judge[j]        (or one of them, by mode)
  a = index of the first j with z[j] == 0, else M   (a token counts only while all before it were accepted)
  next token: from the residual max(0, p_a - q_a), normalised, when a < M;
              from p_M after a fully accepted block; inverse CDF in ascending
              token id with one uniform.

Deterministic variants of the standard test (Sec. 3.2 measures acceptance with a greedily
decoded target; Sec. 5.1 "Training-free baseline" defines top-K verification): with rule="topk" the
candidate x_j passes the standard test iff it is among the K highest-valued entries of p_j
(K = 1 is greedy verification, K = V accepts everything), and the next token is the target's
greedy token argmax p_a, at a rejection as well as after a fully accepted block. No uniform is
drawn and the draft distribution plays no role. Equal logits are ordered by token id (lower id
ranks higher), so "among the K highest" and "argmax" are unique.

Final RMS normalisation (Sec. 4.1 "Model design and training": the judge reads the last embedding
ahead of the model's final RMS norm and LM head): with rms_eps given, the LM head sees
H[b,j] / sqrt(mean_k H[b,j,k]^2 + rms_eps) while the judge still reads H[b,j+1] itself. The
normalisation gain is taken as folded into W beforehand.

8-bit head (the paper runs its targets with 8-bit weights, Table 1 caption and App. B.3): with
w_scale given, W holds FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no
infinities) and the logical weight is w_scale[v] * e4m3(W[v,k]). The rows of H are quantised the
same way before the LM head, one scale per row: with a_r = max_k |H[r,k]|, the scale is
s_r = a_r / 448 and h8[r,k] is the E4M3 value nearest to H[r,k] * 448 / a_r (ties to the even
mantissa, saturating at +-448; an all-zero row gives zeros and s_r = 0). The logit is
w_scale[v] * s_r * sum_k e4m3(W[v,k]) * h8[r,k]; the judge still reads the unquantised row.

Readings taken where the paper is silent (all restated in the design notes):
  * the judge for draft token j reads row j+1 of H, the embedding produced by
    feeding that token (Sec. 4.1 speaks of the embedding of the current token);
  * the token at the first rejection comes from the residual distribution, the
    form that keeps standard speculative sampling lossless; the paper's wording taken
    literally (draw from p_i itself) is available as resample="target_p";
  * Eq. 4 is evaluated division-free, u*q < p, which equals u < min(1, p/q)
    for u in [0, 1); q(x) = 0 accepts iff p(x) > 0;
  * the judge comparison is strict; tau = 1 never accepts, so the OR mode
    reduces to the standard test (Sec. 4.1, last sentence);
  * uniforms: Philox4x32-10 (Salmon et al., SC'11), key = the 64-bit seed split
    in two words, counter = (b, slot, stream, 0), first output word, top 24
    bits: u = (word >> 8) * 2**-24.  stream 0 feeds the acceptance test of slot
    j, stream 1 the token draw at slot a;
  * an all-zero residual (p_a == q_a) falls back to sampling from p_a;
  * inverse CDF: T = u' * sum(r); token = min{t : r[0] + .. + r[t] > T}; if
    rounding leaves no such t, the last token with r > 0.

Pins (tests/test_oracle_*.py): Philox known-answer vectors printed with the
generator's publication; closed forms of the acceptance law and of the emitted
token law by exhaustive enumeration on tiny vocabularies; q = p accepts all;
tau = 1 and mode "standard" equal a separate textbook routine; chi-square of the
emitted token against p; judge special cases (w = 0, w = unit vector); the
prefix rule over all 2^M masks; OR monotonicity; one-hot residuals.
Parity unpinned: nothing about real-model behaviour (acceptance lengths or
accuracy with trained weights) is checked anywhere.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import numpy as np

MODE_STANDARD, MODE_JUDGE, MODE_JUDGE_OR_STANDARD = 0, 1, 2
RESAMPLE_RESIDUAL, RESAMPLE_TARGET_P = 0, 1
STREAM_ACCEPT, STREAM_SAMPLE = 0, 1

RULE_SAMPLING, RULE_TOPK = 0, 1

_MODES = {"standard": MODE_STANDARD, "judge": MODE_JUDGE, "judge_or_standard": MODE_JUDGE_OR_STANDARD}
_RESAMPLE = {"residual": RESAMPLE_RESIDUAL, "target_p": RESAMPLE_TARGET_P}


# --------------------------------------------------------------------------
# Philox4x32-10, from its published definition (Salmon, Moraes, Dror, Shaw:
# "Parallel random numbers: as easy as 1, 2, 3", SC'11, Sec. 3.3 / Table 2).
# --------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9   # golden ratio
_PHILOX_W1 = 0xBB67AE85   # sqrt(3) - 1
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> tuple:
    """One Philox4x32-10 block: 4 counter words, 2 key words -> 4 output words."""
    c0, c1, c2, c3 = (int(c) & _MASK32 for c in counter)
    k0, k1 = (int(k) & _MASK32 for k in key)
    for rnd in range(10):
        if rnd > 0:                      # the key is bumped between rounds (9 bumps)
            k0 = (k0 + _PHILOX_W0) & _MASK32
            k1 = (k1 + _PHILOX_W1) & _MASK32
        prod0 = _PHILOX_M0 * c0          # 64-bit products
        prod1 = _PHILOX_M1 * c2
        hi0, lo0 = prod0 >> 32, prod0 & _MASK32
        hi1, lo1 = prod1 >> 32, prod1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return c0, c1, c2, c3


def uniform24(seed: int, b: int, slot: int, stream: int) -> float:
    """u in [0, 1) on the 2**-24 grid, keyed by (seed; b, slot, stream)."""
    key = (seed & _MASK32, (seed >> 32) & _MASK32)
    word0 = philox4x32_10((b, slot, stream, 0), key)[0]
    return (word0 >> 8) * 2.0 ** -24


# --------------------------------------------------------------------------
# storage widening (own copy: the checker shares no helper with anything else)
# --------------------------------------------------------------------------
def _to_f64(a: np.ndarray) -> np.ndarray:
    """float64 values of a stored array: uint16 = bfloat16 bit patterns, else floats."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


# --------------------------------------------------------------------------
# the steps
# --------------------------------------------------------------------------
# --------------------------------------------------------------------------
# FP8 E4M3 ("fn": finite, no infinities; 0x7F / 0xFF are NaN), from the format's definition
# --------------------------------------------------------------------------
def _e4m3_value(c: int) -> float:
    """Value of one E4M3 code: (-1)^s 2^(e-7) (1 + m/8); e = 0: (-1)^s 2^-6 m/8; 0x7F / 0xFF: NaN."""
    s, e, m = c >> 7, (c >> 3) & 0xF, c & 0x7
    if e == 0xF and m == 0x7:
        return float("nan")
    mag = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return -mag if s else mag


_E4M3_TABLE = np.array([_e4m3_value(c) for c in range(256)], dtype=np.float64)


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """float64 values of E4M3 codes (uint8): the 256 values of the format, looked up by code."""
    return _E4M3_TABLE[np.asarray(codes, dtype=np.uint8)]


def e4m3_round(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 value of every entry of x (float64), ties to the even mantissa, saturating at
    +-448; float64."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), 448.0)
    # spacing of the E4M3 grid around a: 2^(floor(log2 a) - 3), but never finer than 2^-9
    ex = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    q = np.ldexp(1.0, (ex - 3).astype(np.int64))
    r = np.round(a / q) * q                   # numpy rounds halves to even; a / q is exact (q = 2^n)
    return np.copysign(np.minimum(r, 448.0), x)


def quantise_rows_e4m3(Hb: np.ndarray) -> tuple:
    """Per-row E4M3 quantisation: returns (values [rows, d] float64 on the E4M3 grid, scale [rows]
    float64) with H ~ scale * values; scale = row amax / 448, values = nearest E4M3 value of
    H * 448 / amax."""
    Hd = _to_f64(Hb)
    amax = np.max(np.abs(Hd), axis=-1, keepdims=True)
    safe = np.where(amax > 0, amax, 1.0)
    vals = e4m3_round(Hd * 448.0 / safe)       # H * 448 is exact in float64 for bf16 / f32 inputs
    return vals, (amax / 448.0)[..., 0]


def rms_normalise(Hb: np.ndarray, eps: float) -> np.ndarray:
    """Rows of Hb divided by sqrt(mean of squares + eps), float64 (RMSNorm without its gain)."""
    Hd = _to_f64(Hb)
    return Hd / np.sqrt(np.mean(Hd * Hd, axis=-1, keepdims=True) + eps)


def project_logits(W: np.ndarray, Hb: np.ndarray, vocab_chunk: int = 8192) -> np.ndarray:
    """L[j, v] = sum_k H[j, k] * W[v, k] in float64 (Eq. 2, LM head).

    W is widened to float64 a slab of vocabulary rows at a time only to bound
    memory; every L[j, v] is still one full-length dot product."""
    Hd = _to_f64(Hb)                                    # [rows, d]
    V = W.shape[0]
    L = np.empty((Hd.shape[0], V), dtype=np.float64)
    for v0 in range(0, V, vocab_chunk):
        v1 = min(V, v0 + vocab_chunk)
        L[:, v0:v1] = Hd @ _to_f64(W[v0:v1]).T
    return L


def logsumexp(row: np.ndarray) -> tuple:
    """(max, log sum exp) of one row, float64."""
    m = float(np.max(row))
    return m, m + float(np.log(np.sum(np.exp(row - m))))


def sigmoid(t: float) -> float:
    return 1.0 / (1.0 + float(np.exp(-t)))


def accepted_prefix_length(z: Sequence[int]) -> int:
    """Index of the first rejected slot, or len(z) when every slot is accepted."""
    for j, zj in enumerate(z):
        if not zj:
            return j
    return len(z)


def combine_masks(z_std: int, z_judge: int, mode: int) -> int:
    if mode == MODE_STANDARD:
        return int(z_std)
    if mode == MODE_JUDGE:
        return int(z_judge)
    return int(z_std or z_judge)


def inverse_cdf(r: np.ndarray, u: float) -> tuple:
    """token = min{t : r[0]+..+r[t] > u * sum(r)}; returns (token, T, cdf)."""
    cdf = np.cumsum(r, dtype=np.float64)                # sequential float64 prefix sums
    total = float(cdf[-1])
    T = u * total
    t = int(np.searchsorted(cdf, T, side="right"))      # first index with cdf > T
    if t >= len(r):                                      # rounding: take the last token with mass
        t = int(np.max(np.nonzero(r > 0)[0]))
    return t, T, cdf


@dataclasses.dataclass
class OracleResult:
    sequences: list                 # which b were computed (all by default)
    accept_len: np.ndarray          # [B] int32 (-1 where not computed)
    next_token: np.ndarray          # [B] int32 (-1 where not computed)
    judge_scores: np.ndarray        # [B, M] float64
    p_draft: np.ndarray             # [B, M] float64  p_j[x_j]
    q_draft: np.ndarray             # [B, M] float64  q_j[x_j]
    masks: np.ndarray               # [B, M] uint8: bit0 standard test, bit1 judge test
    row_max: np.ndarray             # [B, M+1] float64  max_v L
    row_lse: np.ndarray             # [B, M+1] float64  logsumexp_v L
    u_accept: np.ndarray            # [B, M] float64 uniforms of the acceptance test
    u_sample: np.ndarray            # [B] float64 uniform of the token draw
    margin_accept: np.ndarray       # [B, M] |u - min(1, p/q)|
    margin_judge: np.ndarray        # [B, M] |s - tau|
    margin_cdf: np.ndarray          # [B] distance of T to the nearest CDF edge of the token, / sum(r);
                                    #     rule "topk": gap between the two largest logits of row a, scaled
    sample_T: np.ndarray            # [B] T = u' * sum(r)
    sample_mass: np.ndarray         # [B] sum(r)
    sample_weights: dict            # b -> r[V] float64 (un-normalised sampling weights)
    logits: dict                    # b -> L[M+1, V] float64 (kept only when keep_logits)

    def token_interval(self, b: int, token: int) -> tuple:
        """CDF interval [lo, hi) of ``token`` in sequence b's sampling weights."""
        r = self.sample_weights[b]
        cdf = np.cumsum(r, dtype=np.float64)
        lo = float(cdf[token - 1]) if token > 0 else 0.0
        return lo, float(cdf[token])


def rank_in_row(row: np.ndarray, x: int) -> int:
    """Position of token x when the row is sorted by value, highest first, equal values by
    ascending token id: the number of entries that rank above x."""
    lx = row[x]
    return int(np.count_nonzero(row > lx) + np.count_nonzero(row[:x] == lx))


def jd_oracle_verify(W, w_judge, b_judge: float, H, draft_tokens, draft_logits, tau: float,
                     seed: int, mode="judge_or_standard", resample="residual",
                     sequences: Optional[Sequence[int]] = None, keep_logits: bool = False,
                     u_accept: Optional[np.ndarray] = None,
                     u_sample: Optional[np.ndarray] = None,
                     rule="sampling", top_k: int = 1, rms_eps: Optional[float] = None,
                     w_scale: Optional[np.ndarray] = None) -> OracleResult:
    """One verification call, step by step, in float64.

    ``u_accept`` [B, M] / ``u_sample`` [B], when given, replace the Philox
    uniforms (used by the enumeration tests, which sweep u over a dyadic grid).
    ``sequences`` restricts the work to some b (sampled checks at full size)."""
    rule = {"sampling": RULE_SAMPLING, "greedy": RULE_TOPK, "topk": RULE_TOPK}[rule] if isinstance(rule, str) else int(rule)
    if rule == RULE_TOPK and top_k < 1:
        raise ValueError("top_k must be >= 1")
    mode = _MODES[mode] if isinstance(mode, str) else int(mode)
    resample = _RESAMPLE[resample] if isinstance(resample, str) else int(resample)
    H = np.asarray(H)
    B, Mp1, d = H.shape
    M = Mp1 - 1
    x = np.asarray(draft_tokens).reshape(B, M)
    dl = np.asarray(draft_logits).reshape(B, M, -1)
    V = W.shape[0]
    wj = _to_f64(w_judge)
    seqs = list(range(B)) if sequences is None else list(sequences)

    res = OracleResult(
        sequences=seqs,
        accept_len=np.full(B, -1, np.int32), next_token=np.full(B, -1, np.int32),
        judge_scores=np.full((B, M), np.nan), p_draft=np.full((B, M), np.nan),
        q_draft=np.full((B, M), np.nan), masks=np.zeros((B, M), np.uint8),
        row_max=np.full((B, M + 1), np.nan), row_lse=np.full((B, M + 1), np.nan),
        u_accept=np.full((B, M), np.nan), u_sample=np.full(B, np.nan),
        margin_accept=np.full((B, M), np.nan), margin_judge=np.full((B, M), np.nan),
        margin_cdf=np.full(B, np.nan), sample_T=np.full(B, np.nan), sample_mass=np.full(B, np.nan),
        sample_weights={}, logits={})

    for b in seqs:
        Hb = _to_f64(H[b])                               # [M+1, d]
        # [M+1, V] (Eq. 2); the LM head sees the RMS-normalised rows when rms_eps is given
        if w_scale is None:
            L = project_logits(W, H[b] if rms_eps is None else rms_normalise(H[b], rms_eps))
        else:
            # 8-bit head: E4M3 weights with per-row scales, rows of H quantised per row
            h8, s_h = quantise_rows_e4m3(H[b])
            L = np.empty((M + 1, V), dtype=np.float64)
            for v0 in range(0, V, 8192):
                v1 = min(V, v0 + 8192)
                L[:, v0:v1] = h8 @ e4m3_decode(W[v0:v1]).T
            L *= np.asarray(w_scale, dtype=np.float64)[None, :] * s_h[:, None]
            if rms_eps is not None:
                Hd = _to_f64(H[b])
                L /= np.sqrt(np.mean(Hd * Hd, axis=-1, keepdims=True) + rms_eps)
        lse_p = np.empty(M + 1)
        for j in range(M + 1):
            res.row_max[b, j], lse_p[j] = logsumexp(L[j])
        res.row_lse[b] = lse_p

        lse_q = np.empty(M)
        z = []
        for j in range(M):
            dlj = dl[b, j].astype(np.float64)
            _, lse_q[j] = logsumexp(dlj)                                    # (Eq. 3: q_j)
            xj = int(x[b, j])
            P = float(np.exp(L[j, xj] - lse_p[j]))                          # p_j[x_j]
            Q = float(np.exp(dlj[xj] - lse_q[j]))                           # q_j[x_j]
            if rule == RULE_TOPK:
                u = float("nan")
                z_std = int(rank_in_row(L[j], xj) < top_k)                  # among the K highest of p_j
            else:
                u = float(u_accept[b, j]) if u_accept is not None else uniform24(seed, b, j, STREAM_ACCEPT)
                z_std = int(u * Q < P)                                      # (Eq. 4)
            s = sigmoid(float(wj @ Hb[j + 1]) + b_judge)                    # judge on x_j's embedding
            z_judge = int(s > tau)                                          # (Sec. 4.1)
            z.append(combine_masks(z_std, z_judge, mode))
            res.p_draft[b, j], res.q_draft[b, j], res.judge_scores[b, j] = P, Q, s
            res.masks[b, j] = z_std | (z_judge << 1)
            res.u_accept[b, j] = u
            if rule == RULE_TOPK:
                # distance of the candidate's logit to the value it would have to cross, in units
                # of the row's logit scale
                srt = np.sort(L[j])[::-1]
                scale = max(abs(float(srt[0])), float(np.sqrt(np.mean(L[j] * L[j]))))
                if z_std:
                    edge = float(srt[top_k]) if top_k < V else -np.inf
                    res.margin_accept[b, j] = (float(L[j, xj]) - edge) / scale
                else:
                    res.margin_accept[b, j] = (float(srt[top_k - 1]) - float(L[j, xj])) / scale
            else:
                ratio = 1.0 if Q == 0.0 else min(1.0, P / Q)
                res.margin_accept[b, j] = abs(u - ratio)
            res.margin_judge[b, j] = abs(s - tau)

        a = accepted_prefix_length(z)                                       # prefix rule
        res.accept_len[b] = a

        if rule == RULE_TOPK:
            # the target's greedy token, at a rejection and after a fully accepted block alike
            t = int(np.argmax(L[a]))                                        # first index among equal maxima
            res.next_token[b] = t
            top2 = np.partition(L[a], -2)[-2:] if V > 1 else np.array([L[a, t], L[a, t]])
            scale = max(abs(float(L[a, t])), float(np.sqrt(np.mean(L[a] * L[a]))))
            res.margin_cdf[b] = float(top2[1] - top2[0]) / scale
            w1 = np.zeros(V)
            w1[t] = 1.0
            res.sample_weights[b] = w1
            res.sample_T[b], res.sample_mass[b] = 0.0, 1.0
            if keep_logits:
                res.logits[b] = L
            continue

        p_a = np.exp(L[a] - lse_p[a])
        if a < M and resample == RESAMPLE_RESIDUAL:
            q_a = np.exp(dl[b, a].astype(np.float64) - lse_q[a])
            r = np.maximum(0.0, p_a - q_a)
            if not np.any(r > 0):                                           # p_a == q_a
                r = p_a
        else:
            r = p_a                                                         # bonus token, or literal reading
        u2 = float(u_sample[b]) if u_sample is not None else uniform24(seed, b, a, STREAM_SAMPLE)
        t, T, cdf = inverse_cdf(r, u2)
        res.next_token[b] = t
        res.u_sample[b] = u2
        res.sample_T[b], res.sample_mass[b] = T, float(cdf[-1])
        lo = float(cdf[t - 1]) if t > 0 else 0.0
        res.margin_cdf[b] = min(abs(T - lo), abs(float(cdf[t]) - T)) / float(cdf[-1])
        res.sample_weights[b] = r
        if keep_logits:
            res.logits[b] = L
    return res
