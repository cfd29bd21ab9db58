"""Helpers shared by the GPU parity tests: upload a workload, run the library through its
C ABI, run the CPU checker on the same inputs, and compare under the stated tolerances.

Tolerances (floating point): logits, row max, log-normalisers and p(x_j) within relative
2e-3 (bf16 inputs, fp32 accumulation), logits relative to max(|ref|, rms of the row);
judge scores within 2e-5 absolute.  Integers (masks, accepted length, next token) must be
equal, except where the checker reports a decision margin below 1e-5 (u against min(1, p/q),
score against tau, T against a CDF edge); those cases are counted and returned.
"""
from __future__ import annotations

import dataclasses

import numpy as np

from oracle import jd_oracle as O
from paper_2501_19309_b200 import inputs as I

REL_TOL = 2e-3
JUDGE_ABS_TOL = 2e-5
MARGIN = 1e-5
# Top-K / greedy rule: a decision is a comparison of two logits, each of which is only required to
# be right within REL_TOL of the row's logit scale, so comparisons closer than twice that are exempt
# (the checker reports the gap in the same scaled units).
MARGIN_LOGIT = 2 * REL_TOL


def torch_mod():
    import torch
    return torch


def upload(inp: I.Inputs, device="cuda:0"):
    """Device tensors of one workload (bf16 bit patterns are reinterpreted, not converted)."""
    torch = torch_mod()

    def store(a):
        t = torch.from_numpy(a)
        if a.dtype == np.uint16:
            t = t.view(torch.bfloat16)
        return t.to(device)

    ws = None if inp.w_scale is None else torch.from_numpy(inp.w_scale).to(device)
    return dict(W=store(inp.W), H=store(inp.H), w=store(inp.w_judge), w_scale=ws,
                x=torch.from_numpy(inp.draft_tokens).to(device),
                dl=torch.from_numpy(inp.draft_logits).to(device))


def make_verifier(inp: I.Inputs, dev: dict, max_B=None, max_M=None):
    from paper_2501_19309_b200 import jd
    wl = inp.wl
    v = jd.Verifier(max_B or wl.B, max_M or wl.M, wl.d, wl.V, wl.dtype)
    v.set_head(dev["W"], dev["w"], inp.b_judge, w_scale=dev.get("w_scale"))
    return v


def to_numpy(out: dict) -> dict:
    torch = torch_mod()
    torch.cuda.synchronize()
    return {k: v.detach().cpu().numpy() for k, v in out.items()}


def run_oracle(inp: I.Inputs, mode, seed=None, tau=None, resample="residual", sequences=None, keep_logits=False,
               rule="sampling", top_k=1, rms_eps=None):
    return O.jd_oracle_verify(inp.W, inp.w_judge, inp.b_judge, inp.H, inp.draft_tokens, inp.draft_logits,
                              inp.tau if tau is None else tau, inp.seed if seed is None else seed,
                              mode, resample, sequences=sequences, keep_logits=keep_logits, rule=rule, top_k=top_k,
                              rms_eps=rms_eps, w_scale=inp.w_scale)


def fp8_row_code_mismatches(inp: I.Inputs, dev: dict) -> int:
    """Runs the library's per-row E4M3 quantiser on the workload's H and counts the elements whose
    code decodes to another value than the checker's quantiser gives; also checks the row scales."""
    torch = torch_mod()
    from paper_2501_19309_b200 import jd
    H = dev["H"]
    rows, d = H.shape[0] * H.shape[1], H.shape[2]
    codes = torch.empty((rows, d), dtype=torch.uint8, device=H.device)
    scale = torch.empty(rows, dtype=torch.float32, device=H.device)
    st = jd.jd_quantize_rows_e4m3(H.data_ptr(), rows, d, codes.data_ptr(), scale.data_ptr(),
                                  torch.cuda.current_stream().cuda_stream)
    assert st == jd.JD_OK
    torch.cuda.synchronize()
    vals, s_ref = O.quantise_rows_e4m3(inp.H.reshape(rows, d))
    got = O.e4m3_decode(codes.cpu().numpy())
    assert np.allclose(scale.cpu().numpy(), s_ref, rtol=1e-6, atol=0)
    return int(np.count_nonzero(got != vals))


@dataclasses.dataclass
class Report:
    sequences: int = 0
    slots: int = 0
    exempt_accept: int = 0      # standard-test bits that differ within the margin
    exempt_judge: int = 0       # judge bits that differ within the margin
    exempt_len: int = 0         # accepted lengths that differ because of an exempt bit
    token_exact: int = 0        # next tokens equal to the checker's
    token_in_margin: int = 0    # next tokens different but inside the widened CDF interval
    max_rel_p: float = 0.0
    max_rel_lse: float = 0.0
    max_abs_judge: float = 0.0
    max_rel_logit: float = 0.0


# Parity counts per workload, gathered over the whole test session; tests/conftest.py prints them in
# the terminal summary and writes them to parity_counts.json (folder: $JD_REPORT_DIR, default
# <repository>/parity_reports).
SESSION_REPORTS: dict = {}
EXEMPT_SHARE_BOUND = 0.01   # of the slots of a workload may differ inside a decision margin


def record(name: str, rep: Report, bound: bool = True) -> Report:
    """Adds one test's counts to the session's table for workload `name`; with `bound`, also asserts
    that at most EXEMPT_SHARE_BOUND of its test bits (never less than one) fell inside a margin.
    The share of exactly equal next tokens is reported, not bounded: with V = 128256 near-flat
    distributions the CDF steps are narrower than the margin itself."""
    agg = SESSION_REPORTS.setdefault(name, Report())
    for f in dataclasses.fields(Report):
        a, b = getattr(agg, f.name), getattr(rep, f.name)
        setattr(agg, f.name, max(a, b) if f.name.startswith("max_") else a + b)
    if bound:
        assert rep.exempt_accept + rep.exempt_judge <= max(1.0, EXEMPT_SHARE_BOUND * rep.slots), (name, rep)
    return agg


def combine(bits: int, mode: str) -> int:
    if mode == "standard":
        return bits & 1
    if mode == "judge":
        return (bits >> 1) & 1
    return 1 if bits else 0


def compare(got: dict, ref: O.OracleResult, mode: str, M: int, report: Report = None, rule: str = "sampling") -> Report:
    """Asserts parity of one call's outputs with the checker on the sequences it computed."""
    rep = report or Report()
    margin_std = MARGIN if rule == "sampling" else MARGIN_LOGIT
    for b in ref.sequences:
        rep.sequences += 1
        # floating-point outputs
        for name, tol in (("row_max", REL_TOL), ("row_lse", REL_TOL)):
            g, r = got[name][b].astype(np.float64), getattr(ref, name)[b]
            rel = np.max(np.abs(g - r) / np.maximum(np.abs(r), 1.0))
            assert rel <= tol, (name, b, rel)
            if name == "row_lse":
                rep.max_rel_lse = max(rep.max_rel_lse, float(rel))
        gp, rp = got["p_draft"][b].astype(np.float64), ref.p_draft[b]
        relp = np.max(np.abs(gp - rp) / np.maximum(rp, 1e-30))
        assert relp <= REL_TOL, ("p_draft", b, relp)
        rep.max_rel_p = max(rep.max_rel_p, float(relp))
        gq, rq = got["q_draft"][b].astype(np.float64), ref.q_draft[b]
        assert np.max(np.abs(gq - rq) / np.maximum(rq, 1e-30)) <= REL_TOL, ("q_draft", b)
        dj = np.max(np.abs(got["judge_scores"][b].astype(np.float64) - ref.judge_scores[b]))
        assert dj <= JUDGE_ABS_TOL, ("judge_scores", b, dj)
        rep.max_abs_judge = max(rep.max_abs_judge, float(dj))

        # decisions
        exempt_bit = False
        for j in range(M):
            rep.slots += 1
            gb, rb = int(got["masks"][b, j]), int(ref.masks[b, j])
            if (gb ^ rb) & 1:
                assert ref.margin_accept[b, j] < margin_std, ("standard test", b, j, ref.margin_accept[b, j])
                rep.exempt_accept += 1
                exempt_bit = True
            if (gb ^ rb) & 2:
                assert ref.margin_judge[b, j] < MARGIN, ("judge test", b, j, ref.margin_judge[b, j])
                rep.exempt_judge += 1
                exempt_bit = True
        # the library's accepted length must follow from its own masks by the prefix rule
        z = [combine(int(v), mode) for v in got["masks"][b]]
        a_gpu = int(got["accept_len"][b])
        assert a_gpu == next((j for j, zj in enumerate(z) if not zj), M), ("prefix rule", b)
        a_ref = int(ref.accept_len[b])
        if a_gpu != a_ref:
            assert exempt_bit, ("accept_len", b, a_gpu, a_ref)
            rep.exempt_len += 1
            continue
        # next token: inside the checker's CDF interval widened by the margin
        tok = int(got["next_token"][b])
        assert 0 <= tok < len(ref.sample_weights[b])
        if tok == int(ref.next_token[b]):
            rep.token_exact += 1
        elif rule != "sampling":
            # greedy token: another token is right only if the two largest logits are that close
            assert ref.margin_cdf[b] < MARGIN_LOGIT, ("greedy next_token", b, tok, int(ref.next_token[b]), ref.margin_cdf[b])
            rep.token_in_margin += 1
        else:
            lo, hi = ref.token_interval(b, tok)
            T, mass = ref.sample_T[b], ref.sample_mass[b]
            assert ref.sample_weights[b][tok] > 0, ("token without mass", b, tok)
            assert lo - MARGIN * mass <= T <= hi + MARGIN * mass, ("next_token", b, tok, int(ref.next_token[b]),
                                                                 (T - lo) / mass, (hi - T) / mass)
            rep.token_in_margin += 1
    return rep


def compare_logits(got_logits: np.ndarray, ref: O.OracleResult, report: Report) -> None:
    for b in ref.sequences:
        L = ref.logits[b]
        g = got_logits[b].astype(np.float64)
        rms = np.sqrt(np.mean(L * L, axis=1, keepdims=True))
        rel = np.max(np.abs(g - L) / np.maximum(np.abs(L), rms))
        assert rel <= REL_TOL, ("logits", b, rel)
        report.max_rel_logit = max(report.max_rel_logit, float(rel))
