"""Seeded synthetic inputs for the judge-decoding verification step.

This module only draws random tensors with the shapes and value distributions
of Llama-3.1-style LM heads (V = 128256, d = 4096 / 8192 / 16384) and of a
draft block of M candidate tokens.  It contains none of the method's
arithmetic (no softmax, no acceptance test, no sampling): both the CUDA
library and the CPU checker are fed from here and share nothing else.

Every array is produced by ``numpy.random.Generator(numpy.random.Philox(key))``
with a key derived from ``(1000 * config_id + data_seed, stream)``, so any part
of a workload can be regenerated independently of the others.  The LM-head
matrix W is drawn in blocks of ``W_BLOCK_ROWS`` vocabulary rows, one key per
block, which lets several host threads fill it in parallel and still give the
same bits for a given (config, seed).

Layout conventions (all C-contiguous):
  W            [V, d]       LM head, one row per vocabulary entry
  H            [B, M+1, d]  row 0 = last context token, row j>=1 = draft token j-1
  draft_tokens [B, M]       int32
  draft_logits [B, M, V]    float32
  w_judge      [d]          judge head weight (dtype of H), b_judge scalar

For dtype "bf16" the arrays W, H and w_judge are returned as uint16 holding
the bfloat16 bit patterns (round-to-nearest-even from float32);
``bf16_bits_to_f32`` widens them back exactly.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

W_BLOCK_ROWS = 2048

# streams of the per-workload key
_S_TOKENS, _S_NOISE, _S_DLOGITS, _S_JUDGE, _S_ALPHA, _S_BOOST, _S_WBLOCK0 = 1, 2, 3, 4, 5, 6, 16


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and recipe of one synthetic verification workload."""

    name: str
    config_id: int
    B: int
    M: int
    d: int
    V: int
    dtype: str = "bf16"            # "bf16" or "f32": storage type of W, H, w_judge; "fp8": W is FP8 E4M3
                                   # codes with one float32 scale per vocabulary row, H and w_judge bf16
    alpha: float = 4.0             # planted-alignment scale (used when alpha_range is None)
    alpha_range: Optional[tuple] = None   # (lo, hi): alpha ~ U[lo, hi]
    alpha_per: str = "seq"         # "seq": one alpha per sequence, "row": one per H row
    sigma: float = 0.5             # std of the additive noise on H
    dl_std: float = 2.0            # std of the draft logits
    boost: float = 4.0             # added to the draft logit of the drafted token
    boost_range: Optional[tuple] = None   # (lo, hi): boost ~ U[lo, hi] per draft slot
    b_judge_std: float = 0.0       # judge bias ~ N(0, b_judge_std^2); 0 -> bias 0
    tau: float = 0.5
    forced_reject_at: Optional[int] = None  # draft slot whose rejection is forced (all modes)

    @property
    def R(self) -> int:
        return self.B * (self.M + 1)

    def scaled(self, name: str, **kw) -> "Workload":
        return dataclasses.replace(self, name=name, **kw)


# The five published workload shapes.
CONFIGS = {
    0: Workload("cfg0-tiny-f32", 0, B=1, M=4, d=256, V=1024, dtype="f32", alpha=3.0, boost=3.0),
    1: Workload("cfg1-8B-head", 1, B=1, M=8, d=4096, V=128256, alpha=4.0, boost=4.0),
    2: Workload("cfg2-70B-head", 2, B=4, M=16, d=8192, V=128256, alpha_range=(1.0, 5.0),
                alpha_per="seq", boost_range=(0.0, 4.0), b_judge_std=0.1),
    3: Workload("cfg3-405B-head", 3, B=1, M=25, d=16384, V=128256, alpha=4.0, boost=4.0,
                forced_reject_at=12),
    4: Workload("cfg4-batched", 4, B=64, M=16, d=8192, V=128256, alpha_range=(0.0, 5.0),
                alpha_per="row", boost=3.0),
}


@dataclasses.dataclass
class Inputs:
    wl: Workload
    data_seed: int
    W: np.ndarray             # [V, d] uint16 (bf16 bits), float32, or uint8 (FP8 E4M3 codes, dtype "fp8")
    H: np.ndarray             # [B, M+1, d] same storage type as W
    w_judge: np.ndarray       # [d] same storage type as W
    b_judge: float
    tau: float
    draft_tokens: np.ndarray  # [B, M] int32
    draft_logits: np.ndarray  # [B, M, V] float32
    seed: int                 # seed handed to the verify call's counter-based RNG
    planted_tokens: np.ndarray  # [B, M+1] int32: token whose W row each H row leans to
    w_scale: Optional[np.ndarray] = None   # [V] float32 row scales of an FP8 head (dtype "fp8")


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32, exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_f32(a: np.ndarray) -> np.ndarray:
    """float32 view of the values of a stored array (bf16 bits or float32)."""
    return bf16_bits_to_f32(a) if a.dtype == np.uint16 else np.asarray(a, dtype=np.float32)


def quantise_rows_fp8(a32: np.ndarray):
    """Per-row FP8 E4M3 storage of a float32 matrix: (codes uint8, scale float32) with
    a ~ scale[:, None] * e4m3(codes); scale = row amax / 448. The float -> E4M3 rounding is
    PyTorch's CPU conversion (nearest, ties to even)."""
    import torch
    a32 = np.ascontiguousarray(a32, dtype=np.float32)
    amax = np.abs(a32).max(axis=1).astype(np.float32)
    scale = (np.where(amax > 0, amax, np.float32(1.0)) / np.float32(448.0)).astype(np.float32)
    q = torch.from_numpy(a32 / scale[:, None]).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn)
    return q.view(torch.uint8).numpy(), scale


def fp8_codes_to_f32(codes: np.ndarray) -> np.ndarray:
    import torch
    return torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).float().numpy()


def _gen(wl: Workload, data_seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[1000 * wl.config_id + data_seed, stream]))


def _store(a32: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(a32) if dtype == "bf16" else np.ascontiguousarray(a32, dtype=np.float32)


def make_W_rows(wl: Workload, data_seed: int, row_lo: int, row_hi: int) -> np.ndarray:
    """Rows [row_lo, row_hi) of W in storage type; rows are N(0, 1/d) rounded to dtype."""
    if wl.dtype == "fp8":
        raise ValueError("FP8 heads are built by make_inputs (codes + row scales)")
    out = np.empty((row_hi - row_lo, wl.d), dtype=np.uint16 if wl.dtype == "bf16" else np.float32)
    scale = np.float32(1.0 / np.sqrt(wl.d))
    blk_lo = row_lo // W_BLOCK_ROWS
    blk_hi = (row_hi + W_BLOCK_ROWS - 1) // W_BLOCK_ROWS
    for blk in range(blk_lo, blk_hi):
        r0 = blk * W_BLOCK_ROWS
        r1 = min(wl.V, r0 + W_BLOCK_ROWS)
        g = _gen(wl, data_seed, _S_WBLOCK0 + blk)
        a = g.standard_normal((r1 - r0, wl.d), dtype=np.float32) * scale
        lo, hi = max(r0, row_lo), min(r1, row_hi)
        out[lo - row_lo:hi - row_lo] = _store(a[lo - r0:hi - r0], wl.dtype)
    return out


def make_W(wl: Workload, data_seed: int, threads: Optional[int] = None) -> np.ndarray:
    """The whole LM head, filled block by block on a few host threads."""
    nblk = (wl.V + W_BLOCK_ROWS - 1) // W_BLOCK_ROWS
    W = np.empty((wl.V, wl.d), dtype=np.uint16 if wl.dtype == "bf16" else np.float32)

    def fill(blk: int) -> None:
        r0 = blk * W_BLOCK_ROWS
        r1 = min(wl.V, r0 + W_BLOCK_ROWS)
        W[r0:r1] = make_W_rows(wl, data_seed, r0, r1)

    threads = threads or min(16, os.cpu_count() or 1)
    if threads <= 1 or nblk == 1:
        for blk in range(nblk):
            fill(blk)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(fill, range(nblk)))
    return W


def make_inputs(wl: Workload, data_seed: int = 0, W: Optional[np.ndarray] = None,
                tau: Optional[float] = None) -> Inputs:
    """Draw one workload.  ``W`` may be passed in when it was already generated
    for this (workload, data_seed); it is not checked."""
    B, M, d, V = wl.B, wl.M, wl.d, wl.V
    w_scale = None
    if wl.dtype == "fp8":
        # the same N(0, 1/d) head as the bf16 workload, stored as FP8 E4M3 with a scale per row
        if W is None:
            base = dataclasses.replace(wl, dtype="f32")
            codes = np.empty((V, d), dtype=np.uint8)
            w_scale = np.empty(V, dtype=np.float32)
            for r0 in range(0, V, 8 * W_BLOCK_ROWS):
                r1 = min(V, r0 + 8 * W_BLOCK_ROWS)
                codes[r0:r1], w_scale[r0:r1] = quantise_rows_fp8(make_W_rows(base, data_seed, r0, r1))
            W = codes
        else:
            W, w_scale = W
    elif W is None:
        W = make_W(wl, data_seed)

    g = _gen(wl, data_seed, _S_TOKENS)
    planted = g.integers(0, V, size=(B, M + 1), dtype=np.int64).astype(np.int32)
    draft_tokens = np.ascontiguousarray(planted[:, :M])

    # per-row planted-alignment scale
    ga = _gen(wl, data_seed, _S_ALPHA)
    if wl.alpha_range is None:
        alpha = np.full((B, M + 1), wl.alpha, dtype=np.float32)
    elif wl.alpha_per == "seq":
        alpha = np.repeat(ga.uniform(*wl.alpha_range, size=(B, 1)), M + 1, axis=1).astype(np.float32)
    else:
        alpha = ga.uniform(*wl.alpha_range, size=(B, M + 1)).astype(np.float32)
    if wl.forced_reject_at is not None:
        alpha[:, wl.forced_reject_at] = 0.0

    # judge head
    gj = _gen(wl, data_seed, _S_JUDGE)
    w32 = gj.standard_normal(d, dtype=np.float32) * np.float32(1.0 / np.sqrt(d))
    b_judge = float(gj.standard_normal() * wl.b_judge_std) if wl.b_judge_std > 0 else 0.0
    act_dtype = "bf16" if wl.dtype == "fp8" else wl.dtype     # storage type of H and w_judge
    w_store = _store(w32, act_dtype)
    w_val = as_f32(w_store).astype(np.float64)

    # H = alpha * unit(W[planted]) + sigma * noise, rounded to the storage type
    gn = _gen(wl, data_seed, _S_NOISE)
    H32 = np.empty((B, M + 1, d), dtype=np.float32)
    for b in range(B):
        if wl.dtype == "fp8":
            rows = (fp8_codes_to_f32(W[planted[b]]) * w_scale[planted[b]][:, None]).astype(np.float64)
        else:
            rows = as_f32(W[planted[b]]).astype(np.float64)             # [M+1, d]
        unit = rows / np.linalg.norm(rows, axis=1, keepdims=True)
        noise = gn.standard_normal((M + 1, d), dtype=np.float32).astype(np.float64) * wl.sigma
        H32[b] = (alpha[b][:, None].astype(np.float64) * unit + noise).astype(np.float32)

    # draft logits
    gd = _gen(wl, data_seed, _S_DLOGITS)
    dl = gd.standard_normal((B, M, V), dtype=np.float32)
    dl *= np.float32(wl.dl_std)
    gb = _gen(wl, data_seed, _S_BOOST)
    if wl.boost_range is None:
        boost = np.full((B, M), wl.boost, dtype=np.float32)
    else:
        boost = gb.uniform(*wl.boost_range, size=(B, M)).astype(np.float32)

    if wl.forced_reject_at is not None:
        # Make slot k fail both tests whatever the uniforms are: the drafted token gets a
        # strongly boosted draft logit while the target row (alpha = 0) does not favour it,
        # and the embedding the judge reads for that slot (row k+1) is shifted along the
        # judge direction so that its judge logit w.h + b equals -4.
        k = wl.forced_reject_at
        boost[:, k] = 8.0
        for b in range(B):
            h = H32[b, k + 1].astype(np.float64)
            cur = float(w_val @ h) + b_judge
            h = h + ((-4.0 - cur) / float(w_val @ w_val)) * w_val
            H32[b, k + 1] = h.astype(np.float32)

    bi, ji = np.meshgrid(np.arange(B), np.arange(M), indexing="ij")
    dl[bi, ji, draft_tokens] += boost

    H = _store(H32, act_dtype)
    return Inputs(wl=wl, data_seed=data_seed, W=W, H=H, w_judge=w_store, b_judge=b_judge,
                  tau=wl.tau if tau is None else tau, draft_tokens=draft_tokens,
                  draft_logits=np.ascontiguousarray(dl), seed=data_seed, planted_tokens=planted, w_scale=w_scale)
