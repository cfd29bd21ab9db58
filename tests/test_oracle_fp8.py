"""Pins for the checker's FP8 E4M3 pieces: the code table and the rounding are checked against an
independent implementation (PyTorch's CPU float8_e4m3fn conversion); the per-row quantiser and the
quantised head against an exhaustive nearest-value search over the format's table in exact
rational arithmetic."""
from fractions import Fraction

import numpy as np
import torch

from oracle import jd_oracle as O


def test_decode_matches_library_table_for_all_codes():
    codes = np.arange(256, dtype=np.uint8)
    mine = O.e4m3_decode(codes)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(np.isnan(mine), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(mine[ok], lib[ok])
    assert mine[0x7E] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6


def test_rounding_matches_library_conversion_and_saturates():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 100, rng.standard_normal(20000) * 0.01,
                        rng.uniform(-460, 460, 20000)]).astype(np.float32)
    grid = O.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    mids = ((grid[:-1] + grid[1:]) / 2).astype(np.float32)          # exact ties
    x = np.concatenate([x, mids, -mids, grid.astype(np.float32)])
    x = x[np.abs(x) <= 464.0]                                        # the library turns larger values into NaN
    mine = O.e4m3_round(x)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(mine, lib)
    assert O.e4m3_round(np.array([1e6, -500.0], np.float32)).tolist() == [448.0, -448.0]


def test_row_quantisation_is_per_row_and_uses_the_full_range():
    rng = np.random.default_rng(1)
    H = (rng.standard_normal((5, 64)) * np.array([[0.01], [1.0], [30.0], [1000.0], [0.0]])).astype(np.float32)
    vals, scale = O.quantise_rows_e4m3(H)
    assert np.all(np.abs(vals[:4]).max(axis=1) == 448.0) and np.all(vals[4] == 0) and scale[4] == 0
    assert np.allclose(scale[:4], np.abs(H[:4]).max(axis=1) / 448.0, rtol=1e-6)
    rel = np.abs(vals[:4] * scale[:4, None] - H[:4]) / np.abs(H[:4]).max(axis=1, keepdims=True)
    assert rel.max() < 2.0 ** -4                                     # half a spacing at the top binade


# The finite non-negative E4M3 values in code order, written out from the format's definition
# (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; exponent field 0 = subnormal; 0x7F = NaN).
E4M3_GRID = [Fraction(c & 7, 8) * Fraction(1, 64) if (c >> 3) == 0
             else Fraction(8 + (c & 7), 8) * Fraction(2) ** ((c >> 3) - 7) for c in range(0x7F)]


def nearest_e4m3_exact(t: Fraction) -> Fraction:
    """Brute force: the table value nearest to t; of two equally near ones the one with the even
    code (= even mantissa); beyond the largest value, the largest value."""
    a = abs(t)
    best = min(range(len(E4M3_GRID)), key=lambda c: (abs(E4M3_GRID[c] - a), c & 1))
    return E4M3_GRID[best] if t >= 0 else -E4M3_GRID[best]


def bf16_round(a):
    u = np.asarray(a, dtype=np.float32).view(np.uint32)
    r = ((u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)).astype(np.uint16)
    return r


def bf16_value(bits) -> float:
    return float((np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32))


def test_grid_written_from_the_definition_has_the_known_corner_values():
    assert E4M3_GRID[0] == 0 and E4M3_GRID[1] == Fraction(1, 512) and E4M3_GRID[7] == Fraction(7, 512)
    assert E4M3_GRID[8] == Fraction(1, 64) and E4M3_GRID[0x38] == 1 and E4M3_GRID[0x7E] == 448
    assert all(E4M3_GRID[c] < E4M3_GRID[c + 1] for c in range(0x7E))


def test_row_quantiser_equals_exact_rational_nearest_value_search():
    """Every element of bf16 rows of very different magnitudes, plus rows built so that many
    elements fall exactly half-way between two table values."""
    rng = np.random.default_rng(5)
    d = 96
    rows = rng.standard_normal((6, d)) * np.array([[1e-3], [0.02], [1.0], [7.0], [300.0], [4e4]])
    bits = bf16_round(rows.astype(np.float32))
    # tie rows: amax = 448 * 2^k (exact in bf16), other elements = mid-points of the grid * 2^k
    mids = [float((E4M3_GRID[c] + E4M3_GRID[c + 1]) / 2) for c in range(0x7E)]
    mids = [m for m in mids if bf16_value(bf16_round(np.float32(m))) == m]      # representable in bf16
    assert len(mids) >= 60
    for k in (-9, 0, 5):
        row = np.zeros(d, dtype=np.float32)
        row[0] = 448.0 * 2.0 ** k
        sel = rng.choice(len(mids), d - 1, replace=len(mids) < d - 1)
        row[1:] = np.array(mids)[sel] * 2.0 ** k * rng.choice([-1.0, 1.0], d - 1)
        bits = np.concatenate([bits, bf16_round(row)[None]], axis=0)
    vals, scale = O.quantise_rows_e4m3(bits)
    ties = 0
    for r in range(bits.shape[0]):
        h = [Fraction(bf16_value(b)) for b in bits[r]]
        amax = max(abs(v) for v in h)
        assert Fraction(float(scale[r])) == Fraction(float(amax / 448))          # a_r / 448, rounded once
        for k in range(d):
            t = h[k] * 448 / amax
            want = nearest_e4m3_exact(t)
            assert Fraction(float(vals[r, k])) == want, (r, k, float(t), float(vals[r, k]), float(want))
            ties += any(abs(t) == (E4M3_GRID[c] + E4M3_GRID[c + 1]) / 2 for c in range(0x7E))
    assert ties >= 200                                                            # the tie rule was exercised


def test_rounding_saturates_and_keeps_sign_in_float64():
    x = np.array([449.0, 1e9, -1e9, 464.0, -447.99, 2.0 ** -10, 2.0 ** -10 * (1 + 1e-9), -0.0])
    got = O.e4m3_round(x)
    assert got.tolist()[:7] == [448.0, 448.0, -448.0, 448.0, -448.0, 0.0, 2.0 ** -9]
    assert np.signbit(got[7])
    # a float64 just above a mid-point must round up although its float32 rounding is the mid-point
    mid = 1.0625                                                                  # between 1.0 and 1.125
    assert O.e4m3_round(np.array([mid, mid * (1 + 1e-12), mid * (1 - 1e-12)])).tolist() == [1.0, 1.125, 1.0]


def test_fp8_head_logits_by_hand():
    rng = np.random.default_rng(2)
    V, d, M = 6, 8, 2
    W8 = rng.integers(0, 0x7E, size=(V, d)).astype(np.uint8) | (rng.integers(0, 2, size=(V, d)).astype(np.uint8) << 7)
    sw = rng.uniform(0.01, 0.1, V).astype(np.float32)
    H = rng.standard_normal((1, M + 1, d)).astype(np.float32)
    x = rng.integers(0, V, size=(1, M)).astype(np.int32)
    dl = rng.standard_normal((1, M, V))
    r = O.jd_oracle_verify(W8, np.zeros(d), 0.0, H, x, dl, 0.5, 0, w_scale=sw, keep_logits=True)
    for j in range(M + 1):
        h = [Fraction(float(v)) for v in H[0, j]]
        amax = max(abs(v) for v in h)
        h8 = [nearest_e4m3_exact(v * 448 / amax) for v in h]
        for v in range(V):
            w = [(-1 if W8[v, k] & 0x80 else 1) * E4M3_GRID[W8[v, k] & 0x7F] for k in range(d)]
            want = float(Fraction(float(sw[v])) * (amax / 448) * sum(a * b for a, b in zip(w, h8)))
            assert abs(r.logits[0][j, v] - want) <= 1e-12 * max(1.0, abs(want))
