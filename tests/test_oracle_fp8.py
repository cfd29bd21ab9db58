"""Pins for the checker's FP8 E4M3 pieces: the code table and the rounding are checked against an
independent implementation (PyTorch's CPU float8_e4m3fn conversion), the quantised head against
hand arithmetic."""
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


def test_fp8_head_logits_by_hand():
    rng = np.random.default_rng(2)
    V, d, M = 6, 8, 2
    W8 = rng.integers(0, 0x7E, size=(V, d)).astype(np.uint8) | (rng.integers(0, 2, size=(V, d)).astype(np.uint8) << 7)
    sw = rng.uniform(0.01, 0.1, V).astype(np.float32)
    H = rng.standard_normal((1, M + 1, d)).astype(np.float32)
    x = rng.integers(0, V, size=(1, M)).astype(np.int32)
    dl = rng.standard_normal((1, M, V))
    r = O.jd_oracle_verify(W8, np.zeros(d), 0.0, H, x, dl, 0.5, 0, w_scale=sw, keep_logits=True)
    tab = O.e4m3_decode(np.arange(256, dtype=np.uint8))
    for j in range(M + 1):
        amax = np.float32(np.abs(H[0, j]).max())
        inv = np.float32(448.0) / amax
        h8 = [float(torch.tensor(np.float32(h * inv)).to(torch.float8_e4m3fn).float()) for h in H[0, j]]
        sh = float(amax / np.float32(448.0))
        for v in range(V):
            want = float(sw[v]) * sh * sum(tab[W8[v, k]] * h8[k] for k in range(d))
            assert abs(r.logits[0][j, v] - want) <= 1e-12 * max(1.0, abs(want))
