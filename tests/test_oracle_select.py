"""Pins for the CPU checker's outlier selection (Section 3.2, Eq. "o").

None of these restates the checker's lexsort: they use a pure-Python tuple
sort over the raw IEEE bit patterns, a closed form on permutations, and
order invariants that hold for any correct exact top-k.
"""
import math
import struct

import numpy as np
import pytest

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import synth


def _bits_abs(g: float) -> int:
    return struct.unpack("<I", struct.pack("<f", g))[0] & 0x7FFFFFFF


def _brute_force(G, k):
    flat = [float(v) for v in G.reshape(-1)]
    order = sorted(range(len(flat)), key=lambda i: (-_bits_abs(flat[i]), i))
    return sorted(order[:k])


def _csr_to_flat(row_ptr, col_idx, K):
    out = []
    for n in range(len(row_ptr) - 1):
        for j in range(row_ptr[n], row_ptr[n + 1]):
            out.append(n * K + int(col_idx[j]))
    return out


@pytest.mark.parametrize("N,K,frac,kind", [
    (8, 32, 0.01, "smooth"), (16, 64, 0.05, "smooth"), (64, 64, 0.01, "smooth"),
    (8, 32, 0.1, "ties"), (64, 64, 0.02, "ties"), (32, 32, 0.5, "ties"),
    (4, 32, 0.3, "two_levels"), (4, 32, 0.999, "smooth"),
])
def test_select_matches_brute_force(N, K, frac, kind):
    W, G = synth.make_weight_and_grad(N, K, seed=3)
    if kind == "ties":
        G = synth.make_tie_heavy_grad(N, K, seed=5, levels=7)
    elif kind == "two_levels":
        G = np.where(np.arange(N * K).reshape(N, K) % 3 == 0, -2.0, 2.0).astype(np.float32)
        G[1, 5] = 3.0
    row_ptr, col_idx, val = orc.select_outliers(W, G, frac)
    k = math.ceil(frac * N * K)
    assert row_ptr[-1] == k == len(col_idx) == len(val)
    want = _brute_force(G, k)
    assert _csr_to_flat(row_ptr, col_idx, K) == want
    wbits = W.view(np.uint16).reshape(-1)
    assert [int(v) for v in val] == [int(wbits[i]) for i in want]


def test_select_permutation_closed_form():
    # G is a seeded permutation of 1..numel: the k largest are numel-k+1..numel.
    N, K = 24, 32
    rng = np.random.default_rng(11)
    perm = rng.permutation(N * K) + 1
    G = perm.reshape(N, K).astype(np.float32) * np.where(rng.random((N, K)) < 0.5, -1, 1).astype(np.float32)
    W = rng.normal(size=(N, K)).astype(np.float16)
    for frac in (0.01, 0.25):
        k = math.ceil(frac * N * K)
        row_ptr, col_idx, _ = orc.select_outliers(W, G, frac)
        got = set(_csr_to_flat(row_ptr, col_idx, K))
        want = set(np.nonzero(perm > N * K - k)[0].tolist())
        assert got == want


def test_select_count_and_edges():
    W, G = synth.make_weight_and_grad(16, 64, seed=1)
    rp, ci, v = orc.select_outliers(W, G, 0.0)
    assert rp.tolist() == [0] * 17 and len(ci) == 0 and len(v) == 0
    rp, ci, v = orc.select_outliers(W, G, 1.0)
    assert rp.tolist() == [64 * i for i in range(17)]
    assert ci.reshape(16, 64).tolist() == [list(range(64))] * 16
    assert np.array_equal(v.reshape(16, 64), W.view(np.uint16))
    # ceil of the literal double product
    assert orc.outlier_count(0.01, 4096 * 4096) == 167773
    assert orc.outlier_count(0.07, 100) == math.ceil(0.07 * 100)
    assert orc.outlier_count(1e-9, 1000) == 1
    with pytest.raises(ValueError):
        orc.outlier_count(1.5, 10)


def test_select_order_invariants_large():
    N, K, frac = 256, 512, 0.01
    W, _ = synth.make_weight_and_grad(N, K, seed=2)
    G = synth.make_tie_heavy_grad(N, K, seed=9, levels=64)
    row_ptr, col_idx, val = orc.select_outliers(W, G, frac)
    mask = orc.outlier_mask(row_ptr, col_idx, N, K).reshape(-1)
    key = np.abs(G).reshape(-1)
    assert mask.sum() == math.ceil(frac * N * K)
    thr = key[mask].min()
    assert thr >= key[~mask].max()
    at_thr = key == thr
    sel_thr = np.nonzero(at_thr & mask)[0]
    unsel_thr = np.nonzero(at_thr & ~mask)[0]
    assert len(unsel_thr) > 0, "test should exercise a tie at the threshold"
    assert sel_thr.max() < unsel_thr.min()
    # columns strictly ascending inside each row
    for n in range(N):
        c = col_idx[row_ptr[n]:row_ptr[n + 1]]
        assert np.all(np.diff(c) > 0)


def test_select_special_values_order():
    # -0 == +0 < denormal < finite < inf < NaN under the bit-pattern order
    base = [0.0, -0.0, 1e-45, -1.0, np.inf, np.nan, 2.0, -np.inf]
    G = np.tile(np.array([base], dtype=np.float32), (1, 4))
    W = np.arange(32, dtype=np.float16).reshape(1, 32)
    nan_cols = [5, 13, 21, 29]
    inf_cols = [4, 7, 12, 15, 20, 23, 28, 31]
    _, ci, _ = orc.select_outliers(W, G, 4 / 32)
    assert ci.tolist() == nan_cols
    _, ci, _ = orc.select_outliers(W, G, 9 / 32)
    assert ci.tolist() == sorted(nan_cols + inf_cols[:5])
    # 4 NaN + 8 inf + 4 (2.0) + 4 (1.0) + 4 denormals = 24; two more must be
    # the two lowest-index zeros, +0 and -0 ranking equal
    _, ci, _ = orc.select_outliers(W, G, 26 / 32)
    zero_cols_taken = [c for c in ci.tolist() if c % 8 in (0, 1)]
    assert len(ci) == 26 and zero_cols_taken == [0, 1]


# ---------------------------------------------------------------- gradient mean over calibration samples (Section 4.3)
def test_gradient_mean_pins():
    rng = np.random.default_rng(21)
    G = rng.normal(size=(6, 8, 32)).astype(np.float32)
    # one sample: the gradient itself
    assert np.array_equal(orc.gradient_mean([G[0]]), G[0])
    # small integers: every float32 sum is exact, so the mean is the exact quotient rounded once
    I = rng.integers(-50, 50, size=(5, 4, 16)).astype(np.float32)
    want = (I.astype(np.float64).sum(axis=0) / 5.0).astype(np.float32)
    assert np.array_equal(orc.gradient_mean(list(I)), want)
    # general values: within count roundings of the float64 mean
    m = orc.gradient_mean(list(G))
    ref = G.astype(np.float64).mean(axis=0)
    assert m.dtype == np.float32
    assert np.all(np.abs(m - ref) <= 6 * 2.0 ** -24 * np.abs(G).astype(np.float64).sum(axis=0) / 6 + 1e-45)
    # a power-of-two count of equal samples returns the sample (doubling and halving are exact)
    assert np.array_equal(orc.gradient_mean([G[1]] * 4), G[1])
