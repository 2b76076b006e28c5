"""Pins for the CPU checker's scale / zero-point / code steps
(Section 3.2, Eqs. "s", "z", "q", "w") and for its packed format.

Pins used: hand-evaluated closed forms (tests/golden/grid_group.json),
properties that single out the intended scale and codes without restating
their formulas (coverage + minimality of the scale, brute-force nearest
level), the library fake-quantize routine as the special case without
outliers, and hand-derived bytes for the packed format.
"""
import json
import os

import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _quant(W, G, frac, bits, group):
    return orc.quantize_layer(W, G, frac, bits, group)


# ---------------------------------------------------------------- closed forms
def test_grid_group_closed_form():
    cases = json.load(open(os.path.join(GOLD, "grid_group.json")))["cases"]
    for c in cases:
        bits, e = c["bits"], c["step_log2"]
        ints = np.arange(c["i_min"], c["i_max"] + 1)
        group = 64
        rng = np.random.default_rng(0)
        # fill a group of 64 with grid values, both extremes present
        vals = np.concatenate([ints, rng.choice(ints, size=group - len(ints))])
        rng.shuffle(vals)
        W = (vals * 2.0 ** e).astype(np.float16).reshape(1, group)
        mask = np.zeros((1, group), dtype=bool)
        s, z = orc.group_stats(W, mask, bits, group)
        assert float(s[0, 0]) == c["scale"] and int(z[0, 0]) == c["zero"]
        q = orc.quantize_codes(W, mask, s, z, bits, group)
        assert np.array_equal(q[0].astype(np.int64), vals - c["i_min"] if c["i_min"] <= 0 else vals)
        empty = (np.zeros(2, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16))
        w_hat = orc.dequantize(q, s, z, group, *empty)
        assert np.array_equal(w_hat, W.astype(np.float64))          # zero error


def test_degenerate_groups():
    # all-zero group and all-outlier group: s = 1, z = 0, codes 0, reconstruction exact
    W = np.zeros((2, 64), dtype=np.float16)
    W[1] = np.linspace(-1, 1, 64).astype(np.float16)
    mask = np.zeros((2, 64), dtype=bool)
    mask[1] = True
    s, z = orc.group_stats(W, mask, 4, 64)
    assert s.view(np.uint16).tolist() == [[0x3C00], [0x3C00]] and z.tolist() == [[0], [0]]
    q = orc.quantize_codes(W, mask, s, z, 4, 64)
    assert not q.any()
    # one surviving positive entry: range is widened to contain 0
    mask[1, 7] = False
    s, z = orc.group_stats(W, mask, 4, 64)
    q = orc.quantize_codes(W, mask, s, z, 4, 64)
    assert z[1, 0] == 0 if W[1, 7] > 0 else z[1, 0] == 15
    assert q[1, 7] in (0, 15) and (np.delete(q[1], 7) == z[1, 0]).all()


# ---------------------------------------------------------------- properties
@pytest.mark.parametrize("bits,group,frac,seed", [(4, 128, 0.01, 0), (3, 64, 0.02, 1), (4, 64, 0.0, 2),
                                                   (3, 128, 0.3, 3), (4, 16, 0.01, 4), (3, 32, 0.02, 5),
                                                   (8, 128, 0.01, 6), (2, 64, 0.01, 7), (8, 16, 0.0, 8)])
def test_scale_covers_range_and_is_minimal(bits, group, frac, seed):
    N, K = 64, 512
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = _quant(W, G, frac, bits, group)
    qmax = 2 ** bits - 1
    w = W.astype(np.float64).reshape(N, K // group, group)
    m = L["mask"].reshape(N, K // group, group)
    lo = np.minimum(np.where(m, 0.0, w).min(axis=2), 0.0)
    hi = np.maximum(np.where(m, 0.0, w).max(axis=2), 0.0)
    s = L["scales"].astype(np.float64)
    live = hi > lo
    # the scale spans the range with qmax steps ...
    assert np.all(s[live] * qmax >= (hi - lo)[live])
    # ... and the next smaller fp16 number would not
    s_prev = np.nextafter(L["scales"], np.float16(0)).astype(np.float64)
    assert np.all(s_prev[live] * qmax < (hi - lo)[live])
    # zero-point: an integer code whose reconstruction is exactly 0 and which
    # places lo within half a step of code 0
    z = L["zeros"].astype(np.float64)
    assert np.all((z >= 0) & (z <= qmax))
    assert np.all(np.abs(lo / s + z)[live] <= 0.5)


@pytest.mark.parametrize("bits,group,frac", [(4, 128, 0.01), (3, 128, 0.01), (4, 64, 0.005), (3, 64, 0.02),
                                             (4, 16, 0.01), (3, 16, 0.01), (4, 32, 0.02), (8, 128, 0.01),
                                             (2, 128, 0.01), (2, 32, 0.02), (8, 64, 0.005)])
def test_error_bound_and_outlier_codes(bits, group, frac):
    N, K = 128, 1024
    W, G = synth.make_weight_and_grad(N, K, seed=4)
    L = _quant(W, G, frac, bits, group)
    s = np.repeat(L["scales"].astype(np.float64), group, axis=1)
    z = np.repeat(L["zeros"], group, axis=1)
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], group, L["row_ptr"], L["col_idx"], L["val"])
    err = np.abs(w_hat - W.astype(np.float64))
    assert np.all(err[~L["mask"]] <= 0.5 * s[~L["mask"]] * (1 + 1e-12))
    assert np.all(err[L["mask"]] == 0.0)                     # outliers kept exactly
    assert np.array_equal(L["codes"][L["mask"]], z[L["mask"]])  # outlier code is the zero-point
    assert L["codes"].max() <= 2 ** bits - 1


def test_codes_are_nearest_level_brute_force():
    # given (s, z), the stored code must minimise |w - s (q - z)| over all levels
    _codes_are_nearest_levels(4, 64)
    _codes_are_nearest_levels(8, 128)
    _codes_are_nearest_levels(2, 32)


def _codes_are_nearest_levels(bits, group):
    N, K = 8, 256
    W, G = synth.make_weight_and_grad(N, K, seed=6)
    L = _quant(W, G, 0.02, bits, group)
    s = np.repeat(L["scales"].astype(np.float64), group, axis=1)
    z = np.repeat(L["zeros"].astype(np.float64), group, axis=1)
    levels = np.arange(2 ** bits, dtype=np.float64)
    cand = s[..., None] * (levels[None, None, :] - z[..., None])
    dist = np.abs(cand - W.astype(np.float64)[..., None])
    best = dist.min(axis=2)
    chosen = np.take_along_axis(dist, L["codes"].astype(np.int64)[..., None], axis=2)[..., 0]
    keep = ~L["mask"]
    assert np.array_equal(chosen[keep], best[keep])


def test_without_outliers_equals_library_fake_quantize():
    # frac = 0 is plain min/max asymmetric round-to-nearest; given the scales
    # and zero-points, torch's per-channel fake-quantize must reproduce the
    # reconstruction (compared away from exact rounding ties, where the
    # library adds the zero-point before rounding).
    N, K, bits, group = 32, 512, 4, 128
    W, G = synth.make_weight_and_grad(N, K, seed=8)
    L = _quant(W, G, 0.0, bits, group)
    assert L["row_ptr"][-1] == 0
    empty = (L["row_ptr"], L["col_idx"], L["val"])
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], group, *empty)
    rows = torch.from_numpy(W.astype(np.float64)).reshape(N * K // group, group)
    sc = torch.from_numpy(L["scales"].astype(np.float64)).reshape(-1)
    zp = torch.from_numpy(L["zeros"].astype(np.int32)).reshape(-1)
    ref = torch.fake_quantize_per_channel_affine(rows.float(), sc.float(), zp, 0, 0, 2 ** bits - 1)
    ref = ref.double().numpy().reshape(N, K)
    s = np.repeat(L["scales"].astype(np.float64), group, axis=1)
    frac_part = np.abs(W.astype(np.float64) / s - np.floor(W.astype(np.float64) / s) - 0.5)
    away = frac_part > 1e-4
    assert away.mean() > 0.99
    assert np.allclose(w_hat[away], ref[away], rtol=0, atol=1e-6)


def test_round_half_even_at_exact_ties():
    # s = 2^-6 exactly (range 15 * 2^-6); entries at (m + 1/2) s must go to the even code offset
    base = np.zeros(64)
    base[0], base[1] = -8, 7                      # fixes s = 2^-6, z = 8
    ties = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, -3.5])
    base[2:10] = ties
    W = (base * 2.0 ** -6).astype(np.float16).reshape(1, 64)
    mask = np.zeros((1, 64), dtype=bool)
    s, z = orc.group_stats(W, mask, 4, 64)
    assert float(s[0, 0]) == 2.0 ** -6 and z[0, 0] == 8
    q = orc.quantize_codes(W, mask, s, z, 4, 64)
    assert (q[0, 2:10].astype(int) - 8).tolist() == [0, 2, 2, 0, -2, -2, 4, -4]


def test_nonfinite_weight_rejected():
    W = np.ones((1, 64), dtype=np.float16)
    W[0, 3] = np.inf
    with pytest.raises(ValueError):
        orc.group_stats(W, np.zeros((1, 64), dtype=bool), 4, 64)


# ---------------------------------------------------------------- packed format
def test_pack_golden_bytes():
    cases = json.load(open(os.path.join(GOLD, "pack_layout.json")))["cases"]
    for c in cases:
        codes = np.array([c["codes"]], dtype=np.uint8)
        words = orc.pack_codes(codes, c["bits"])
        assert [f"{int(w):08X}" for w in words[0]] == c["words_hex"]
        assert np.array_equal(orc.unpack_codes(words, c["bits"], 32), codes)


def _pack_run_scalar(codes32, bits):
    """The written format definition, one column at a time, in plain Python integers."""
    words = [0] * bits
    for i, c in enumerate(codes32):
        c = int(c)
        if bits == 4:
            t, j, e = i // 8, (i % 8) // 2, i % 2
            words[t] |= c << (16 * e + 4 * j)
        elif bits in (2, 8):
            per = 32 // bits
            t, j, e = i // per, (i % per) // 2, i % 2
            words[t] |= c << (16 * e + bits * j)
        else:
            if i < 30:
                w, p_, e = i // 10, (i % 10) // 2, i % 2
                words[w] |= c << (16 * e + 3 * p_)
            else:
                for b in range(3):
                    words[b] |= ((c >> b) & 1) << (15 if i == 30 else 31)
    return words


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_pack_matches_scalar_definition_and_roundtrips(bits):
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 2 ** bits, size=(5, 160), dtype=np.uint8)
    words = orc.pack_codes(codes, bits)
    assert words.shape == (5, 160 * bits // 32) and words.dtype == np.uint32
    for n in range(5):
        for r in range(160 // 32):
            want = _pack_run_scalar(codes[n, 32 * r:32 * r + 32], bits)
            assert [int(w) for w in words[n, bits * r:bits * r + bits]] == want
    assert np.array_equal(orc.unpack_codes(words, bits, 160), codes)
    # every bit of every word is used exactly once: all-ones codes fill the words
    full = orc.pack_codes(np.full((1, 32), 2 ** bits - 1, dtype=np.uint8), bits)
    assert [int(w) for w in full[0]] == [0xFFFFFFFF] * bits
    with pytest.raises(ValueError):
        orc.pack_codes(np.full((1, 32), 2 ** bits, dtype=np.uint16), bits)
