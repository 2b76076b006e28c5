"""Pins for the CPU checker's reconstruction + product
(Section 3.2, Eq. "w"; outliers kept in FP16, Section 1)."""
import numpy as np
import pytest

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import synth


def _layer(N, K, frac, bits, group, seed):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], group, L["row_ptr"], L["col_idx"], L["val"])
    return W, L, w_hat


def test_all_outliers_reproduces_dense_product_exactly():
    W, L, w_hat = _layer(64, 256, 1.0, 4, 64, seed=1)
    assert np.array_equal(w_hat, W.astype(np.float64))
    _, x = synth.make_activations(5, 256, seed=1)
    y, bound = orc.linear(x, w_hat)
    assert np.array_equal(y, x @ W.astype(np.float64).T)
    assert np.all(bound >= np.abs(y))


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64)])
def test_unit_activation_reads_back_columns(bits, group):
    W, L, w_hat = _layer(32, 256, 0.02, bits, group, seed=2)
    cols = [0, 1, 17, 127, 128, 255]
    _, x = synth.unit_activations(cols, 256)
    y, bound = orc.linear(x, w_hat)
    for m, c in enumerate(cols):
        assert np.array_equal(y[m], w_hat[:, c])
        assert np.array_equal(bound[m], np.abs(w_hat[:, c]))


def test_product_against_scalar_definition():
    # y[m, n] = sum_k x[m, k] * (s (q - z) + S)[n, k], written as explicit loops
    W, L, w_hat = _layer(8, 64, 0.05, 4, 64, seed=3)
    _, x = synth.make_activations(3, 64, seed=3)
    y, bound = orc.linear(x, w_hat)
    S = {}
    for n in range(8):
        for j in range(L["row_ptr"][n], L["row_ptr"][n + 1]):
            S[(n, int(L["col_idx"][j]))] = float(np.array(L["val"][j], dtype=np.uint16).view(np.float16))
    for m in range(3):
        for n in range(8):
            acc = 0.0
            accb = 0.0
            for k in range(64):
                s = float(L["scales"][n, k // 64])
                w = s * (int(L["codes"][n, k]) - int(L["zeros"][n, k // 64])) + S.get((n, k), 0.0)
                acc += x[m, k] * w
                accb += abs(x[m, k] * w)
            assert abs(acc - y[m, n]) <= 1e-12 * max(1.0, accb)
            assert abs(accb - bound[m, n]) <= 1e-12 * max(1.0, accb)


def test_linearity_and_grid_aligned_weights():
    # weights on the quantization grid and no outliers: reconstruction is W itself
    rng = np.random.default_rng(5)
    ints = rng.integers(-8, 8, size=(16, 128))
    ints[:, 0], ints[:, 1] = -8, 7
    ints[:, 64], ints[:, 65] = -8, 7
    W = (ints * 2.0 ** -7).astype(np.float16)
    G = rng.normal(size=W.shape).astype(np.float32)
    L = orc.quantize_layer(W, G, 0.0, 4, 64)
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], 64, L["row_ptr"], L["col_idx"], L["val"])
    assert np.array_equal(w_hat, W.astype(np.float64))
    _, x1 = synth.make_activations(2, 128, seed=1)
    _, x2 = synth.make_activations(2, 128, seed=2)
    y1, _ = orc.linear(x1, w_hat)
    y2, _ = orc.linear(x2, w_hat)
    y12, _ = orc.linear(x1 + 2 * x2, w_hat)
    assert np.allclose(y12, y1 + 2 * y2, rtol=1e-13, atol=1e-13)
    assert np.array_equal(y1, x1 @ W.astype(np.float64).T)


def test_outliers_enter_once():
    # the dense term is exactly zero at outlier positions, so w_hat there is the fp16 weight
    W, L, w_hat = _layer(32, 256, 0.1, 3, 64, seed=7)
    m = L["mask"]
    assert m.sum() == L["row_ptr"][-1] and m.sum() > 0
    assert np.array_equal(w_hat[m], W.astype(np.float64)[m])


# ---------------------------------------------------------------- the method's objectives (Section 3.1)
def test_quality_scalar_definition_and_special_cases():
    # explicit loops over a tiny layer
    W, G = synth.make_weight_and_grad(4, 64, seed=9)
    L = orc.quantize_layer(W, G, 0.05, 4, 64)
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], 64, L["row_ptr"], L["col_idx"], L["val"])
    sq, fo = orc.quality(W, G, w_hat)
    a = b = 0.0
    for n in range(4):
        for k in range(64):
            d = float(W[n, k]) - float(w_hat[n, k])
            a += d * d
            b += float(G[n, k]) * d
    assert abs(sq - a) <= 1e-15 * max(1.0, a) and abs(fo - b) <= 1e-12 * max(1.0, abs(b))
    assert sq > 0.0
    # every weight kept as an outlier: nothing is lost
    L1 = orc.quantize_layer(W, G, 1.0, 4, 64)
    w1 = orc.dequantize(L1["codes"], L1["scales"], L1["zeros"], 64, L1["row_ptr"], L1["col_idx"], L1["val"])
    assert orc.quality(W, G, w1) == (0.0, 0.0)
    # with g = sign(W - W_Q) the first-order term is the L1 norm of the error, with g = 0 it vanishes
    d = W.astype(np.float64) - w_hat
    sq2, l1 = orc.quality(W, np.sign(d).astype(np.float32), w_hat)
    assert sq2 == sq and abs(l1 - np.abs(d).sum()) <= 1e-12
    assert orc.quality(W, np.zeros_like(G), w_hat)[1] == 0.0
    # the squared error respects the rounding bound: at most (s / 2)^2 per non-outlier entry
    s = np.repeat(L["scales"].astype(np.float64), 64, axis=1)
    assert sq <= np.sum((0.5 * s[~L["mask"]]) ** 2) * (1 + 1e-12)


def test_quality_closed_form_on_a_known_group():
    # one group whose range fixes s = 2^-6, z = 8; entries a quarter step off the grid lose (s / 4)^2 each
    base = np.zeros(64)
    base[0], base[1] = -8, 7
    base[2:12] = np.arange(10) - 4 + 0.25          # 10 entries, each 0.25 step above a grid point
    W = (base * 2.0 ** -6).astype(np.float16).reshape(1, 64)
    G = np.full((1, 64), 2.0, dtype=np.float32)
    L = orc.quantize_layer(W, G * 0 + np.arange(64, dtype=np.float32)[::-1], 0.0, 4, 64)
    assert float(L["scales"][0, 0]) == 2.0 ** -6 and int(L["zeros"][0, 0]) == 8
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], 64, L["row_ptr"], L["col_idx"], L["val"])
    sq, fo = orc.quality(W, G, w_hat)
    step = 2.0 ** -6
    assert sq == 10 * (0.25 * step) ** 2
    assert fo == 2.0 * 10 * 0.25 * step                # W - W_Q = +s/4 on those ten entries
