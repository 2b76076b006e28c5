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
