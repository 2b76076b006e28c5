"""Parity on Llama-70B-shaped layers (8192 x 8192, 28672 x 8192, 8192 x 28672): both bit widths,
groups of 64 and 128, outlier fractions 0.5 / 1 / 2 %, M in {1, 8, 32, 2048}.  As at the other full
sizes the CPU checker selects the outliers of the whole matrix (compared in full, bit for bit) and
encodes, reconstructs and multiplies ~250 sampled output rows one by one, for every token row."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, to_dev, x_tensor

pytestmark = pytest.mark.gpu


def _sample_rows(N, seed, extra=246):
    rng = np.random.default_rng(seed)
    rows = {0, 1, 7, 8, 15, 16, N - 17, N - 16, N - 2, N - 1}
    rows.update(int(r) for r in rng.integers(0, N, size=extra))
    return sorted(rows)


def _checker_rows(W, row_ptr, col_idx, val, rows, bits, group):
    K = W.shape[1]
    counts = [int(row_ptr[n + 1] - row_ptr[n]) for n in rows]
    sub_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    sub_col = np.concatenate([col_idx[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.int32)
    sub_val = np.concatenate([val[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.uint16)
    mask = orc.outlier_mask(sub_ptr, sub_col, len(rows), K)
    Ws = np.ascontiguousarray(W[rows])
    s, z = orc.group_stats(Ws, mask, bits, group)
    q = orc.quantize_codes(Ws, mask, s, z, bits, group)
    words = orc.pack_codes(q, bits)
    w_hat = orc.dequantize(q, s, z, group, sub_ptr, sub_col, sub_val)
    return s, z, words, w_hat


# (shape index, encodings as (bits, group) pairs, outlier fraction)
CASES = [
    (0, ((4, 64), (3, 128)), 0.02),
    (1, ((3, 128), (4, 128)), 0.005),
    (2, ((4, 128), (3, 64)), 0.01),
]


@pytest.mark.parametrize("shape_index,encodings,frac", CASES)
def test_llama70b_shaped_layer(shape_index, encodings, frac):
    N, K = synth.LLAMA70B_SHAPES[shape_index]
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(4, shape_index))
    row_ptr, col_idx, val = orc.select_outliers(W, G, frac)
    Wd, Gd = to_dev(W), to_dev(G)
    del G
    rows = _sample_rows(N, seed=40 + shape_index)
    for enc_i, (bits, group) in enumerate(encodings):
        S = gwq.gwq_select_outliers(Wd, Gd, frac)
        P = gwq.gwq_pack(Wd, S, bits, group)
        a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
        if enc_i == 0:   # the selection does not depend on the encoding
            assert np.array_equal(a["row_ptr"], row_ptr)
            assert np.array_equal(a["col_idx"], col_idx)
            assert np.array_equal(a["val"].view(np.uint16), val)
        s, z, words, w_hat = _checker_rows(W, row_ptr, col_idx, val, rows, bits, group)
        assert np.array_equal(a["scales"].view(np.uint16)[rows], s.view(np.uint16))
        assert np.array_equal(a["zeros"][rows], z)
        assert np.array_equal(a["words"].view(np.uint32)[rows], words)
        del a
        for M, dtype in ((1, "f16"), (8, "f16"), (32, "bf16"), (2048, "bf16")):
            bits16, xv = synth.make_activations(M, K, seed=4100 + 10 * shape_index + M % 7, dtype=dtype,
                                                heavy_channels=8 if M == 2048 else 0)
            y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
            torch.cuda.synchronize()
            y_ref, bound = orc.linear(xv, w_hat)       # every token row on ~250 sampled output rows
            assert_linear_close(y[:, rows], y_ref, bound)
            del y
        assert gwq.gwq_device_status(P) == 0
        del P, S
