"""Parity on Llama-70B-shaped layers (8192 x 8192, 28672 x 8192, 8192 x 28672): both bit widths,
groups of 64 and 128, outlier fractions 0.5 / 1 / 2 %, M in {1, 8, 32, 2048}.  As at the other full
sizes the CPU checker selects the outliers of the whole matrix (compared in full, bit for bit) and
encodes, reconstructs and multiplies 272 distinct sampled output rows for every token row; for the first encoding
of every shape, 64 seeded token rows of the M = 2048 product are also checked on every output row (the checker
then walks the whole matrix block of rows by block of rows)."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, checker_row_blocks, checker_rows, distinct_rows, to_dev, x_tensor

pytestmark = pytest.mark.gpu


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
    rows = distinct_rows(N, seed=40 + shape_index, count=272)
    assert len(set(rows)) >= 256
    for enc_i, (bits, group) in enumerate(encodings):
        S = gwq.gwq_select_outliers(Wd, Gd, frac)
        P = gwq.gwq_pack(Wd, S, bits, group)
        a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
        if enc_i == 0:   # the selection does not depend on the encoding
            assert np.array_equal(a["row_ptr"], row_ptr)
            assert np.array_equal(a["col_idx"], col_idx)
            assert np.array_equal(a["val"].view(np.uint16), val)
        s, z, words, w_hat = checker_rows(W, row_ptr, col_idx, val, rows, bits, group)
        assert np.array_equal(a["scales"].view(np.uint16)[rows], s.view(np.uint16))
        assert np.array_equal(a["zeros"][rows], z)
        assert np.array_equal(a["words"].view(np.uint32)[rows], words)
        del a
        for M, dtype in ((1, "f16"), (8, "f16"), (32, "bf16"), (2048, "bf16")):
            bits16, xv = synth.make_activations(M, K, seed=4100 + 10 * shape_index + M % 7, dtype=dtype,
                                                heavy_channels=8 if M == 2048 else 0)
            y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
            torch.cuda.synchronize()
            y_ref, bound = orc.linear(xv, w_hat)       # every token row on the sampled output rows
            assert_linear_close(y[:, rows], y_ref, bound)
            if M == 2048 and enc_i == 0:               # 64 seeded token rows on every output row
                toks = np.sort(np.random.default_rng(4200 + shape_index).choice(M, size=64, replace=False))
                y_t = y[torch.from_numpy(toks).to(y.device)].double().cpu()
                for r0, r1, _s, _z, _w, wh in checker_row_blocks(W, row_ptr, col_idx, val, bits, group, block=4096):
                    y_ref, bound = orc.linear(xv[toks], wh)
                    assert_linear_close(y_t[:, r0:r1], y_ref, bound)
            del y
        assert gwq.gwq_device_status(P) == 0
        del P, S
