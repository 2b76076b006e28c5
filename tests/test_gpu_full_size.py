"""Parity at the benchmark's full layer sizes, in the launch configuration the benchmark times
(sibling layers through gwq_linear_multi, replayed from a CUDA graph; the tensor-core path with
bf16 activations and heavy channels).  The CPU checker encodes the whole layer (every row: CSR, scales,
zero-points and packed words are compared bit for bit) and every output is checked for M = 1, 4, 16, 512 and
2048; at M = 8192 all token rows are checked on 256 distinct output rows and 64 seeded token rows on every
output row."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, checker_row_blocks, distinct_rows, to_dev, x_tensor

pytestmark = pytest.mark.gpu

FRAC, GROUP = 0.01, 128


@pytest.mark.parametrize("N,K,bits,layer_index,whole", [(11008, 4096, 4, 4, True), (4096, 11008, 3, 6, True),
                                                         (11008, 4096, 8, 4, False), (4096, 11008, 2, 6, False)])
def test_full_size_layer(N, K, bits, layer_index, whole):
    # whole = False (the widths beside the paper's): the encoding, M = 1, 4, 16 and 2048 only
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(1, layer_index))
    row_ptr, col_idx, val = orc.select_outliers(W, G, FRAC)
    Wd, Gd = to_dev(W), to_dev(G)
    S = gwq.gwq_select_outliers(Wd, Gd, FRAC)
    P = gwq.gwq_pack(Wd, S, bits, GROUP)
    del Gd, G
    a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
    # the outlier set of the whole matrix, bit for bit
    assert np.array_equal(a["row_ptr"], row_ptr)
    assert np.array_equal(a["col_idx"], col_idx)
    assert np.array_equal(a["val"].view(np.uint16), val)
    # codes, scales and zero-points of every row, bit for bit; the reconstruction is kept for the products
    w_hat = np.empty((N, K), dtype=np.float64)
    for r0, r1, s, z, words, wh in checker_row_blocks(W, row_ptr, col_idx, val, bits, GROUP):
        assert np.array_equal(a["scales"].view(np.uint16)[r0:r1], s.view(np.uint16))
        assert np.array_equal(a["zeros"][r0:r1], z)
        assert np.array_equal(a["words"].view(np.uint32)[r0:r1], words)
        w_hat[r0:r1] = wh
    del a

    # decode path as the benchmark launches it: two sibling layers in one call, captured without a warm-up
    # call (nothing on this path allocates or synchronises) and replayed from the graph; every output
    for M in (1, 4, 16):
        bits16, xv = synth.make_activations(M, K, seed=500 + M, dtype="f16")
        x = x_tensor(bits16, "f16")
        ys = [torch.zeros((M, N), dtype=torch.float32, device=x.device) for _ in range(2)]
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                gwq.gwq_linear_multi([P, P], x, outs=ys)
            graph.replay()
            torch.cuda.synchronize()
        y_ref, bound = orc.linear(xv, w_hat)
        for y in ys:
            assert_linear_close(y, y_ref, bound)
        assert gwq.gwq_device_status(P) == 0

    # tensor-core path: bf16 activations with 8 heavy channels, as in the prefill cases; every output
    for M in ((512, 2048) if whole else (2048,)):
        bits16, xv = synth.make_activations(M, K, seed=900 + M, dtype="bf16", heavy_channels=8)
        y = gwq.gwq_linear(P, x_tensor(bits16, "bf16"), out_dtype=torch.float32)
        y_ref, bound = orc.linear(xv, w_hat)
        assert_linear_close(y, y_ref, bound)
        del y, y_ref, bound
    if not whole:
        assert gwq.gwq_device_status(P) == 0
        return
    # M = 8192: all token rows on 256 distinct output rows, and 64 seeded token rows on every output row
    M = 8192
    bits16, xv = synth.make_activations(M, K, seed=900 + M, dtype="bf16", heavy_channels=8)
    y = gwq.gwq_linear(P, x_tensor(bits16, "bf16"), out_dtype=torch.float32)
    rows = distinct_rows(N, seed=layer_index, count=256)
    assert len(set(rows)) >= 256
    y_ref, bound = orc.linear(xv, w_hat[rows])
    assert_linear_close(y[:, rows], y_ref, bound)
    toks = np.sort(np.random.default_rng(70 + layer_index).choice(M, size=64, replace=False))
    y_ref, bound = orc.linear(xv[toks], w_hat)
    assert_linear_close(y[torch.from_numpy(toks).to(y.device)], y_ref, bound)
    assert gwq.gwq_device_status(P) == 0
