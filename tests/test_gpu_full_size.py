"""Parity at the benchmark's full layer sizes, in the launch configuration the benchmark times
(sibling layers through gwq_linear_multi, replayed from a CUDA graph; the tensor-core path with
bf16 activations and heavy channels).  The CPU checker selects the outliers of the whole matrix
(the selection is global) and then encodes, reconstructs and multiplies SAMPLED rows one by one;
the CSR is compared in full, everything else on the sampled rows."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, to_dev, x_tensor

pytestmark = pytest.mark.gpu

FRAC, GROUP = 0.01, 128


def _sample_rows(N, seed):
    rng = np.random.default_rng(seed)
    rows = {0, 1, 7, 8, 15, 16, N - 17, N - 16, N - 2, N - 1}
    rows.update(int(r) for r in rng.integers(0, N, size=14))
    return sorted(rows)


def _checker_rows(W, row_ptr, col_idx, val, rows, bits):
    """Encode and reconstruct the sampled rows with the checker, given the whole matrix's outliers."""
    K = W.shape[1]
    counts = [int(row_ptr[n + 1] - row_ptr[n]) for n in rows]
    sub_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    sub_col = np.concatenate([col_idx[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.int32)
    sub_val = np.concatenate([val[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.uint16)
    mask = orc.outlier_mask(sub_ptr, sub_col, len(rows), K)
    Ws = np.ascontiguousarray(W[rows])
    s, z = orc.group_stats(Ws, mask, bits, GROUP)
    q = orc.quantize_codes(Ws, mask, s, z, bits, GROUP)
    words = orc.pack_codes(q, bits)
    w_hat = orc.dequantize(q, s, z, GROUP, sub_ptr, sub_col, sub_val)
    return s, z, words, w_hat


@pytest.mark.parametrize("N,K,bits,layer_index", [(11008, 4096, 4, 4), (4096, 11008, 3, 6)])
def test_full_size_layer(N, K, bits, layer_index):
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(1, layer_index))
    row_ptr, col_idx, val = orc.select_outliers(W, G, FRAC)
    Wd, Gd = to_dev(W), to_dev(G)
    S = gwq.gwq_select_outliers(Wd, Gd, FRAC)
    P = gwq.gwq_pack(Wd, S, bits, GROUP)
    del Gd
    a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
    # the outlier set of the whole matrix, bit for bit
    assert np.array_equal(a["row_ptr"], row_ptr)
    assert np.array_equal(a["col_idx"], col_idx)
    assert np.array_equal(a["val"].view(np.uint16), val)
    # codes, scales and zero-points of the sampled rows, bit for bit
    rows = _sample_rows(N, seed=layer_index)
    s, z, words, w_hat = _checker_rows(W, row_ptr, col_idx, val, rows, bits)
    assert np.array_equal(a["scales"].view(np.uint16)[rows], s.view(np.uint16))
    assert np.array_equal(a["zeros"][rows], z)
    assert np.array_equal(a["words"].view(np.uint32)[rows], words)

    # decode path as the benchmark launches it: two sibling layers in one call, replayed from a graph
    for M in (1, 4, 16):
        bits16, xv = synth.make_activations(M, K, seed=500 + M, dtype="f16")
        x = x_tensor(bits16, "f16")
        ys = [torch.zeros((M, N), dtype=torch.float32, device=x.device) for _ in range(2)]
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            gwq.gwq_linear_multi([P, P], x, outs=ys)      # also sizes the scratch outside the capture
            torch.cuda.synchronize()
            for y in ys:
                y.zero_()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                gwq.gwq_linear_multi([P, P], x, outs=ys)
            graph.replay()
            torch.cuda.synchronize()
        y_ref, bound = orc.linear(xv, w_hat)
        for y in ys:
            assert_linear_close(y[:, rows], y_ref, bound)
        assert gwq.gwq_device_status(P) == 0

    # tensor-core path: bf16 activations with 8 heavy channels, as in the prefill cases
    for M in (512, 2048, 8192):
        bits16, xv = synth.make_activations(M, K, seed=900 + M, dtype="bf16", heavy_channels=8)
        y = gwq.gwq_linear(P, x_tensor(bits16, "bf16"), out_dtype=torch.float32)
        y_ref, bound = orc.linear(xv, w_hat)
        assert_linear_close(y[:, rows], y_ref, bound)
        del y
    assert gwq.gwq_device_status(P) == 0
