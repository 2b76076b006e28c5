"""GPU parity of outlier selection + group quantization + packing against the CPU
checker: bit-exact row_ptr / col_idx / val / scales / zero-points / packed words."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_packed_equal, quantize_on_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K,frac,bits,group,seed", [
    (256, 512, 0.01, 4, 128, 0),
    (256, 512, 0.01, 3, 128, 1),
    (192, 1024, 0.02, 4, 64, 2),
    (192, 1024, 0.005, 3, 64, 3),
    (1000, 2176, 0.01, 4, 128, 4),     # N not a multiple of any tile, K = 17 * 128
    (1000, 2176, 0.01, 3, 64, 5),
    (64, 4096, 0.3, 4, 128, 6),        # dense outliers
    (2048, 2048, 0.01, 4, 128, 7),
    (300, 1056, 0.01, 4, 16, 8),       # the paper's own group size (Section 3.2: beta = 16); K = 33 * 32
    (300, 1056, 0.02, 3, 16, 9),
    (192, 1024, 0.01, 4, 32, 10),
    (192, 1024, 0.3, 3, 32, 11),
])
def test_encode_matches_checker(N, K, frac, bits, group, seed):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    P = quantize_on_gpu(W, G, frac, bits, group)
    assert P.nnz == L["row_ptr"][-1]
    assert_packed_equal(P, L)
    P.free()


@pytest.mark.parametrize("levels,frac", [(64, 0.01), (7, 0.2), (2, 0.5), (1, 0.37)])
def test_tie_heavy_gradient(levels, frac):
    N, K = 300, 1024
    W, _ = synth.make_weight_and_grad(N, K, 11)
    G = synth.make_tie_heavy_grad(N, K, seed=12, levels=levels)
    L = orc.quantize_layer(W, G, frac, 4, 128)
    P = quantize_on_gpu(W, G, frac, 4, 128)
    assert_packed_equal(P, L)
    P.free()


@pytest.mark.parametrize("frac", [0.0, 1.0, 1e-9, 1.0 / (128 * 256)])
def test_fraction_edges(frac):
    N, K = 128, 256
    W, G = synth.make_weight_and_grad(N, K, 13)
    L = orc.quantize_layer(W, G, frac, 4, 64)
    P = quantize_on_gpu(W, G, frac, 4, 64)
    assert_packed_equal(P, L)
    P.free()


def test_special_gradient_values_and_signed_zero():
    N, K = 64, 256
    W, G = synth.make_weight_and_grad(N, K, 14)
    rng = np.random.default_rng(14)
    flat = G.reshape(-1)
    idx = rng.choice(N * K, size=600, replace=False)
    flat[idx[:100]] = np.inf
    flat[idx[100:200]] = -np.inf
    flat[idx[200:300]] = np.nan
    flat[idx[300:450]] = 0.0
    flat[idx[450:600]] = -0.0
    for frac in (0.005, 0.015, 0.99):
        L = orc.quantize_layer(W, G, frac, 3, 64)
        P = quantize_on_gpu(W, G, frac, 3, 64)
        assert_packed_equal(P, L)
        P.free()


def test_structured_rows_and_groups():
    # rows with no outliers, a row that is all outliers, groups that are all outliers,
    # all-positive / all-negative / constant / zero groups
    N, K, group = 32, 512, 128
    rng = np.random.default_rng(15)
    W = rng.normal(0, 0.02, size=(N, K)).astype(np.float16)
    W[3, :128] = np.abs(W[3, :128])
    W[4, 128:256] = -np.abs(W[4, 128:256])
    W[5, :128] = np.float16(0.0371)
    W[6, 256:384] = 0
    W[7, :] = 0
    G = rng.normal(0, 1e-3, size=(N, K)).astype(np.float32)
    G[9, :] = 50.0            # whole row outliers
    G[11, 128:256] = 60.0     # one whole group
    G[3, 5] = 70.0
    frac = (K + 128 + 1 + 40) / (N * K)
    for bits in (3, 4):
        L = orc.quantize_layer(W, G, frac, bits, group)
        P = quantize_on_gpu(W, G, frac, bits, group)
        assert_packed_equal(P, L)
        P.free()


def test_nonfinite_weight_is_an_error_and_bad_arguments():
    N, K = 32, 256
    W, G = synth.make_weight_and_grad(N, K, 16)
    W[5, 17] = np.inf
    Wd, Gd = to_dev(W), to_dev(G)
    S = gwq.gwq_select_outliers(Wd, Gd, 0.01)
    with pytest.raises(gwq.GwqError) as e:
        gwq.gwq_pack(Wd, S, 4, 128)
    assert e.value.status == 4
    S.free()
    with pytest.raises(gwq.GwqError) as e:
        gwq.gwq_select_outliers(Wd, Gd, 1.5)
    assert e.value.status == 1
    S = gwq.gwq_select_outliers(Wd, Gd, 0.01)
    for bits, group, want in ((5, 128, 2), (4, 8, 2), (4, 96, 2)):
        with pytest.raises(gwq.GwqError) as e:
            gwq.gwq_pack(Wd, S, bits, group)
        assert e.value.status == want
    S.free()
    torch.cuda.synchronize()


def test_rows_of_an_outlier_matrix_pack_like_the_rows_of_the_whole():
    # the selection ranks the whole matrix; a rank that owns rows [128, 300) cuts them out and packs them alone
    N, K, r0, r1 = 300, 512, 128, 300
    W, G = synth.make_weight_and_grad(N, K, 55)
    L = orc.quantize_layer(W, G, 0.02, 3, 64)
    Wd, Gd = torch.from_numpy(W).to("cuda:0"), torch.from_numpy(G).to("cuda:0")
    S = gwq.gwq_select_outliers(Wd, Gd, 0.02)
    S_loc = gwq.gwq_outliers_rows(S, r0, r1)
    rp, ci, va = (t.cpu().numpy() for t in S_loc.arrays())
    lo, hi = int(L["row_ptr"][r0]), int(L["row_ptr"][r1])
    assert np.array_equal(rp, L["row_ptr"][r0:r1 + 1] - lo)
    assert np.array_equal(ci, L["col_idx"][lo:hi]) and np.array_equal(va.view(np.uint16), L["val"][lo:hi])
    P = gwq.gwq_pack(Wd[r0:r1].contiguous(), S_loc, 3, 64)
    a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
    assert np.array_equal(a["words"].view(np.uint32), L["words"][r0:r1])
    assert np.array_equal(a["scales"].view(np.uint16), L["scales"].view(np.uint16)[r0:r1])
    assert np.array_equal(a["zeros"], L["zeros"][r0:r1])
    with pytest.raises(gwq.GwqError):
        gwq.gwq_outliers_rows(S, 10, 10)
    P.free()
    S.free()
