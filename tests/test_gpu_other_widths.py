"""GPU parity for 2- and 8-bit codes (Section 3.2, Eqs. "s", "z", "q", "w" with b = 2 and b = 8; the paper's
experiments use 3 and 4 bits): bit-exact encoding, and the product on every kernel that serves these widths,
|y_gpu - y_ref| <= 1e-3 * sum_k |x_k w_hat_k| + 1e-5 per output."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import (assert_linear_close, assert_packed_equal, oracle_w_hat, quantize_on_gpu, to_dev, x_tensor)

pytestmark = pytest.mark.gpu

_cache = {}


def _layer(N, K, frac, bits, group, seed):
    key = (N, K, frac, bits, group, seed)
    if key not in _cache:
        W, G = synth.make_weight_and_grad(N, K, seed)
        L = orc.quantize_layer(W, G, frac, bits, group)
        P = quantize_on_gpu(W, G, frac, bits, group)
        assert_packed_equal(P, L)
        _cache[key] = (P, L, oracle_w_hat(L))
    return _cache[key]


@pytest.mark.parametrize("N,K,frac,bits,group,seed", [
    (256, 512, 0.01, 8, 128, 70),
    (256, 512, 0.01, 2, 128, 71),
    (1000, 2176, 0.02, 8, 64, 72),     # N not a multiple of any tile, K = 17 * 128
    (1000, 2176, 0.005, 2, 64, 73),
    (64, 4096, 0.3, 2, 128, 74),       # dense outliers
    (300, 1056, 0.01, 8, 16, 75),      # the group size Section 3.2 names; K = 33 * 32
    (300, 1056, 0.02, 2, 16, 76),
    (192, 1024, 0.01, 8, 32, 77),
    (192, 1024, 0.0, 2, 32, 78),
    (128, 256, 1.0, 8, 128, 79),       # every entry an outlier: s = 1, z = 0, all codes 0
])
def test_encode_matches_checker(N, K, frac, bits, group, seed):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    P = quantize_on_gpu(W, G, frac, bits, group)
    assert P.nnz == L["row_ptr"][-1]
    assert_packed_equal(P, L)
    assert int(L["codes"].max()) <= 2 ** bits - 1
    if frac < 1.0:
        assert int(L["codes"].max()) == 2 ** bits - 1    # the top level is in use: the range check means something
    P.free()


def test_all_code_values_survive_the_packed_words():
    # weights on an exact grid that uses every one of the 256 levels in every group: codes = grid index
    N, K, group = 48, 512, 256 // 2
    rng = np.random.default_rng(80)
    idx = np.stack([rng.permutation(256)[:group] for _ in range(N * (K // group))]).reshape(N, K)
    idx[:, 0::group] = 0
    idx[:, 1::group] = 255        # both extremes in every group
    W = ((idx - 128) * 2.0 ** -9).astype(np.float16)
    G = np.zeros((N, K), dtype=np.float32)
    L = orc.quantize_layer(W, G, 0.0, 8, group)
    assert np.array_equal(L["codes"], idx.astype(np.uint8))
    P = quantize_on_gpu(W, G, 0.0, 8, group)
    assert_packed_equal(P, L)
    x16, xv = synth.unit_activations([0, 1, 2, 3, 127, 128, 255, 511], K, "f16")
    y = gwq.gwq_linear(P, x_tensor(x16, "f16"), out_dtype=torch.float32)
    assert np.array_equal(y.double().cpu().numpy(), xv @ W.astype(np.float64).T)   # zero error on the grid
    P.free()


LAYERS = [
    (1024, 1024, 0.01, 8, 128, 81),
    (1024, 1024, 0.01, 2, 128, 82),
    (1000, 2176, 0.02, 8, 64, 83),     # ragged last row block, groups of 64
    (1000, 2176, 0.005, 2, 64, 84),
    (528, 4096, 0.01, 2, 128, 85),
]


@pytest.mark.parametrize("layer", LAYERS)
@pytest.mark.parametrize("M", [1, 2, 4, 7, 8, 16, 17, 32])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_decode_sizes(layer, M, dtype):
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=M, dtype=dtype)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)
    y16 = gwq.gwq_linear(P, x_tensor(bits16, dtype))
    assert_linear_close(y16, y_ref, bound, extra_rel=2.0 ** -8 if dtype == "bf16" else 0.0)
    again = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert torch.equal(y, again)


@pytest.mark.parametrize("layer", LAYERS[:4])
def test_unit_activations_read_back_weight_columns(layer):
    P, L, w_hat = _layer(*layer)
    cols = [0, 1, 2, 3, 15, 16, 31, 32, 63, 64, 127, 128, P.K - 1]
    cols += [int(c) for c in L["col_idx"][:7]]          # some outlier columns
    bits16, xv = synth.unit_activations(cols, P.K, "f16")
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


@pytest.mark.parametrize("layer", LAYERS[:4])
@pytest.mark.parametrize("M,dtype", [(33, "f16"), (64, "bf16"), (200, "bf16"), (257, "bf16"), (700, "f16")])
def test_tensor_core_paths(layer, M, dtype):
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=100 + M, dtype=dtype, heavy_channels=8)
    y_ref, bound = orc.linear(xv, w_hat)
    x = x_tensor(bits16, dtype)
    y = gwq.gwq_linear(P, x, out_dtype=torch.float32)     # the binding's workspace: the two-phase path
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)
    # the fused kernel: a workspace without room for the expanded weights (none at all for fp16 activations)
    lib = gwq.load_library()
    xd = gwq.GWQ_F16 if dtype == "f16" else gwq.GWQ_BF16
    ws_bytes = ((M * P.K * 2 + 255) // 256 + (M * 4 + 255) // 256) * 256 if dtype == "bf16" else 0
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=x.device)
    yf = torch.zeros((M, P.N), dtype=torch.float32, device=x.device)
    st = lib.gwq_linear_ws(P._h, x.data_ptr(), xd, M, yf.data_ptr(), gwq.GWQ_F32, ws.data_ptr() if ws_bytes else None,
                           ws_bytes, torch.cuda.current_stream().cuda_stream)
    assert st == 0
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(yf, y_ref, bound)


@pytest.mark.parametrize("N,K,M,bits,dtype", [(600, 320, 2300, 8, "f16"), (2700, 192, 2100, 2, "bf16"),
                                              (1500, 4096, 700, 8, "bf16")])
def test_two_phase_path_ragged_tiles(N, K, M, bits, dtype):
    # K not a multiple of 128 takes the run-by-run expansion, the others the block expansion
    P, L, w_hat = _layer(N, K, 0.01, bits, 64, 86)
    bits16, xv = synth.make_activations(M, P.K, seed=M, dtype=dtype, heavy_channels=4)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)


SMALL_GROUP_LAYERS = [
    (520, 1024, 0.01, 8, 16, 87),      # the group size Section 3.2 names, ragged last tile
    (520, 1024, 0.02, 2, 16, 88),
    (384, 2048, 0.01, 8, 32, 89),
    (384, 2048, 0.005, 2, 32, 90),
    (200, 1056, 0.01, 8, 16, 91),      # K = 33 * 32: the general kernel
    (200, 1056, 0.01, 2, 32, 92),
]


@pytest.mark.parametrize("layer", SMALL_GROUP_LAYERS)
@pytest.mark.parametrize("M,dtype", [(1, "f16"), (1, "bf16"), (4, "bf16"), (8, "f16"), (32, "bf16"), (40, "f16"),
                                     (300, "bf16")])
def test_small_groups(layer, M, dtype):
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=160 + M, dtype=dtype, heavy_channels=8 if M > 32 else 0)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)


def test_sibling_layers_in_one_launch():
    layers = [_layer(1024, 1024, 0.01, 8, 128, 81), _layer(512, 1024, 0.01, 8, 128, 93)]
    for M in (1, 8):
        bits16, xv = synth.make_activations(M, 1024, seed=M, dtype="f16")
        x = x_tensor(bits16, "f16")
        ys = gwq.gwq_linear_multi([l[0] for l in layers], x, out_dtype=torch.float32)
        for (P, L, w_hat), y in zip(layers, ys):
            assert torch.equal(y, gwq.gwq_linear(P, x, out_dtype=torch.float32))
            y_ref, bound = orc.linear(xv, w_hat)
            assert_linear_close(y, y_ref, bound)


@pytest.mark.parametrize("N,K,frac,bits,group,seed", [(100, 2176, 0.02, 8, 64, 94), (64, 1024, 0.01, 2, 128, 95),
                                                      (100, 1056, 0.01, 2, 16, 96)])
def test_quality_matches_checker(N, K, frac, bits, group, seed):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    P = quantize_on_gpu(W, G, frac, bits, group)
    w_hat = oracle_w_hat(L)
    sq_ref, fo_ref = orc.quality(W, G, w_hat)
    sq, fo = gwq.gwq_quality(to_dev(W), to_dev(G), P)
    d = W.astype(np.float64) - w_hat
    eps = 2.0 ** -52
    assert abs(sq - sq_ref) <= 1024 * eps * float(np.sum(d * d)) + 1e-300
    assert abs(fo - fo_ref) <= 1024 * eps * float(np.sum(np.abs(G.astype(np.float64) * d))) + 1e-300
    P.free()


def test_other_widths_are_refused():
    W, G = synth.make_weight_and_grad(32, 256, 97)
    Wd, Gd = to_dev(W), to_dev(G)
    for bits in (1, 5, 6, 7, 16):
        S = gwq.gwq_select_outliers(Wd, Gd, 0.01)
        with pytest.raises(gwq.GwqError):
            gwq.gwq_pack(Wd, S, bits, 128)
