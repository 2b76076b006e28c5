"""GPU parity of y = x (deq(Wq) + S)^T against the CPU checker:
|y_gpu - y_ref| <= 1e-3 * sum_k |x_k w_hat_k| + 1e-5 per output."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import (assert_linear_close, assert_packed_equal, oracle_w_hat, quantize_on_gpu, x_tensor)

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


DECODE_LAYERS = [
    (1024, 1024, 0.01, 4, 128, 20),
    (1024, 1024, 0.01, 3, 128, 21),
    (1000, 2176, 0.02, 4, 64, 22),
    (1000, 2176, 0.005, 3, 64, 23),
    (528, 4096, 0.01, 4, 128, 24),
]


@pytest.mark.parametrize("layer", DECODE_LAYERS)
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


@pytest.mark.parametrize("layer", DECODE_LAYERS[:4])
def test_unit_activations_read_back_weight_columns(layer):
    P, L, w_hat = _layer(*layer)
    cols = [0, 1, 31, 32, 63, 64, 127, 128, P.K - 1]
    cols += [int(c) for c in L["col_idx"][:7]]          # some outlier columns
    bits16, xv = synth.unit_activations(cols, P.K, "f16")
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


@pytest.mark.parametrize("M", [33, 63, 64, 100, 128, 300])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_larger_batches(M, dtype):
    P, L, w_hat = _layer(*DECODE_LAYERS[0])
    bits16, xv = synth.make_activations(M, P.K, seed=M, dtype=dtype, heavy_channels=8)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


PREFILL_LAYERS = [
    (1024, 1024, 0.01, 4, 128, 20),
    (1024, 1024, 0.01, 3, 128, 21),
    (1000, 2176, 0.02, 4, 64, 22),      # N not a multiple of the 128-row tile, group 64
    (1000, 2176, 0.005, 3, 64, 23),
    (256, 4096, 0.3, 4, 128, 25),       # outlier-heavy rows
]


@pytest.mark.parametrize("layer", PREFILL_LAYERS)
@pytest.mark.parametrize("M,dtype", [(33, "f16"), (64, "bf16"), (65, "f16"), (200, "bf16"), (256, "f16"),
                                     (257, "bf16"), (700, "f16")])
def test_tensor_core_path(layer, M, dtype):
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
    # room for the fp16 copy of bf16 activations and the token scales, none for the weights
    ws_bytes = ((M * P.K * 2 + 255) // 256 + (M * 4 + 255) // 256) * 256 if dtype == "bf16" else 0
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=x.device)
    yf = torch.zeros((M, P.N), dtype=torch.float32, device=x.device)
    st = lib.gwq_linear_ws(P._h, x.data_ptr(), xd, M, yf.data_ptr(), gwq.GWQ_F32, ws.data_ptr() if ws_bytes else None,
                           ws_bytes, torch.cuda.current_stream().cuda_stream)
    assert st == 0
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(yf, y_ref, bound)
    y16 = gwq.gwq_linear(P, x_tensor(bits16, dtype))
    assert_linear_close(y16, y_ref, bound, extra_rel=2.0 ** -8 if dtype == "bf16" else 0.0)


@pytest.mark.parametrize("bits,dtype", [(4, "f16"), (3, "bf16")])
@pytest.mark.parametrize("expanded", [False, True])
def test_persistent_ctas_with_several_tiles_each(bits, dtype, expanded):
    # N = 4096, K = 256, M = 4096: 32 x 16 = 512 tiles of 128 rows x 256 tokens on at most 148 persistent CTAs, so
    # every CTA computes three or four tiles: both accumulators are reused (the wait for the epilogue to drain
    # them), the stage ring wraps across tiles, and every output is checked.  Once with the weights expanded
    # beforehand (workspace with room for them), once through the fused kernel (workspace for the fp16 copy of
    # bf16 activations only, none for fp16 activations).
    N, K, M = 4096, 256, 4096
    W, G = synth.make_weight_and_grad(N, K, 26)
    L = orc.quantize_layer(W, G, 0.01, bits, 128)
    P = quantize_on_gpu(W, G, 0.01, bits, 128)
    assert_packed_equal(P, L)
    w_hat = oracle_w_hat(L)
    bits16, xv = synth.make_activations(M, K, seed=126, dtype=dtype, heavy_channels=8)
    y_ref, bound = orc.linear(xv, w_hat)
    x = x_tensor(bits16, dtype)
    lib = gwq.load_library()
    xd = gwq.GWQ_F16 if dtype == "f16" else gwq.GWQ_BF16
    full = int(lib.gwq_linear_workspace_bytes(P._h, xd, M))
    assert full >= N * K * 2                                     # 4096 tokens: the expansion is asked for
    ws_bytes = full if expanded else full - N * K * 2            # without room for the weights: the fused kernel
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=x.device)
    y = torch.zeros((M, N), dtype=torch.float32, device=x.device)
    st = lib.gwq_linear_ws(P._h, x.data_ptr(), xd, M, y.data_ptr(), gwq.GWQ_F32, ws.data_ptr() if ws_bytes else None,
                           ws_bytes, torch.cuda.current_stream().cuda_stream)
    assert st == 0
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)
    P.free()


@pytest.mark.parametrize("N,K,M,bits,dtype", [(600, 320, 2300, 4, "f16"), (2700, 192, 2100, 3, "bf16"), (96, 64, 2048, 4, "f16"),
                                                   (600, 384, 2300, 4, "bf16"), (300, 256, 2100, 3, "f16"), (9472, 128, 512, 4, "f16"),
                                                   (1500, 4096, 700, 4, "bf16"), (2560, 6144, 520, 3, "f16"), (520, 4096, 300, 4, "f16")])
def test_two_phase_path_ragged_tiles_and_bands(N, K, M, bits, dtype):
    # the contraction on CTA pairs (tiles of 256 rows x 256 tokens, reached with many tokens and room for the
    # expanded weights): ragged last tiles in both directions, 11 weight tiles (a full band of 8 and a narrower one),
    # a layer smaller than one tile; K a multiple of 128 (the weights expanded block by block) and not; token tiles of
    # 128 (the small layers) and of 256 (9472 rows x 512 tokens: one tile per pair of SMs); left-over tiles cut into
    # K-slices whose partial sums a second kernel adds (the last three: 18, 30 and 6 tiles on 74 pairs); every output
    W, G = synth.make_weight_and_grad(N, K, 27)
    L = orc.quantize_layer(W, G, 0.01, bits, 64)
    P = quantize_on_gpu(W, G, 0.01, bits, 64)
    assert_packed_equal(P, L)
    w_hat = oracle_w_hat(L)
    bits16, xv = synth.make_activations(M, K, seed=127, dtype=dtype, heavy_channels=4)
    y_ref, bound = orc.linear(xv, w_hat)
    x = x_tensor(bits16, dtype)
    lib = gwq.load_library()
    xd = gwq.GWQ_F16 if dtype == "f16" else gwq.GWQ_BF16
    assert int(lib.gwq_linear_workspace_bytes(P._h, xd, M)) >= N * K * 2
    y = gwq.gwq_linear(P, x, out_dtype=torch.float32)          # the binding supplies the workspace
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)
    # 2-byte outputs: rows of y that start on 16-byte boundaries leave through TMA stores, the others (N = 300, 2700
    # with 2 bytes per element) through plain stores
    y16 = gwq.gwq_linear(P, x)
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y16, y_ref, bound, extra_rel=2.0 ** -8 if dtype == "bf16" else 0.0)
    P.free()


def test_single_layer_config_seed_0():
    # the single-layer configuration as written: 4096 x 4096, seed 0, 4 bits, groups of 128, 1 % outliers, fp16
    # activations, one token; encoding bit for bit and every output
    N = K = 4096
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(0, 0))
    L = orc.quantize_layer(W, G, 0.01, 4, 128)
    assert int(L["row_ptr"][-1]) == 167773
    P = quantize_on_gpu(W, G, 0.01, 4, 128)
    assert_packed_equal(P, L)
    w_hat = oracle_w_hat(L)
    bits16, xv = synth.make_activations(1, K, seed=synth.layer_seed(0, 0), dtype="f16")
    y_ref, bound = orc.linear(xv, w_hat)
    for out_dtype in (torch.float32, torch.float16):
        y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=out_dtype)
        assert_linear_close(y, y_ref, bound)
    P.free()


def test_tensor_core_path_reads_back_columns_exactly_in_fp16():
    # one-hot fp16 activations: y[m] is column c of the reconstructed weight, outliers included
    P, L, w_hat = _layer(*PREFILL_LAYERS[0])
    cols = list(range(0, 1024, 17)) + [int(c) for c in L["col_idx"][:20]]
    bits16, xv = synth.unit_activations(cols, P.K, "f16")
    assert len(cols) > 64
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


@pytest.mark.parametrize("layer", [(200, 1056, 0.01, 4, 16, 30), (200, 1056, 0.02, 3, 16, 31), (96, 1024, 0.01, 4, 32, 32)])
@pytest.mark.parametrize("M,dtype", [(1, "f16"), (5, "bf16"), (16, "f16"), (40, "bf16"), (70, "f16")])
def test_small_groups(layer, M, dtype):
    # groups of 16 (the paper's own value, Section 3.2) and 32: the general kernel serves every M
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=60 + M, dtype=dtype)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


SMALL_GROUP_LAYERS = [
    (520, 1024, 0.01, 4, 16, 33),      # the paper's own group size (Section 3.2), ragged last tile
    (520, 1024, 0.02, 3, 16, 34),
    (384, 2048, 0.01, 4, 32, 35),
    (384, 2048, 0.005, 3, 32, 36),
]


@pytest.mark.parametrize("layer", SMALL_GROUP_LAYERS)
@pytest.mark.parametrize("M,dtype", [(1, "f16"), (1, "bf16"), (2, "f16"), (4, "bf16"), (8, "f16"), (17, "f16"), (32, "bf16"),
                                     (33, "f16"), (300, "bf16"), (2100, "f16")])
def test_small_groups_on_the_fast_paths(layer, M, dtype):
    # K a multiple of 128: groups of 16 and 32 run on the tensor cores (one scale per 16 or 32 columns inside the
    # 64-column k-block; the weights expanded beforehand for many tokens) and, for one token, on the streaming kernel
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=160 + M, dtype=dtype, heavy_channels=8 if M > 32 else 0)
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)


@pytest.mark.parametrize("layer", [DECODE_LAYERS[0], DECODE_LAYERS[3]])
@pytest.mark.parametrize("M", [1, 8, 16, 32, 200])
def test_repeated_calls_give_the_same_bits(layer, M):
    # fixed summation order everywhere (no floating-point atomics): the same call twice is bit-identical
    P, L, w_hat = _layer(*layer)
    bits16, _ = synth.make_activations(M, P.K, seed=300 + M, dtype="f16", heavy_channels=8 if M > 32 else 0)
    x = x_tensor(bits16, "f16")
    y1 = gwq.gwq_linear(P, x, out_dtype=torch.float32).clone()
    y2 = gwq.gwq_linear(P, x, out_dtype=torch.float32)
    assert torch.equal(y1, y2)


def test_all_outliers_is_the_dense_product():
    N, K = 128, 512
    W, G = synth.make_weight_and_grad(N, K, 30)
    P = quantize_on_gpu(W, G, 1.0, 4, 128)
    bits16, xv = synth.make_activations(3, K, seed=30)
    y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=torch.float32)
    y_ref = xv @ W.astype(np.float64).T
    bound = np.abs(xv) @ np.abs(W.astype(np.float64)).T
    assert_linear_close(y, y_ref, bound)
    P.free()


def test_host_buffer_entry_point_and_argument_errors():
    P, L, w_hat = _layer(*DECODE_LAYERS[0])
    bits16, xv = synth.make_activations(4, P.K, seed=5)
    y_ref, bound = orc.linear(xv, w_hat)
    xh = torch.from_numpy(bits16.view(np.int16).copy()).view(torch.float16).pin_memory()
    yh = torch.empty((4, P.N), dtype=torch.float32).pin_memory()
    gwq.gwq_linear_host(P, xh, yh)
    assert_linear_close(yh, y_ref, bound)
    # the asynchronous variant: two calls in a row on the same layer, results valid after one synchronisation
    ya, yb = (torch.zeros((4, P.N), dtype=torch.float32).pin_memory() for _ in range(2))
    gwq.gwq_linear_host_async(P, xh, ya)
    gwq.gwq_linear_host_async(P, xh, yb)
    torch.cuda.synchronize()
    assert_linear_close(ya, y_ref, bound)
    assert torch.equal(ya, yb)
    with pytest.raises(gwq.GwqError) as e:
        gwq.gwq_linear(P, torch.zeros((2, P.K), dtype=torch.float32, device="cuda:0"))
    assert e.value.status == 2
