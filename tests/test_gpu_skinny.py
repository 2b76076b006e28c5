"""GPU parity of the tcgen05 streaming kernel (fp16 activations, 17 to 32 tokens, reached through gwq_linear_ws)
against the CPU checker: every output, |y_gpu - y_ref| <= 1e-3 * sum_k |x_k w_hat_k| + 1e-5.  The layers are chosen
so that the ranges of steps the CTAs take cut tiles in every way: tiles shared by several CTAs (partial sums added
by the second kernel), CTAs that own whole tiles plus a head and a tail, a ragged last tile, one step per CTA."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, assert_packed_equal, oracle_w_hat, quantize_on_gpu, x_tensor

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


LAYERS = [
    (1024, 1024, 0.01, 4, 128, 120),     # 8 tiles x 8 steps = 64 steps: one step per CTA, every tile shared by 8 CTAs
    (1000, 2176, 0.02, 3, 128, 121),     # ragged last tile, 17 steps per tile
    (1000, 2176, 0.02, 4, 64, 122),      # groups of 64: two accumulators per step
    (640, 1152, 0.005, 3, 64, 123),
    (19072, 256, 0.01, 4, 128, 124),     # 149 tiles x 2 steps on 148 CTAs: whole tiles, heads and tails
    (256, 8192, 0.3, 4, 128, 125),       # outlier-heavy rows (about 2400 per row)
    (96, 128, 0.05, 4, 128, 126),        # a single step
]


@pytest.mark.parametrize("layer", LAYERS)
@pytest.mark.parametrize("M", [17, 24, 32])
def test_streaming_tensor_core_kernel(layer, M):
    P, L, w_hat = _layer(*layer)
    bits16, xv = synth.make_activations(M, P.K, seed=200 + M, dtype="f16")
    x = x_tensor(bits16, "f16")
    assert gwq.load_library().gwq_linear_workspace_bytes(P._h, gwq.GWQ_F16, M) > 0
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x, out_dtype=torch.float32)          # the binding supplies the workspace
    assert gwq.gwq_device_status(P) == 0
    assert_linear_close(y, y_ref, bound)
    y2 = gwq.gwq_linear(P, x, out_dtype=torch.float32)          # fixed summation order: the same bits again
    assert torch.equal(y, y2)
    y16 = gwq.gwq_linear(P, x)
    assert_linear_close(y16, y_ref, bound)


def test_one_hot_activations_read_back_weight_columns():
    P, L, w_hat = _layer(*LAYERS[1])
    cols = [0, 1, 31, 32, 63, 64, 127, 128, 129, P.K - 1] + [int(c) for c in L["col_idx"][:12]]
    bits16, xv = synth.unit_activations(cols, P.K, "f16")
    y_ref, bound = orc.linear(xv, w_hat)
    y = gwq.gwq_linear(P, x_tensor(bits16, "f16"), out_dtype=torch.float32)
    assert_linear_close(y, y_ref, bound)


def test_without_a_workspace_the_older_kernels_serve_the_call():
    P, L, w_hat = _layer(*LAYERS[0])
    bits16, xv = synth.make_activations(20, P.K, seed=77, dtype="f16")
    x = x_tensor(bits16, "f16")
    y = torch.empty((20, P.N), dtype=torch.float32, device=x.device)
    st = gwq.load_library().gwq_linear(P._h, x.data_ptr(), gwq.GWQ_F16, 20, y.data_ptr(), gwq.GWQ_F32, None)
    torch.cuda.synchronize()
    assert st == 0
    y_ref, bound = orc.linear(xv, w_hat)
    assert_linear_close(y, y_ref, bound)


def test_give_up_path_of_the_streaming_kernel():
    # spin limit zero: the first wait that is not satisfied at once gives up; the kernel returns, reports it, and
    # the layer works again afterwards
    P, L, w_hat = _layer(*LAYERS[0])
    bits16, xv = synth.make_activations(20, P.K, seed=78, dtype="f16")
    x = x_tensor(bits16, "f16")
    gwq.gwq_set_wait_limit(P, 0)
    gwq.gwq_linear(P, x, out_dtype=torch.float32)
    assert gwq.gwq_device_status(P) == gwq.GWQ_ERR_TIMEOUT
    gwq.gwq_set_wait_limit(P, -1)
    y = gwq.gwq_linear(P, x, out_dtype=torch.float32)
    assert gwq.gwq_device_status(P) == 0
    y_ref, bound = orc.linear(xv, w_hat)
    assert_linear_close(y, y_ref, bound)
