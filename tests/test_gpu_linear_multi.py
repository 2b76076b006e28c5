"""GPU parity of gwq_linear_multi (several layers that read the same activations, one call) against the
CPU checker, and bit-equality with the per-layer call whose products it must reproduce."""
import ctypes as C

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


# sibling projections: same K, different (ragged) N; the last row block of the first two layers is partial
def _siblings(bits, K=1024, group=128):
    return [_layer(N, K, 0.01, bits, group, 40 + i) for i, N in enumerate((200, 72, 1000))]


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("M", [1, 3, 8, 16, 32])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_fused_siblings_match_checker_and_single_calls(bits, M, dtype):
    sib = _siblings(bits)
    Ps = [s[0] for s in sib]
    bits16, xv = synth.make_activations(M, Ps[0].K, seed=100 + M, dtype=dtype)
    x = x_tensor(bits16, dtype)
    ys = gwq.gwq_linear_multi(Ps, x, out_dtype=torch.float32)
    assert len(ys) == len(Ps)
    for (P, L, w_hat), y in zip(sib, ys):
        assert tuple(y.shape) == (M, P.N)
        y_ref, bound = orc.linear(xv, w_hat)
        assert_linear_close(y, y_ref, bound)
        # the fused launch runs the same arithmetic per row block as the single call
        assert torch.equal(y, gwq.gwq_linear(P, x, out_dtype=torch.float32))
    for P in Ps:
        assert gwq.gwq_device_status(P) == 0


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("M,dtype", [(1, "f16"), (4, "bf16"), (8, "f16"), (12, "f16")])
def test_fused_siblings_with_groups_of_64(bits, M, dtype):
    # one launch up to 8 tokens; beyond, one launch per layer on the tensor-core kernel
    sib = [_layer(N, 2176, 0.01, bits, 64, 50 + i) for i, N in enumerate((200, 72))]
    Ps = [s[0] for s in sib]
    bits16, xv = synth.make_activations(M, 2176, seed=200 + M, dtype=dtype)
    x = x_tensor(bits16, dtype)
    ys = gwq.gwq_linear_multi(Ps, x, out_dtype=torch.float32)
    for (P, L, w_hat), y in zip(sib, ys):
        y_ref, bound = orc.linear(xv, w_hat)
        assert_linear_close(y, y_ref, bound)
        assert torch.equal(y, gwq.gwq_linear(P, x, out_dtype=torch.float32))


def test_tall_siblings_beyond_16_tokens_follow_the_single_call():
    # layers of 10240 rows or more go to the tensor-core kernel from 17 tokens on, in the fused call too
    sib = [_layer(10240, 256, 0.01, 4, 128, 52), _layer(10368, 256, 0.01, 4, 128, 53)]
    for M in (16, 20):
        bits16, xv = synth.make_activations(M, 256, seed=210 + M, dtype="f16")
        x = x_tensor(bits16, "f16")
        ys = gwq.gwq_linear_multi([s[0] for s in sib], x, out_dtype=torch.float32)
        for (P, L, w_hat), y in zip(sib, ys):
            y_ref, bound = orc.linear(xv, w_hat)
            assert_linear_close(y, y_ref, bound)
            assert torch.equal(y, gwq.gwq_linear(P, x, out_dtype=torch.float32))
            assert gwq.gwq_device_status(P) == 0


def test_two_and_four_layers_and_16_bit_outputs():
    sib = _siblings(4) + [_layer(48, 1024, 0.02, 4, 128, 47)]
    bits16, xv = synth.make_activations(4, 1024, seed=7, dtype="f16")
    x = x_tensor(bits16, "f16")
    for n in (1, 2, 4):
        ys = gwq.gwq_linear_multi([s[0] for s in sib[:n]], x)
        for (P, L, w_hat), y in zip(sib[:n], ys):
            assert y.dtype == torch.float16
            y_ref, bound = orc.linear(xv, w_hat)
            assert_linear_close(y, y_ref, bound)


def test_layers_that_cannot_share_a_launch_still_give_every_product():
    # different bit widths, differing group sizes, and M > 32: the call falls back to one launch per layer
    a = _layer(200, 1024, 0.01, 4, 128, 40)
    b = _layer(72, 1024, 0.01, 3, 128, 41)
    c = _layer(96, 1024, 0.01, 4, 64, 48)
    for M, dtype in ((4, "f16"), (40, "bf16")):
        bits16, xv = synth.make_activations(M, 1024, seed=11 + M, dtype=dtype)
        ys = gwq.gwq_linear_multi([a[0], b[0], c[0]], x_tensor(bits16, dtype), out_dtype=torch.float32)
        for (P, L, w_hat), y in zip((a, b, c), ys):
            y_ref, bound = orc.linear(xv, w_hat)
            assert_linear_close(y, y_ref, bound)


def test_argument_errors():
    a = _layer(200, 1024, 0.01, 4, 128, 40)[0]
    other_k = _layer(64, 512, 0.01, 4, 128, 49)[0]
    lib = gwq.load_library()
    bits16, _ = synth.make_activations(2, 1024, seed=1, dtype="f16")
    x = x_tensor(bits16, "f16")
    y = torch.empty((2, 1000), dtype=torch.float16, device=x.device)

    def call(handles, count):
        hs = (C.POINTER(gwq.gwq_packed) * len(handles))(*handles)
        ys = (C.c_void_p * len(handles))(*[y.data_ptr()] * len(handles))
        return lib.gwq_linear_multi(hs, count, x.data_ptr(), gwq.GWQ_F16, 2, ys, gwq.GWQ_F16, None)

    assert call([a._h], 0) == gwq.GWQ_ERR_INVALID_ARG
    assert call([a._h] * (gwq.GWQ_MULTI_MAX + 1), gwq.GWQ_MULTI_MAX + 1) == gwq.GWQ_ERR_INVALID_ARG
    assert call([a._h, other_k._h], 2) == gwq.GWQ_ERR_INVALID_ARG      # differing K
    with pytest.raises(ValueError):
        gwq.gwq_linear_multi([a, other_k], x)
