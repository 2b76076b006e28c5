"""Edge cases of the forward product on the GPU against the CPU checker: the largest K each path
takes, layers smaller than one tile, no outliers at all, rows with more outliers than a warp keeps
in registers, and all of them through both the streaming and the tensor-core path where they apply."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import (assert_linear_close, assert_packed_equal, oracle_w_hat, quantize_on_gpu, x_tensor)

pytestmark = pytest.mark.gpu


def _check(N, K, frac, bits, group, seed, cases):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    P = quantize_on_gpu(W, G, frac, bits, group)
    assert_packed_equal(P, L)
    w_hat = oracle_w_hat(L)
    for M, dtype in cases:
        bits16, xv = synth.make_activations(M, K, seed=seed + M, dtype=dtype)
        y_ref, bound = orc.linear(xv, w_hat)
        y = gwq.gwq_linear(P, x_tensor(bits16, dtype), out_dtype=torch.float32)
        assert_linear_close(y, y_ref, bound)
    assert gwq.gwq_device_status(P) == 0
    P.free()


def test_largest_k_with_16_bit_outlier_columns():
    # K = 65536: the last K the streaming and tensor-core kernels take (outlier columns in 16 bits)
    _check(40, 65536, 0.01, 4, 128, 70, [(1, "f16"), (16, "bf16"), (32, "f16"), (64, "f16")])


def test_wide_layers_at_32_tokens():
    # the tables of a wide layer and the activation tiles of 32 tokens compete for shared memory
    _check(48, 16384, 0.01, 3, 128, 78, [(32, "f16"), (17, "bf16")])
    _check(48, 32768, 0.01, 4, 128, 79, [(32, "bf16")])


def test_k_beyond_16_bit_columns_takes_the_general_kernel():
    _check(16, 131072, 0.005, 3, 128, 71, [(1, "f16"), (40, "bf16")])


@pytest.mark.parametrize("N", [1, 15, 17])
def test_fewer_rows_than_a_tile(N):
    _check(N, 1024, 0.02, 4, 128, 72 + N, [(1, "f16"), (32, "bf16"), (33, "f16"), (300, "bf16")])


@pytest.mark.parametrize("bits", [4, 3])
def test_no_outliers(bits):
    _check(272, 2048, 0.0, bits, 128, 75, [(1, "f16"), (4, "bf16"), (16, "f16"), (128, "bf16")])


def test_rows_with_hundreds_of_outliers():
    # 30 % outliers: ~1200 per row, far more than the 96 entries a warp keeps in registers on the streaming
    # path and than the look-ahead window of the tensor-core path
    _check(64, 4096, 0.3, 3, 128, 76, [(1, "f16"), (8, "bf16"), (16, "f16"), (17, "bf16"), (96, "f16")])


def test_one_group_per_row():
    # K = 128: a single group, seven of the eight warps of a streaming CTA have nothing to do
    _check(96, 128, 0.05, 4, 128, 77, [(1, "f16"), (16, "f16"), (64, "bf16")])


@pytest.mark.parametrize("bits", [4, 3])
def test_groups_of_64_on_the_streaming_path(bits):
    # a warp step of 128 columns holds two groups of 64, kept apart in two halves of the token block: wide rows whose
    # activations are not staged up front (per-warp tiles), a partial last row block, up to 16 tokens (four token blocks
    # beyond 8); with more tokens the tensor-core kernel takes over
    _check(72, 8192, 0.01, bits, 64, 80 + bits, [(1, "f16"), (1, "bf16"), (3, "f16"), (5, "bf16"), (8, "f16"), (8, "bf16"),
                                                 (9, "f16"), (13, "bf16"), (16, "f16"), (16, "bf16"), (17, "f16"), (32, "bf16")])
    _check(40, 28672, 0.005, bits, 64, 84 + bits, [(1, "f16"), (4, "bf16"), (7, "f16"), (16, "bf16")])


def test_groups_of_64_with_an_odd_number_of_groups():
    # K = 192 is not a whole number of 128-column steps: the general kernel
    _check(48, 192, 0.02, 4, 64, 88, [(1, "f16"), (3, "bf16"), (20, "f16")])


def test_tall_layers_take_the_tensor_core_kernel_from_17_tokens():
    # N >= 10240 with groups of 128: 17 to 32 tokens go to the tensor-core kernel's 32-token tile, fewer tokens
    # and shorter layers stay on the streaming kernel; fused siblings follow the same rule
    _check(10368, 512, 0.01, 4, 128, 90, [(16, "f16"), (17, "f16"), (24, "bf16"), (32, "f16"), (32, "bf16")])
    _check(10240, 256, 0.01, 3, 128, 91, [(17, "bf16"), (32, "f16")])


@pytest.mark.parametrize("bits", [4, 3])
def test_two_tiles_per_cta(bits):
    # 8192 rows: more 16-row blocks than one wave of CTAs, at most one wave of 32-row blocks, so up to 8 tokens the
    # streaming kernel runs with two m16 tiles per CTA (staged activations here; a ragged last block: 8200 rows)
    _check(8192, 256, 0.01, bits, 128, 92 + bits, [(1, "f16"), (1, "bf16"), (3, "f16"), (8, "f16"), (8, "bf16"), (16, "f16")])
    _check(8200, 128, 0.02, bits, 128, 96 + bits, [(1, "f16"), (5, "bf16")])


def test_two_tiles_per_cta_with_activation_ring():
    # 8 tokens of 6144 activations do not fit up front: per-warp rings, two tiles per CTA (7168 rows)
    _check(7168, 6144, 0.01, 4, 128, 99, [(8, "f16"), (7, "bf16"), (1, "f16")])
