"""Seeded synthetic inputs for the GWQ linear layer.

This module only *draws numbers*: it contains none of the method's arithmetic
(no ranking, no scales, no codes, no products).  It serves the CUDA path, the
tests and the CPU checker alike, so that all of them see the same tensors.

The tensors stand in for LLM linear layers and a calibration gradient
(Llama-7B / 70B shaped projections):

* ``W``: fp16, normal(0, 0.02) with 0.1 % of the entries multiplied by 20
  (heavy-tailed weights).
* ``G``: fp32, Laplace(0, 1) scaled per input column by a lognormal(0, 1)
  factor, so that large gradients line up along channels, which is the
  structure the paper reports for gradient-located outliers (Section 3.1).
* ``x``: normal(0, 1) rounded to fp16 or bf16; the prefill variant multiplies
  8 seeded channels by 50.

Draw order is fixed: W, heavy positions, Laplace field, column scales, then
(separately seeded) x.
"""
from __future__ import annotations

import numpy as np

# Llama-shaped linear layers as (N = out features, K = in features).
LLAMA7B_LAYER_SET = (
    ("q_proj", 4096, 4096),
    ("k_proj", 4096, 4096),
    ("v_proj", 4096, 4096),
    ("o_proj", 4096, 4096),
    ("gate_proj", 11008, 4096),
    ("up_proj", 11008, 4096),
    ("down_proj", 4096, 11008),
)
LLAMA70B_SHAPES = ((8192, 8192), (28672, 8192), (8192, 28672))


def layer_seed(config_index: int, layer_index: int) -> int:
    """Seed convention: config 0 uses seed 0; others 1000*config + layer."""
    return 0 if config_index == 0 else 1000 * config_index + layer_index


def make_weight_and_grad(N: int, K: int, seed: int):
    """Return (W fp16 [N,K], G fp32 [N,K]) for one layer."""
    rng = np.random.default_rng(seed)
    numel = N * K
    W = rng.normal(0.0, 0.02, size=(N, K))
    n_heavy = int(round(0.001 * numel))
    if n_heavy > 0:
        pos = rng.choice(numel, size=n_heavy, replace=False)
        W.reshape(-1)[pos] *= 20.0
    W16 = W.astype(np.float16)
    del W
    L = rng.laplace(0.0, 1.0, size=(N, K))
    c = np.exp(rng.normal(0.0, 1.0, size=(K,)))
    G = (L * c[None, :]).astype(np.float32)
    return W16, G


def make_tie_heavy_grad(N: int, K: int, seed: int, levels: int = 64):
    """Gradient with only ``levels`` distinct magnitudes, random signs, so that
    many entries share the threshold magnitude of any top-k cut."""
    rng = np.random.default_rng(seed)
    table = np.abs(rng.normal(0.0, 1.0, size=(levels,))).astype(np.float32)
    idx = rng.integers(0, levels, size=(N, K))
    sign = rng.integers(0, 2, size=(N, K)).astype(np.float32) * 2.0 - 1.0
    return (table[idx] * sign).astype(np.float32)


def round_to_bf16_bits(a32: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns the 16-bit
    patterns as uint16.  Pure format conversion for the input tensors."""
    u = np.ascontiguousarray(a32, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_activations(M: int, K: int, seed: int, dtype: str = "f16", heavy_channels: int = 0):
    """Return (bits uint16 [M,K], values float64 [M,K]).

    ``bits`` are the fp16 or bf16 patterns handed to the GPU; ``values`` are
    the exact real numbers those patterns denote.
    """
    rng = np.random.default_rng(seed + 7_000_000)
    x = rng.normal(0.0, 1.0, size=(M, K))
    if heavy_channels > 0:
        ch = rng.choice(K, size=heavy_channels, replace=False)
        x[:, ch] *= 50.0
    if dtype == "f16":
        h = x.astype(np.float16)
        return h.view(np.uint16).copy(), h.astype(np.float64)
    if dtype == "bf16":
        bits = round_to_bf16_bits(x.astype(np.float32))
        return bits, bf16_bits_to_f32(bits).astype(np.float64)
    raise ValueError(f"unknown activation dtype {dtype!r}")


def unit_activations(cols, K: int, dtype: str = "f16"):
    """One-hot rows x[m] = e_{cols[m]}: the product then reads back single
    columns of the reconstructed weight."""
    M = len(cols)
    one = np.uint16(0x3C00) if dtype == "f16" else np.uint16(0x3F80)
    bits = np.zeros((M, K), dtype=np.uint16)
    vals = np.zeros((M, K), dtype=np.float64)
    for m, c in enumerate(cols):
        bits[m, c] = one
        vals[m, c] = 1.0
    return bits, vals
