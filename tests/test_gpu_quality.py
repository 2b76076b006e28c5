"""GPU parity of gwq_quality (Section 3.1: squared error, Eq. "Q"; first-order loss change, Eq. "Taylor")
against the CPU checker.  Both sides sum exact FP64 terms; only the order of the additions differs, so
the tolerance is 1024 units of FP64 rounding of the sum of magnitudes (a thread adds ~500 terms in a row)."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_packed_equal, oracle_w_hat, quantize_on_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,K,frac,bits,group,seed", [
    (64, 512, 0.01, 4, 128, 60), (100, 2176, 0.02, 3, 64, 61), (528, 4096, 0.01, 4, 128, 62),
    (33, 1024, 0.0, 3, 128, 63), (16, 256, 1.0, 4, 64, 64), (1000, 2176, 0.3, 4, 64, 65),
    (100, 1056, 0.01, 4, 16, 66), (64, 1024, 0.02, 3, 32, 67),
])
def test_quality_matches_checker(N, K, frac, bits, group, seed):
    W, G = synth.make_weight_and_grad(N, K, seed)
    L = orc.quantize_layer(W, G, frac, bits, group)
    P = quantize_on_gpu(W, G, frac, bits, group)
    assert_packed_equal(P, L)
    w_hat = oracle_w_hat(L)
    sq_ref, fo_ref = orc.quality(W, G, w_hat)
    sq, fo = gwq.gwq_quality(to_dev(W), to_dev(G), P)
    d = W.astype(np.float64) - w_hat
    eps = 2.0 ** -52
    assert abs(sq - sq_ref) <= 1024 * eps * float(np.sum(d * d)) + 1e-300
    assert abs(fo - fo_ref) <= 1024 * eps * float(np.sum(np.abs(G.astype(np.float64) * d))) + 1e-300
    if frac == 1.0:
        assert sq == 0.0 and fo == 0.0
    # a second call gives the same bits (fixed summation order)
    assert gwq.gwq_quality(to_dev(W), to_dev(G), P) == (sq, fo)


def test_quality_argument_checks():
    W, G = synth.make_weight_and_grad(16, 256, 66)
    P = quantize_on_gpu(W, G, 0.01, 4, 128)
    with pytest.raises(ValueError):
        gwq.gwq_quality(to_dev(W[:8]), to_dev(G[:8]), P)
    with pytest.raises(ValueError):
        gwq.gwq_quality(to_dev(W).float(), to_dev(G), P)
