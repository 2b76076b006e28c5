"""The give-up path of the tensor-core kernel's bounded waits, walked without any fault: the spin limit is
set to zero on an otherwise ordinary small problem, so the first wait that is not satisfied at once gives
up; the kernel must record GWQ_ERR_TIMEOUT, drain what it has in flight, free its tensor memory and return,
and the next call with the default limit must be correct again."""
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import assert_linear_close, oracle_w_hat, quantize_on_gpu, x_tensor

pytestmark = pytest.mark.gpu


# the last case takes the two-phase path (the contraction on CTA pairs)
@pytest.mark.parametrize("N,K,M", [(128, 256, 64), (384, 2048, 300), (600, 512, 2200)])
def test_zero_spin_limit_gives_up_cleanly_and_the_layer_stays_usable(N, K, M):
    W, G = synth.make_weight_and_grad(N, K, 95)
    L = orc.quantize_layer(W, G, 0.01, 4, 128)
    P = quantize_on_gpu(W, G, 0.01, 4, 128)
    w_hat = oracle_w_hat(L)
    bits16, xv = synth.make_activations(M, K, seed=95, dtype="f16")
    x = x_tensor(bits16, "f16")
    y_ref, bound = orc.linear(xv, w_hat)

    gwq.gwq_set_wait_limit(P, 0)
    gwq.gwq_linear(P, x, out_dtype=torch.float32)          # returns: every wait is bounded
    assert gwq.gwq_device_status(P) == gwq.GWQ_ERR_TIMEOUT  # recorded, and cleared by the read
    assert gwq.gwq_device_status(P) == 0

    gwq.gwq_set_wait_limit(P, -1)                           # the default again
    for _ in range(2):
        y = gwq.gwq_linear(P, x, out_dtype=torch.float32)
        assert gwq.gwq_device_status(P) == 0
        assert_linear_close(y, y_ref, bound)
    P.free()
