"""GPU parity of gwq_gradient_mean (Section 4.3: outliers located on the mean of the calibration
samples' gradients) against the CPU checker: same FP32 additions in the same order, so bit for bit,
and the outlier set selected on the mean."""
import numpy as np
import pytest
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("count", [1, 2, 5, 16])
def test_mean_and_selection_on_it(count):
    N, K = 96, 1056                                  # numel not a multiple of the launch width
    W, _ = synth.make_weight_and_grad(N, K, 80)
    Gs = [synth.make_weight_and_grad(N, K, 81 + i)[1] for i in range(count)]
    mean_ref = orc.gradient_mean(Gs)
    mean = gwq.gwq_gradient_mean([to_dev(G) for G in Gs])
    assert np.array_equal(mean.cpu().numpy().view(np.uint32), mean_ref.view(np.uint32))
    row_ptr, col_idx, val = orc.select_outliers(W, mean_ref, 0.01)
    S = gwq.gwq_select_outliers(to_dev(W), mean, 0.01)
    rp, ci, v = (t.cpu().numpy() for t in S.arrays())
    assert np.array_equal(rp, row_ptr) and np.array_equal(ci, col_idx)
    assert np.array_equal(v.view(np.uint16), val)
    S.free()


def test_in_place_and_argument_errors():
    Gs = [to_dev(synth.make_weight_and_grad(8, 64, 90 + i)[1]) for i in range(3)]
    want = gwq.gwq_gradient_mean(Gs).clone()
    got = gwq.gwq_gradient_mean(Gs, out=Gs[0])       # the output may be one of the inputs
    assert torch.equal(got, want)
    with pytest.raises(ValueError):
        gwq.gwq_gradient_mean([])
    with pytest.raises(gwq.GwqError):
        gwq.gwq_gradient_mean([want] * 17)            # more samples than one call takes
