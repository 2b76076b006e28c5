"""The allocation-free selection entry point gives the same CSR as gwq_select_outliers.

Some users of this library cannot let it allocate: their process has given all device
memory to its own pool, or a cudaMalloc in the middle of serving would stall every
stream.  For them gwq_select_outliers_static works out of a fixed array inside the
library and writes into buffers they pass in.  That array is shared by all calls and
keeps the previous call's contents, so the check is made on two calls in a row with
different matrices (the second smaller than the first, so stale counters would show).
This file sorts last so that a failure here cannot hide the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(N, K, frac, seed, ties=False):
    W, G = synth.make_weight_and_grad(N, K, seed)
    if ties:
        G = synth.make_tie_heavy_grad(N, K, seed, levels=5)
    Wd, Gd = torch.from_numpy(W).to(DEV), torch.from_numpy(G).to(DEV)
    S = gwq.gwq_select_outliers(Wd, Gd, frac)
    want = [t.cpu().numpy() for t in S.arrays()]
    S.free()
    cap = int(np.ceil(frac * N * K)) + 5
    row_ptr = torch.full((N + 1,), -7, dtype=torch.int32, device=DEV)
    col_idx = torch.full((cap,), -7, dtype=torch.int32, device=DEV)
    val = torch.full((cap,), -7, dtype=torch.int16, device=DEV)
    nnz = gwq.gwq_select_outliers_static(Wd, Gd, frac, row_ptr, col_idx, val)
    torch.cuda.synchronize()
    assert nnz == want[0][-1] == len(want[1])
    assert np.array_equal(row_ptr.cpu().numpy(), want[0])
    assert np.array_equal(col_idx.cpu().numpy()[:nnz], want[1])
    assert np.array_equal(val.cpu().numpy()[:nnz], want[2])
    assert np.all(col_idx.cpu().numpy()[nnz:] == -7)          # nothing written past nnz


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    _both(768, 1024, 0.01, seed=41)
    _both(200, 512, 0.03, seed=42, ties=True)     # smaller: stale per-row counters must not leak in
    _both(768, 1024, 0.01, seed=41)


def test_limits_are_reported_not_faulted():
    N, K = 64, 256
    W, G = synth.make_weight_and_grad(N, K, 43)
    Wd, Gd = torch.from_numpy(W).to(DEV), torch.from_numpy(G).to(DEV)
    row_ptr = torch.zeros(N + 1, dtype=torch.int32, device=DEV)
    small = torch.zeros(8, dtype=torch.int32, device=DEV)
    small16 = torch.zeros(8, dtype=torch.int16, device=DEV)
    with pytest.raises(gwq.GwqError) as e:          # capacity below ceil(frac * N * K)
        gwq.gwq_select_outliers_static(Wd, Gd, 0.01, row_ptr, small, small16)
    assert e.value.status == 1
    lib = gwq.load_library()                         # more rows than the fixed work area covers
    import ctypes as C
    nnz = C.c_int64(0)
    st = lib.gwq_select_outliers_static(Wd.data_ptr(), Gd.data_ptr(), 40000, 32, 0.0, row_ptr.data_ptr(),
                                        small.data_ptr(), small16.data_ptr(), 8, C.byref(nnz), None)
    assert st == 2
    assert gwq.gwq_select_outliers_static(Wd, Gd, 0.0, row_ptr, small, small16) == 0
    assert not row_ptr.any()
