"""The allocation-free selection entry point gives the same CSR as gwq_select_outliers and as the CPU checker.

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

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq
from paper_2411_00850_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(N, K, frac, seed, ties=False, check_memory=False):
    W, G = synth.make_weight_and_grad(N, K, seed)
    if ties:
        G = synth.make_tie_heavy_grad(N, K, seed, levels=5)
    Wd, Gd = torch.from_numpy(W).to(DEV), torch.from_numpy(G).to(DEV)
    S = gwq.gwq_select_outliers(Wd, Gd, frac)
    want = [t.cpu().numpy() for t in S.arrays()]
    S.free()
    ref = orc.select_outliers(W, G, frac)                      # the CPU checker, directly
    cap = int(np.ceil(frac * N * K)) + 5
    row_ptr = torch.full((N + 1,), -7, dtype=torch.int32, device=DEV)
    col_idx = torch.full((cap,), -7, dtype=torch.int32, device=DEV)
    val = torch.full((cap,), -7, dtype=torch.int16, device=DEV)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    nnz = gwq.gwq_select_outliers_static(Wd, Gd, frac, row_ptr, col_idx, val)
    torch.cuda.synchronize()
    if check_memory:   # the call took no device memory (the driver's own figure, not torch's pool)
        assert torch.cuda.mem_get_info()[0] == free_before
    assert nnz == want[0][-1] == len(want[1]) == len(ref[1])
    got = (row_ptr.cpu().numpy(), col_idx.cpu().numpy(), val.cpu().numpy())
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[0], ref[0])
    assert np.array_equal(got[1][:nnz], want[1]) and np.array_equal(got[1][:nnz], ref[1])
    assert np.array_equal(got[2][:nnz], want[2]) and np.array_equal(got[2][:nnz].view(np.uint16), ref[2])
    assert np.all(got[1][nnz:] == -7) and np.all(got[2][nnz:] == -7)      # nothing written past nnz


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    _both(768, 1024, 0.01, seed=41)
    _both(200, 512, 0.03, seed=42, ties=True, check_memory=True)   # smaller: stale per-row counters must not leak in
    _both(768, 1024, 0.01, seed=41, check_memory=True)


def test_largest_row_count_the_work_area_covers():
    _both(32768, 32, 0.01, seed=44)               # N = 32768 is accepted (32769 is refused, below)


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
    st = lib.gwq_select_outliers_static(Wd.data_ptr(), Gd.data_ptr(), 32769, 32, 0.0, row_ptr.data_ptr(),
                                        small.data_ptr(), small16.data_ptr(), 8, C.byref(nnz), None)
    assert st == 2                                   # nothing was read or written: the size check comes first
    st = lib.gwq_select_outliers_static(Wd.data_ptr(), Gd.data_ptr(), N, K, 0.01, row_ptr.data_ptr(),
                                        small.data_ptr(), small16.data_ptr(), 8, C.byref(nnz), None)
    assert st == 1 and nnz.value == int(np.ceil(0.01 * N * K))   # too short: the needed size is reported
    assert gwq.gwq_select_outliers_static(Wd, Gd, 0.0, row_ptr, small, small16) == 0
    assert not row_ptr.any()
