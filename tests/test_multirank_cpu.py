"""The N > 1 path of the benchmark is "replicas only": no data-path collective, one max-reduction of
the per-rank step time.  Covered here with two gloo ranks on the CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 2.0 + 3.0 * rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local)
    value = bench.whole_job_gbs(10 ** 9, ms, world)
    dist.barrier()
    out[rank] = (ms, value)
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms, value = res[rank]
        assert ms == 5.0                                   # max over ranks, on every rank
        assert value == pytest.approx(2 * 1e9 / 5e-3 / 1e9)  # both replicas' bytes over the slowest time


def test_single_process_is_its_own_maximum():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.whole_job_gbs(2 * 10 ** 9, 1.0, 1) == pytest.approx(2000.0)


# ---------------------------------------------------------------- a layer whose rows are split over two ranks
class _CheckerOps:
    """The per-rank steps of RowShardedLinear carried out by the CPU checker (NumPy float64)."""

    @staticmethod
    def select(W, G, frac):
        from oracle import gwq_oracle as orc
        return orc.select_outliers(W, G, frac)

    @staticmethod
    def rows(S, row0, row1):
        row_ptr, col_idx, val = S
        lo, hi = int(row_ptr[row0]), int(row_ptr[row1])
        return (row_ptr[row0:row1 + 1] - row_ptr[row0]), col_idx[lo:hi], val[lo:hi]

    @staticmethod
    def pack(W_local, S_local, bits, group):
        import numpy as np
        from oracle import gwq_oracle as orc
        row_ptr, col_idx, val = S_local
        n, K = W_local.shape
        mask = orc.outlier_mask(row_ptr, col_idx, n, K)
        s, z = orc.group_stats(np.ascontiguousarray(W_local), mask, bits, group)
        q = orc.quantize_codes(W_local, mask, s, z, bits, group)
        return orc.dequantize(q, s, z, group, row_ptr, col_idx, val)

    @staticmethod
    def linear(w_hat, x):
        from oracle import gwq_oracle as orc
        return torch.from_numpy(orc.linear(x.numpy(), w_hat)[0])


def _sharded_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import gwq_oracle as orc
    from paper_2411_00850_b200 import sharded, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, K, M = 300, 256, 5                       # 3 units of 128 rows: rank 0 owns one, rank 1 two (the last ragged)
    W, G = synth.make_weight_and_grad(N, K, 77)
    _, xv = synth.make_activations(M, K, seed=77)
    layer = sharded.RowShardedLinear(W, G, 0.02, 4, 64, _CheckerOps)
    y = layer.forward(torch.from_numpy(xv))
    L = orc.quantize_layer(W, G, 0.02, 4, 64)   # the whole layer on one rank
    w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], 64, L["row_ptr"], L["col_idx"], L["val"])
    y_ref, bound = orc.linear(xv, w_hat)
    out[rank] = ((layer.row0, layer.row1), float(np.max(np.abs(y.numpy() - y_ref) / (bound + 1e-30))), tuple(y.shape))
    dist.barrier()
    dist.destroy_process_group()


def test_row_sharded_layer_on_two_ranks_equals_the_whole_layer():
    world = 2
    port = 31500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_sharded_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == (0, 128) and res[1][0] == (128, 300)
    for rank in (0, 1):
        assert res[rank][2] == (5, 300)
        assert res[rank][1] < 1e-14          # float64 products of the same reconstructed rows


def test_row_ranges_tile_the_rows():
    sys.path.insert(0, ROOT)
    from paper_2411_00850_b200 import sharded
    for N in (1, 127, 128, 300, 4096, 11008, 28672):
        for world in (1, 2, 3, 4, 8):
            ranges = [sharded.row_range(N, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == N
            for (a0, a1), (b0, b1) in zip(ranges, ranges[1:]):
                assert a1 == b0 and a0 <= a1
            assert all(r0 % 128 == 0 for r0, _ in ranges)
