"""Runs gwq_linear a few times on one synthetic layer: the small, self-contained case that the
profiler captures are taken on (python -m paper_2411_00850_b200.profile_case N K bits M dtype [copies [group]]).

`copies` packed copies of the layer are cycled through so that the weights read by one launch
are not in L2 from the previous one.  Prints the mean time per launch measured with CUDA events.
"""
from __future__ import annotations

import sys

import numpy as np
import torch

from . import binding as gwq
from . import build, synth


def main(argv):
    N, K, bits, M = (int(a) for a in argv[:4])
    dtype = argv[4] if len(argv) > 4 else "f16"
    copies = int(argv[5]) if len(argv) > 5 else 4
    group = int(argv[6]) if len(argv) > 6 else 128
    build.build()
    dev = "cuda:0"
    W, G = synth.make_weight_and_grad(N, K, 1)
    Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
    packed = [gwq.gwq_pack(Wd, gwq.gwq_select_outliers(Wd, Gd, 0.01), bits, group) for _ in range(copies)]
    bits16, _ = synth.make_activations(M, K, 1, dtype=dtype, heavy_channels=8 if M > 32 else 0)
    x = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16 if dtype == "f16" else torch.bfloat16)
    y = torch.empty((M, N), dtype=x.dtype, device=dev)
    for _ in range(3):
        for P in packed:
            gwq.gwq_linear(P, x, out=y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for P in packed:
        gwq.gwq_linear(P, x, out=y)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / copies
    nnz = packed[0].nnz
    print(f"N={N} K={K} bits={bits} group={group} M={M} {dtype}: {us:.2f} us per launch (stream order, no graph), "
          f"{2 * M * (N * K + nnz) / us / 1e6:.1f} TFLOP/s, status {gwq.gwq_device_status(packed[0])}")


if __name__ == "__main__":
    main(sys.argv[1:])
