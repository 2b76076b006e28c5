"""Helpers shared by the GPU parity tests: run the CUDA path and the CPU checker on the
same seeded inputs and compare."""
import numpy as np
import torch

from oracle import gwq_oracle as orc
from paper_2411_00850_b200 import binding as gwq

DEV = "cuda:0"
REL_TOL, ABS_TOL = 1e-3, 1e-5   # |y_gpu - y_ref| <= REL_TOL * sum_k |x_k w_hat_k| + ABS_TOL


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def quantize_on_gpu(W: np.ndarray, G: np.ndarray, frac: float, bits: int, group: int):
    Wd, Gd = to_dev(W), to_dev(G)
    S = gwq.gwq_select_outliers(Wd, Gd, frac)
    P = gwq.gwq_pack(Wd, S, bits, group)
    return P


def assert_packed_equal(P, L):
    """Bit-exact comparison of everything the encoder produces."""
    a = {k: v.cpu().numpy() for k, v in P.arrays().items()}
    assert np.array_equal(a["row_ptr"], L["row_ptr"]), "row_ptr"
    assert np.array_equal(a["col_idx"], L["col_idx"]), "col_idx"
    assert np.array_equal(a["val"].view(np.uint16), L["val"]), "val"
    assert np.array_equal(a["scales"].view(np.uint16), L["scales"].view(np.uint16)), "scales"
    assert np.array_equal(a["zeros"], L["zeros"]), "zeros"
    assert np.array_equal(a["words"].view(np.uint32), L["words"]), "codes"


def x_tensor(bits16: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(bits16.view(np.int16).copy()).to(DEV)
    return t.view(torch.float16 if dtype == "f16" else torch.bfloat16)


def assert_linear_close(y_gpu: torch.Tensor, y_ref: np.ndarray, bound: np.ndarray, extra_rel: float = 0.0):
    """extra_rel accounts for the rounding of a 16-bit OUTPUT (half an ulp of |y|)."""
    yg = y_gpu.double().cpu().numpy()
    tol = REL_TOL * bound + ABS_TOL + extra_rel * np.abs(y_ref)
    err = np.abs(yg - y_ref)
    worst = np.unravel_index(np.argmax(err - tol), err.shape)
    assert np.all(err <= tol), f"worst at {worst}: err {err[worst]:.3e} tol {tol[worst]:.3e} y {y_ref[worst]:.4e}"
    return float((err / (REL_TOL * bound + ABS_TOL)).max())


def oracle_w_hat(L):
    return orc.dequantize(L["codes"], L["scales"], L["zeros"], L["group"], L["row_ptr"], L["col_idx"], L["val"])


def checker_rows(W, row_ptr, col_idx, val, rows, bits, group):
    """Encode and reconstruct the given rows with the CPU checker, the outliers of the whole matrix given
    (the selection is global, everything after it is per row).  Returns (scales, zeros, words, w_hat)."""
    K = W.shape[1]
    rows = np.asarray(rows, dtype=np.int64)
    counts = (row_ptr[rows + 1] - row_ptr[rows]).astype(np.int64)
    sub_ptr = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    if len(rows) and np.all(np.diff(rows) == 1):          # a contiguous block of rows: one slice of the CSR
        lo, hi = int(row_ptr[rows[0]]), int(row_ptr[rows[-1] + 1])
        sub_col, sub_val = col_idx[lo:hi].astype(np.int32), val[lo:hi].astype(np.uint16)
    else:
        sub_col = np.concatenate([col_idx[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.int32)
        sub_val = np.concatenate([val[row_ptr[n]:row_ptr[n + 1]] for n in rows]).astype(np.uint16)
    mask = orc.outlier_mask(sub_ptr, sub_col, len(rows), K)
    Ws = np.ascontiguousarray(W[rows])
    s, z = orc.group_stats(Ws, mask, bits, group)
    q = orc.quantize_codes(Ws, mask, s, z, bits, group)
    words = orc.pack_codes(q, bits)
    w_hat = orc.dequantize(q, s, z, group, sub_ptr, sub_col, sub_val)
    return s, z, words, w_hat


def checker_row_blocks(W, row_ptr, col_idx, val, bits, group, block=2048):
    """checker_rows over the whole matrix, block of rows by block of rows (bounded host memory)."""
    N = W.shape[0]
    for r0 in range(0, N, block):
        r1 = min(N, r0 + block)
        yield (r0, r1) + checker_rows(W, row_ptr, col_idx, val, np.arange(r0, r1), bits, group)


def distinct_rows(N, seed, count):
    """`count` distinct row indices: the first and last rows of the 16-row and 128-row tiles plus seeded draws."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 7, 8, 15, 16, 127, 128, N - 129, N - 128, N - 17, N - 16, N - 2, N - 1]
    rows = {r for r in fixed if 0 <= r < N}
    for r in rng.permutation(N):
        if len(rows) >= count:
            break
        rows.add(int(r))
    return sorted(rows)
