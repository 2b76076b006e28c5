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
