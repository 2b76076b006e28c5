"""CPU checker for the GWQ mixed-precision linear layer (arXiv 2411.00850).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is compared against.  It shares no code with the CUDA path and
must never be imported by it; only the test-suite, the smoke check and the
CPU-baseline leg of the benchmark call it.

Everything is NumPy in float64 (the inputs are fp16 / fp32 values, all of
which are exact in float64).  The method is an encoding followed by a product,
so the functions below take the paper's steps in the paper's order:

  Section 3.2, Eq. "o"   select_outliers   mask of the largest |gradient|
  Section 3.2, Eq. "s"   group_stats       per-group scale
  Section 3.2, Eq. "z"   group_stats       per-group zero-point
  Section 3.2, Eq. "q"   quantize_codes    round-to-nearest codes
  Section 3.2, Eq. "w"   dequantize        s * (q - z), plus the kept outliers
  Abstract / Section 1   linear            y = x (deq(Wq) + S)^T, outliers in FP16

Readings taken where the paper is silent, garbled or ambiguous (each is a
choice of this implementation, listed again in the design notes):

  R1  Eq. "s" prints the denominator as 2^{b-1}; read as 2^b - 1 (the number of
      steps between code 0 and code 2^b-1), otherwise most codes are unused.
  R2  Eq. "z" gives a real number; the stored zero-point is
      clip(rint(-lo / s), 0, 2^b - 1).
  R3  The range used for a group always contains 0: lo = min(0, min w),
      hi = max(0, max w); only then is an integer zero-point in range.
  R4  "round" is round-half-to-even on the float64 quotient.
  R5  Codes are clipped to [0, 2^b - 1].
  R6  The scale is stored in fp16, rounded toward +inf from the float64
      quotient, so that (hi - lo) / s never exceeds 2^b - 1.
  R7  A group with hi == lo (all remaining entries zero, or every entry an
      outlier) gets s = 1, z = 0.
  R8  Eq. "o" (>= quantile) is read as an exact count: the
      ceil(frac * numel) entries of largest |g| in the matrix, equal
      magnitudes resolved in favour of the lower flat index n*K + k.  The
      order on magnitudes is the order of the IEEE-754 bit patterns of |g|
      (so -0 == +0 < finite < inf < NaN).
  R9  Groups are runs of `group` consecutive input features (k) inside one
      output row; outliers take no part in min / max and get code z, so their
      dense reconstruction is exactly 0.
  R10 The product accumulates in float64 here; the kept outliers enter with
      their exact fp16 values.

Parity status: every function below is pinned by tests that do not restate its
formula (brute force, closed forms, invariants, library special cases); see
tests/test_oracle_*.py.  The paper prints no worked numeric example, and never
defines its "GWQ-O"/"GWQ-R" variants nor the storage format behind its average
bit-widths: the bit layout of `pack_codes` is this project's own documented
format (parity with the paper unpinned for the format alone).
"""
from __future__ import annotations

import math

import numpy as np

__all__ = [
    "gradient_mean",
    "outlier_count",
    "select_outliers",
    "outlier_mask",
    "group_stats",
    "quantize_codes",
    "pack_codes",
    "unpack_codes",
    "dequantize",
    "quality",
    "linear",
    "quantize_layer",
]


# --------------------------------------------------------------------------
# Eq. "o": outlier location
# --------------------------------------------------------------------------
def gradient_mean(G_list) -> np.ndarray:
    """Gradient mean over calibration samples (Section 4.3, "Effect on Number of Calibration"):
    float32 additions in list order, then one float32 division by the count."""
    acc = np.array(G_list[0], dtype=np.float32, copy=True)
    for G in G_list[1:]:
        acc = (acc + np.asarray(G, dtype=np.float32)).astype(np.float32)
    return (acc / np.float32(len(G_list))).astype(np.float32)


def outlier_count(frac: float, numel: int) -> int:
    """Number of kept outliers: ceil(frac * numel) in IEEE double, clamped."""
    if not (0.0 <= frac <= 1.0):
        raise ValueError("frac must lie in [0, 1]")
    k = int(math.ceil(float(frac) * float(numel)))
    return max(0, min(int(numel), k))


def _abs_key(G: np.ndarray) -> np.ndarray:
    """Bit pattern of |g| as an unsigned integer; its integer order is the
    order used for ranking (reading R8)."""
    g = np.ascontiguousarray(G, dtype=np.float32)
    return g.view(np.uint32).reshape(-1) & np.uint32(0x7FFFFFFF)


def select_outliers(W: np.ndarray, G: np.ndarray, frac: float):
    """Eq. "o" with reading R8.

    W: fp16 [N, K]; G: fp32 [N, K].
    Returns (row_ptr int32 [N+1], col_idx int32 [nnz], val uint16 [nnz]): the
    CSR matrix S holding W's bit patterns at the selected positions, columns
    ascending inside every row.
    """
    if W.shape != G.shape or W.ndim != 2:
        raise ValueError("W and G must be 2-D and of equal shape")
    if W.dtype != np.float16 or G.dtype != np.float32:
        raise ValueError("W must be fp16 and G fp32")
    N, K = W.shape
    numel = N * K
    k_out = outlier_count(frac, numel)
    key = _abs_key(G)
    flat = np.arange(numel, dtype=np.int64)
    # sort by magnitude descending, then flat index ascending
    order = np.lexsort((flat, -key.astype(np.int64)))
    chosen = np.sort(order[:k_out])
    rows = chosen // K
    cols = chosen % K
    row_ptr = np.zeros(N + 1, dtype=np.int64)
    np.add.at(row_ptr, rows + 1, 1)
    row_ptr = np.cumsum(row_ptr)
    val = np.ascontiguousarray(W).view(np.uint16).reshape(-1)[chosen]
    return row_ptr.astype(np.int32), cols.astype(np.int32), val.astype(np.uint16)


def outlier_mask(row_ptr: np.ndarray, col_idx: np.ndarray, N: int, K: int) -> np.ndarray:
    """Dense boolean mask O [N, K] of the CSR pattern."""
    mask = np.zeros((N, K), dtype=bool)
    counts = np.diff(row_ptr.astype(np.int64))
    rows = np.repeat(np.arange(N, dtype=np.int64), counts)
    mask[rows, col_idx.astype(np.int64)] = True
    return mask


# --------------------------------------------------------------------------
# Eqs. "s", "z": per-group scale and zero-point
# --------------------------------------------------------------------------
def _fp16_round_up(v: np.ndarray) -> np.ndarray:
    """Smallest fp16 value >= v (v float64, finite, >= 0)."""
    h = v.astype(np.float16)
    low = h.astype(np.float64) < v
    h_up = np.nextafter(h, np.float16(np.inf))
    return np.where(low, h_up, h).astype(np.float16)


def group_stats(W: np.ndarray, mask: np.ndarray, bits: int, group: int):
    """Eqs. "s" and "z" with readings R1-R3, R6, R7, R9.

    Returns (scales fp16 [N, K/group], zeros uint8 [N, K/group]).
    """
    N, K = W.shape
    if K % group != 0:
        raise ValueError("K must be a multiple of the group size")
    if not np.all(np.isfinite(W)):
        raise ValueError("non-finite weight")
    qmax = float(2 ** bits - 1)
    ng = K // group
    w = W.astype(np.float64).reshape(N, ng, group)
    m = mask.reshape(N, ng, group)
    lo = np.where(m, np.inf, w).min(axis=2)
    hi = np.where(m, -np.inf, w).max(axis=2)
    lo = np.minimum(lo, 0.0)
    hi = np.maximum(hi, 0.0)
    flat_range = hi == lo
    s64 = (hi - lo) / qmax
    s16 = _fp16_round_up(np.where(flat_range, 1.0, s64))
    s = s16.astype(np.float64)
    z = np.clip(np.rint(-lo / s), 0.0, qmax)
    z = np.where(flat_range, 0.0, z)
    return s16, z.astype(np.uint8)


# --------------------------------------------------------------------------
# Eq. "q": codes
# --------------------------------------------------------------------------
def quantize_codes(W, mask, scales, zeros, bits: int, group: int) -> np.ndarray:
    """Eq. "q" with readings R4, R5, R9.  Returns codes uint8 [N, K]."""
    N, K = W.shape
    qmax = float(2 ** bits - 1)
    s = np.repeat(scales.astype(np.float64), group, axis=1)
    z = np.repeat(zeros.astype(np.float64), group, axis=1)
    q = np.clip(np.rint(W.astype(np.float64) / s) + z, 0.0, qmax)
    q = np.where(mask, z, q)
    return q.astype(np.uint8)


# --------------------------------------------------------------------------
# Storage format (this project's own; the paper specifies none)
# --------------------------------------------------------------------------
def _bit_positions(bits: int):
    """For column i of a 32-column run: list of (word, bit offset, code bit) triples,
    one per code bit, following the written format definition (see pack_codes)."""
    pos = []
    for i in range(32):
        if bits == 4:
            t, r = divmod(i, 8)          # word t holds columns 8t..8t+7
            j, e = divmod(r, 2)          # column 8t + 2j + e
            pos.append([(t, 16 * e + 4 * j + b, b) for b in range(4)])
        elif bits == 3:
            if i < 30:
                w, r = divmod(i, 10)     # word w holds columns 10w..10w+9
                p_, e = divmod(r, 2)     # column 10w + 2p + e
                pos.append([(w, 16 * e + 3 * p_ + b, b) for b in range(3)])
            else:
                e = i - 30               # columns 30 / 31: bit b lives in word b, bit 15 / 31
                pos.append([(b, 16 * e + 15, b) for b in range(3)])
        elif bits in (2, 8):
            per = 32 // bits             # columns per word
            t, r = divmod(i, per)        # word t holds columns per*t .. per*t + per - 1
            j, e = divmod(r, 2)          # column per*t + 2j + e
            pos.append([(t, 16 * e + bits * j + b, b) for b in range(bits)])
        else:
            raise ValueError("bits must be 2, 3, 4 or 8")
    return pos


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Pack codes [N, K] into 32-bit words, `bits` words per run of 32 columns.

    Pair-interleaved order: in every word the low 16 bits hold even columns and
    the high 16 bits hold the odd columns that follow them, so that one mask
    yields a (column 2j, column 2j+1) pair in the two halves of a register.
      4 bits: word t of a row holds columns 8t..8t+7; column 8t + 2j + e
              (j = 0..3, e = 0,1) sits in bits [16e + 4j, 16e + 4j + 4).
      2 and 8 bits, likewise: word t holds columns ct..ct+c-1 with c = 32/bits;
              column ct + 2j + e sits in bits [16e + bits j, 16e + bits j + bits).
      3 bits: word w (0..2) of run r holds columns 32r + 10w + 2p + e
              (p = 0..4, e = 0,1) in bits [16e + 3p, 16e + 3p + 3); bit b of the
              codes of columns 32r+30 and 32r+31 sits in bit 15 and bit 31 of
              word b.
    Returns uint32 [N, K*bits/32].
    """
    N, K = codes.shape
    if K % 32 != 0:
        raise ValueError("K must be a multiple of 32")
    if codes.max(initial=0) > 2 ** bits - 1:
        raise ValueError("code out of range")
    out = np.zeros((N, K // 32, bits), dtype=np.uint32)
    c = codes.reshape(N, K // 32, 32).astype(np.uint32)
    for i, triples in enumerate(_bit_positions(bits)):
        for (word, off, b) in triples:
            out[:, :, word] |= ((c[:, :, i] >> np.uint32(b)) & np.uint32(1)) << np.uint32(off)
    return out.reshape(N, K * bits // 32)


def unpack_codes(words: np.ndarray, bits: int, K: int) -> np.ndarray:
    """Inverse of pack_codes.  Returns codes uint8 [N, K]."""
    N = words.shape[0]
    w = words.reshape(N, K // 32, bits).astype(np.uint32)
    codes = np.zeros((N, K // 32, 32), dtype=np.uint32)
    for i, triples in enumerate(_bit_positions(bits)):
        for (word, off, b) in triples:
            codes[:, :, i] |= ((w[:, :, word] >> np.uint32(off)) & np.uint32(1)) << np.uint32(b)
    return codes.reshape(N, K).astype(np.uint8)


# --------------------------------------------------------------------------
# Eq. "w": reconstruction, and the layer product
# --------------------------------------------------------------------------
def dequantize(codes, scales, zeros, group: int, row_ptr, col_idx, val) -> np.ndarray:
    """Eq. "w" plus the kept FP16 outliers: w_hat = s*(q - z) + S, float64 [N,K]."""
    N, K = codes.shape
    s = np.repeat(scales.astype(np.float64), group, axis=1)
    z = np.repeat(zeros.astype(np.float64), group, axis=1)
    w_hat = s * (codes.astype(np.float64) - z)
    counts = np.diff(row_ptr.astype(np.int64))
    rows = np.repeat(np.arange(N, dtype=np.int64), counts)
    S = np.zeros((N, K), dtype=np.float64)
    S[rows, col_idx.astype(np.int64)] = val.view(np.float16).astype(np.float64)
    return w_hat + S


def quality(W: np.ndarray, G: np.ndarray, w_hat: np.ndarray):
    """The two objectives the method states for a quantized layer (Section 3.1):
    the squared error ||W - W_Q||_2^2 (Eq. "Q") and the first-order change of the loss
    g^T (W - W_Q) (Eq. "Taylor" / "final_OPO"), with W_Q = w_hat.  Plain float64 sums."""
    d = W.astype(np.float64) - w_hat
    return float(np.sum(d * d)), float(np.sum(G.astype(np.float64) * d))


def linear(x: np.ndarray, w_hat: np.ndarray):
    """y = x w_hat^T in float64, and bound = |x| |w_hat|^T (the per-output sum
    of |x_k * w_hat_k| that the floating-point tolerance is stated against)."""
    x64 = np.asarray(x, dtype=np.float64)
    y = x64 @ w_hat.T
    bound = np.abs(x64) @ np.abs(w_hat).T
    return y, bound


def quantize_layer(W, G, frac: float, bits: int, group: int) -> dict:
    """All encoding steps in order; returns every intermediate by name."""
    N, K = W.shape
    row_ptr, col_idx, val = select_outliers(W, G, frac)
    mask = outlier_mask(row_ptr, col_idx, N, K)
    scales, zeros = group_stats(W, mask, bits, group)
    codes = quantize_codes(W, mask, scales, zeros, bits, group)
    words = pack_codes(codes, bits)
    return dict(N=N, K=K, bits=bits, group=group, row_ptr=row_ptr, col_idx=col_idx,
                val=val, mask=mask, scales=scales, zeros=zeros, codes=codes, words=words)
