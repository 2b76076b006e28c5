/*
 * gwq.h - C ABI of the GWQ mixed-precision linear layer for NVIDIA B200 (sm_100a).
 *
 * Method: "GWQ: Gradient-Aware Weight Quantization for Large Language Models"
 * (arXiv 2411.00850).  A weight matrix W [N, K] (N output features, K input
 * features) is split by the magnitude of a calibration gradient G of the same
 * shape: the largest ~1 % of |g| mark "outlier" weights that stay in FP16
 * (Section 3.2, Eq. "o"; Section 1); all other weights are quantized to b = 3 or
 * 4 bits with one scale s and one zero-point z per group of consecutive input
 * features (Section 3.2, Eqs. "s", "z", "q"), and the layer computes
 *
 *        y = x (s (q - z) + S)^T                      (Section 3.2, Eq. "w")
 *
 * where S is the sparse FP16 outlier matrix.
 *
 * Conventions for every call
 *  - Pointers are DEVICE pointers unless an argument says "host".
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *  - Caller-owned buffers (W, G, x, y) are never freed by the library and only
 *    y is written.  Objects returned through `out` are owned by the library and
 *    released with gwq_free().
 *  - Nothing aborts or throws: every failure is a gwq_status.  There is no CPU
 *    fallback: without a CUDA device the calls return GWQ_ERR_CUDA.
 *  - Matrices are row-major.  fp16 / bf16 data are passed as uint16_t bit
 *    patterns.  Device pointers must be 16-byte aligned.
 */
#ifndef GWQ_H_
#define GWQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GWQ_OK = 0,
  GWQ_ERR_INVALID_ARG = 1, /* null or misaligned pointer, non-positive size, frac outside [0,1] */
  GWQ_ERR_UNSUPPORTED = 2, /* bits not in {2,3,4,8}, group not in {16,32,64,128}, K % group != 0 */
  GWQ_ERR_ALLOC = 3,       /* device or host allocation failed                                  */
  GWQ_ERR_NONFINITE = 4,   /* W holds an inf or NaN                                             */
  GWQ_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (kernel returned early)        */
  GWQ_ERR_CUDA = 6,        /* a CUDA runtime call failed                                        */
  GWQ_ERR_WORKSPACE = 7    /* the call needs scratch memory: see gwq_linear_ws                  */
} gwq_status;

typedef enum { GWQ_F16 = 0, GWQ_BF16 = 1, GWQ_F32 = 2 } gwq_dtype;

/* Sparse FP16 outlier matrix S in CSR form (Section 3.2, Eq. "o": the mask O; the
 * values are the original FP16 weights at the masked positions).                    */
typedef struct gwq_outliers {
  uint32_t tag;      /* library-private type tag, do not modify                          */
  int32_t N, K;      /* shape of W                                                       */
  int64_t nnz;       /* = ceil(frac * N * K)                                             */
  int32_t* row_ptr;  /* device [N+1]                                                     */
  int32_t* col_idx;  /* device [nnz], strictly ascending inside each row                 */
  uint16_t* val;     /* device [nnz], fp16 bit patterns copied from W                    */
} gwq_outliers;

/* Packed layer.
 * codes: uint32 [N, K*bits/32], `bits` words per run of 32 consecutive columns, in
 *   pair-interleaved order: the low 16 bits of a word hold even columns, the high 16 bits
 *   the odd columns that follow them.
 *     4 bits: word t of a row holds columns 8t..8t+7; column 8t + 2j + e (j = 0..3,
 *             e = 0,1) is in bits [16e + 4j, 16e + 4j + 4).
 *     2 and 8 bits, likewise: word t holds the c = 32 / bits columns ct..ct+c-1; column ct + 2j + e is in
 *             bits [16e + bits j, 16e + bits j + bits).
 *     3 bits: word w (0..2) of run r holds columns 32r + 10w + 2p + e (p = 0..4, e = 0,1)
 *             in bits [16e + 3p, 16e + 3p + 3); bit b of the codes of columns 32r+30 and
 *             32r+31 is in bit 15 and bit 31 of word b.
 * scales: fp16 [N, K/group]; zeros: uint8 [N, K/group], each in [0, 2^bits - 1].
 * An outlier position stores the code z of its group, so its dense term is exactly 0. */
typedef struct gwq_packed {
  uint32_t tag;
  int32_t N, K, bits, group;
  uint32_t* codes;
  uint16_t* scales;
  uint8_t* zeros;
  gwq_outliers* S; /* owned by this object                                               */
  void* priv;      /* kernel-private derived tables and staging; opaque                  */
} gwq_packed;

/* Outlier location (Section 3.2, Eq. "o"; Figure 2: "the top 1% with the largest |g|").
 * Selects exactly ceil(frac * N*K) entries (the product evaluated in IEEE double) with
 * the largest |G| over the whole matrix; entries of equal magnitude are taken in
 * ascending flat index n*K + k.  Magnitudes are ordered by the bit pattern of |g|
 * (so -0 == +0 < finite < inf < NaN); G may hold any bit pattern.
 *   W_f16 [N,K] fp16, G_f32 [N,K] fp32: device, caller-owned, read only.
 *   *out: new library-owned CSR object.  The call synchronises `stream` before it
 *   returns.
 * Errors: INVALID_ARG (null / misaligned pointer, N or K <= 0, N*K >= 2^31, frac outside
 *   [0,1]), UNSUPPORTED (K % 32 != 0), ALLOC, CUDA.  On error *out is NULL.             */
gwq_status gwq_select_outliers(const uint16_t* W_f16, const float* G_f32, int32_t N, int32_t K,
                               double frac, gwq_outliers** out, void* stream);

/* Outlier selection for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of gwq_select_outliers with identical
 * results.)
 *
 * Who needs it: processes that have handed the whole device to their own memory pool or
 * run under a fixed memory budget, so that a cudaMalloc inside a library call would
 * fail, fragment the pool, or stall every stream of the process while the driver
 * synchronises; and callers on a latency-critical path that may not take that stall.
 * This call performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 *   row_ptr [N+1], col_idx [capacity], val [capacity]: device buffers supplied by the
 *   caller; capacity must be >= ceil(frac * N*K), which is written to *nnz_host (host),
 *   also when the call fails because capacity is too small (0 on every other failure).
 *   The work area is a fixed 392 KiB array inside the library image, present on every
 *   GPU that loads the library; it bounds the row count: N <= 32768, otherwise
 *   GWQ_ERR_UNSUPPORTED.  All calls on one GPU share that array, so two calls that
 *   overlap on the GPU (different streams or threads) corrupt each other; serialise
 *   them.  The first call on each device looks up the array's device address; make that
 *   first call outside any stream capture.  Synchronises `stream` before returning.
 * Errors: as gwq_select_outliers, plus INVALID_ARG when capacity is too small.           */
gwq_status gwq_select_outliers_static(const uint16_t* W_f16, const float* G_f32, int32_t N, int32_t K,
                                      double frac, int32_t* row_ptr, int32_t* col_idx, uint16_t* val,
                                      int64_t capacity, int64_t* nnz_host, void* stream);

/* Rows [row0, row1) of an outlier matrix as an object of its own (N = row1 - row0, same K, columns and values
 * copied, row pointers re-based).  The outlier location of Eq. "o" ranks the whole matrix, so a layer whose
 * rows are split over several GPUs is selected as a whole and then cut: every rank packs and multiplies its own
 * rows, and one all-gather of y puts the product together (the paper runs on one GPU and has no counterpart).
 *   *out: new library-owned object; S is unchanged.  Synchronises `stream`.
 * Errors: INVALID_ARG (bad object, row range outside [0, N] or empty), ALLOC, CUDA.  On error *out is NULL. */
gwq_status gwq_outliers_rows(const gwq_outliers* S, int32_t row0, int32_t row1, gwq_outliers** out, void* stream);

/* Group-wise asymmetric quantization of the non-outliers (Section 3.2, Eqs. "s", "z",
 * "q") and bit-packing.  Per (row, group of `group` consecutive k), over non-outlier
 * entries only: lo = min(0, min w), hi = max(0, max w); s = (hi - lo) / (2^bits - 1)
 * rounded up to fp16 (the paper's printed denominator 2^{b-1} is read as 2^b - 1);
 * z = clip(rint(-lo / s), 0, 2^bits - 1); q = clip(rint(w / s) + z, 0, 2^bits - 1),
 * round-half-to-even; outliers get q = z.  A group with hi == lo gets s = 1, z = 0.
 *   bits: 3 or 4 (the widths of the paper's experiments), or 2 or 8 (Eqs. "s", "z", "q" hold for any b).
 *   group: 16 (the value Section 3.2 names), 32, 64 or 128; K a multiple of 32 and of group.  Which kernel of gwq_linear serves a layer depends on its shape: with K a multiple of 128 (up to
 *      65536) the streaming kernels take groups of 128 up to 32 tokens, of 64 up to 16, of 32 up to 4 and of 16
 *      for one token; with K a multiple of 64 the tensor-core kernel takes every group size and token count;
 *      anything else is served by a general (slow) kernel.
 *   W_f16: device, caller-owned, read only.
 *   S: from gwq_select_outliers with the same N, K; on success its ownership moves into
 *      *out (do not free it separately); on failure it stays with the caller.
 *   *out: new library-owned packed layer.  Synchronises `stream` before returning.
 * Errors: INVALID_ARG, UNSUPPORTED (bits, group, K % group, K > 131072), NONFINITE (W has
 *   inf/NaN), ALLOC, CUDA.  On error *out is NULL.                                       */
gwq_status gwq_pack(const uint16_t* W_f16, gwq_outliers* S, int32_t N, int32_t K, int32_t bits,
                    int32_t group, gwq_packed** out, void* stream);

/* Forward product y = x (s (q - z) + S)^T (Section 3.2, Eq. "w", outliers in FP16).
 *   x: device [M, K], fp16 or bf16 (x_dtype).  y: device [M, N], y_dtype one of
 *   F16 / BF16 / F32.  Accumulation is FP32.  M >= 1.  Up to 32 tokens take a bandwidth-bound streaming
 *   kernel (mma.sync; with a workspace, 17 to 32 fp16 tokens take a tcgen05 one: see gwq_linear_ws), more tokens
 *   the tensor-core kernel (TMA, tcgen05, tensor memory), which with a workspace and enough tokens (more than 256;
 *   always for layers with fewer 128-row tiles than the device has SMs) expands the weights once instead of
 *   once per token tile and contracts on pairs of CTAs (tcgen05 cta_group::2, tiles of 256 features x 256 tokens).
 *   Asynchronous on `stream`: the call only enqueues kernels.  It never allocates and never
 *   synchronises, so it may be captured into a CUDA graph from its first use.  Calls that share P
 *   must be enqueued on one stream (or otherwise ordered): with 9 to 32 tokens they share a small
 *   scratch buffer that gwq_pack created inside P.
 *   A call that cannot do without scratch (bf16 activations on the tensor-core path need an fp16 copy of
 *   x) returns GWQ_ERR_WORKSPACE and does nothing: make it through gwq_linear_ws.  Calls that merely run
 *   faster with scratch take their slower kernel here.
 * Errors: INVALID_ARG, UNSUPPORTED (x_dtype F32), WORKSPACE, CUDA (launch failure).      */
gwq_status gwq_linear(const gwq_packed* P, const void* x, gwq_dtype x_dtype, int32_t M, void* y,
                      gwq_dtype y_dtype, void* stream);

/* gwq_linear with scratch memory supplied by the caller.  gwq_linear_workspace_bytes returns the bytes
 * the product (P, x_dtype, M) needs (0 when it needs none); `workspace` must be a device buffer of at
 * least that size, 256-byte aligned, and must not be used by anything else until the kernels enqueued by
 * the call have finished (calls on one stream may share it).  Otherwise exactly gwq_linear.
 * Errors: as gwq_linear; WORKSPACE when workspace_bytes is too small or the buffer is misaligned.  */
size_t gwq_linear_workspace_bytes(const gwq_packed* P, gwq_dtype x_dtype, int32_t M);
gwq_status gwq_linear_ws(const gwq_packed* P, const void* x, gwq_dtype x_dtype, int32_t M, void* y,
                         gwq_dtype y_dtype, void* workspace, size_t workspace_bytes, void* stream);

/* Several forward products that read the same activations, in one call: y[i] = x (deq(P[i]) + S_i)^T for
 * i < count.  This is launch-level fusion of sibling projections (q | k | v, or gate | up, of a decoder
 * block: Section 4.2, "Model Efficiency Comparison", times whole-model generation, where these run back to back); each product is
 * exactly the one gwq_linear computes, bit for bit.
 *   P: host array of `count` packed layers (1 <= count <= GWQ_MULTI_MAX) with the same K.
 *   x: device [M, K]; y: host array of `count` device pointers, y[i] is [M, P[i]->N], all of y_dtype.
 *   With M <= 32, one group size (64 or 128) and one bit width for all layers, the products run as ONE kernel
 *   launch wherever the streaming kernel takes that shape (layer 0 lends its scratch: do not overlap with
 *   another call that uses P[0]); otherwise the call is the same as `count` calls of gwq_linear in order
 *   (and like them returns GWQ_ERR_WORKSPACE where a product needs scratch: call gwq_linear_ws per layer
 *   then).  Asynchronous on `stream`; never allocates, never synchronises.
 * Errors: INVALID_ARG (count, null entries, differing K, alignment), otherwise as gwq_linear.          */
#define GWQ_MULTI_MAX 4
gwq_status gwq_linear_multi(const gwq_packed* const* P, int32_t count, const void* x, gwq_dtype x_dtype,
                            int32_t M, void* const* y, gwq_dtype y_dtype, void* stream);

/* Mean of the gradients of `count` calibration samples (Section 4.3, "Effect on Number of Calibration":
 * the outliers are located on the gradient mean); the result feeds gwq_select_outliers.
 * G_mean[i] = (((G_0[i] + G_1[i]) + G_2[i]) + ...) / count, FP32, additions in sample order, round to
 * nearest, one division: reproducible bit for bit.
 *   G_list: host array of `count` device pointers (1 <= count <= GWQ_GRAD_SAMPLES_MAX), each [numel] fp32.
 *   G_mean: device [numel] fp32, caller-owned; may be one of the inputs.  Asynchronous on `stream`.
 * Errors: INVALID_ARG, CUDA.                                                                          */
#define GWQ_GRAD_SAMPLES_MAX 16
gwq_status gwq_gradient_mean(const float* const* G_list, int32_t count, int64_t numel, float* G_mean,
                             void* stream);

/* The two objectives the method states for a quantized layer (Section 3.1): the squared error
 * ||W - W_Q||_2^2 (Eq. "Q") and the first-order change of the loss g^T (W - W_Q) (Eq. "Taylor",
 * Eq. "final_OPO"), with W_Q = s (q - z) + S as gwq_linear uses it.  Terms and sums in FP64, in a fixed
 * order.  W_f16 [N,K], G_f32 [N,K]: device, the arrays P was made from (any other pair of that shape gives
 * the same formulas on them).  *sq_err, *first_order: host.  Allocates 16 N bytes for the call,
 * synchronises `stream`.  Errors: INVALID_ARG, ALLOC, CUDA.                                             */
gwq_status gwq_quality(const uint16_t* W_f16, const float* G_f32, const gwq_packed* P, double* sq_err,
                       double* first_order, void* stream);

/* Same product with HOST buffers: copies x_host [M,K] to a staging buffer kept inside P,
 * runs gwq_linear, copies y back into y_host [M,N] and synchronises `stream`.
 * For best copy speed the host buffers should be page-locked.  The staging buffers (and the scratch
 * of gwq_linear_ws, where needed) grow on demand (cudaMalloc) and are shared by all calls on P: not
 * re-entrant per P.                                                                    */
gwq_status gwq_linear_host(gwq_packed* P, const void* x_host, gwq_dtype x_dtype, int32_t M,
                           void* y_host, gwq_dtype y_dtype, void* stream);

/* gwq_linear_host without the final synchronisation: the copy of x, the product and the copy of y are
 * enqueued on `stream` and the call returns; y_host is valid, and x_host may be reused, once the caller
 * has synchronised the stream (one synchronisation can serve many calls).  Calls that share P must be
 * on one stream (they share P's staging buffers, and stream order keeps them apart).  Use page-locked
 * host buffers, or the copies are not asynchronous.  A call that has to grow the staging buffers
 * synchronises the stream and allocates.  Errors: as gwq_linear_host.                              */
gwq_status gwq_linear_host_async(gwq_packed* P, const void* x_host, gwq_dtype x_dtype, int32_t M,
                                 void* y_host, gwq_dtype y_dtype, void* stream);

/* Device-side status of the gwq_linear calls made on P so far: synchronises `stream`, returns
 * GWQ_OK or the error a kernel recorded (GWQ_ERR_TIMEOUT when a bounded wait inside the
 * tensor-core path ran out and the kernel returned early; y is then undefined, and later
 * tensor-core calls on P do no work until the status has been read) and clears it.            */
gwq_status gwq_device_status(const gwq_packed* P, void* stream);

/* Diagnostic, no counterpart in the paper: the number of SM clock cycles a bounded device-side wait of the
 * tensor-core path may spin before the kernel gives up with GWQ_ERR_TIMEOUT (default: 10^9, about half a
 * second).  cycles < 0 restores the default; 0 makes the first wait that is not satisfied at once give up,
 * which lets a test walk the give-up path (the kernel drains what it has in flight, frees its tensor memory
 * and returns) without any fault.  Takes effect for the calls on P made afterwards.
 * Errors: INVALID_ARG.                                                                              */
gwq_status gwq_set_wait_limit(gwq_packed* P, int64_t cycles);

/* Releases a gwq_outliers* or a gwq_packed* (and everything it owns).  NULL is a no-op. */
void gwq_free(void* obj);

/* Static, NUL-terminated name of a status code.                                        */
const char* gwq_status_string(gwq_status s);

#ifdef __cplusplus
}
#endif
#endif /* GWQ_H_ */
