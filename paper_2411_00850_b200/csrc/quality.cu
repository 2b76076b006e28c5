// The two objectives the method states for a quantized layer (Section 3.1), evaluated on the device:
//   squared error        ||W - W_Q||_2^2          (Eq. "Q")
//   first-order change   g^T (W - W_Q)            (Eq. "Taylor": L(W_Q) ~ L(W) - g^T (W - W_Q); Eq. "final_OPO")
// with W_Q = s (q - z) + S, the outliers S being the kept FP16 weights.  Every term is formed and
// summed in FP64 (fp16 / fp32 inputs convert exactly, s (q - z) is exact in FP64), rows are reduced in a
// fixed order, so the two numbers do not depend on scheduling.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;

// One CTA per row: thread t takes the runs of 32 columns t, t + 256, ...; outlier positions are marked in
// a bit map (one word per run) and handled from the CSR entries instead.
__global__ void __launch_bounds__(kThreads)
quality_row_kernel(const uint16_t* __restrict__ W, const float* __restrict__ G, const uint32_t* __restrict__ codes,
                   const uint16_t* __restrict__ scales, const uint8_t* __restrict__ zeros,
                   const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                   const uint16_t* __restrict__ val, int K, int bits, int group, double* __restrict__ rows) {
  extern __shared__ unsigned mask[];   // [K / 32]
  __shared__ double red[2][kThreads / 32];
  const int n = blockIdx.x, tid = threadIdx.x;
  const int nruns = K / 32, ngroups = K / group;
  const uint16_t* wrow = W + (size_t)n * K;
  const float* grow = G + (size_t)n * K;
  const uint32_t* crow = codes + (size_t)n * nruns * bits;
  for (int r = tid; r < nruns; r += kThreads) mask[r] = 0u;
  __syncthreads();
  const int jb = row_ptr[n], je = row_ptr[n + 1];
  double sq = 0.0, fo = 0.0;
  for (int j = jb + tid; j < je; j += kThreads) {
    const int c = col_idx[j];
    atomicOr(&mask[c >> 5], 1u << (c & 31));
    const double d = (double)__half2float(__ushort_as_half(wrow[c])) - (double)__half2float(__ushort_as_half(val[j]));
    sq += d * d;
    fo += (double)grow[c] * d;
  }
  __syncthreads();
  for (int r = tid; r < nruns; r += kThreads) {
    unsigned w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int j = 0; j < bits; ++j) w[j] = __ldg(crow + r * bits + j);
    const unsigned m = mask[r];
    for (int i = 0; i < 32; ++i) {
      if ((m >> i) & 1u) continue;
      // pair-interleaved packed order (see include/gwq.h)
      unsigned code;
      const int e = i & 1;
      if (bits == 4) {
        code = (w[i >> 3] >> (16 * e + 4 * ((i & 7) >> 1))) & 15u;
      } else if (bits != 3) {   // 2 and 8 bits: 32 / bits columns per word
        const int per = 32 / bits;
        code = (w[i / per] >> (16 * e + bits * ((i % per) >> 1))) & ((1u << bits) - 1u);
      } else if (i < 30) {
        const int wi = i / 10, r10 = i - 10 * wi;
        code = (w[wi] >> (16 * e + 3 * (r10 >> 1))) & 7u;
      } else {
        const int sh = 15 + 16 * e;
        code = ((w[0] >> sh) & 1u) | (((w[1] >> sh) & 1u) << 1) | (((w[2] >> sh) & 1u) << 2);
      }
      const int k = r * 32 + i, g = k / group;
      const double s = (double)__half2float(__ushort_as_half(scales[(size_t)n * ngroups + g]));
      const int z = zeros[(size_t)n * ngroups + g];
      const double d = (double)__half2float(__ushort_as_half(wrow[k])) - s * (double)((int)code - z);
      sq += d * d;
      fo += (double)grow[k] * d;
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
    fo += __shfl_xor_sync(0xFFFFFFFFu, fo, o);
  }
  if ((tid & 31) == 0) {
    red[0][tid >> 5] = sq;
    red[1][tid >> 5] = fo;
  }
  __syncthreads();
  if (tid == 0) {
    double a = 0.0, b = 0.0;
    for (int w8 = 0; w8 < kThreads / 32; ++w8) {
      a += red[0][w8];
      b += red[1][w8];
    }
    rows[2 * (size_t)n] = a;
    rows[2 * (size_t)n + 1] = b;
  }
}

// Sum of the per-row pairs in a fixed order: thread t adds rows t, t + 1024, ..., then a tree over the threads.
__global__ void __launch_bounds__(1024) quality_sum_kernel(const double* __restrict__ rows, int N, double* __restrict__ out) {
  __shared__ double sa[1024], sb[1024];
  double a = 0.0, b = 0.0;
  for (int n = threadIdx.x; n < N; n += 1024) {
    a += rows[2 * (size_t)n];
    b += rows[2 * (size_t)n + 1];
  }
  sa[threadIdx.x] = a;
  sb[threadIdx.x] = b;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) {
      sa[threadIdx.x] += sa[threadIdx.x + o];
      sb[threadIdx.x] += sb[threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    out[0] = sa[0];
    out[1] = sb[0];
  }
}

}  // namespace

extern "C" gwq_status gwq_quality(const uint16_t* W, const float* G, const gwq_packed* P, double* sq_err,
                                  double* first_order, void* stream_) {
  if (!W || !G || !P || P->tag != GWQ_TAG_PACKED || !P->S || !sq_err || !first_order) return GWQ_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  gwq_status st = GWQ_OK;
  double* rows = nullptr;
  double host[2] = {0.0, 0.0};
  const size_t smem = (size_t)(P->K / 32) * sizeof(unsigned);
  GWQ_CUDA_TRY(cudaMalloc(&rows, ((size_t)P->N * 2 + 2) * sizeof(double)));
  quality_row_kernel<<<P->N, kThreads, smem, stream>>>(W, G, P->codes, P->scales, P->zeros, P->S->row_ptr,
                                                      P->S->col_idx, P->S->val, P->K, P->bits, P->group, rows);
  GWQ_CUDA_TRY(cudaGetLastError());
  quality_sum_kernel<<<1, 1024, 0, stream>>>(rows, P->N, rows + (size_t)P->N * 2);
  GWQ_CUDA_TRY(cudaGetLastError());
  GWQ_CUDA_TRY(cudaMemcpyAsync(host, rows + (size_t)P->N * 2, sizeof(host), cudaMemcpyDeviceToHost, stream));
  GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  *sq_err = host[0];
  *first_order = host[1];
fail:
  if (rows) cudaFree(rows);
  return st;
}
