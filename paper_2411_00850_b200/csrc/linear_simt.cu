// General CUDA-core path of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w").
//
// One warp owns one output row at a time: each lane takes runs of 32 columns (the
// unit of the packed format), unpacks the codes one by one, accumulates
// sum_k x_k (q_k - z) per run in FP32 and scales it by s once per run; the row's CSR
// outliers are appended, then the lanes are reduced with shuffles.  It handles every
// M by looping over tiles of 4 tokens and serves the shapes the specialised paths do
// not take.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int MT = 4;  // tokens per pass

template <bool BF16>
__device__ __forceinline__ float ld_act(const uint16_t* p) {
  if (BF16) return __uint_as_float((unsigned int)(*p) << 16);
  return __half2float(__ushort_as_half(*p));
}

__device__ __forceinline__ void st_out(void* y, gwq_dtype yd, long long idx, float v) {
  if (yd == GWQ_F32) {
    reinterpret_cast<float*>(y)[idx] = v;
  } else if (yd == GWQ_F16) {
    reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
  } else {
    reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
  }
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads)
linear_simt_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ scales,
                   const uint8_t* __restrict__ zeros, const int32_t* __restrict__ row_ptr,
                   const int32_t* __restrict__ col_idx, const uint16_t* __restrict__ val,
                   const uint16_t* __restrict__ x, void* __restrict__ y, gwq_dtype yd, int N, int K,
                   int M, int bits, int group) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (kThreads / 32);
  const int wid = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  const int nruns = K / 32;
  const int ngroups = K / group;
  for (int row = wid; row < N; row += warps_total) {
    const uint32_t* crow = codes + (long long)row * nruns * bits;
    const int jb = row_ptr[row], je = row_ptr[row + 1];
    for (int m0 = 0; m0 < M; m0 += MT) {
      float acc[MT];
#pragma unroll
      for (int t = 0; t < MT; ++t) acc[t] = 0.f;
      const int gsz = group < 32 ? group : 32;   // columns of a run that share one scale and zero-point
      for (int r = lane; r < nruns; r += 32) {
        unsigned int w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int j = 0; j < bits; ++j) w[j] = __ldg(crow + r * bits + j);
        for (int seg = 0; seg < 32; seg += gsz) {
          const int g = (r * 32 + seg) / group;
          const float s = __half2float(__ushort_as_half(scales[(long long)row * ngroups + g]));
          const float z = (float)zeros[(long long)row * ngroups + g];
          float part[MT];
#pragma unroll
          for (int t = 0; t < MT; ++t) part[t] = 0.f;
          for (int i = seg; i < seg + gsz; ++i) {
            // pair-interleaved packed order (see include/gwq.h)
            unsigned int code;
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
            const float qz = (float)(int)code - z;
#pragma unroll
            for (int t = 0; t < MT; ++t) {
              if (m0 + t < M) part[t] = fmaf(ld_act<BF16>(x + (long long)(m0 + t) * K + r * 32 + i), qz, part[t]);
            }
          }
#pragma unroll
          for (int t = 0; t < MT; ++t) acc[t] = fmaf(s, part[t], acc[t]);
        }
      }
      for (int j = jb + lane; j < je; j += 32) {
        const float v = __half2float(__ushort_as_half(val[j]));
        const int c = col_idx[j];
#pragma unroll
        for (int t = 0; t < MT; ++t)
          if (m0 + t < M) acc[t] = fmaf(v, ld_act<BF16>(x + (long long)(m0 + t) * K + c), acc[t]);
      }
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        float v = acc[t];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == 0 && m0 + t < M) st_out(y, yd, (long long)(m0 + t) * N + row, v);
      }
    }
  }
}

}  // namespace

gwq_status gwq_launch_simt(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y,
                           gwq_dtype yd, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const int warps_per_block = kThreads / 32;
  int grid = (P->N + warps_per_block - 1) / warps_per_block;
  const int cap = pv->sm_count * 8;
  if (grid > cap) grid = cap;
  const gwq_outliers* S = P->S;
  if (xd == GWQ_BF16)
    linear_simt_kernel<true><<<grid, kThreads, 0, stream>>>(P->codes, P->scales, P->zeros, S->row_ptr, S->col_idx,
                                                            S->val, static_cast<const uint16_t*>(x), y, yd, P->N,
                                                            P->K, M, P->bits, P->group);
  else
    linear_simt_kernel<false><<<grid, kThreads, 0, stream>>>(P->codes, P->scales, P->zeros, S->row_ptr, S->col_idx,
                                                             S->val, static_cast<const uint16_t*>(x), y, yd, P->N,
                                                             P->K, M, P->bits, P->group);
  return cudaGetLastError() == cudaSuccess ? GWQ_OK : GWQ_ERR_CUDA;
}
