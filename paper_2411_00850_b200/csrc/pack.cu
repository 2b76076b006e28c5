// Group-wise asymmetric quantization of the non-outliers and bit-packing
// (Section 3.2, Eqs. "s", "z", "q"; outliers excluded from the group range).
//
// One CTA per output row (the weights of a warp's first four passes are requested before
// anything else).  The row's outlier columns are expanded into a bitmask in
// shared memory, each warp then quantizes whole groups (min / max by shuffles, the
// scale and zero-point in FP64 so that every rounding is fixed bit for bit), codes go
// to shared memory as bytes and are finally packed into 32-bit words.
#include <new>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ bool half_bits_finite(unsigned int h) { return (h & 0x7C00u) != 0x7C00u; }

template <int GROUP>
__global__ void __launch_bounds__(kThreads)
pack_row_kernel(const uint16_t* __restrict__ W, const int32_t* __restrict__ row_ptr,
                const int32_t* __restrict__ col_idx, int K, int bits, uint32_t* __restrict__ codes,
                uint16_t* __restrict__ scales, uint8_t* __restrict__ zeros, int32_t* __restrict__ status) {
  extern __shared__ unsigned char smem[];
  unsigned int* mask = reinterpret_cast<unsigned int*>(smem);  // K/32 words
  unsigned char* q8 = smem + (K / 32) * 4;                      // K bytes
  const int row = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // A warp takes one group per pass (GROUP >= 32: GROUP / 32 consecutive elements per lane) or 32 / GROUP
  // neighbouring groups per pass (GROUP = 16: one element per lane, 16 lanes per group).
  constexpr int LPG = GROUP >= 32 ? 32 : GROUP;   // lanes per group
  constexpr int EPL = GROUP / LPG;                // consecutive elements per lane
  constexpr int GPP = 32 / LPG;                   // groups per warp and pass
  constexpr int kAhead = 4;                       // passes whose weights are requested together
  constexpr int kPassStride = (kThreads / 32) * GPP;
  const int ngroups = K / GROUP;
  const uint16_t* wrow = W + (long long)row * K;
  auto load_raw = [&](int g0) {   // this lane's EPL weights of the pass that starts at group g0
    const int g = min(g0 + lane / LPG, ngroups - 1);   // K is a multiple of 32, so every group of a pass exists
    const int c0 = g * GROUP + (lane % LPG) * EPL;
    uint2 v = make_uint2(0u, 0u);
    if (EPL == 4) v = *reinterpret_cast<const uint2*>(wrow + c0);
    else if (EPL == 2) v.x = *reinterpret_cast<const unsigned int*>(wrow + c0);
    else v.x = wrow[c0];
    return v;
  };
  // the first passes' weights are on their way while the mask is built
  uint2 raw[kAhead];
#pragma unroll
  for (int u = 0; u < kAhead; ++u) {
    const int g0 = warp * GPP + u * kPassStride;
    raw[u] = g0 < ngroups ? load_raw(g0) : make_uint2(0u, 0u);
  }
  for (int i = threadIdx.x; i < K / 32; i += kThreads) mask[i] = 0;
  __syncthreads();
  const int jb = row_ptr[row], je = row_ptr[row + 1];
  for (int j = jb + threadIdx.x; j < je; j += kThreads) {
    const int c = col_idx[j];
    if (c >= 0 && c < K) atomicOr(&mask[c >> 5], 1u << (c & 31));
  }
  __syncthreads();

  const double qmax = (double)((1 << bits) - 1);
  bool bad = false;
  auto quantize_pass = [&](const int g0, const uint2 v) {
    const int g = min(g0 + lane / LPG, ngroups - 1);
    const int c0 = g * GROUP + (lane % LPG) * EPL;
    unsigned int hb[EPL];
    if (EPL == 4) {
      hb[0] = v.x & 0xFFFFu; hb[1 % EPL] = v.x >> 16; hb[(EPL - 2 + EPL) % EPL] = v.y & 0xFFFFu; hb[EPL - 1] = v.y >> 16;
    } else if (EPL == 2) {
      hb[0] = v.x & 0xFFFFu; hb[EPL - 1] = v.x >> 16;
    } else {
      hb[0] = v.x & 0xFFFFu;
    }
    // this lane's EPL mask bits: c0 is a multiple of EPL, so they sit in one mask word
    const unsigned int mbits = (mask[c0 >> 5] >> (c0 & 31)) & ((1u << EPL) - 1u);
    float w[EPL];
    float lo = 0.f, hi = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      bad |= !half_bits_finite(hb[e]);
      w[e] = __half2float(__ushort_as_half((unsigned short)hb[e]));
      if (!((mbits >> e) & 1u)) {
        lo = fminf(lo, w[e]);
        hi = fmaxf(hi, w[e]);
      }
    }
#pragma unroll
    for (int o = LPG / 2; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    }
    __half sh = __ushort_as_half((unsigned short)0x3C00u);  // 1.0
    double z = 0.0;
    if (hi > lo) {
      const double s64 = ((double)hi - (double)lo) / qmax;
      // smallest fp16 >= s64: two directed roundings compose to one
      sh = __float2half_ru(__double2float_ru(s64));
      const double s = (double)__half2float(sh);
      z = fmin(fmax(rint(-(double)lo / s), 0.0), qmax);
    }
    // Codes: rint(w / s) with the quotient rounded to FP32 equals the same with the FP64 quotient.  w and s are fp16
    // values (integers of at most 11 bits times powers of two), so the exact quotient is either a half-integer,
    // which both formats hold exactly, or at least 2^-13 away from every half-integer, while the FP32 rounding of a
    // quotient below 1024 moves it by at most 2^-15 (non-outliers satisfy |w / s| <= 2^bits): the rounding decision
    // is the same, at a fraction of the cost of an FP64 divide per weight.
    const float sf = __half2float(sh), zf = (float)z, qmaxf = (float)qmax;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      float q = zf;
      if (!((mbits >> e) & 1u)) q = fminf(fmaxf(rintf(__fdiv_rn(w[e], sf)) + zf, 0.f), qmaxf);
      q8[c0 + e] = (unsigned char)(int)q;
    }
    if (lane % LPG == 0) {
      scales[(long long)row * ngroups + g] = __half_as_ushort(sh);
      zeros[(long long)row * ngroups + g] = (uint8_t)(int)z;
    }
  };
  for (int gb = warp * GPP; gb < ngroups; gb += kAhead * kPassStride) {
    if (gb != warp * GPP) {   // later batches (rows of more than kAhead passes per warp)
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        const int g0 = gb + u * kPassStride;
        raw[u] = g0 < ngroups ? load_raw(g0) : make_uint2(0u, 0u);
      }
    }
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      const int g0 = gb + u * kPassStride;
      if (g0 < ngroups) quantize_pass(g0, raw[u]);   // warp-uniform
    }
  }
  if (bad) atomicExch(status, (int32_t)GWQ_ERR_NONFINITE);
  __syncthreads();

  // pack (pair-interleaved order: even columns in the low half-word, odd in the high):
  //  4 bits: word j of a run holds its columns 8j..8j+7, column 8j+2p+e in bits [16e+4p, +4)
  //          (2 and 8 bits likewise: 16 / 4 columns per word, column 16j+2p+e / 4j+2p+e in bits [16e+bits p, +bits))
  //  3 bits: word j holds columns 10j..10j+9, column 10j+2p+e in bits [16e+3p, +3); bit j of the
  //          codes of columns 30 / 31 goes to bit 15 / 31 of word j
  const int nwords = K / 32 * bits;
  uint32_t* crow = codes + (long long)row * nwords;
  for (int wi = threadIdx.x; wi < nwords; wi += kThreads) {
    const int run = wi / bits, j = wi - run * bits;
    const unsigned char* r = q8 + run * 32;
    unsigned int word = 0;
    if (bits == 4) {
      const unsigned char* c = r + 8 * j;
#pragma unroll
      for (int p = 0; p < 4; ++p)
        word |= ((unsigned int)c[2 * p] << (4 * p)) | ((unsigned int)c[2 * p + 1] << (16 + 4 * p));
    } else if (bits != 3) {   // 2 and 8 bits: the 4-bit rule with 32 / bits columns per word
      const int per = 32 / bits;
      const unsigned char* c = r + per * j;
      for (int p = 0; p < per / 2; ++p)
        word |= ((unsigned int)c[2 * p] << (bits * p)) | ((unsigned int)c[2 * p + 1] << (16 + bits * p));
    } else {
      const unsigned char* c = r + 10 * j;
#pragma unroll
      for (int p = 0; p < 5; ++p)
        word |= ((unsigned int)c[2 * p] << (3 * p)) | ((unsigned int)c[2 * p + 1] << (16 + 3 * p));
      word |= (((unsigned int)r[30] >> j) & 1u) << 15;
      word |= (((unsigned int)r[31] >> j) & 1u) << 31;
    }
    crow[wi] = word;
  }
}

// Decode-side copy of the CSR payload: one 32-bit word per outlier, value << 16 | column.
__global__ void fuse_col_val_kernel(const int32_t* __restrict__ col, const uint16_t* __restrict__ val,
                                    uint32_t* __restrict__ cv, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) cv[i] = ((uint32_t)val[i] << 16) | ((uint32_t)col[i] & 0xFFFFu);
}

// Block-ordered copy of the outliers for the tcgen05 streaming kernel: the matrix is cut into blocks of 128 rows x
// 128 columns, numbered tile * (K / 128) + column block; ob_ptr[b] .. ob_ptr[b + 1] are the entries of block b, each
// packed as row-in-block << 23 | column-in-block << 16 | fp16 value.  Three passes: count, scan, fill (the order of
// the entries inside a block is whatever the atomics give; every entry has its own position, so it does not matter).
__global__ void ob_count_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col, int N, int G,
                                unsigned int* __restrict__ cnt) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= N) return;
  unsigned int* c = cnt + (size_t)(row >> 7) * G;
  for (int j = row_ptr[row]; j < row_ptr[row + 1]; ++j) atomicAdd(c + (col[j] >> 7), 1u);
}
// exclusive scan of cnt[0..n) into ptr[0..n], one block; cnt is cleared for the fill pass
__global__ void __launch_bounds__(1024) ob_scan_kernel(unsigned int* __restrict__ cnt, int32_t* __restrict__ ptr, int n) {
  __shared__ unsigned int part[1024];
  const int t = threadIdx.x;
  const int per = (n + 1023) / 1024, lo = min(n, t * per), hi = min(n, lo + per);
  unsigned int sum = 0;
  for (int i = lo; i < hi; ++i) sum += cnt[i];
  part[t] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    const unsigned int v = t >= off ? part[t - off] : 0u;
    __syncthreads();
    part[t] += v;
    __syncthreads();
  }
  unsigned int run = part[t] - sum;
  for (int i = lo; i < hi; ++i) {
    ptr[i] = (int32_t)run;
    run += cnt[i];
    cnt[i] = 0u;
  }
  if (t == 1023) ptr[n] = (int32_t)part[1023];
}
__global__ void ob_fill_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                               const uint16_t* __restrict__ val, int N, int G, const int32_t* __restrict__ ptr,
                               unsigned int* __restrict__ cursor, uint32_t* __restrict__ ob) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= N) return;
  const size_t b0 = (size_t)(row >> 7) * G;
  for (int j = row_ptr[row]; j < row_ptr[row + 1]; ++j) {
    const int c = col[j];
    const size_t b = b0 + (c >> 7);
    const unsigned int pos = atomicAdd(cursor + b, 1u);
    ob[(size_t)ptr[b] + pos] = ((uint32_t)(row & 127) << 23) | ((uint32_t)(c & 127) << 16) | (uint32_t)val[j];
  }
}

// Tensor-core-side copy of the group tables, transposed to [group][row] so that the 128 rows of a
// tile read 128 neighbouring words.
__global__ void transpose_scale_zero_kernel(const uint16_t* __restrict__ scales, const uint8_t* __restrict__ zeros,
                                            uint32_t* __restrict__ sz_t, int N, int ngroups) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // output index g * N + n
  if (i < (long long)N * ngroups) {
    const int g = (int)(i / N), n = (int)(i - (long long)g * N);
    sz_t[i] = (uint32_t)scales[(size_t)n * ngroups + g] | ((uint32_t)zeros[(size_t)n * ngroups + g] << 16);
  }
}

}  // namespace

extern "C" gwq_status gwq_pack(const uint16_t* W, gwq_outliers* S, int32_t N, int32_t K, int32_t bits,
                               int32_t group, gwq_packed** out, void* stream_) {
  if (out) *out = nullptr;
  if (!W || !S || !out || N <= 0 || K <= 0) return GWQ_ERR_INVALID_ARG;
  if (S->tag != GWQ_TAG_OUTLIERS || S->N != N || S->K != K) return GWQ_ERR_INVALID_ARG;
  if (!gwq_aligned16(W)) return GWQ_ERR_INVALID_ARG;
  if (bits != 2 && bits != 3 && bits != 4 && bits != 8) return GWQ_ERR_UNSUPPORTED;
  if (group != 16 && group != 32 && group != 64 && group != 128) return GWQ_ERR_UNSUPPORTED;
  if (K % group != 0 || K > 131072) return GWQ_ERR_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);

  gwq_status st = GWQ_OK;
  int32_t host_status = 0;
  const size_t ngroups = (size_t)N * (K / group);
  const size_t nwords = (size_t)N * (K / 32) * bits;
  const size_t smem = (size_t)(K / 32) * 4 + (size_t)K;
  gwq_packed* P = new (std::nothrow) gwq_packed();
  gwq_priv* pv = new (std::nothrow) gwq_priv();
  if (!P || !pv) {
    delete P;
    delete pv;
    return GWQ_ERR_ALLOC;
  }
  *pv = gwq_priv{};
  pv->wait_cycles = GWQ_DEFAULT_WAIT_CYCLES;
  P->tag = GWQ_TAG_PACKED;
  P->N = N; P->K = K; P->bits = bits; P->group = group;
  P->codes = nullptr; P->scales = nullptr; P->zeros = nullptr; P->S = nullptr; P->priv = pv;
  int dev = 0;
  GWQ_CUDA_TRY(cudaGetDevice(&dev));
  GWQ_CUDA_TRY(cudaDeviceGetAttribute(&pv->sm_count, cudaDevAttrMultiProcessorCount, dev));
  GWQ_CUDA_TRY(cudaMalloc(&P->codes, nwords * sizeof(uint32_t)));
  GWQ_CUDA_TRY(cudaMalloc(&P->scales, ngroups * sizeof(uint16_t) + 16));
  GWQ_CUDA_TRY(cudaMalloc(&P->zeros, ngroups + 16));
  GWQ_CUDA_TRY(cudaMalloc(&pv->dev_status, 64));
  GWQ_CUDA_TRY(cudaMemsetAsync(pv->dev_status, 0, 64, stream));
#define GWQ_PACK_LAUNCH(G)                                                                                              \
  do {                                                                                                                  \
    GWQ_CUDA_TRY(cudaFuncSetAttribute(pack_row_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));     \
    pack_row_kernel<G><<<N, kThreads, smem, stream>>>(W, S->row_ptr, S->col_idx, K, bits, P->codes, P->scales,           \
                                                      P->zeros, pv->dev_status);                                        \
  } while (0)
  if (group == 128) GWQ_PACK_LAUNCH(128);
  else if (group == 64) GWQ_PACK_LAUNCH(64);
  else if (group == 32) GWQ_PACK_LAUNCH(32);
  else GWQ_PACK_LAUNCH(16);
#undef GWQ_PACK_LAUNCH
  GWQ_CUDA_TRY(cudaGetLastError());
  if (K <= 65536) {
    const long long nnz = S->nnz;
    GWQ_CUDA_TRY(cudaMalloc(&pv->cv, (size_t)(nnz > 0 ? nnz : 1) * sizeof(uint32_t) + 16));
    if (nnz > 0) {
      fuse_col_val_kernel<<<(unsigned)((nnz + 255) / 256), 256, 0, stream>>>(S->col_idx, S->val, pv->cv, nnz);
      GWQ_CUDA_TRY(cudaGetLastError());
    }
  }
  if (K <= 65536 && group >= 64 && K % 128 == 0) {   // block-ordered outliers of the tcgen05 streaming kernel
    const long long nnz = S->nnz;
    const int G = K / 128;
    const size_t nblocks = (size_t)((N + 127) / 128) * G;
    unsigned int* cnt = nullptr;
    GWQ_CUDA_TRY(cudaMalloc(&pv->ob, (size_t)(nnz > 0 ? nnz : 1) * sizeof(uint32_t) + 16));
    GWQ_CUDA_TRY(cudaMalloc(&pv->ob_ptr, (nblocks + 1) * sizeof(int32_t)));
    GWQ_CUDA_TRY(cudaMalloc(&cnt, nblocks * sizeof(unsigned int)));
    pv->ob_scratch = cnt;   // released once the stream has been synchronised below
    GWQ_CUDA_TRY(cudaMemsetAsync(cnt, 0, nblocks * sizeof(unsigned int), stream));
    ob_count_kernel<<<(N + 255) / 256, 256, 0, stream>>>(S->row_ptr, S->col_idx, N, G, cnt);
    ob_scan_kernel<<<1, 1024, 0, stream>>>(cnt, pv->ob_ptr, (int)nblocks);
    ob_fill_kernel<<<(N + 255) / 256, 256, 0, stream>>>(S->row_ptr, S->col_idx, S->val, N, G, pv->ob_ptr, cnt, pv->ob);
    GWQ_CUDA_TRY(cudaGetLastError());
  }
  if (K <= 65536 && group >= 64 && K % 128 == 0) {   // scratch of the streaming path with more than 8 tokens
    GWQ_CUDA_TRY(cudaMalloc(&pv->xt, gwq_decode_scratch_bytes(K)));
    pv->xt_bytes = gwq_decode_scratch_bytes(K);
  }
  {   // group table of the tensor-core and streaming paths, transposed
    GWQ_CUDA_TRY(cudaMalloc(&pv->sz_t, ngroups * sizeof(uint32_t) + 16));
    transpose_scale_zero_kernel<<<(unsigned)((ngroups + 255) / 256), 256, 0, stream>>>(P->scales, P->zeros, pv->sz_t,
                                                                                       N, K / group);
    GWQ_CUDA_TRY(cudaGetLastError());
  }
  GWQ_CUDA_TRY(cudaMemcpyAsync(&host_status, pv->dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  if (pv->ob_scratch) {
    cudaFree(pv->ob_scratch);
    pv->ob_scratch = nullptr;
  }
  if (host_status != 0) {
    st = (gwq_status)host_status;
    goto fail;
  }
  GWQ_CUDA_TRY(cudaMemsetAsync(pv->dev_status, 0, 64, stream));
  P->S = S;
  *out = P;
  return GWQ_OK;
fail:
  if (P->codes) cudaFree(P->codes);
  if (P->scales) cudaFree(P->scales);
  if (P->zeros) cudaFree(P->zeros);
  if (pv->cv) cudaFree(pv->cv);
  if (pv->sz_t) cudaFree(pv->sz_t);
  if (pv->xt) cudaFree(pv->xt);
  if (pv->ob) cudaFree(pv->ob);
  if (pv->ob_ptr) cudaFree(pv->ob_ptr);
  if (pv->ob_scratch) cudaFree(pv->ob_scratch);
  if (pv->dev_status) cudaFree(pv->dev_status);
  delete pv;
  delete P;
  return st;
}
