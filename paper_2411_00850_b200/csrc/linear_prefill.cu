// Prefill path (M > 32) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w"): a dense contraction
// on the 5th-generation tensor cores.
//
// One CTA computes a tile of 128 output features x TOK tokens.  The weight rows are the M side
// of the MMA (A operand), the tokens its N side (B operand); both are K-major in shared memory
// in the 128-byte-swizzled layout, the FP32 accumulator lives in tensor memory.
//   warp 0, one thread : TMA loads of the activation tile (TOK x 64) per k-block
//   warp 1, one thread : tcgen05.mma (4 x K=16 per k-block), tcgen05.commit frees the stage
//   warps 2..13        : 3 groups of 4 warps, group g taking the k-blocks g, g+3, ...; in a group
//                        one thread per weight row: packed codes from global memory -> exact
//                        q - z by a magic-number subtract -> times the group scale -> 128 bytes
//                        of the swizzled A tile; the row's CSR outliers are written over their
//                        (exactly zero) dense entries, so the tensor cores also do the SpMM;
//   warps 14..17       : epilogue, one thread per output feature: tcgen05.ld, conversion, stores
// The CTAs are persistent (one per SM, tiles handed out round-robin) and keep two accumulators in
// tensor memory, so the epilogue of a tile runs under the main loop of the next one.
// The tensor cores always run in fp16: bf16 activations are first rewritten, one pass, as
// fp16 x 2^-e with one power of two per token (exact for every element within 2^-14 of the
// token's largest, i.e. for everything that matters), because weights rounded to bf16 (8 bits)
// cannot meet the 1e-3 tolerance when a few activation channels dominate a sum; the epilogue
// multiplies the token's column by 2^e again.  fp16 also keeps the FP16 outliers exact.
// Stages are handed over with mbarriers; every wait is bounded and, when it runs out, the CTA
// records GWQ_ERR_TIMEOUT, leaves its loops, frees its tensor memory and returns.
#include "tc_common.cuh"

namespace {
using namespace gwq_tc;

constexpr int kTileN = 128;      // weight rows per CTA (UMMA M)
constexpr int kBlockK = 64;      // k-block: 128 bytes of 16-bit operands
constexpr int kDequantWarps = 4;   // warps of one dequantisation group (one thread per tile row)
constexpr int kDequantGroups = 3;  // groups; group g takes the k-blocks g, g + 3, ... (numbered over all tiles)
constexpr int kEpilogueWarps = 4;  // one thread per tile row
constexpr int kCtaThreads = 32 * (2 + kDequantWarps * kDequantGroups + kEpilogueWarps);
constexpr int kMaxStages = 8;

struct PrefillArgs {
  const uint32_t* codes;
  const uint16_t* scales;
  const uint8_t* zeros;
  const int32_t* row_ptr;
  const uint32_t* sz_t; // [K/group][N]: scale fp16 bits | zero-point << 16
  const uint32_t* cv;   // per outlier: fp16 value << 16 | column
  void* y;
  gwq_dtype yd;
  int32_t* status;
  const float* tok_scale;   // per token 2^e, or null (activations were fp16 already)
  int N, K, M, group;
  long long wait_cycles;    // limit of every hand-over wait (the waits of the give-up path keep the default)
};

// bf16 [M,K] -> fp16 [M,K] scaled per token row by a power of two that puts the row's largest
// magnitude just below 2^15; tok_scale[m] receives the inverse factor.  One CTA per token.
__global__ void __launch_bounds__(256) bf16_rows_to_scaled_f16(const uint16_t* __restrict__ x, uint16_t* __restrict__ x16,
                                                               float* __restrict__ tok_scale, int K) {
  __shared__ float red[8];
  const uint16_t* row = x + (size_t)blockIdx.x * K;
  uint16_t* out = x16 + (size_t)blockIdx.x * K;
  unsigned amax = 0;   // largest |x| as a bf16 bit pattern (monotone in magnitude)
  for (int i = threadIdx.x; i < K / 8; i += 256) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(row) + i);
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      amax = max(amax, w[j] & 0x7FFFu);
      amax = max(amax, (w[j] >> 16) & 0x7FFFu);
    }
  }
  for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = __uint_as_float(amax);
  __syncthreads();
  for (int w = 0; w < 8; ++w) amax = max(amax, __float_as_uint(red[w]));
  // exponent of the largest magnitude (non-finite inputs keep e = 0 and simply propagate)
  const int ex = (int)(amax >> 7) & 0xFF;
  int e = (ex == 0 || ex == 0xFF) ? 0 : ex - 127 - 14;
  e = max(-100, min(100, e));
  const float down = __uint_as_float((unsigned)(127 - e) << 23);   // 2^-e
  if (threadIdx.x == 0) tok_scale[blockIdx.x] = __uint_as_float((unsigned)(127 + e) << 23);
  for (int i = threadIdx.x; i < K / 8; i += 256) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(row) + i);
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
    unsigned o4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = __uint_as_float(w[j] << 16) * down, hi = __uint_as_float(w[j] & 0xFFFF0000u) * down;
      const __half2 h = __floats2half2_rn(lo, hi);
      o4[j] = *reinterpret_cast<const unsigned*>(&h);
    }
    reinterpret_cast<uint4*>(out)[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
  }
}


// Packed words of one row for one k-block (8 words for 4 bits, 6 for 3 bits) with the widest loads
// the alignment allows: a thread reads its own row, so every load instruction of a warp touches 32
// different lines, and the number of load instructions is what the load pipe pays for.
template <int WPB>
__device__ __forceinline__ void load_words(const uint32_t* __restrict__ p, unsigned (&w)[WPB]) {
  if (WPB == 8) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(p)), b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4 % WPB] = b.x; w[5 % WPB] = b.y; w[6 % WPB] = b.z; w[7 % WPB] = b.w;
  } else {   // 24 bytes, 8-byte aligned
    const uint2 a = __ldg(reinterpret_cast<const uint2*>(p)), b = __ldg(reinterpret_cast<const uint2*>(p) + 1),
                c = __ldg(reinterpret_cast<const uint2*>(p) + 2);
    w[0] = a.x; w[1] = a.y; w[2] = b.x; w[3] = b.y; w[4] = c.x; w[5] = c.y;
  }
}

template <bool BF16>
__device__ __forceinline__ unsigned mul_scale(unsigned d, unsigned s_hi2, unsigned s_lo2) {
  if (BF16) {
    // s = s_hi + s_lo exactly (both bf16): d s_hi + (d s_lo) keeps the bits of s that bf16 alone would drop
    const __nv_bfloat162 dd = *reinterpret_cast<const __nv_bfloat162*>(&d);
    const __nv_bfloat162 r = __hfma2(dd, *reinterpret_cast<const __nv_bfloat162*>(&s_hi2),
                                     __hmul2(dd, *reinterpret_cast<const __nv_bfloat162*>(&s_lo2)));
    return *reinterpret_cast<const unsigned*>(&r);
  } else {
    const __half2 r = __hmul2(*reinterpret_cast<const __half2*>(&d), *reinterpret_cast<const __half2*>(&s_hi2));
    return *reinterpret_cast<const unsigned*>(&r);
  }
}
template <bool BF16>
__device__ __forceinline__ unsigned sub_magic(unsigned qm, unsigned zm) {
  if (BF16) {
    const __nv_bfloat162 r =
        __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&qm), *reinterpret_cast<const __nv_bfloat162*>(&zm));
    return *reinterpret_cast<const unsigned*>(&r);
  } else {
    const __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&qm), *reinterpret_cast<const __half2*>(&zm));
    return *reinterpret_cast<const unsigned*>(&r);
  }
}

// EXP: the weights have been expanded to fp16 [N, K] beforehand (expand_kernel): the producer loads the weight tile
// by TMA as well and the dequantisation warps have nothing to do.
// GPK: scale groups per 64-column k-block: 1 (groups of 64 and 128), 2 (groups of 32), 4 (groups of 16).
template <int BITS, int TOK, bool BF16, bool EXP, int GPK>
__global__ void __launch_bounds__(kCtaThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmw, const PrefillArgs p,
               const int stages, const int ntn, const int ntiles) {
  constexpr int kABytes = kTileN * kBlockK * 2;   // 16 KB
  constexpr int kBBytes = TOK * kBlockK * 2;
  constexpr int kAccCols = TOK < 32 ? 32 : TOK;   // tensor-memory columns of one accumulator
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* tiles =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) unsigned long long bars[3 * kMaxStages + 5];
  __shared__ unsigned tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nkb = p.K / kBlockK;
  const unsigned bar0 = smem_u32(bars);
  auto full_b = [&](int s) { return bar0 + 8u * s; };
  auto full_a = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto empty = [&](int s) { return bar0 + 8u * (2 * kMaxStages + s); };
  auto acc_full = [&](int a) { return bar0 + 8u * (3 * kMaxStages + a); };
  auto acc_empty = [&](int a) { return bar0 + 8u * (3 * kMaxStages + 2 + a); };
  const unsigned drain_bar = bar0 + 8u * (3 * kMaxStages + 4);   // give-up path: completion of the MMAs in flight
  const long long lim = p.wait_cycles;
  auto a_tile = [&](int s) { return tiles + (size_t)s * (kABytes + kBBytes); };
  auto b_tile = [&](int s) { return tiles + (size_t)s * (kABytes + kBBytes) + kABytes; };
  // this CTA's tiles: blockIdx.x, blockIdx.x + gridDim.x, ...; the feature tile runs fastest, so the CTAs
  // that are busy at the same time share their activation rows in L2
  const int my_tiles = blockIdx.x < ntiles ? (ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (tid == 0) {
    abort_s = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_b(s), 1);
      mbar_init(full_a(s), kDequantWarps);
      mbar_init(empty(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full(a), 1);
      mbar_init(acc_empty(a), kEpilogueWarps);
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor memory: two accumulators of kAccCols columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                 "r"(2 * kAccCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_acc = tmem_base_s;
  bool ok = *reinterpret_cast<volatile int32_t*>(p.status) == 0;   // an earlier CTA gave up: do no work
  int issued = 0;   // k-block copies started (producer thread only), counted over all tiles

  if (warp == 0) {
    // ------------------------------------------------------------------ activation tiles by TMA
    if (lane == 0) {
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const int tile = blockIdx.x + ti * gridDim.x;
        const int m0 = (tile / ntn) * TOK;
        for (int kb = 0; kb < nkb && ok; ++kb) {
          const int it = ti * nkb + kb, s = it % stages, round = it / stages;
          if (round > 0) ok = mbar_wait(empty(s), (round - 1) & 1, abort_flag, lim);
          if (!ok) break;
          mbar_expect_tx(full_b(s), EXP ? kBBytes + kABytes : kBBytes);
          tma_load_2d(smem_u32(b_tile(s)), &tmx, kb * kBlockK, m0, full_b(s));
          if (EXP) tma_load_2d(smem_u32(a_tile(s)), &tmw, kb * kBlockK, (tile % ntn) * kTileN, full_b(s));
          issued = it + 1;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      // instruction descriptor: FP32 accumulate, A and B both fp16 or both bf16, K-major, N = TOK, M = 128
      const unsigned idesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) |
                             ((unsigned)(TOK >> 3) << 17) | ((unsigned)(kTileN >> 4) << 24);
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const int a = ti & 1;
        if (ti >= 2) ok = mbar_wait(acc_empty(a), ((ti >> 1) - 1) & 1, abort_flag, lim);   // drained by the epilogue
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned acc = tmem_acc + (unsigned)(a * kAccCols);
        for (int kb = 0; kb < nkb && ok; ++kb) {
          const int it = ti * nkb + kb, s = it % stages, round = it / stages;
          ok = (EXP || mbar_wait(full_a(s), round & 1, abort_flag, lim)) && mbar_wait(full_b(s), round & 1, abort_flag, lim);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t da = umma_desc(smem_u32(a_tile(s))), db = umma_desc(smem_u32(b_tile(s)));
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)   // 32 bytes further along K inside the swizzle atom
            umma_f16(acc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0);
          umma_commit(empty(s));
        }
        if (ok) umma_commit(acc_full(a));
      }
    }
  } else if (warp < 2 + kDequantWarps * kDequantGroups) {
    // ------------------------------------------------------------------ dequantisation
    constexpr int G = kDequantGroups;
    const int gq = (warp - 2) >> 2;            // group: global k-block numbers gq, gq + G, ...
    const int r = (warp & 3) * 32 + lane;      // row inside the tile
    constexpr int WPB = kBlockK * BITS / 32;   // packed words per row per k-block (8 or 6)
    constexpr unsigned MAGIC = BF16 ? 0x43004300u : 0x64006400u;   // 128.0 / 1024.0: ulp = 1
    constexpr int kOutWin = 8;                 // outliers of the row kept this many entries ahead
    for (int ti = 0; ti < (EXP ? 0 : my_tiles) && ok; ++ti) {
      const int tile = blockIdx.x + ti * gridDim.x;
      const int row = (tile % ntn) * kTileN + r;
      const bool live = row < p.N;
      const int rowc = live ? row : p.N - 1;
      const uint32_t* crow = p.codes + (size_t)rowc * (p.K / 32) * BITS;
      const uint32_t* szcol = p.sz_t + rowc;   // [group][row] table: neighbouring rows are neighbouring words
      int j = 0, je = 0;
      if (live) {
        j = p.row_ptr[row];
        je = p.row_ptr[row + 1];
      }
      unsigned win[kOutWin];
#pragma unroll
      for (int i = 0; i < kOutWin; ++i) win[i] = j + i < je ? __ldg(p.cv + j + i) : 0xFFFFFFFFu;
      // first k-block of this tile that belongs to the group
      int kb = ((gq - ti * nkb) % G + G) % G;
      unsigned wq[WPB];
      unsigned sz_nx[GPK];   // scale (fp16 bits) | zero-point << 16 of the groups of the next k-block
#pragma unroll
      for (int g = 0; g < GPK; ++g) sz_nx[g] = 0;
      if (kb < nkb) {
        load_words<WPB>(crow + (size_t)kb * WPB, wq);
#pragma unroll
        for (int g = 0; g < GPK; ++g) sz_nx[g] = __ldg(szcol + (size_t)((kb * kBlockK) / p.group + g) * p.N);
      }
      for (; kb < nkb && ok; kb += G) {
        const int it = ti * nkb + kb, s = it % stages, round = it / stages;
        unsigned s_hi2[GPK], s_lo2[GPK], zm[GPK];   // per group of the k-block; pair h belongs to group h GPK / 32
#pragma unroll
        for (int g = 0; g < GPK; ++g) {
          const float sc = live ? __half2float(__ushort_as_half((unsigned short)(sz_nx[g] & 0xFFFFu))) : 0.f;
          s_lo2[g] = 0;
          if (BF16) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(sc);
            const __nv_bfloat16 lo = __float2bfloat16_rn(sc - __bfloat162float(hi));
            s_hi2[g] = (unsigned)__bfloat16_as_ushort(hi) * 0x00010001u;
            s_lo2[g] = (unsigned)__bfloat16_as_ushort(lo) * 0x00010001u;
          } else {
            s_hi2[g] = (unsigned)__half_as_ushort(__float2half_rn(sc)) * 0x00010001u;
          }
          zm[g] = MAGIC | ((sz_nx[g] >> 16) * 0x00010001u);
        }
        unsigned cur[WPB];
#pragma unroll
        for (int i = 0; i < WPB; ++i) cur[i] = wq[i];
        if (kb + G < nkb) {   // codes, scale and zero-point of this group's next k-block
          load_words<WPB>(crow + (size_t)(kb + G) * WPB, wq);
#pragma unroll
          for (int g = 0; g < GPK; ++g) sz_nx[g] = __ldg(szcol + (size_t)(((kb + G) * kBlockK) / p.group + g) * p.N);
        }
        // 64 codes -> 32 pairs (columns 2h, 2h+1) -> 8 chunks of 16 bytes
        unsigned out[32];
        if (BITS == 4) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
              out[4 * i + q4] = mul_scale<BF16>(
                  sub_magic<BF16>(((cur[i % WPB] >> (4 * q4)) & 0x000F000Fu) | MAGIC, zm[(4 * i + q4) * GPK / 32]),
                  s_hi2[(4 * i + q4) * GPK / 32], s_lo2[(4 * i + q4) * GPK / 32]);
        } else {
#pragma unroll
          for (int run = 0; run < 2; ++run) {
            const unsigned* w3 = cur + (run * 3) % WPB;
#pragma unroll
            for (int i = 0; i < 3; ++i)
#pragma unroll
              for (int pp = 0; pp < 5; ++pp)
                out[16 * run + 5 * i + pp] =
                    mul_scale<BF16>(sub_magic<BF16>(((w3[i] >> (3 * pp)) & 0x00070007u) | MAGIC,
                                                    zm[(16 * run + 5 * i + pp) * GPK / 32]),
                                    s_hi2[(16 * run + 5 * i + pp) * GPK / 32], s_lo2[(16 * run + 5 * i + pp) * GPK / 32]);
            const unsigned last =
                ((w3[0] >> 15) & 0x00010001u) | ((w3[1] >> 14) & 0x00020002u) | ((w3[2] >> 13) & 0x00040004u);
            out[16 * run + 15] = mul_scale<BF16>(sub_magic<BF16>(last | MAGIC, zm[(16 * run + 15) * GPK / 32]),
                                                 s_hi2[(16 * run + 15) * GPK / 32], s_lo2[(16 * run + 15) * GPK / 32]);
          }
        }
        if (round > 0) ok = mbar_wait_warp(empty(s), (round - 1) & 1, abort_flag, lim);
        if (!ok) break;
        unsigned char* arow = a_tile(s) + r * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<uint4*>(arow + ((c ^ (r & 7)) << 4)) =
              make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
        // the row's outliers inside this k-block replace their dense entries (which are exactly 0)
        const unsigned k_end = (unsigned)(kb + 1) * kBlockK;
        while (j < je && (win[0] & 0xFFFFu) < k_end) {   // entries of other groups' k-blocks are skipped
          const unsigned e = win[0];
          if ((e & 0xFFFFu) >= k_end - kBlockK) {
            const unsigned col = (e & 0xFFFFu) - (unsigned)kb * kBlockK;
            unsigned short v16 = (unsigned short)(e >> 16);
            if (BF16) v16 = __bfloat16_as_ushort(__float2bfloat16_rn(__half2float(__ushort_as_half(v16))));
            *reinterpret_cast<unsigned short*>(arow + ((((col >> 3) ^ (r & 7)) << 4) | ((col & 7) << 1))) = v16;
          }
          ++j;
#pragma unroll
          for (int i = 0; i + 1 < kOutWin; ++i) win[i] = win[i + 1];
          win[kOutWin - 1] = j + kOutWin - 1 < je ? __ldg(p.cv + j + kOutWin - 1) : 0xFFFFFFFFu;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(full_a(s));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one thread per output feature
    const int quad = warp & 3;                 // tensor-memory lane quarter this warp may access
    const int r = quad * 32 + lane;
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
      const int tile = blockIdx.x + ti * gridDim.x;
      const int row = (tile % ntn) * kTileN + r, m0 = (tile / ntn) * TOK;
      const bool live = row < p.N;
      const int a = ti & 1;
      ok = mbar_wait_warp(acc_full(a), (ti >> 1) & 1, abort_flag, lim);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c0 = 0; c0 < TOK; c0 += 32) {
        if (m0 + c0 >= p.M) break;             // warp-uniform
        unsigned v[32];
        tmem_ld32(tmem_acc + ((unsigned)(quad * 32) << 16) + (unsigned)(a * kAccCols + c0), v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (live) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int m = m0 + c0 + i;
            if (m < p.M) {
              float f = __uint_as_float(v[i]);
              if (p.tok_scale) f *= __ldg(p.tok_scale + m);
              const size_t idx = (size_t)m * p.N + row;
              if (p.yd == GWQ_F32) reinterpret_cast<float*>(p.y)[idx] = f;
              else if (p.yd == GWQ_F16) reinterpret_cast<__half*>(p.y)[idx] = __float2half_rn(f);
              else reinterpret_cast<__nv_bfloat16*>(p.y)[idx] = __float2bfloat16_rn(f);
            }
          }
        }
      }
      // the accumulator may be overwritten by the tile after next
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(a));
    }
  }
  if (!ok) {
    *abort_flag = 1;
    atomicExch(p.status, (int32_t)GWQ_ERR_TIMEOUT);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0 && lane == 0 && abort_s) {
    // bulk copies that were issued must land before the shared memory is given back: wait (bounded)
    // for the last phase armed on every stage
    int zero = 0;
    for (int s = 0; s < stages; ++s) {
      if (issued > s) {
        const int last_it = ((issued - 1 - s) / stages) * stages + s;   // last copy issued on stage s
        (void)mbar_wait(full_b(s), (last_it / stages) & 1, &zero, kSpinCycles);
      }
    }
  }
  if (warp == 1 && lane == 0 && abort_s) {
    // MMAs that were issued may still read the stages and write tensor memory: one more commit arrives when all
    // of them have completed; wait (bounded) for it before the tensor memory is freed
    int zero = 0;
    umma_commit(drain_bar);
    (void)mbar_wait(drain_bar, 0, &zero, kSpinCycles);
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(2 * kAccCols) : "memory");
  }
}

// Two-phase path for many tokens: every token tile of the fused kernel expands the same weights again (M / 256
// times), so beyond a few tiles the weights are expanded once, to fp16 [N, K] in the caller's workspace (the same
// values the fused kernel writes into its tiles: exact q - z, one fp16 rounding of the product with the scale, the
// FP16 outliers over their zero entries), and the contraction streams both operands by TMA.
template <int BITS>
__global__ void __launch_bounds__(256) expand_kernel(const uint32_t* __restrict__ codes, const uint32_t* __restrict__ sz_t,
                                                     uint16_t* __restrict__ w16, int N, int K, int group) {
  const int runs = K >> 5;                                   // runs of 32 columns per row
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= (long long)N * runs) return;
  const int row = (int)(i / runs), run = (int)(i % runs);
  const uint32_t* src = codes + ((size_t)row * runs + run) * BITS;
  unsigned w[BITS];
  if (BITS == 4) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[BITS - 1] = v.w;
  } else {
#pragma unroll
    for (int k = 0; k < BITS; ++k) w[k] = __ldg(src + k);
  }
  // scale and zero-point of the run's two halves of 16 columns (one group unless the groups are 16 wide)
  unsigned s2[2], zm[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const unsigned sz = __ldg(sz_t + (size_t)((run * 32 + 16 * h) / group) * N + row);
    s2[h] = (sz & 0xFFFFu) * 0x00010001u;
    zm[h] = 0x64006400u | ((sz >> 16) * 0x00010001u);
  }
  unsigned out[16];   // pair p (columns 2p, 2p+1 of the run) belongs to half p / 8
  if (BITS == 4) {
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        out[4 * t + j] = mul_scale<false>(sub_magic<false>(((w[t % BITS] >> (4 * j)) & 0x000F000Fu) | 0x64006400u, zm[t / 2]),
                                          s2[t / 2], 0);
  } else {
#pragma unroll
    for (int k = 0; k < 3; ++k)
#pragma unroll
      for (int pp = 0; pp < 5; ++pp)
        out[5 * k + pp] = mul_scale<false>(sub_magic<false>(((w[k] >> (3 * pp)) & 0x00070007u) | 0x64006400u, zm[(5 * k + pp) / 8]),
                                           s2[(5 * k + pp) / 8], 0);
    const unsigned last = ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[BITS - 1] >> 13) & 0x00040004u);
    out[15] = mul_scale<false>(sub_magic<false>(last | 0x64006400u, zm[1]), s2[1], 0);
  }
  uint4* dst = reinterpret_cast<uint4*>(w16 + (size_t)row * K + run * 32);
#pragma unroll
  for (int c = 0; c < 4; ++c) dst[c] = make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
}
// the FP16 outliers over their (exactly zero) expanded entries; one warp per row
__global__ void __launch_bounds__(256) expand_outliers_kernel(const int32_t* __restrict__ row_ptr, const uint32_t* __restrict__ cv,
                                                              uint16_t* __restrict__ w16, int N, int K) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= N) return;
  uint16_t* dst = w16 + (size_t)row * K;
  for (int j = row_ptr[row] + (threadIdx.x & 31); j < row_ptr[row + 1]; j += 32) {
    const unsigned e = __ldg(cv + j);
    dst[e & 0xFFFFu] = (uint16_t)(e >> 16);
  }
}

template <int BITS, int TOK, bool EXP, int GPK = 1>
gwq_status launch(const gwq_packed* P, const void* x, const float* tok_scale, const void* w16, int M, void* y, gwq_dtype yd,
                  cudaStream_t stream) {
  constexpr bool BF16 = false;   // operands are always fp16 here (see the file header)
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  EncodeTiledFn enc = encode_fn();
  if (!enc) return GWQ_ERR_CUDA;
  CUtensorMap tmx, tmw;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)P->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)P->K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)TOK};
    if (enc(&tmx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  tmw = tmx;
  if (EXP) {
    const cuuint64_t dims[2] = {(cuuint64_t)P->K, (cuuint64_t)P->N};
    const cuuint64_t strides[1] = {(cuuint64_t)P->K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileN};
    if (enc(&tmw, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(w16), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  const int stage_bytes = kTileN * kBlockK * 2 + TOK * kBlockK * 2;
  int stages = (220 * 1024 - 1024) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  if (cudaFuncSetAttribute(prefill_kernel<BITS, TOK, BF16, EXP, GPK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return GWQ_ERR_CUDA;
  PrefillArgs a;
  a.codes = P->codes; a.scales = P->scales; a.zeros = P->zeros; a.row_ptr = P->S->row_ptr; a.cv = pv->cv; a.sz_t = pv->sz_t;
  a.y = y; a.yd = yd; a.status = pv->dev_status; a.tok_scale = tok_scale; a.N = P->N; a.K = P->K; a.M = M; a.group = P->group;
  a.wait_cycles = pv->wait_cycles;
  const int ntn = (P->N + kTileN - 1) / kTileN, ntiles = ntn * ((M + TOK - 1) / TOK);
  const int grid = ntiles < pv->sm_count ? ntiles : pv->sm_count;   // persistent: at most one CTA per SM
  prefill_kernel<BITS, TOK, BF16, EXP, GPK><<<grid, kCtaThreads, smem, stream>>>(tmx, tmw, a, stages, ntn, ntiles);
  return cudaGetLastError() == cudaSuccess ? GWQ_OK : GWQ_ERR_CUDA;
}

template <int BITS>
gwq_status launch_tok(const gwq_packed* P, const void* x, const float* tok_scale, int M, void* y, gwq_dtype yd,
                      cudaStream_t stream) {
  if (P->group == 32) {   // small groups: the smallest and the largest token tile only
    if (M <= 32) return launch<BITS, 32, false, 2>(P, x, tok_scale, nullptr, M, y, yd, stream);
    return launch<BITS, 256, false, 2>(P, x, tok_scale, nullptr, M, y, yd, stream);
  }
  if (P->group == 16) {
    if (M <= 32) return launch<BITS, 32, false, 4>(P, x, tok_scale, nullptr, M, y, yd, stream);
    return launch<BITS, 256, false, 4>(P, x, tok_scale, nullptr, M, y, yd, stream);
  }
  if (M <= 32) return launch<BITS, 32, false>(P, x, tok_scale, nullptr, M, y, yd, stream);
  if (M <= 64) return launch<BITS, 64, false>(P, x, tok_scale, nullptr, M, y, yd, stream);
  if (M <= 128) return launch<BITS, 128, false>(P, x, tok_scale, nullptr, M, y, yd, stream);
  return launch<BITS, 256, false>(P, x, tok_scale, nullptr, M, y, yd, stream);
}

// Tokens from which the weights are expanded once instead of once per token tile.  The expansion costs a pass of
// 2.5 bytes per weight (about 40 us for 11008 x 4096) and the two-operand contraction is faster per tile than the
// fused kernel only with 256-token tiles (128-token tiles ask L2 for 114 bytes per clock and SM); measured, bf16
// activations, 4 bit: 835 against 731 TFLOP/s at 2048 tokens and 1044 against 895 at 8192 on 11008 x 4096, 796
// against 693 and 1105 against 906 on 4096 x 11008; at 512 and 1024 tokens the fused kernel is level or ahead.
constexpr int kExpandMinTokens = 2048;

// Expanded weights: the expansion, the outliers over it, then the contraction with token tiles of 256.
gwq_status launch_expanded(const gwq_packed* P, const void* x, const float* tok_scale, uint16_t* w16, int M, void* y,
                           gwq_dtype yd, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const long long runs = (long long)P->N * (P->K / 32);
  if (P->bits == 4)
    expand_kernel<4><<<(unsigned)((runs + 255) / 256), 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group);
  else
    expand_kernel<3><<<(unsigned)((runs + 255) / 256), 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group);
  expand_outliers_kernel<<<(P->N + 7) / 8, 256, 0, stream>>>(P->S->row_ptr, pv->cv, w16, P->N, P->K);
  if (cudaGetLastError() != cudaSuccess) return GWQ_ERR_CUDA;
  return launch<4, 256, true>(P, x, tok_scale, w16, M, y, yd, stream);
}

}  // namespace

// Scratch of the tensor-core path: bf16 activations need an fp16 copy of x and one scale per token; from
// kExpandMinTokens tokens on, the fp16 expansion of the weights [N, K] follows.
static size_t x16_bytes(const gwq_packed* P, gwq_dtype xd, int M) {
  if (xd != GWQ_BF16) return 0;
  return (((size_t)M * P->K * 2 + 255) & ~(size_t)255) + (((size_t)M * 4 + 255) & ~(size_t)255);
}
size_t gwq_prefill_workspace_bytes(const gwq_packed* P, gwq_dtype xd, int M) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  if (!pv->cv || !pv->sz_t || P->K % kBlockK != 0) return 0;   // the general kernel needs none
  return x16_bytes(P, xd, M) + (M >= kExpandMinTokens ? (((size_t)P->N * P->K * 2 + 255) & ~(size_t)255) : 0);
}

// Prefill launcher: K <= 65536 (16-bit outlier columns).  Other shapes go to the general kernel.
// bf16 activations are first rewritten into the caller's workspace (fp16 copy of x and the token scales); with room
// for the expanded weights behind them, many tokens take the two-phase path, else the fused kernel.
gwq_status gwq_launch_prefill(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y, gwq_dtype yd,
                              void* ws, size_t ws_bytes, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  if (!pv->cv || !pv->sz_t || P->K % kBlockK != 0) return gwq_launch_simt(P, x, xd, M, y, yd, stream);
  const float* tok_scale = nullptr;
  const size_t xb = x16_bytes(P, xd, M);
  if ((xb > 0 && (!ws || ws_bytes < xb)) || (ws && (reinterpret_cast<uintptr_t>(ws) & 255u) != 0)) return GWQ_ERR_WORKSPACE;
  if (xd == GWQ_BF16) {
    uint16_t* x16 = static_cast<uint16_t*>(ws);
    float* ts = reinterpret_cast<float*>(static_cast<char*>(ws) + (((size_t)M * P->K * 2 + 255) & ~(size_t)255));
    bf16_rows_to_scaled_f16<<<M, 256, 0, stream>>>(static_cast<const uint16_t*>(x), x16, ts, P->K);
    if (cudaGetLastError() != cudaSuccess) return GWQ_ERR_CUDA;
    x = x16;
    tok_scale = ts;
  }
  if (M >= kExpandMinTokens && ws && ws_bytes >= gwq_prefill_workspace_bytes(P, xd, M))
    return launch_expanded(P, x, tok_scale, reinterpret_cast<uint16_t*>(static_cast<char*>(ws) + xb), M, y, yd, stream);
  if (P->bits == 4) return launch_tok<4>(P, x, tok_scale, M, y, yd, stream);
  return launch_tok<3>(P, x, tok_scale, M, y, yd, stream);
}
