// Prefill path (M > 32) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w"): a dense contraction
// on the 5th-generation tensor cores, in two forms: a fused kernel that dequantises into its weight tiles (few
// tokens; described here) and, further down, a two-phase path that expands the weights once and contracts on pairs
// of CTAs.
//
// Fused kernel: one CTA computes a tile of 128 output features x TOK tokens.  The weight rows are the M side
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
#include <atomic>

#include "tc_common.cuh"

namespace {
using namespace gwq_tc;

// The kernels of the two-phase path are launched with programmatic stream serialization: each lets its successor
// start at once (griddepcontrol.launch_dependents) and waits for its predecessor to complete (griddepcontrol.wait)
// before it touches anything a kernel before it writes or still reads; what depends on the weights alone comes first.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_sync() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kTileN = 128;      // weight rows per CTA (UMMA M)
constexpr int kBlockK = 64;      // k-block: 128 bytes of 16-bit operands
constexpr int kDequantWarps = 4;   // warps of one dequantisation group (one thread per tile row)
constexpr int kDequantGroups = 3;  // groups; group g takes the k-blocks g, g + 3, ... (numbered over all tiles)
constexpr int kEpilogueWarps = 4;  // one thread per tile row
constexpr int kCtaThreads = 32 * (2 + kDequantWarps * kDequantGroups + kEpilogueWarps);
constexpr int kMaxStages = 8;   // of the fused kernel
// stages of the fused kernel's ring for a token tile: what 219 KB hold, at most kMaxStages (a compile-time constant in
// the kernel: the stage of a k-block is a remainder that every role takes per k-block)
__host__ __device__ constexpr int fused_stages(int tok) {
  return (220 * 1024 - 1024) / (128 * 64 * 2 + tok * 64 * 2) > kMaxStages ? kMaxStages
                                                                           : (220 * 1024 - 1024) / (128 * 64 * 2 + tok * 64 * 2);
}

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
  pdl_trigger();
  pdl_sync();   // x may still be being written
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


// Packed words of one row for one k-block (8 words for 4 bits, 6 for 3, 4 for 2, 16 for 8) with the widest loads
// the alignment allows: a thread reads its own row, so every load instruction of a warp touches 32
// different lines, and the number of load instructions is what the load pipe pays for.
template <int WPB>
__device__ __forceinline__ void load_words(const uint32_t* __restrict__ p, unsigned (&w)[WPB]) {
  if (WPB == 8) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(p)), b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4 % WPB] = b.x; w[5 % WPB] = b.y; w[6 % WPB] = b.z; w[7 % WPB] = b.w;
  } else if (WPB == 16 || WPB == 4) {   // 8 bits: 64 bytes; 2 bits: 16 bytes
#pragma unroll
    for (int i = 0; i < WPB / 4; ++i) {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(p) + i);
      w[(4 * i) % WPB] = a.x; w[(4 * i + 1) % WPB] = a.y; w[(4 * i + 2) % WPB] = a.z; w[(4 * i + 3) % WPB] = a.w;
    }
  } else {   // 24 bytes, 8-byte aligned
    const uint2 a = __ldg(reinterpret_cast<const uint2*>(p)), b = __ldg(reinterpret_cast<const uint2*>(p) + 1),
                c = __ldg(reinterpret_cast<const uint2*>(p) + 2);
    w[0] = a.x; w[1] = a.y; w[2 % WPB] = b.x; w[3 % WPB] = b.y; w[4 % WPB] = c.x; w[5 % WPB] = c.y;
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

// GPK: scale groups per 64-column k-block: 1 (groups of 64 and 128), 2 (groups of 32), 4 (groups of 16).
template <int BITS, int TOK, bool BF16, int GPK>
__global__ void __launch_bounds__(kCtaThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tmx, const PrefillArgs p,
               const int ntn, const int ntiles) {
  constexpr int stages = fused_stages(TOK);
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
          mbar_expect_tx(full_b(s), kBBytes);
          tma_load_2d(smem_u32(b_tile(s)), &tmx, kb * kBlockK, m0, full_b(s));
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
          ok = mbar_wait(full_a(s), round & 1, abort_flag, lim) && mbar_wait(full_b(s), round & 1, abort_flag, lim);
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
    const int gshift = __ffs(p.group) - 1;     // the group size is a power of two: no division per k-block
    for (int ti = 0; ti < my_tiles && ok; ++ti) {
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
        for (int g = 0; g < GPK; ++g) sz_nx[g] = __ldg(szcol + (size_t)(((kb * kBlockK) >> gshift) + g) * p.N);
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
          for (int g = 0; g < GPK; ++g) sz_nx[g] = __ldg(szcol + (size_t)((((kb + G) * kBlockK) >> gshift) + g) * p.N);
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
        } else if (BITS == 2 || BITS == 8) {   // pair h: word h / (16 / BITS), BITS (h % (16 / BITS)) bits up
          constexpr int PPW = 16 / BITS;
          constexpr unsigned CMASK = ((1u << BITS) - 1u) * 0x00010001u;
#pragma unroll
          for (int h = 0; h < 32; ++h)
            out[h] = mul_scale<BF16>(
                sub_magic<BF16>(((cur[(h / PPW) % WPB] >> (BITS * (h % PPW))) & CMASK) | MAGIC, zm[h * GPK / 32]),
                s_hi2[h * GPK / 32], s_lo2[h * GPK / 32]);
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
// FP16 outliers over their zero entries), and the contraction (pair_kernel) streams both operands by TMA.
// expand_kernel + expand_outliers_kernel serve the layers without a block-ordered outlier list (groups of 16 or 32,
// K not a multiple of 128); the others take expand_block_kernel.
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
    w[0] = v.x; w[1 % BITS] = v.y; w[2 % BITS] = v.z; w[3 % BITS] = v.w;
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
  } else if (BITS == 2 || BITS == 8) {
    constexpr int PPW = 16 / BITS;
    constexpr unsigned CMASK = ((1u << BITS) - 1u) * 0x00010001u;
#pragma unroll
    for (int h = 0; h < 16; ++h)
      out[h] = mul_scale<false>(sub_magic<false>(((w[(h / PPW) % BITS] >> (BITS * (h % PPW))) & CMASK) | 0x64006400u, zm[h / 8]),
                                s2[h / 8], 0);
  } else {
#pragma unroll
    for (int k = 0; k < 3; ++k)
#pragma unroll
      for (int pp = 0; pp < 5; ++pp)
        out[5 * k + pp] = mul_scale<false>(sub_magic<false>(((w[k % BITS] >> (3 * pp)) & 0x00070007u) | 0x64006400u, zm[(5 * k + pp) / 8]),
                                           s2[(5 * k + pp) / 8], 0);
    const unsigned last = ((w[0] >> 15) & 0x00010001u) | ((w[1 % BITS] >> 14) & 0x00020002u) | ((w[BITS - 1] >> 13) & 0x00040004u);
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

// ---------------------------------------------------------------------------------------------------------------
// Contraction of the two-phase path on pairs of CTAs (a cluster of two SMs, tcgen05 cta_group::2): one MMA spans
// 256 weight rows x 256 tokens, each CTA of the pair holding its 128 weight rows (A) and its 128 of the 256 token
// rows (B) of a k-block in its own shared memory: 32 KB per k-block and SM instead of the 48 KB of a 128 x 256 tile,
// which is what the contraction is bound by (the operands come out of L2).  Each CTA keeps the accumulators of
// its 128 rows in its own tensor memory (two of 256 columns, so the epilogue of a tile runs under the next tile).
//   warp 0, one thread : TMA (no multicast) of the CTA's two half tiles per k-block; the bytes of both CTAs are
//                        counted by the `full` barrier of the pair's first CTA, which arms it;
//   warp 1, one thread : in the pair's first CTA only: tcgen05.mma cta_group::2, and tcgen05.commit to both CTAs'
//                        `empty` / `acc_full` barriers; in both CTAs the warp owns the tensor-memory allocation;
//   warps 2..5         : epilogue, one thread per weight row of the CTA: tcgen05.ld, token scale, conversion into a
//                        shared-memory tile of 32 tokens x 128 features that one thread hands to a TMA store (whole
//                        256-byte rows of y instead of 2 bytes per thread); both CTAs' epilogue warps tell the first
//                        CTA when an accumulator is free again.
// Every wait is bounded (see the fused kernel); the two CTAs leave together through a cluster barrier.
constexpr int kPairThreads = 32 * 6;
// TOK tokens per tile of a pair (UMMA N; 256, or 128 where that fills the pairs better), half of them loaded by each CTA
template <int TOK> struct PairCfg {
  static constexpr int kStageBytes = kTileN * kBlockK * 2 + (TOK / 2) * kBlockK * 2;   // A half and B half of a k-block
  static constexpr int kStages = TOK == 256 ? 6 : 8;                                   // 192 KB of stages
};
constexpr int kOutStageBytes = 32 * kTileN * 4;             // 32 tokens x 128 features, up to 4 bytes each

__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address, in the pair's first CTA, of the object at this CTA's shared address `addr`
__device__ __forceinline__ unsigned in_first_cta(unsigned addr) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(addr));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of a CTA pair: the data lands in this CTA's shared memory, the bytes are counted by `bar_cluster`
__device__ __forceinline__ void tma_load_2d_pair(unsigned dst, const CUtensorMap* map, int c0, int c1, unsigned bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void umma_f16_pair(unsigned tmem_d, uint64_t da, uint64_t db, unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives, when the MMAs issued so far have completed, on this CTA's barrier
__device__ __forceinline__ void umma_commit_pair_local(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// arrives, when the MMAs issued so far have completed, on the barrier at this shared address in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3)
               : "memory");
}

// Order of a pair's tiles: bands of kBandTiles weight tiles, inside a band the weight tile runs fastest and the
// token tile slowest.  The pairs work on neighbouring tiles at the same time, so what they read together is one
// band of the weights (which stays in L2 for the whole band) and a few token tiles, instead of all of the weights
// for every group of token tiles.
constexpr int kBandTiles = 8;   // (4 to 16 measure alike; one band of all the weight tiles is 7 % slower)
__host__ __device__ __forceinline__ void pair_tile(int t, int ntn, int ntm, int& tn, int& tm) {
  const int per_band = kBandTiles * ntm;
  const int band = t / per_band, i = t - band * per_band;
  const int left = ntn - band * kBandTiles;
  const int width = kBandTiles < left ? kBandTiles : left;   // the last band may be narrower
  tm = i / width;
  tn = band * kBandTiles + (i - tm * width);
}

struct PairArgs {
  void* y;
  gwq_dtype yd;
  int32_t* status;
  const float* tok_scale;   // per token 2^e, or null
  int N, K, M;
  int tma_store;            // y is written through tmy (its rows start on 16-byte boundaries), else by plain stores
  long long wait_cycles;
};

// tmx: x16 [M][K] with boxes of 64 columns x 128 rows; tmw: expanded weights [N][K], same boxes.
// tmy: y [M][N] with boxes of 128 output features x 32 tokens.
// ntn: tiles of 256 weight rows; ntiles: all tiles (order: pair_tile); pairs: clusters of the launch.
// SLICED: the left-over tiles of the last round are cut into `split` K-slices (a build of its own, so that the
// common case carries none of it).
template <int TOK, bool SLICED>
__global__ void __launch_bounds__(kPairThreads, 1)
pair_kernel(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmw,
            const __grid_constant__ CUtensorMap tmy, const __grid_constant__ CUtensorMap tmp, const PairArgs p, const int ntn,
            const int ntiles, const int pairs, const int split) {
  constexpr int kHalfBytes = kTileN * kBlockK * 2;   // 16 KB: 128 rows x 128 bytes
  constexpr int kPairStages = PairCfg<TOK>::kStages, kPairStageBytes = PairCfg<TOK>::kStageBytes, kPairTok = TOK;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* tiles =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) unsigned long long bars[2 * 8 + 5];
  __shared__ unsigned tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned rank = cluster_ctarank();       // 0: the pair's first CTA, which issues the MMAs
  const int pair = blockIdx.x >> 1;
  const int nkb = p.K / kBlockK;
  const unsigned bar0 = smem_u32(bars);
  auto full = [&](int s) { return bar0 + 8u * s; };                       // first CTA's: bytes of both CTAs
  auto empty = [&](int s) { return bar0 + 8u * (kPairStages + s); };      // each CTA's own
  auto acc_full = [&](int a) { return bar0 + 8u * (2 * kPairStages + a); };      // each CTA's own
  auto acc_empty = [&](int a) { return bar0 + 8u * (2 * kPairStages + 2 + a); }; // first CTA's: both epilogues
  const unsigned drain_bar = bar0 + 8u * (2 * kPairStages + 4);
  const long long lim = p.wait_cycles;
  auto a_tile = [&](int s) { return tiles + (size_t)s * kPairStageBytes; };
  auto b_tile = [&](int s) { return tiles + (size_t)s * kPairStageBytes + kHalfBytes; };
  unsigned char* out_stage = tiles + (size_t)kPairStages * kPairStageBytes;   // two tiles of 32 tokens x 128 features
  const int ntm = ntiles / ntn;   // token tiles
  // Work items of this pair: the tiles pair, pair + pairs, ... of the full rounds; then, when the tiles left over for
  // the last round are at most half as many as the pairs (split > 1), one K-slice of a left-over tile (its partial sums
  // go to the workspace as FP32 and a second kernel adds the slices), else that tile whole.
  const int full_rounds = ntiles / pairs, rem = ntiles - full_rounds * pairs;
  const int my_items = full_rounds + ((SLICED ? pair < rem * split : pair < rem) ? 1 : 0);
  auto item = [&](int w, int& tile, int& kb0, int& kb1) {   // returns true for a K-slice
    if (!SLICED || w < full_rounds) {
      tile = pair + w * pairs; kb0 = 0; kb1 = nkb;
      return false;
    }
    const int sl = pair % split;
    tile = full_rounds * pairs + pair / split;
    kb0 = (int)((long long)nkb * sl / split);
    kb1 = (int)((long long)nkb * (sl + 1) / split);
    return true;
  };

  if (tid == 0) {
    abort_s = 0;
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(full(s), 1);
      mbar_init(empty(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(acc_full(a), 1);
      mbar_init(acc_empty(a), 2 * kEpilogueWarps);
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // tensor memory of both CTAs: two accumulators of TOK columns x 128 lanes each
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(2 * TOK)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers exist before either signals the other
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_acc = tmem_base_s;
  pdl_trigger();
  pdl_sync();   // the operands are written, and y may still be read, by the kernels before
  bool ok = *reinterpret_cast<volatile int32_t*>(p.status) == 0;   // an earlier CTA gave up: do no work
  int issued = 0;   // k-block copies started (producer thread only), counted over all tiles

  if (warp == 0) {
    // ------------------------------------------------------------------ this CTA's halves of the operand tiles by TMA
    if (lane == 0) {
      int it = 0;
      for (int w = 0; w < my_items && ok; ++w) {
        int tile, kb0, kb1, tn, tm;
        item(w, tile, kb0, kb1);
        pair_tile(tile, ntn, ntm, tn, tm);
        const int n0 = tn * (2 * kTileN) + (int)rank * kTileN;
        const int m0 = tm * kPairTok + (int)rank * (kPairTok / 2);
        for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
          const int s = it % kPairStages, round = it / kPairStages;
          if (round > 0) ok = mbar_wait(empty(s), (round - 1) & 1, abort_flag, lim);
          if (!ok) break;
          if (rank == 0) mbar_expect_tx(full(s), 2 * kPairStageBytes);   // both CTAs' halves
          const unsigned fb = in_first_cta(full(s));
          tma_load_2d_pair(smem_u32(a_tile(s)), &tmw, kb * kBlockK, n0, fb);
          tma_load_2d_pair(smem_u32(b_tile(s)), &tmx, kb * kBlockK, m0, fb);
          issued = it + 1;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue (first CTA of the pair)
    if (lane == 0 && rank == 0) {
      // instruction descriptor: FP32 accumulate, A and B fp16, K-major, N = 256, M = 256 (128 rows per CTA)
      const unsigned idesc = (1u << 4) | ((unsigned)(kPairTok >> 3) << 17) | ((unsigned)((2 * kTileN) >> 4) << 24);
      int it = 0;
      for (int w = 0; w < my_items && ok; ++w) {
        int tile, kb0, kb1;
        item(w, tile, kb0, kb1);
        const int a = w & 1;
        if (w >= 2) ok = mbar_wait(acc_empty(a), ((w >> 1) - 1) & 1, abort_flag, lim);   // drained by both epilogues
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned acc = tmem_acc + (unsigned)(a * kPairTok);
        for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
          const int s = it % kPairStages, round = it / kPairStages;
          ok = mbar_wait(full(s), round & 1, abort_flag, lim);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t da = umma_desc(smem_u32(a_tile(s))), db = umma_desc(smem_u32(b_tile(s)));
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)   // 32 bytes further along K inside the swizzle atom
            umma_f16_pair(acc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > kb0 || k != 0) ? 1u : 0u);
          umma_commit_pair(empty(s));
        }
        if (ok) umma_commit_pair(acc_full(a));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one thread per weight row of the CTA
    const int quad = warp & 3;                 // tensor-memory lane quarter this warp may access
    const int r = quad * 32 + lane;
    int chunk = 0;                             // chunks handed to the TMA store so far
    for (int w = 0; w < my_items && ok; ++w) {
      int tile, kb0, kb1, tn, tm;
      const bool slice = item(w, tile, kb0, kb1) && SLICED;
      pair_tile(tile, ntn, ntm, tn, tm);
      const int row = tn * (2 * kTileN) + (int)rank * kTileN + r, m0 = tm * kPairTok;
      const bool live = row < p.N;
      const int a = w & 1;
      ok = mbar_wait_warp(acc_full(a), (w >> 1) & 1, abort_flag, lim);
      {   // one verdict for the four epilogue warps: they meet at barriers inside the tile
        unsigned all;
        asm volatile("{\n .reg .pred q, r;\n setp.ne.b32 q, %1, 0;\n bar.red.and.pred r, 1, 128, q;\n selp.b32 %0, 1, 0, r;\n}\n"
                     : "=r"(all) : "r"((unsigned)ok) : "memory");
        ok = all != 0;
      }
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c0 = 0; c0 < kPairTok; c0 += 32) {
        if (m0 + c0 >= p.M) break;             // warp-uniform
        unsigned v[32];
        tmem_ld32(tmem_acc + ((unsigned)(quad * 32) << 16) + (unsigned)(a * kPairTok + c0), v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (p.tma_store || slice) {
          // the chunk goes through a shared-memory tile [32 tokens][128 features] (two of them, used in turn)
          unsigned char* st = out_stage + (chunk & 1) * kOutStageBytes;
          if (chunk >= 2) {   // the store that read this tile two chunks ago has finished reading it
            if (warp == 2 && lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            asm volatile("bar.sync 1, 128;" ::: "memory");
          }
          // token scales of the chunk (one vector load per four tokens while the chunk lies inside M)
          float ts[32];
          if (p.tok_scale) {
            if (m0 + c0 + 32 <= p.M) {
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const float4 t4 = __ldg(reinterpret_cast<const float4*>(p.tok_scale + m0 + c0) + q);
                ts[4 * q] = t4.x; ts[4 * q + 1] = t4.y; ts[4 * q + 2] = t4.z; ts[4 * q + 3] = t4.w;
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) ts[i] = __ldg(p.tok_scale + min(m0 + c0 + i, p.M - 1));
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) ts[i] = 1.f;
          }
          if (slice) {   // raw FP32 partial sums of this K-slice; scale and conversion follow in the second kernel
#pragma unroll
            for (int i = 0; i < 32; ++i) reinterpret_cast<unsigned*>(st)[i * kTileN + r] = v[i];
          } else if (p.yd == GWQ_F32) {
#pragma unroll
            for (int i = 0; i < 32; ++i) reinterpret_cast<float*>(st)[i * kTileN + r] = __uint_as_float(v[i]) * ts[i];
          } else {
            // 2-byte outputs: neighbouring lanes (features r, r + 1) swap one of every two tokens, so that each lane
            // converts and stores a pair of neighbouring features of one token as one word
            const bool odd = (lane & 1) != 0;
            unsigned* st32 = reinterpret_cast<unsigned*>(st);
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float f0 = __uint_as_float(v[i]) * ts[i], f1 = __uint_as_float(v[i + 1]) * ts[i + 1];
              const float got = __shfl_xor_sync(0xFFFFFFFFu, odd ? f0 : f1, 1);
              const float lo = odd ? got : f0, hi = odd ? f1 : got;   // features (r & ~1), (r | 1) of token i + odd
              unsigned w;
              if (p.yd == GWQ_F16) {
                const __half2 h = __floats2half2_rn(lo, hi);
                w = *reinterpret_cast<const unsigned*>(&h);
              } else {
                const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
                w = *reinterpret_cast<const unsigned*>(&h);
              }
              st32[((i + (odd ? 1 : 0)) * kTileN + (r & ~1)) >> 1] = w;
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the TMA
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (warp == 2 && lane == 0 && slice) {   // slot `pair` of the partial tiles: [TOK tokens][256 features] FP32
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(&tmp), "r"((int)rank * kTileN), "r"(pair * kPairTok + c0), "r"(smem_u32(st))
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          } else if (warp == 2 && lane == 0) {   // rows past N and tokens past M are clipped by the copy
            // y is written once and not read again here: its lines are the first to leave L2, not the operands'
            asm volatile(
                "{\n .reg .b64 pol;\n createpolicy.fractional.L2::evict_first.b64 pol, 1.0;\n"
                " cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], pol;\n}\n"
                ::"l"(&tmy), "r"(tn * (2 * kTileN) + (int)rank * kTileN), "r"(m0 + c0), "r"(smem_u32(st))
                : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          ++chunk;
        } else if (live) {
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
      // the accumulator may be overwritten by the tile after next: both CTAs tell the first one
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(in_first_cta(acc_empty(a)));
    }
    // the stores still in flight read this CTA's shared memory
    if (warp == 2 && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
  if (!ok) {
    *abort_flag = 1;
    atomicExch(p.status, (int32_t)GWQ_ERR_TIMEOUT);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (abort_s) {
    // give-up path.  Bulk copies that were issued must land before the shared memory is given back; their bytes are
    // counted in the first CTA, so this CTA waits a fixed time that is long against a copy instead (bounded).
    if (warp == 0 && lane == 0 && issued > 0) {
      const long long t0 = clock64();
      while (clock64() - t0 < 200000) {}
    }
    // MMAs that were issued may still read both CTAs' stages and write both tensor memories: one more commit arrives
    // when all of them have completed; wait (bounded) for it before the pair leaves
    if (warp == 1 && lane == 0 && rank == 0) {
      int zero = 0;
      umma_commit_pair_local(drain_bar);
      (void)mbar_wait(drain_bar, 0, &zero, kSpinCycles);
    }
  }
  __syncthreads();
  cluster_sync_all();   // neither CTA frees its tensor memory, or exits, while the other may still signal or write it
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(2 * TOK) : "memory");
  }
}

// K-slices of a left-over tile: split = pairs / left-over tiles when these are at most half as many as the pairs
// (at least 8 k-blocks per slice, at most 8 slices) and the slices save more than adding them up costs, else 1.
static int pair_split(int ntiles, int pairs, int nkb) {
  const int rem = ntiles % pairs;
  if (rem == 0 || 2 * rem > pairs) return 1;
  int split = pairs / rem;
  if (split > 8) split = 8;
  while (split > 1 && nkb / split < 8) --split;
  // the second kernel and the partial tiles cost about as much as 43 k-blocks of a tile (measured: 4096 x 4096 at 512
  // tokens, two slices of 32 k-blocks: 47 against 41 us; 11008 x 4096, six slices: 75 against 80 us; 4096 x 11008, two
  // slices of 86: 83 against 93 us, 65 against 90 us at 256 tokens)
  if ((long long)nkb * (split - 1) < 43LL * split) return 1;
  return split;
}
// bytes of the FP32 partial tiles: one slot of TOK tokens x 256 features per pair
static size_t pair_partial_bytes(int sms) { return (size_t)(sms / 2 > 0 ? sms / 2 : 1) * 256 * 256 * sizeof(float); }

// Adds the K-slices of the left-over tiles (slots t split .. t split + split - 1 of left-over tile t, in slice order:
// the same bits every time), applies the token scale and stores y.  One CTA per tile and 4 tokens, one thread per
// (feature, token); the loads of a sum are requested together.
template <int TOK>
__global__ void __launch_bounds__(1024) pair_fixup_kernel(const float* __restrict__ partial, void* y, gwq_dtype yd,
                                                          const float* __restrict__ tok_scale, int N, int M, int ntn, int ntm,
                                                          int first_tile, int split) {
  pdl_trigger();
  pdl_sync();
  int tn, tm;
  pair_tile(first_tile + blockIdx.x, ntn, ntm, tn, tm);
  const int n = tn * 256 + threadIdx.x, ml = blockIdx.y * 4 + threadIdx.y, m = tm * TOK + ml;
  if (n >= N || m >= M) return;
  const float* src = partial + ((size_t)blockIdx.x * split * TOK + ml) * 256 + threadIdx.x;
  float t[8];
#pragma unroll
  for (int sl = 0; sl < 8; ++sl) t[sl] = sl < split ? __ldg(src + (size_t)sl * TOK * 256) : 0.f;
  float v = t[0];
#pragma unroll
  for (int sl = 1; sl < 8; ++sl) v += t[sl];   // slice order
  if (tok_scale) v *= __ldg(tok_scale + m);
  const size_t idx = (size_t)m * N + n;
  if (yd == GWQ_F32) reinterpret_cast<float*>(y)[idx] = v;
  else if (yd == GWQ_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
  else reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
}

// Launch of the pair kernel on the expanded weights w16 [N][K] and fp16 activations x [M][K].
template <int TOK>
gwq_status launch_pairs_tok(const gwq_packed* P, const void* x, const float* tok_scale, const void* w16, float* partial, int M,
                            void* y, gwq_dtype yd, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  EncodeTiledFn enc = encode_fn();
  if (!enc) return GWQ_ERR_CUDA;
  CUtensorMap tmx, tmw;
  const cuuint32_t estr[2] = {1, 1};
  const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileN};
  {
    const cuuint32_t xbox[2] = {(cuuint32_t)kBlockK, (cuuint32_t)(TOK / 2)};
    const cuuint64_t dims[2] = {(cuuint64_t)P->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)P->K * 2};
    if (enc(&tmx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, xbox, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)P->K, (cuuint64_t)P->N};
    const cuuint64_t strides[1] = {(cuuint64_t)P->K * 2};
    if (enc(&tmw, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(w16), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  const size_t esz = yd == GWQ_F32 ? 4 : 2;
  const int tma_store = ((size_t)P->N * esz) % 16 == 0 ? 1 : 0;   // y itself is 16-byte aligned (checked at the entry point)
  CUtensorMap tmy = tmx;
  if (tma_store) {
    const cuuint64_t dims[2] = {(cuuint64_t)P->N, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)P->N * esz};
    const cuuint32_t obox[2] = {(cuuint32_t)kTileN, 32};
    const CUtensorMapDataType dt = yd == GWQ_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                 : (yd == GWQ_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
    if (enc(&tmy, dt, 2, y, dims, strides, obox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  CUtensorMap tmp = tmx;   // FP32 partial tiles: rows = slot * TOK + token, 256 features each
  if (partial) {
    const int slots = pv->sm_count / 2 > 0 ? pv->sm_count / 2 : 1;
    const cuuint64_t dims[2] = {256, (cuuint64_t)slots * TOK};
    const cuuint64_t strides[1] = {256 * sizeof(float)};
    const cuuint32_t obox[2] = {(cuuint32_t)kTileN, 32};
    if (enc(&tmp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, partial, dims, strides, obox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  const size_t smem = (size_t)PairCfg<TOK>::kStages * PairCfg<TOK>::kStageBytes + 2 * kOutStageBytes + 1024;
  if (cudaFuncSetAttribute(pair_kernel<TOK, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaFuncSetAttribute(pair_kernel<TOK, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return GWQ_ERR_CUDA;
  PairArgs a;
  a.y = y; a.yd = yd; a.status = pv->dev_status; a.tok_scale = tok_scale; a.N = P->N; a.K = P->K; a.M = M;
  a.tma_store = tma_store;
  a.wait_cycles = pv->wait_cycles;
  const int ntn = (P->N + 2 * kTileN - 1) / (2 * kTileN), ntiles = ntn * ((M + TOK - 1) / TOK);
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // persistent: as many pairs as the device holds at once (pairs sit inside one GPC, so this may be fewer than SMs / 2)
  cfg.gridDim = dim3(2u * (unsigned)(pv->sm_count / 2));
  // (asked once per device and token-tile size: the answer depends on nothing else)
  static std::atomic<int> resident_on[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 63;
  int resident = resident_on[dev].load(std::memory_order_relaxed);
  if (resident == 0) {
    if (cudaOccupancyMaxActiveClusters(&resident, pair_kernel<TOK, false>, &cfg) != cudaSuccess || resident < 1) {
      (void)cudaGetLastError();
      resident = -1;
    }
    resident_on[dev].store(resident, std::memory_order_relaxed);
  }
  if (resident < 1) return GWQ_ERR_UNSUPPORTED;
  int pairs = resident < pv->sm_count / 2 ? resident : pv->sm_count / 2;
  const int split = partial ? pair_split(ntiles, pairs, P->K / kBlockK) : 1;   // fewer tiles than pairs: all of them left over
  if (split == 1 && pairs > ntiles) pairs = ntiles;
  cfg.gridDim = dim3(2u * (unsigned)pairs);
  const cudaError_t le = split > 1 ? cudaLaunchKernelEx(&cfg, pair_kernel<TOK, true>, tmx, tmw, tmy, tmp, a, ntn, ntiles, pairs, split)
                                   : cudaLaunchKernelEx(&cfg, pair_kernel<TOK, false>, tmx, tmw, tmy, tmp, a, ntn, ntiles, pairs, split);
  if (le != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  if (split > 1) {
    const int rem = ntiles % pairs;
    if (launch_pdl(pair_fixup_kernel<TOK>, dim3((unsigned)rem, TOK / 4), dim3(256, 4), 0, stream, (const float*)partial, y, yd, tok_scale,
                   P->N, M, ntn, ntiles / ntn, ntiles - rem, split) != cudaSuccess) {
      (void)cudaGetLastError();
      return GWQ_ERR_CUDA;
    }
  }
  return GWQ_OK;
}

// Tokens per tile: the pairs work in rounds of one tile each (the last round in K-slices when few tiles are left over).
// A 128-token tile loads 24 KB per k-block for half the multiplies of a 256-token tile's 32 KB, and the operands come
// out of L2, so it takes about 0.8 of the time, not half (measured, 512 tokens: 66 against 76 us where both need one
// round, 4096 x 11008; 69 against 64 us with three rounds against two, 11008 x 4096): it is taken only where it needs
// hardly more rounds than the larger tile.
gwq_status launch_pairs(const gwq_packed* P, const void* x, const float* tok_scale, const void* w16, float* partial, int M, void* y,
                        gwq_dtype yd, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const int pairs = pv->sm_count / 2 > 0 ? pv->sm_count / 2 : 1;
  const int ntn = (P->N + 2 * kTileN - 1) / (2 * kTileN), nkb = P->K / kBlockK;
  auto rounds = [&](int tok) {   // in units of one tile's time
    const int ntiles = ntn * ((M + tok - 1) / tok);
    const int split = partial ? pair_split(ntiles, pairs, nkb) : 1;
    return (double)(ntiles / pairs) + (ntiles % pairs ? 1.0 / split : 0.0);
  };
  if (0.8 * rounds(128) < rounds(256)) return launch_pairs_tok<128>(P, x, tok_scale, w16, partial, M, y, yd, stream);
  return launch_pairs_tok<256>(P, x, tok_scale, w16, partial, M, y, yd, stream);
}

template <int BITS, int TOK, int GPK = 1>
gwq_status launch(const gwq_packed* P, const void* x, const float* tok_scale, int M, void* y, gwq_dtype yd, cudaStream_t stream) {
  constexpr bool BF16 = false;   // operands are always fp16 here (see the file header)
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  EncodeTiledFn enc = encode_fn();
  if (!enc) return GWQ_ERR_CUDA;
  CUtensorMap tmx;
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
  const int stage_bytes = kTileN * kBlockK * 2 + TOK * kBlockK * 2;
  static_assert(kTileN == 128 && kBlockK == 64, "fused_stages() is written for these tile sizes");
  constexpr int stages = fused_stages(TOK);
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  if (cudaFuncSetAttribute(prefill_kernel<BITS, TOK, BF16, GPK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return GWQ_ERR_CUDA;
  PrefillArgs a;
  a.codes = P->codes; a.scales = P->scales; a.zeros = P->zeros; a.row_ptr = P->S->row_ptr; a.cv = pv->cv; a.sz_t = pv->sz_t;
  a.y = y; a.yd = yd; a.status = pv->dev_status; a.tok_scale = tok_scale; a.N = P->N; a.K = P->K; a.M = M; a.group = P->group;
  a.wait_cycles = pv->wait_cycles;
  const int ntn = (P->N + kTileN - 1) / kTileN, ntiles = ntn * ((M + TOK - 1) / TOK);
  const int grid = ntiles < pv->sm_count ? ntiles : pv->sm_count;   // persistent: at most one CTA per SM
  prefill_kernel<BITS, TOK, BF16, GPK><<<grid, kCtaThreads, smem, stream>>>(tmx, a, ntn, ntiles);
  return cudaGetLastError() == cudaSuccess ? GWQ_OK : GWQ_ERR_CUDA;
}

template <int BITS>
gwq_status launch_tok(const gwq_packed* P, const void* x, const float* tok_scale, int M, void* y, gwq_dtype yd,
                      cudaStream_t stream) {
  if (P->group == 32) {   // small groups: the smallest and the largest token tile only
    if (M <= 32) return launch<BITS, 32, 2>(P, x, tok_scale, M, y, yd, stream);
    return launch<BITS, 256, 2>(P, x, tok_scale, M, y, yd, stream);
  }
  if (P->group == 16) {
    if (M <= 32) return launch<BITS, 32, 4>(P, x, tok_scale, M, y, yd, stream);
    return launch<BITS, 256, 4>(P, x, tok_scale, M, y, yd, stream);
  }
  if (M <= 32) return launch<BITS, 32>(P, x, tok_scale, M, y, yd, stream);
  if (M <= 64) return launch<BITS, 64>(P, x, tok_scale, M, y, yd, stream);
  if (M <= 128) return launch<BITS, 128>(P, x, tok_scale, M, y, yd, stream);
  return launch<BITS, 256>(P, x, tok_scale, M, y, yd, stream);
}

// The same expansion by blocks of 128 rows x 128 columns, for layers that carry the block-ordered outlier list
// (groups of 64 or 128, K a multiple of 128): one CTA expands a block into shared memory, drops the block's FP16
// outliers over their zero entries there and writes whole 256-byte row segments: one pass, no 2-byte stores to
// global memory.
template <int BITS>
__global__ void __launch_bounds__(256) expand_block_kernel(const uint32_t* __restrict__ codes, const uint32_t* __restrict__ sz_t,
                                                           const uint32_t* __restrict__ ob, const int32_t* __restrict__ ob_ptr,
                                                           uint16_t* __restrict__ w16, int N, int K, int group) {
  constexpr int kPitch = 128 + 8;                  // halves per row of the tile: 16 bytes of padding
  __shared__ __align__(16) uint16_t tile[128 * kPitch];
  pdl_trigger();
  const int G = K >> 7;
  const int blk = blockIdx.x, row0 = (blk / G) * 128, g = blk % G;
  const int e0 = __ldg(ob_ptr + blk), e1 = __ldg(ob_ptr + blk + 1);
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int idx = threadIdx.x + 256 * u, r = idx >> 2, q = idx & 3;   // row of the block, run of 32 columns
    const int row = min(row0 + r, N - 1);
    const uint32_t* src = codes + ((size_t)row * (K >> 5) + g * 4 + q) * BITS;
    unsigned w[BITS];
    if (BITS == 4) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
      w[0] = v.x; w[1 % BITS] = v.y; w[2 % BITS] = v.z; w[3 % BITS] = v.w;
    } else {
#pragma unroll
      for (int k = 0; k < BITS; ++k) w[k] = __ldg(src + k);
    }
    unsigned s2[2], zm[2];   // scale and zero-point of the run's two halves of 16 columns
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const unsigned sz = __ldg(sz_t + (size_t)((g * 128 + q * 32 + 16 * h) / group) * N + row);
      s2[h] = (sz & 0xFFFFu) * 0x00010001u;
      zm[h] = 0x64006400u | ((sz >> 16) * 0x00010001u);
    }
    unsigned out[16];
    if (BITS == 4) {
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          out[4 * t + j] = mul_scale<false>(sub_magic<false>(((w[t % BITS] >> (4 * j)) & 0x000F000Fu) | 0x64006400u, zm[t / 2]),
                                            s2[t / 2], 0);
    } else if (BITS == 2 || BITS == 8) {
      constexpr int PPW = 16 / BITS;
      constexpr unsigned CMASK = ((1u << BITS) - 1u) * 0x00010001u;
#pragma unroll
      for (int h = 0; h < 16; ++h)
        out[h] = mul_scale<false>(sub_magic<false>(((w[(h / PPW) % BITS] >> (BITS * (h % PPW))) & CMASK) | 0x64006400u, zm[h / 8]),
                                  s2[h / 8], 0);
    } else {
#pragma unroll
      for (int k = 0; k < 3; ++k)
#pragma unroll
        for (int pp = 0; pp < 5; ++pp)
          out[5 * k + pp] = mul_scale<false>(sub_magic<false>(((w[k % BITS] >> (3 * pp)) & 0x00070007u) | 0x64006400u, zm[(5 * k + pp) / 8]),
                                             s2[(5 * k + pp) / 8], 0);
      const unsigned last = ((w[0] >> 15) & 0x00010001u) | ((w[1 % BITS] >> 14) & 0x00020002u) | ((w[BITS - 1] >> 13) & 0x00040004u);
      out[15] = mul_scale<false>(sub_magic<false>(last | 0x64006400u, zm[1]), s2[1], 0);
    }
    uint4* dst = reinterpret_cast<uint4*>(tile + r * kPitch + q * 32);
#pragma unroll
    for (int c = 0; c < 4; ++c) dst[c] = make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
  }
  __syncthreads();
  for (int e = e0 + threadIdx.x; e < e1; e += 256) {
    const unsigned v = __ldg(ob + e);
    tile[((v >> 23) & 127u) * kPitch + ((v >> 16) & 127u)] = (uint16_t)v;
  }
  __syncthreads();
  pdl_sync();   // the workspace may still be read by the kernel before (everything above depends on the weights alone)
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int id = threadIdx.x + 256 * u, r = id >> 4, pc = id & 15;   // 16-byte piece pc of row r
    if (row0 + r < N)
      *reinterpret_cast<uint4*>(w16 + (size_t)(row0 + r) * K + g * 128 + pc * 8) =
          *reinterpret_cast<const uint4*>(tile + r * kPitch + pc * 8);
  }
}

// When the weights are expanded once instead of once per token tile.  The expansion is a pass of 2.5 bytes per weight
// (24 us for 45 M weights, 125 us for 235 M); the contraction on CTA pairs then runs at 1000 to 1500 TFLOP/s, where the
// fused kernel is bound by its dequantisation warps (250 to 770), expands the weights again for every token tile of
// 256 and leaves SMs idle when the layer has fewer 128-row tiles than the device has SMs.  So: more than 256 tokens
// always; any number of tokens of this path (33 on) where the 128-row tiles do not fill the SMs.  Measured, bf16 activations, 4 bit, fused
// against two-phase (us): 11008 x 4096: 49 / 51 at 33 tokens, 52 / 52 at 64, 58 / 54 at 128, 75 / 59 at 256, 114 / 78 at 512;
// 4096 x 11008: 122 / 82 at 33, 123 / 83 at 64, 147 / 86 at 256, 144 / 89 at 512; 4096 x 4096: 51 / 36 at 33, 53 / 35 at 64, 74 / 39 at 256;
// 8192 x 8192: 99 / 82 at 128, 117 / 84 at 256, 116 / 92 at 512; 28672 x 8192 (224 tiles on 148 SMs): 180 / 228 at 128,
// 207 / 239 at 256, 361 / 307 at 384, 374 / 312 at 512.
constexpr int kExpandAlwaysTokens = 257;   // more than one token tile of the fused kernel
constexpr int kExpandMinTokens = 33;       // ... every call of this path where the fused kernel's tiles leave SMs idle
static bool wants_expansion(const gwq_packed* P, int M) {
#ifdef GWQ_TUNE_EXPAND_MIN
  return M >= GWQ_TUNE_EXPAND_MIN;
#endif
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const int sms = pv->sm_count > 0 ? pv->sm_count : 148;
  return M >= kExpandAlwaysTokens || (M >= kExpandMinTokens && (P->N + kTileN - 1) / kTileN < sms);
}

// Expanded weights: the expansion, the outliers over it, then the contraction with token tiles of 256.
gwq_status launch_expanded(const gwq_packed* P, const void* x, const float* tok_scale, uint16_t* w16, float* partial, int M,
                           void* y, gwq_dtype yd, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  if (pv->ob && pv->ob_ptr && P->K % 128 == 0) {
    const unsigned blocks = (unsigned)((P->N + 127) / 128) * (unsigned)(P->K / 128);
#define GWQ_EXPAND_BLOCK(B)                                                                                                  \
  (void)launch_pdl(expand_block_kernel<B>, dim3(blocks), dim3(256), 0, stream, (const uint32_t*)P->codes, (const uint32_t*)pv->sz_t, \
                   (const uint32_t*)pv->ob, (const int32_t*)pv->ob_ptr, w16, P->N, P->K, P->group)
    switch (P->bits) {
      case 4: GWQ_EXPAND_BLOCK(4); break;
      case 3: GWQ_EXPAND_BLOCK(3); break;
      case 8: GWQ_EXPAND_BLOCK(8); break;
      default: GWQ_EXPAND_BLOCK(2); break;
    }
#undef GWQ_EXPAND_BLOCK
  } else {
    const long long runs = (long long)P->N * (P->K / 32);
    const unsigned grid = (unsigned)((runs + 255) / 256);
    switch (P->bits) {
      case 4: expand_kernel<4><<<grid, 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group); break;
      case 3: expand_kernel<3><<<grid, 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group); break;
      case 8: expand_kernel<8><<<grid, 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group); break;
      default: expand_kernel<2><<<grid, 256, 0, stream>>>(P->codes, pv->sz_t, w16, P->N, P->K, P->group); break;
    }
    expand_outliers_kernel<<<(P->N + 7) / 8, 256, 0, stream>>>(P->S->row_ptr, pv->cv, w16, P->N, P->K);
  }
  if (cudaGetLastError() != cudaSuccess) return GWQ_ERR_CUDA;
  return launch_pairs(P, x, tok_scale, w16, partial, M, y, yd, stream);
}

}  // namespace

// Scratch of the tensor-core path: bf16 activations need an fp16 copy of x and one scale per token; from
// the token count where the two-phase path takes over (wants_expansion), the fp16 expansion of the weights follows.
static size_t x16_bytes(const gwq_packed* P, gwq_dtype xd, int M) {
  if (xd != GWQ_BF16) return 0;
  return (((size_t)M * P->K * 2 + 255) & ~(size_t)255) + (((size_t)M * 4 + 255) & ~(size_t)255);
}
size_t gwq_prefill_workspace_bytes(const gwq_packed* P, gwq_dtype xd, int M) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  if (!pv->cv || !pv->sz_t || P->K % kBlockK != 0) return 0;   // the general kernel needs none
  // (the expanded weights are followed by the FP32 partial tiles of the K-slices)
  return x16_bytes(P, xd, M) +
         (wants_expansion(P, M) ? (((size_t)P->N * P->K * 2 + 255) & ~(size_t)255) + pair_partial_bytes(pv->sm_count) : 0);
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
    if (launch_pdl(bf16_rows_to_scaled_f16, dim3((unsigned)M), dim3(256), 0, stream, static_cast<const uint16_t*>(x), x16, ts, P->K) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return GWQ_ERR_CUDA;
    }
    x = x16;
    tok_scale = ts;
  }
  if (wants_expansion(P, M) && ws && ws_bytes >= gwq_prefill_workspace_bytes(P, xd, M))
  {
    char* w16 = static_cast<char*>(ws) + xb;
    float* partial = reinterpret_cast<float*>(w16 + (((size_t)P->N * P->K * 2 + 255) & ~(size_t)255));
    const gwq_status st = launch_expanded(P, x, tok_scale, reinterpret_cast<uint16_t*>(w16), partial, M, y, yd, stream);
    if (st != GWQ_ERR_UNSUPPORTED) return st;   // a device that holds no cluster of two such CTAs: the fused kernel
  }
  switch (P->bits) {
    case 4: return launch_tok<4>(P, x, tok_scale, M, y, yd, stream);
    case 3: return launch_tok<3>(P, x, tok_scale, M, y, yd, stream);
    case 8: return launch_tok<8>(P, x, tok_scale, M, y, yd, stream);
    case 2: return launch_tok<2>(P, x, tok_scale, M, y, yd, stream);
  }
  return GWQ_ERR_UNSUPPORTED;
}
