// Skinny path (fp16 activations, up to 32 tokens) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w") on the
// 5th-generation tensor cores: bandwidth-bound, so everything is arranged around the number of instructions a
// packed byte costs.
//
// Work is cut into steps of 128 output rows x 128 columns.  The steps of a layer, tile after tile, form one
// sequence that is divided evenly over one CTA per SM; a CTA walks its range as a pipeline of warp roles:
//   warp 0, one thread : TMA (no multicast): the packed codes of the step (128 rows x 64 or 48 bytes) and the
//                        activation tile (tokens x 128 columns, two 128-byte-swizzled k-blocks) into a stage;
//   warps 2..9         : two sets of four warps that take alternate steps, one thread per row: the row's codes
//                        from shared memory -> masked in place into fp16 subnormals q 2^-24 (no arithmetic on the
//                        codes) -> tensor memory (tcgen05.st), the A operand of the step;
//   warps 15, 16       : one per set: the FP16 outliers of the step's block (a block-ordered copy of the CSR entries,
//                        made by gwq_pack) are dropped into an otherwise all-zero shared-memory tile and taken out
//                        again once the MMAs have read it;
//   warp 1, one thread : tcgen05.mma kind::f16, M = 128 rows, N = tokens: 8 MMAs (K = 16) with A from tensor
//                        memory into the step's accumulator, 8 more with the outlier tile as A into an
//                        accumulator that runs over the whole tile (the tensor cores do the sparse product);
//   warp 14            : sums of x over the step's groups for every token (mma.sync against all ones);
//   warps 10..13       : one thread per row: the step's accumulator from tensor memory, y += s 2^24 D - s z sum(x)
//                        per group (scale and zero-point never touch a weight); at the end of a tile the outlier
//                        accumulator is added and the row is stored.
// A tile that falls into the ranges of several CTAs is stored as FP32 partial sums (at most two per CTA) in the
// caller's workspace and a second, small kernel adds them in CTA order: no atomics, the same bits every time.
// Every wait is bounded; when one runs out the CTA records GWQ_ERR_TIMEOUT, drains its copies and MMAs, frees its
// tensor memory and returns.
#include "tc_common.cuh"

namespace {
using namespace gwq_tc;

constexpr int kRows = 128;        // rows of a tile (UMMA M)
// ring of codes + activation tiles (measured, 32 tokens: 4 / 6 / 8 stages: 163 / 158 / 163 us on 28672 x 8192,
// 155 / 149 / 155 us on 8192 x 28672, 38 / 37 / 37 us on 11008 x 4096)
constexpr int kStages = 6;
constexpr int kSets = 2;          // expansion warp sets, one tensor-memory A buffer and one outlier tile each
constexpr int kXs = 8;            // ring of group-sum slots
constexpr int kWarpProducer = 0, kWarpMma = 1, kWarpExpand0 = 2, kWarpEpi0 = 2 + 4 * kSets, kWarpSums = kWarpEpi0 + 4;
constexpr int kWarpOut0 = kWarpSums + 1;
constexpr int kThreads = 32 * (kWarpOut0 + kSets);
constexpr int kOutTileBytes = kRows * 128 * 2;   // outlier tile of a step: 128 rows x 128 columns fp16 (two k-blocks)
constexpr int kTmemCols = 256;

struct SkinnyArgs {
  const uint32_t* szt;      // [K / group][N]: scale fp16 bits | zero-point << 16
  const uint32_t* ob;       // outliers by block: row-in-block << 23 | column-in-block << 16 | fp16 value
  const int32_t* ob_ptr;    // extents of the blocks in ob; block = tile * G + step of the tile = index of the step
  void* y;
  float* partial;           // [2 * gridDim][TOK][128] partial sums of tiles shared with other CTAs
  int32_t* status;
  gwq_dtype yd;
  int N, K, M;
  int G;                    // steps per tile (K / 128)
  long long total;          // steps of the layer (tiles * G)
  long long wait_cycles;
};

__device__ __forceinline__ void umma_ts(unsigned tmem_d, unsigned tmem_a, uint64_t db, unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tmem_st16(unsigned taddr, const unsigned* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(unsigned taddr, unsigned (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void mma16816_ones(float (&d)[4], unsigned b0, unsigned b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%4,%4,%4}, {%5,%6}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(0x3C003C00u), "r"(b0), "r"(b1));
}

// first step of CTA p of P over `total` steps
__device__ __host__ __forceinline__ long long range_begin(long long total, int P, int p) { return total * p / P; }

// BITS: 3 or 4.  TOK: tokens of a tile (UMMA N; 32 is the one instantiated).  G64: groups of 64 columns (two accumulators per step).
template <int BITS, int TOK, bool G64>
__global__ void __launch_bounds__(kThreads, 1)
skinny_kernel(const __grid_constant__ CUtensorMap tmc, const __grid_constant__ CUtensorMap tmx, const SkinnyArgs p) {
  constexpr int CB = 16 * BITS;                    // bytes of packed codes per row and step
  constexpr int kCodeBytes = kRows * CB;
  constexpr int kXBytes = 2 * TOK * 128;           // two k-blocks of TOK rows x 128 bytes
  constexpr int kStageBytes = 8192 + 8192;         // activation tiles first (1024-byte aligned), then the codes
  constexpr int AS = G64 ? 2 : 1;                  // accumulator steps (scale groups) per step
  static_assert(kXBytes <= 8192 && kCodeBytes <= 8192, "stage layout");
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  unsigned char* out_tiles = base + kStages * kStageBytes;                       // kSets x 32 KB
  float* xsum = reinterpret_cast<float*>(out_tiles + kSets * kOutTileBytes);     // [kXs][AS][TOK]
  __shared__ __align__(8) unsigned long long bars[2 * kStages + 2 * kSets + 4 + 4 + 2 * kXs + 1];
  __shared__ unsigned tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned bar0 = smem_u32(bars);
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto a_full = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto a_empty = [&](int b) { return bar0 + 8u * (2 * kStages + kSets + b); };
  auto d_full = [&](int d) { return bar0 + 8u * (2 * kStages + 2 * kSets + d); };
  auto d_empty = [&](int d) { return bar0 + 8u * (2 * kStages + 2 * kSets + 2 + d); };
  auto o_full = [&](int o) { return bar0 + 8u * (2 * kStages + 2 * kSets + 4 + o); };
  auto o_empty = [&](int o) { return bar0 + 8u * (2 * kStages + 2 * kSets + 6 + o); };
  auto xs_full = [&](int q) { return bar0 + 8u * (2 * kStages + 2 * kSets + 8 + q); };
  auto xs_empty = [&](int q) { return bar0 + 8u * (2 * kStages + 2 * kSets + 8 + kXs + q); };
  const unsigned drain_bar = bar0 + 8u * (2 * kStages + 2 * kSets + 8 + 2 * kXs);
  auto x_tile = [&](int s, int kb) { return base + s * kStageBytes + kb * (TOK * 128); };
  auto code_tile = [&](int s) { return base + s * kStageBytes + 8192; };
  const long long lim = p.wait_cycles;

  // this CTA's range of steps
  const long long it0 = range_begin(p.total, gridDim.x, blockIdx.x), it1 = range_begin(p.total, gridDim.x, blockIdx.x + 1);
  const int nsteps = (int)(it1 - it0);
  const int G = p.G;
  // tile and group of step j of this CTA with 32-bit arithmetic: a 64-bit division per step and role costs several
  // hundred cycles of a single warp, which is what the step has
  const unsigned tile0 = (unsigned)(it0 / G), grp0 = (unsigned)(it0 % G);
  auto tile_of = [&](int j) { return (int)(tile0 + (grp0 + (unsigned)j) / (unsigned)G); };
  auto grp_of = [&](int j) { return (int)((grp0 + (unsigned)j) % (unsigned)G); };

  if (tid == 0) {
    abort_s = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full(s), 1);
      mbar_init(empty(s), 6);   // the step's four expansion warps, the MMA commit, the sums warp
    }
    for (int b = 0; b < kSets; ++b) {
      mbar_init(a_full(b), 5);   // four expansion warps and the set's outlier warp
      mbar_init(a_empty(b), 1);
    }
    for (int d = 0; d < 2; ++d) {
      mbar_init(d_full(d), 1);
      mbar_init(d_empty(d), 4);
      mbar_init(o_full(d), 1);
      mbar_init(o_empty(d), 4);
    }
    for (int q = 0; q < kXs; ++q) {
      mbar_init(xs_full(q), 1);
      mbar_init(xs_empty(q), 4);
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the outlier tiles start as all zeros
  for (int i = tid; i < kSets * kOutTileBytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(out_tiles)[i] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem0 = tmem_base_s;
  // tensor-memory columns: A buffers 0 .. 127 (64 each), step accumulators, outlier accumulators
  auto tm_a = [&](int b) { return tmem0 + (unsigned)(b * 64); };
  auto tm_d = [&](int d) { return tmem0 + (unsigned)(128 + d * TOK); };
  auto tm_o = [&](int o) { return tmem0 + (unsigned)(128 + 2 * TOK + o * TOK); };
  asm volatile("griddepcontrol.launch_dependents;");
  bool ok = *reinterpret_cast<volatile int32_t*>(p.status) == 0;   // an earlier launch gave up: do no work
  int issued = 0;   // stages armed by the producer

  if (warp == kWarpProducer) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      // the codes of the first stages do not depend on the previous kernel: they are requested before the wait
      const int pre = nsteps < kStages ? nsteps : kStages;
      for (int j = 0; j < pre && ok; ++j) {
        const int tile = tile_of(j), grp = grp_of(j);
        mbar_expect_tx(full(j), kCodeBytes + kXBytes);
        tma_load_2d(smem_u32(code_tile(j)), &tmc, grp * 4 * BITS, tile * kRows, full(j));
        issued = j + 1;
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int j = 0; j < nsteps && ok; ++j) {
        const int tile = tile_of(j), grp = grp_of(j);
        const int s = j % kStages;
        if (j >= kStages) {
          ok = mbar_wait(empty(s), ((j / kStages) - 1) & 1, abort_flag, lim);
          if (!ok) break;
          mbar_expect_tx(full(s), kCodeBytes + kXBytes);
          tma_load_2d(smem_u32(code_tile(s)), &tmc, grp * 4 * BITS, tile * kRows, full(s));
          issued = j + 1;
        }
        tma_load_2d(smem_u32(x_tile(s, 0)), &tmx, grp * 128, 0, full(s));
        tma_load_2d(smem_u32(x_tile(s, 1)), &tmx, grp * 128 + 64, 0, full(s));
      }
    }
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      // instruction descriptor: FP32 accumulate, A and B fp16, K-major, N = TOK, M = 128
      const unsigned idesc = (1u << 4) | ((unsigned)(TOK >> 3) << 17) | ((unsigned)(kRows >> 4) << 24);
      int piece = 0;
      for (int j = 0; j < nsteps && ok; ++j) {
        const int grp = grp_of(j);
        const int s = j % kStages, b = j % kSets;
        const bool first = j == 0 || grp == 0, last = j == nsteps - 1 || grp == G - 1;
        const int o = piece & 1;
        ok = mbar_wait(full(s), (j / kStages) & 1, abort_flag, lim) && mbar_wait(a_full(b), (j / kSets) & 1, abort_flag, lim);
        if (ok && first && piece >= 2) ok = mbar_wait(o_empty(o), ((piece >> 1) - 1) & 1, abort_flag, lim);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t dx0 = umma_desc(smem_u32(x_tile(s, 0))), dx1 = umma_desc(smem_u32(x_tile(s, 1)));
        const uint64_t do0 = umma_desc(smem_u32(out_tiles + b * kOutTileBytes)),
                       do1 = umma_desc(smem_u32(out_tiles + b * kOutTileBytes + kOutTileBytes / 2));
        // MMAs into one accumulator depend on one another (a chain of K = 16 slices), so the step's chains are issued
        // interleaved: the step accumulator(s) and the outlier accumulator advance together
#pragma unroll
        for (int h = 0; h < AS; ++h) {
          const int q = j * AS + h, d = q & 1;
          if (q >= 2) ok = mbar_wait(d_empty(d), ((q >> 1) - 1) & 1, abort_flag, lim);
          if (!ok) break;
        }
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int k = 0; k < 8 / AS; ++k) {
#pragma unroll
          for (int h = 0; h < AS; ++h) {
            const int kk = h * (8 / AS) + k;   // K = 16 slice of the step
            umma_ts(tm_d((j * AS + h) & 1), tm_a(b) + (unsigned)(8 * kk), (kk < 4 ? dx0 : dx1) + (uint64_t)(2 * (kk & 3)), idesc,
                    k != 0);
            umma_f16(tm_o(o), (kk < 4 ? do0 : do1) + (uint64_t)(2 * (kk & 3)), (kk < 4 ? dx0 : dx1) + (uint64_t)(2 * (kk & 3)),
                     idesc, !(first && k == 0 && h == 0));
          }
        }
#pragma unroll
        for (int h = 0; h < AS; ++h) umma_commit(d_full((j * AS + h) & 1));
        umma_commit(a_empty(b));
        umma_commit(empty(s));
        if (last) {
          umma_commit(o_full(o));
          ++piece;
        }
      }
    }
  } else if (warp >= kWarpExpand0 && warp < kWarpEpi0) {
    // ------------------------------------------------------------------ expansion: codes -> tensor memory, outliers -> tile
    const int set = (warp - kWarpExpand0) >> 2;
    const int quad = warp & 3;                 // tensor-memory lane quarter this warp may access
    const int r = quad * 32 + lane;            // row inside the tile
    for (int j = set; j < nsteps && ok; j += kSets) {
      const int s = j % kStages;
      ok = mbar_wait_warp(full(s), (j / kStages) & 1, abort_flag, lim);
      if (!ok) break;
      // the row's packed words of the step
      unsigned w[4 * BITS];
      {
        const unsigned char* crow = code_tile(s) + r * CB;
#pragma unroll
        for (int c = 0; c < BITS; ++c) {
          const int pc = BITS == 4 ? (c ^ ((r >> 1) & 3)) : c;   // 64-byte rows are stored with the 64-byte swizzle
          const uint4 v = *reinterpret_cast<const uint4*>(crow + pc * 16);
          w[4 * c] = v.x; w[4 * c + 1] = v.y; w[4 * c + 2] = v.z; w[4 * c + 3] = v.w;
        }
      }
      // pairs (columns 2h, 2h+1) as fp16 subnormals at mantissa position 0: column pair h of the step -> word h
      unsigned a[64];
      if (BITS == 4) {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          a[4 * t] = w[t] & 0x000F000Fu;
          a[4 * t + 1] = (w[t] >> 4) & 0x000F000Fu;
          a[4 * t + 2] = (w[t] >> 8) & 0x000F000Fu;
          a[4 * t + 3] = (w[t] >> 12) & 0x000F000Fu;
        }
      } else {
#pragma unroll
        for (int run = 0; run < 4; ++run) {
          const unsigned* w3 = w + 3 * run;
#pragma unroll
          for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int pp = 0; pp < 5; ++pp) a[16 * run + 5 * i + pp] = (w3[i] >> (3 * pp)) & 0x00070007u;
          a[16 * run + 15] = ((w3[0] >> 15) & 0x00010001u) | ((w3[1] >> 14) & 0x00020002u) | ((w3[2] >> 13) & 0x00040004u);
        }
      }
      // the A buffer and the outlier tile of this set are free once the MMAs of two steps ago have completed
      if (j >= kSets) ok = mbar_wait_warp(a_empty(set), ((j / kSets) - 1) & 1, abort_flag, lim);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      {
        const unsigned ta = tm_a(set) + ((unsigned)(quad * 32) << 16);
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st16(ta + (unsigned)(16 * c), a + 16 * c);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(a_full(set));
        mbar_arrive(empty(s));
      }
    }
  } else if (warp >= kWarpEpi0 && warp < kWarpSums) {
    // ------------------------------------------------------------------ epilogue: one thread per row
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    float yacc[TOK];
#pragma unroll
    for (int m = 0; m < TOK; ++m) yacc[m] = 0.f;
    int piece = 0;
    bool head = true;   // the current piece contains the first step of this CTA
    // scale and zero-point words of the next three steps: requested that far ahead, so that no step waits for memory
    constexpr int kAhead = 3;
    unsigned sz_ring[kAhead][AS];
    auto load_sz = [&](int j, unsigned (&dst)[AS]) {
      if (j < nsteps) {
        const int rown = tile_of(j) * kRows + r, grpn = grp_of(j);
#pragma unroll
        for (int h = 0; h < AS; ++h) dst[h] = __ldg(p.szt + (size_t)(grpn * AS + h) * p.N + (rown < p.N ? rown : p.N - 1));
      }
    };
#pragma unroll
    for (int a = 0; a < kAhead; ++a) load_sz(a, sz_ring[a]);
    asm volatile("griddepcontrol.wait;" ::: "memory");   // y and the workspace may still be in use by the previous kernel
    for (int j = 0; j < nsteps && ok; ++j) {
      const int tile = tile_of(j), grp = grp_of(j);
      const int row = tile * kRows + r;
      const bool last = j == nsteps - 1 || grp == G - 1;
      const int xq = j % kXs;
      unsigned sz[AS];
#pragma unroll
      for (int h = 0; h < AS; ++h) sz[h] = sz_ring[0][h];
#pragma unroll
      for (int a = 0; a + 1 < kAhead; ++a)
#pragma unroll
        for (int h = 0; h < AS; ++h) sz_ring[a][h] = sz_ring[a + 1][h];
      load_sz(j + kAhead, sz_ring[kAhead - 1]);
      ok = mbar_wait_warp(xs_full(xq), (j / kXs) & 1, abort_flag, lim);
      if (!ok) break;
#pragma unroll
      for (int h = 0; h < AS; ++h) {
        const int q = j * AS + h, d = q & 1;
        const float sc = __half2float(__ushort_as_half((unsigned short)(sz[h] & 0xFFFFu)));
        const float s2 = sc * 16777216.f, szf = sc * (float)(sz[h] >> 16);
        ok = mbar_wait_warp(d_full(d), (q >> 1) & 1, abort_flag, lim);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        unsigned v[TOK];
#pragma unroll
        for (int c = 0; c < TOK / 16; ++c)
          tmem_ld16(tm_d(d) + ((unsigned)(quad * 32) << 16) + (unsigned)(16 * c), reinterpret_cast<unsigned(&)[16]>(v[16 * c]));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(d_empty(d));
        const float4* xs4 = reinterpret_cast<const float4*>(xsum + (xq * AS + h) * TOK);
#pragma unroll
        for (int m4 = 0; m4 < TOK / 4; ++m4) {
          const float4 xs = xs4[m4];
          yacc[4 * m4] = fmaf(s2, __uint_as_float(v[4 * m4]), fmaf(-szf, xs.x, yacc[4 * m4]));
          yacc[4 * m4 + 1] = fmaf(s2, __uint_as_float(v[4 * m4 + 1]), fmaf(-szf, xs.y, yacc[4 * m4 + 1]));
          yacc[4 * m4 + 2] = fmaf(s2, __uint_as_float(v[4 * m4 + 2]), fmaf(-szf, xs.z, yacc[4 * m4 + 2]));
          yacc[4 * m4 + 3] = fmaf(s2, __uint_as_float(v[4 * m4 + 3]), fmaf(-szf, xs.w, yacc[4 * m4 + 3]));
        }
      }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(xs_empty(xq));
      if (last) {
        const int o = piece & 1;
        ok = mbar_wait_warp(o_full(o), (piece >> 1) & 1, abort_flag, lim);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        unsigned v[TOK];
#pragma unroll
        for (int c = 0; c < TOK / 16; ++c)
          tmem_ld16(tm_o(o) + ((unsigned)(quad * 32) << 16) + (unsigned)(16 * c), reinterpret_cast<unsigned(&)[16]>(v[16 * c]));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(o_empty(o));
        const bool whole = grp == G - 1 && (head ? grp0 == 0u : true) && (j + 1 >= G);   // the piece is the whole tile
        if (whole) {
          if (row < p.N) {
#pragma unroll
            for (int m = 0; m < TOK; ++m) {
              if (m < p.M) {
                const float f = yacc[m] + __uint_as_float(v[m]);
                const size_t idx = (size_t)m * p.N + row;
                if (p.yd == GWQ_F32) reinterpret_cast<float*>(p.y)[idx] = f;
                else if (p.yd == GWQ_F16) reinterpret_cast<__half*>(p.y)[idx] = __float2half_rn(f);
                else reinterpret_cast<__nv_bfloat16*>(p.y)[idx] = __float2bfloat16_rn(f);
              }
            }
          }
        } else {
          float* slot = p.partial + (size_t)(2 * blockIdx.x + (head ? 0 : 1)) * (TOK * kRows);
#pragma unroll
          for (int m = 0; m < TOK; ++m) slot[m * kRows + r] = yacc[m] + __uint_as_float(v[m]);
        }
#pragma unroll
        for (int m = 0; m < TOK; ++m) yacc[m] = 0.f;
        ++piece;
        head = false;
      }
    }
  } else if (warp == kWarpSums) {
    // ------------------------------------------------------------------ sums of x over the step's groups, per token
    const int gid = lane >> 2, t = lane & 3;
    for (int j = 0; j < nsteps && ok; ++j) {
      const int s = j % kStages, xq = j % kXs;
      ok = mbar_wait_warp(full(s), (j / kStages) & 1, abort_flag, lim);
      if (ok && j >= kXs) ok = mbar_wait_warp(xs_empty(xq), ((j / kXs) - 1) & 1, abort_flag, lim);
      if (!ok) break;
      float acc[AS][TOK / 8][4];
#pragma unroll
      for (int h = 0; h < AS; ++h)
#pragma unroll
        for (int nb = 0; nb < TOK / 8; ++nb)
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[h][nb][i] = 0.f;
#pragma unroll
      for (int kb = 0; kb < 2; ++kb) {
        const unsigned char* xt = x_tile(s, kb);
#pragma unroll
        for (int nb = 0; nb < TOK / 8; ++nb) {
          const int n = nb * 8 + gid;   // token row of the tile
          const unsigned char* xrow = xt + n * 128 + 4 * t;
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16) {
            const unsigned b0 = *reinterpret_cast<const unsigned*>(xrow + (((2 * k16) ^ (n & 7)) << 4));
            const unsigned b1 = *reinterpret_cast<const unsigned*>(xrow + (((2 * k16 + 1) ^ (n & 7)) << 4));
            mma16816_ones(acc[G64 ? kb : 0][nb], b0, b1);
          }
        }
      }
      if (gid == 0) {
#pragma unroll
        for (int h = 0; h < AS; ++h)
#pragma unroll
          for (int nb = 0; nb < TOK / 8; ++nb)
            *reinterpret_cast<float2*>(xsum + (xq * AS + h) * TOK + nb * 8 + 2 * t) = make_float2(acc[h][nb][0], acc[h][nb][1]);
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(xs_full(xq));
        mbar_arrive(empty(s));
      }
    }
  } else {
    // ------------------------------------------------------------------ outliers of the step's block -> the set's tile
    const int set = warp - kWarpOut0;
    unsigned char* otile = out_tiles + set * kOutTileBytes;
    constexpr int kHeld = 8;                   // entries per lane kept in registers (256 per block; the rest is re-read)
    unsigned held[kHeld];                      // the block's first entries; after the step: what has to be taken out again
    int e0 = 0, e1 = 0, c0 = 0, c1 = 0;        // entries of this step's block, and of the block this set dropped last
    // byte offset of entry v inside an outlier tile: two k-blocks, rows of 128 bytes, 128-byte swizzle
    auto out_off = [&](unsigned v) {
      const unsigned r = (v >> 23) & 127u, c = (v >> 16) & 127u;
      return (c >> 6) * (unsigned)(kOutTileBytes / 2) + r * 128u + ((((c & 63u) >> 3) ^ (r & 7u)) << 4) + ((c & 7u) << 1);
    };
    int n0 = 0, n1 = 0;                        // extents of the block after next of this set (requested two steps ahead)
    auto fetch_extents = [&](int j) {
      if (j < nsteps) {
        n0 = __ldg(p.ob_ptr + it0 + j);
        n1 = __ldg(p.ob_ptr + it0 + j + 1);
      }
    };
    auto fetch = [&](int j) {   // first entries of the block of step j, whose extents are in (n0, n1) by now
      e0 = e1 = 0;
      if (j < nsteps) {
        e0 = n0;
        e1 = n1;
#pragma unroll
        for (int i = 0; i < kHeld; ++i) held[i] = e0 + lane + 32 * i < e1 ? __ldg(p.ob + e0 + lane + 32 * i) : 0xFFFFFFFFu;
      }
    };
    unsigned prev[kHeld];
#pragma unroll
    for (int i = 0; i < kHeld; ++i) prev[i] = 0xFFFFFFFFu;
    fetch_extents(set);
    fetch(set);
    fetch_extents(set + kSets);
    for (int j = set; j < nsteps && ok; j += kSets) {
      if (j >= kSets) ok = mbar_wait_warp(a_empty(set), ((j / kSets) - 1) & 1, abort_flag, lim);   // MMAs of two steps ago done
      if (!ok) break;
      // take out what the last step of this set dropped in, then drop in this step's entries
#pragma unroll
      for (int i = 0; i < kHeld; ++i)
        if (prev[i] != 0xFFFFFFFFu) *reinterpret_cast<unsigned short*>(otile + out_off(prev[i])) = 0;
      for (int e = c0 + lane + 32 * kHeld; e < c1; e += 32)
        *reinterpret_cast<unsigned short*>(otile + out_off(__ldg(p.ob + e))) = 0;
#pragma unroll
      for (int i = 0; i < kHeld; ++i) {
        prev[i] = held[i];
        if (held[i] != 0xFFFFFFFFu) *reinterpret_cast<unsigned short*>(otile + out_off(held[i])) = (unsigned short)held[i];
      }
      for (int e = e0 + lane + 32 * kHeld; e < e1; e += 32) {
        const unsigned v = __ldg(p.ob + e);
        *reinterpret_cast<unsigned short*>(otile + out_off(v)) = (unsigned short)v;
      }
      c0 = e0;
      c1 = e1;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
      __syncwarp();
      if (lane == 0) mbar_arrive(a_full(set));
      fetch(j + kSets);   // behind the proxy fence, which would have waited for these loads
      fetch_extents(j + 2 * kSets);
    }
  }
  if (!ok) {
    *abort_flag = 1;
    atomicExch(p.status, (int32_t)GWQ_ERR_TIMEOUT);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kWarpProducer && lane == 0 && abort_s) {
    // bulk copies that were issued must land before the shared memory is given back
    int zero = 0;
    for (int s = 0; s < kStages; ++s) {
      if (issued > s) {
        const int last_j = ((issued - 1 - s) / kStages) * kStages + s;   // last step armed on stage s
        (void)mbar_wait(full(s), (last_j / kStages) & 1, &zero, kSpinCycles);
      }
    }
  }
  if (warp == kWarpMma && lane == 0 && abort_s) {
    // MMAs in flight still read the stages and write tensor memory: one more commit arrives when all have completed
    int zero = 0;
    umma_commit(drain_bar);
    (void)mbar_wait(drain_bar, 0, &zero, kSpinCycles);
  }
  __syncthreads();
  if (warp == kWarpMma) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem0), "r"(kTmemCols) : "memory");
  }
}

// Adds the partial sums of the tiles that several CTAs share, in CTA order, and stores the rows.  One CTA per tile
// and block of 8 tokens, one thread per (row, token); the loads of a sum are requested four at a time.
template <int TOK>
__global__ void __launch_bounds__(kRows * 8) skinny_fixup_kernel(const float* __restrict__ partial, void* y, gwq_dtype yd,
                                                                int N, int M, int G, long long total, int P) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int tile = blockIdx.x, r = threadIdx.x, m = blockIdx.y * 8 + threadIdx.y;
  const long long first = (long long)tile * G, last = first + G - 1;
  // owner of a step: the last CTA whose range begins at or before it
  const int p_first = (int)(((first + 1) * P + total - 1) / total) - 1, p_last = (int)(((last + 1) * P + total - 1) / total) - 1;
  if (p_first == p_last) return;   // one CTA had the whole tile and stored it
  const int row = tile * kRows + r;
  if (row >= N || m >= M) return;
  // CTA q's piece of this tile is its first piece (slot 2q) when its range begins inside the tile: every q but
  // possibly the first one, whose range may have begun in the tile before (then this is its last piece, slot 2q + 1)
  const int first_slot = 2 * p_first + (range_begin(total, P, p_first) < first ? 1 : 0);
  float v = 0.f;
  for (int q0 = p_first; q0 <= p_last; q0 += 4) {
    float t[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q = q0 + u;
      const int slot = q == p_first ? first_slot : 2 * q;
      t[u] = q <= p_last ? __ldg(partial + ((size_t)slot * TOK + m) * kRows + r) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) v += t[u];   // CTA order: the same bits every time
  }
  const size_t idx = (size_t)m * N + row;
  if (yd == GWQ_F32) reinterpret_cast<float*>(y)[idx] = v;
  else if (yd == GWQ_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
  else reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
}

template <int BITS, int TOK, bool G64>
gwq_status launch(const gwq_packed* P, const void* x, int M, void* y, gwq_dtype yd, void* ws, cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  EncodeTiledFn enc = encode_fn();
  if (!enc) return GWQ_ERR_CUDA;
  CUtensorMap tmx, tmc;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)P->K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)P->K * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)TOK};
    if (enc(&tmx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)(P->K / 32) * BITS, (cuuint64_t)P->N};
    const cuuint64_t strides[1] = {(cuuint64_t)(P->K / 32) * BITS * 4};
    const cuuint32_t box[2] = {(cuuint32_t)(4 * BITS), (cuuint32_t)kRows};
    if (enc(&tmc, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, P->codes, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            BITS == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GWQ_ERR_CUDA;
  }
  const int tiles = (P->N + kRows - 1) / kRows;
  SkinnyArgs a;
  a.szt = pv->sz_t; a.ob = pv->ob; a.ob_ptr = pv->ob_ptr; a.y = y; a.partial = static_cast<float*>(ws);
  a.status = pv->dev_status; a.yd = yd; a.N = P->N; a.K = P->K; a.M = M; a.G = P->K / 128;
  a.total = (long long)tiles * a.G; a.wait_cycles = pv->wait_cycles;
  const int sms = pv->sm_count > 0 ? pv->sm_count : 148;
  const int grid = a.total < sms ? (int)a.total : sms;
  const size_t smem = 1024 + (size_t)kStages * 16384 + (size_t)kSets * kOutTileBytes + (size_t)kXs * 2 * 32 * 4;
  if (cudaFuncSetAttribute(skinny_kernel<BITS, TOK, G64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return GWQ_ERR_CUDA;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, skinny_kernel<BITS, TOK, G64>, tmc, tmx, a) != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)((M + 7) / 8));
  cfg.blockDim = dim3(kRows, 8);
  cfg.dynamicSmemBytes = 0;
  if (cudaLaunchKernelEx(&cfg, skinny_fixup_kernel<TOK>, (const float*)a.partial, y, yd, P->N, M, a.G, a.total, grid) != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  return GWQ_OK;
}

}  // namespace

// The skinny kernel takes fp16 activations, up to 32 tokens, groups of 64 or 128, K a multiple of 128 up to 65536.
bool gwq_skinny_takes(const gwq_packed* P, gwq_dtype xd, int M) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  return xd == GWQ_F16 && (P->bits == 3 || P->bits == 4) && M >= 1 && M <= 32 && (P->group == 64 || P->group == 128) && P->K % 128 == 0 && P->K <= 65536 &&
         pv->ob && pv->ob_ptr && pv->sz_t;
}

// Workspace: two partial tiles per CTA.
size_t gwq_skinny_workspace_bytes(const gwq_packed* P, int M) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const int sms = pv->sm_count > 0 ? pv->sm_count : 148;
  (void)M;
  return (size_t)2 * sms * 32 * kRows * sizeof(float);   // token tiles of 32
}

gwq_status gwq_launch_skinny(const gwq_packed* P, const void* x, int M, void* y, gwq_dtype yd, void* ws, size_t ws_bytes,
                             cudaStream_t stream) {
  if (!ws || ws_bytes < gwq_skinny_workspace_bytes(P, M) || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0)
    return GWQ_ERR_WORKSPACE;
  const bool g64 = P->group == 64;
  if (P->bits == 4)
    return g64 ? launch<4, 32, true>(P, x, M, y, yd, ws, stream) : launch<4, 32, false>(P, x, M, y, yd, ws, stream);
  return g64 ? launch<3, 32, true>(P, x, M, y, yd, ws, stream) : launch<3, 32, false>(P, x, M, y, yd, ws, stream);
}
