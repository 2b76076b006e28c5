// Decode path (M <= 32) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w"): bandwidth-bound.
//
// One CTA owns 16 output rows; its 8 warps split K by quantization group (128 columns).
// Per group a warp streams the packed codes of its 16 rows straight from global memory
// into registers (each lane: one run of 32 columns for rows g and g+8), masks them into
// 16-bit floating-point integers and multiplies them with the activations on the tensor
// cores (mma.sync m16n8k16: the 16 weight rows are the A operand, 8 tokens the B operand,
// FP32 accumulators).  Scale and zero-point are applied once per group to the
// accumulator, y += s (sum x q) - s z (sum x), so no scaled weight is ever rounded:
//  * fp16 activations: the raw code bits are used as fp16 subnormals q 2^-24 (one shift
//    and one mask per pair of codes) and sum x comes from a second MMA whose A operand is
//    all ones;
//  * bf16 activations: (bits | magic) - (z | magic) gives q - z exactly (one more packed
//    subtract per pair), no second MMA.
// The pair-interleaved packed order makes both operands natural: pair h of a lane's run
// holds columns (2h, 2h+1), the same pair as 32-bit word h of its activation segment.
// Activations are staged in shared memory chunk by chunk (8 groups, double buffered, padded
// against bank conflicts); the CSR outliers of a row are added, chunk by chunk and from the
// same staged activations, by the warp that owns the row.  After the K loop the warps'
// partial sums meet in shared memory and y is stored.  The kernel is launched with programmatic stream serialization: its weight
// prefetch may overlap the previous kernel, everything that touches x or y comes after
// griddepcontrol.wait.
#include <type_traits>

#include "common.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kRows = 16;   // rows per CTA (one m16 tile)
constexpr int kDepth = 4;   // groups of codes in flight per warp
constexpr int kMaxTokens64 = 16;  // groups of 64: tokens one launch takes
// Groups of 64 with 9 to 16 tokens need four token blocks (184 to 229 registers, one CTA per SM): faster than the
// tensor-core kernel's 32-token tile up to about this many weights (measured: 59.8 against 84.8 us on 8192 x 8192,
// 184.5 against 163.1 us on 28672 x 8192), slower beyond.
constexpr long long kMaxWeights64Wide = 160LL * 1000 * 1000;

template <bool BF16>
__device__ __forceinline__ void mma16816(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
  if (BF16) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}

// (q | magic) - (z | magic) on both halves: exact small integers q - z.
template <bool BF16>
__device__ __forceinline__ unsigned sub_zero(unsigned qm, unsigned zm) {
  if (BF16) {
    __nv_bfloat162 r = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&qm), *reinterpret_cast<__nv_bfloat162*>(&zm));
    return *reinterpret_cast<unsigned*>(&r);
  } else {
    __half2 r = __hsub2(*reinterpret_cast<__half2*>(&qm), *reinterpret_cast<__half2*>(&zm));
    return *reinterpret_cast<unsigned*>(&r);
  }
}

// ---------------------------------------------------------------------------------------------
// One group step of a warp: 8 (x NB) weight MMAs for the 16 rows x 128 columns whose packed words
// are qa (row g) and qb (row g + 8) of this lane, against the activation words xr[nb][0..15]
// (word h = columns 2h, 2h+1 of the lane's run).
//
// Raw variant (fp16 activations).  The masked code bits are used directly as fp16 subnormals:
// a code at mantissa bit position p is the number q 2^(p-24).  Integer instructions are the
// scarce resource of this kernel (half-rate pipe), so codes are masked where they sit and only
// one shift per word moves the upper byte down; the positions that occur (0 and 4 for 4 bits,
// 0, 3 and 6 for 3 bits) each get their own accumulator, merged with the right power of two in
// the group epilogue.  With ONES, `xs` accumulates sum_k x_k through an A operand of all ones
// (otherwise the caller supplies that sum).
template <int NB>
struct AccRaw4 {
  float c0[NB][4], c4[NB][4], xs[NB][4];
};
template <int NB>
struct AccRaw3 {
  float c0[NB][4], c3[NB][4], c6[NB][4], xs[NB][4];
};
template <int NB>
struct AccSub {
  float c[NB][4];
};

#define GWQ_ONES 0x3C003C00u

template <int NB, bool ONES>
__device__ __forceinline__ void step_raw4(const unsigned (&qa)[4], const unsigned (&qb)[4],
                                          const unsigned (&xr)[NB][16], AccRaw4<NB>& acc) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const unsigned ta = qa[i] >> 8, tb = qb[i] >> 8;
    const unsigned a00 = qa[i] & 0x000F000Fu, b00 = qb[i] & 0x000F000Fu;  // pair 4i   (position 0)
    const unsigned a01 = qa[i] & 0x00F000F0u, b01 = qb[i] & 0x00F000F0u;  // pair 4i+1 (position 4)
    const unsigned a02 = ta & 0x000F000Fu, b02 = tb & 0x000F000Fu;        // pair 4i+2 (position 0)
    const unsigned a03 = ta & 0x00F000F0u, b03 = tb & 0x00F000F0u;        // pair 4i+3 (position 4)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      mma16816<false>(acc.c0[nb], a00, b00, a02, b02, xr[nb][4 * i], xr[nb][4 * i + 2]);
      mma16816<false>(acc.c4[nb], a01, b01, a03, b03, xr[nb][4 * i + 1], xr[nb][4 * i + 3]);
      if (ONES) {
        mma16816<false>(acc.xs[nb], GWQ_ONES, GWQ_ONES, GWQ_ONES, GWQ_ONES, xr[nb][4 * i], xr[nb][4 * i + 2]);
        mma16816<false>(acc.xs[nb], GWQ_ONES, GWQ_ONES, GWQ_ONES, GWQ_ONES, xr[nb][4 * i + 1], xr[nb][4 * i + 3]);
      }
    }
  }
}

template <int NB, bool ONES>
__device__ __forceinline__ void step_raw3(const unsigned (&qa)[3], const unsigned (&qb)[3],
                                          const unsigned (&xr)[NB][16], AccRaw3<NB>& acc) {
  unsigned a[16], b[16];  // pair h of rows g / g + 8; positions: h%5 in {0,3} -> 0, {1,4} -> 3, {2} -> 6, h=15 -> 6
  unsigned ta[3], tb[3];
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    ta[i] = qa[i] >> 9;
    tb[i] = qb[i] >> 9;
    a[5 * i] = qa[i] & 0x00070007u;     b[5 * i] = qb[i] & 0x00070007u;
    a[5 * i + 1] = qa[i] & 0x00380038u; b[5 * i + 1] = qb[i] & 0x00380038u;
    a[5 * i + 2] = qa[i] & 0x01C001C0u; b[5 * i + 2] = qb[i] & 0x01C001C0u;
    a[5 * i + 3] = ta[i] & 0x00070007u; b[5 * i + 3] = tb[i] & 0x00070007u;
    a[5 * i + 4] = ta[i] & 0x00380038u; b[5 * i + 4] = tb[i] & 0x00380038u;
  }
  // columns 30, 31: bit w of their codes is bit 15 / 31 of word w; assembled at position 6
  a[15] = (ta[0] & 0x00400040u) | ((qa[1] >> 8) & 0x00800080u) | ((qa[2] >> 7) & 0x01000100u);
  b[15] = (tb[0] & 0x00400040u) | ((qb[1] >> 8) & 0x00800080u) | ((qb[2] >> 7) & 0x01000100u);
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
#define GWQ_M3(ACC, H1, H2) \
  mma16816<false>(ACC[nb], a[H1], b[H1], a[H2], b[H2], xr[nb][H1], xr[nb][H2]); \
  if (ONES) mma16816<false>(acc.xs[nb], GWQ_ONES, GWQ_ONES, GWQ_ONES, GWQ_ONES, xr[nb][H1], xr[nb][H2]);
    GWQ_M3(acc.c0, 0, 3) GWQ_M3(acc.c0, 5, 8) GWQ_M3(acc.c0, 10, 13)
    GWQ_M3(acc.c3, 1, 4) GWQ_M3(acc.c3, 6, 9) GWQ_M3(acc.c3, 11, 14)
    GWQ_M3(acc.c6, 2, 7) GWQ_M3(acc.c6, 12, 15)
#undef GWQ_M3
  }
}

// Subtract variant (bf16 activations): (bits | magic) - (z | magic) = q - z exactly in bf16; one
// accumulator, no ones operand.  zma / zmb hold magic | z in both halves.
template <int BITS, int NB>
__device__ __forceinline__ void step_sub(const unsigned (&qa)[BITS], const unsigned (&qb)[BITS], unsigned zma,
                                         unsigned zmb, const unsigned (&xr)[NB][16], AccSub<NB>& acc) {
  constexpr unsigned MAGIC = 0x43004300u;  // bf16 128.0: ulp = 1
  unsigned a[16], b[16];
  if (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        a[4 * i + j] = sub_zero<true>(((qa[i] >> (4 * j)) & 0x000F000Fu) | MAGIC, zma);
        b[4 * i + j] = sub_zero<true>(((qb[i] >> (4 * j)) & 0x000F000Fu) | MAGIC, zmb);
      }
  } else {
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
      for (int p = 0; p < 5; ++p) {
        a[5 * i + p] = sub_zero<true>(((qa[i] >> (3 * p)) & 0x00070007u) | MAGIC, zma);
        b[5 * i + p] = sub_zero<true>(((qb[i] >> (3 * p)) & 0x00070007u) | MAGIC, zmb);
      }
    const unsigned la = ((qa[0] >> 15) & 0x00010001u) | ((qa[1] >> 14) & 0x00020002u) |
                        ((qa[BITS - 1] >> 13) & 0x00040004u);
    const unsigned lb = ((qb[0] >> 15) & 0x00010001u) | ((qb[1] >> 14) & 0x00020002u) |
                        ((qb[BITS - 1] >> 13) & 0x00040004u);
    a[15] = sub_zero<true>(la | MAGIC, zma);
    b[15] = sub_zero<true>(lb | MAGIC, zmb);
  }
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int m8 = 0; m8 < 8; ++m8)
      mma16816<true>(acc.c[nb], a[2 * m8], b[2 * m8], a[2 * m8 + 1], b[2 * m8 + 1], xr[nb][2 * m8],
                     xr[nb][2 * m8 + 1]);
}

template <int BITS>
__device__ __forceinline__ void load_run(const uint32_t* __restrict__ base, unsigned off, unsigned (&w)[BITS]) {
  const uint32_t* p = base + off;
  if (BITS == 4) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));  // streamed once: evict first
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[BITS - 1] = v.w;
  } else {
#pragma unroll
    for (int i = 0; i < BITS; ++i) w[i] = __ldcs(p + i);
  }
}

// Same load, executed only where `pred` holds (predicated instructions, no branch).
template <int BITS>
__device__ __forceinline__ void load_run_if(const uint32_t* __restrict__ base, unsigned off, unsigned (&w)[BITS],
                                            bool pred) {
  const uint32_t* p = base + off;
  if (BITS == 4) {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %5, 0;\n @q ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];\n}\n"
        : "+r"(w[0]), "+r"(w[1]), "+r"(w[2]), "+r"(w[BITS - 1])
        : "l"(p), "r"((int)pred));
  } else {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %4, 0;\n @q ld.global.cs.u32 %0, [%3];\n @q ld.global.cs.u32 %1, [%3+4];\n"
        " @q ld.global.cs.u32 %2, [%3+8];\n}\n"
        : "+r"(w[0]), "+r"(w[1]), "+r"(w[2])
        : "l"(p), "r"((int)pred));
  }
}

__device__ __forceinline__ void store_y(void* y, gwq_dtype yd, long long idx, float v) {
  if (yd == GWQ_F32) reinterpret_cast<float*>(y)[idx] = v;
  else if (yd == GWQ_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
  else reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
}

template <bool BF16>
__device__ __forceinline__ float act_to_float(uint16_t b) {
  if (BF16) return __uint_as_float((unsigned)b << 16);
  return __half2float(__ushort_as_half(b));
}

struct DecodeArgs {
  const uint32_t* codes;
  const uint32_t* szt;   // [K / group][N]: scale (fp16 bits) | zero-point << 16
  const int32_t* row_ptr;
  const uint32_t* cv;  // per outlier: fp16 value << 16 | column
  const uint16_t* x;
  const uint16_t* xt;  // [K][TP] copy of x (ring mode with more than one token), else null
  const float* xg;     // [K/128][TP] sums of x over each group of columns (same mode), else null
  void* y;
  gwq_dtype yd;
  int N, K, M;
};

// One launch may serve several layers that read the same activations (sibling projections): the grid is the
// concatenation of the layers' row blocks, layer l owning the blocks [first_block[l], first_block[l + 1]).
constexpr int kMaxLayers = GWQ_MULTI_MAX;
struct LayerArgs {
  const uint32_t* codes;
  const uint32_t* szt;
  const int32_t* row_ptr;
  const uint32_t* cv;
  void* y;
  int N;
};
struct MultiArgs {
  LayerArgs layer[kMaxLayers];
  int first_block[kMaxLayers + 1];
  int count;
  int sm_count;
  const uint16_t* x;
  const uint16_t* xt;
  const float* xg;
  gwq_dtype yd;
  int K, M;
};

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// Activations are staged chunk by chunk: one chunk is 8 groups (1024 columns), one group per warp,
// double buffered, so shared memory stays small for every M and K and the B fragments never come
// from global memory.  16-byte piece c of token row m sits at piece c + (c >> 3) + 2 (m & 1) of its
// row (one pad piece per 128 bytes, odd rows shifted by two): the 64-byte segments of the four lanes
// of a quad and of two neighbouring token rows then fall into all eight 16-byte bank groups.
constexpr int kOutSlots = 3;                          // outlier entries per lane kept in registers
constexpr int kChunkGroups = kWarps;                 // groups per chunk
constexpr int kChunkPieces = kChunkGroups * 16;      // 16-byte pieces per token row per chunk
constexpr int kRowPitch = kChunkPieces + kChunkPieces / 8 + 4;   // pieces, with padding
__device__ __forceinline__ int xs_piece(int c, int m) { return m * kRowPitch + c + (c >> 3) + ((m & 1) << 1); }

// Sum, over the lanes that hold the same token group, VT per-lane values: TS token groups are
// interleaved over the lanes (group = lane % TS).  Afterwards lane L holds, in v[0], the total of
// token (L % TS) * VT + value index, the value index being L / (32 / VT) for VT < 8 ... see below.
template <int VT, int TS>
__device__ __forceinline__ void reduce_tokens(float (&v)[VT], int lane) {
  int n = VT;
#pragma unroll
  for (int o = 16; o >= TS; o >>= 1) {
    if (n > 1) {
      const int half = n >> 1;
      const bool up = (lane & o) != 0;
#pragma unroll
      for (int i = 0; i < (VT > 1 ? VT / 2 : 1); ++i) {
        if (i < half) {
          const float send = up ? v[i] : v[i + half];
          const float keep = up ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, o);
        }
      }
      n = half;
    } else {
      v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], o);
    }
  }
}

template <int BITS, int NB, bool BF16>
struct StepAcc;
template <int NB> struct StepAcc<4, NB, false> { using type = AccRaw4<NB>; };
template <int NB> struct StepAcc<3, NB, false> { using type = AccRaw3<NB>; };
template <int BITS, int NB> struct StepAcc<BITS, NB, true> { using type = AccSub<NB>; };

// TP = tokens rounded up to 1, 4, 8, 16 or 32.  Group size 128.
// NBUF = 0: the activations of all chunks are staged up front by the whole CTA (small M K).
// NBUF = 2, 3: every warp keeps a private ring of NBUF buffers with the activations of its own group only
//           (M x 128 columns), copied one step ahead with cp.async; no CTA barrier in the K loop.
constexpr int kTilePitch = 16;   // pieces per token row of a warp tile: no padding, the pieces of a row are permuted
// piece p (16 bytes) of token row m of a warp tile: the XOR keeps the four lanes of a quad and four neighbouring
// token rows in different 16-byte bank groups
__device__ __forceinline__ int tile_piece(int pc, int m) { return m * kTilePitch + (pc ^ (pc >> 3) ^ ((m & 3) << 1)); }
// G64: groups of 64 columns.  A warp step still covers 128 columns, i.e. two groups: the runs of lanes t = 0, 1 belong
// to the first, those of t = 2, 3 to the second.  An MMA sums over all four lanes, so the two groups are kept apart on
// the token side: a token block holds 4 tokens, output column n < 4 is token n with the activations of the second
// group replaced by zeros (lanes t >= 2 read the zero page), column n >= 4 is token n - 4 with those of the first
// group replaced by zeros.  Accumulator columns 2t, 2t+1 of lane t then belong to the lane's own group (t >> 1), whose
// scale and zero-point it applies; the two halves of a token meet in the final sum.  With more than one token the sums
// of x come from the all-ones MMA (which sees the same zeros); a single token's are reduced over half a warp each.
// TP <= 16.
template <int TP, bool G64>
struct TokenBlocks { static constexpr int value = G64 ? (TP <= 4 ? 1 : TP / 4) : (TP <= 8 ? 1 : TP / 8); };
template <int BITS, int TP, bool BF16, int NBUF, bool G64>
__global__ void __launch_bounds__(kThreads, TokenBlocks<TP, G64>::value == 1 ? 3 : (TokenBlocks<TP, G64>::value == 2 ? 2 : 1))
decode_kernel(const MultiArgs ma) {
  // the layer this CTA works for and its row block inside that layer
  DecodeArgs p;
  int blk = blockIdx.x;
  {
    int l = 0;
#pragma unroll
    for (int i = 1; i < kMaxLayers; ++i)
      if (i < ma.count && (int)blockIdx.x >= ma.first_block[i]) l = i;
#pragma unroll
    for (int i = 0; i < kMaxLayers; ++i) {
      if (i == l) {
        p.codes = ma.layer[i].codes; p.szt = ma.layer[i].szt;
        p.row_ptr = ma.layer[i].row_ptr; p.cv = ma.layer[i].cv; p.y = ma.layer[i].y; p.N = ma.layer[i].N;
        blk = (int)blockIdx.x - ma.first_block[i];
      }
    }
    p.x = ma.x; p.xt = ma.xt; p.xg = ma.xg; p.yd = ma.yd; p.K = ma.K; p.M = ma.M;
  }
  constexpr int NB = TokenBlocks<TP, G64>::value;   // token blocks of the MMA (8 tokens; 4 with groups of 64)
  constexpr int WPR = BITS;                   // words per run of 32 columns
  // raw path: sum_k x_k of a group from shared memory (one token), from the table that comes with the
  // token-major copy (ring mode), else from a second MMA with an all-ones A operand
  constexpr bool ONES = !BF16 && TP != 1 && (G64 || NBUF == 0);
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int ngroups = p.K >> 7;               // warp steps of 128 columns in a row
  const int ntab = G64 ? 2 * ngroups : ngroups;   // scale / zero-point entries in a row
  // shared: zero page 64 B | scale and zero-point table [ntab][16 rows] u32 | red [kWarps][NB][16][8] f32 |
  //         outl [16][TP] f32 | x chunk buffers 2 x [M][kRowPitch] pieces
  // (the table is group-major: the eight rows a load instruction asks for are eight neighbouring words, no bank
  // conflicts however wide the layer is)
  uint32_t* sm_tab = reinterpret_cast<uint32_t*>(smem_raw + 64);
  float* sm_red = reinterpret_cast<float*>(sm_tab + kRows * ntab);
  float* sm_out = sm_red + kWarps * NB * 128;
  uint4* sm_x = reinterpret_cast<uint4*>(sm_out + kRows * TP);
  const int buf_pieces = p.M * kRowPitch;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, t = lane & 3;
  const int r0 = blk * kRows;
  const int ra = min(r0 + gid, p.N - 1), rb = min(r0 + gid + 8, p.N - 1);
  const unsigned row_words = (unsigned)(p.K >> 5) * WPR;
  constexpr unsigned kStepWords = kWarps * 4 * WPR;  // codes of 8 groups
  unsigned oa = (unsigned)ra * row_words + (unsigned)(warp * 4 + t) * WPR;  // group `warp`, this lane's run
  unsigned ob = (unsigned)rb * row_words + (unsigned)(warp * 4 + t) * WPR;
  const int nsteps = (ngroups - warp + kWarps - 1) / kWarps;  // this warp's groups: warp, warp + 8, ...
  const int nchunks = (ngroups + kChunkGroups - 1) / kChunkGroups;

  pdl_launch_dependents();

  // ---- everything that does not depend on the previous kernel: all loads are issued before any is awaited
  // CSR extents of the two rows this warp owns (rows 2 warp and 2 warp + 1 of the CTA)
  int rp = 0;
  if (lane < 3) rp = __ldg(p.row_ptr + min(r0 + 2 * warp + lane, p.N));
  {
    // scales and zero-points of the 16 rows: 64 contiguous bytes per group of the group-major table
    const int rows_here = min(kRows, p.N - r0);
    if (rows_here == kRows && (p.N & 3) == 0) {
      const unsigned dst0 = (unsigned)__cvta_generic_to_shared(sm_tab);
      for (int c = tid; c < 4 * ntab; c += kThreads) {   // piece c: rows 4 (c & 3) .. + 3 of group c >> 2
        const uint32_t* src = p.szt + (size_t)(c >> 2) * p.N + r0 + 4 * (c & 3);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (unsigned)c * 16u), "l"(src));
      }
    } else {   // partial last CTA, or rows that do not start on 16-byte boundaries: rows past N read as scale 0
      for (int i = tid; i < kRows * ntab; i += kThreads) {
        const int r = i & 15, g = i >> 4;
        sm_tab[i] = r < rows_here ? __ldg(p.szt + (size_t)g * p.N + r0 + r) : 0u;
      }
    }
  }
  unsigned wa[kDepth][BITS], wb[kDepth][BITS];
#pragma unroll
  for (int d = 0; d < kDepth; ++d) {
    if (d < nsteps) {
      load_run<BITS>(p.codes, oa + d * kStepWords, wa[d]);
      load_run<BITS>(p.codes, ob + d * kStepWords, wb[d]);
    }
  }
  if (tid < 16) reinterpret_cast<unsigned*>(smem_raw)[tid] = 0u;

  // CSR extents of the two owned rows.  Ring mode needs them now (lane = (entry, group of VT tokens): the first
  // kPre batches of outlier entries of both rows are requested before the wait on the previous kernel, they are
  // weights); with everything staged they are taken after the activations have been requested, so that waiting
  // for the row pointers delays nothing.
  int j0 = 0, j1 = 0, j2 = 0;
  if (NBUF != 0) {
    j0 = __shfl_sync(0xFFFFFFFFu, rp, 0);
    j1 = __shfl_sync(0xFFFFFFFFu, rp, 1);
    j2 = __shfl_sync(0xFFFFFFFFu, rp, 2);
  }
  constexpr int VT = TP < 8 ? TP : 8, TS = TP / VT, EPB = 32 / TS;
  constexpr int kPre = TP <= 8 ? 2 : 3;   // batches of EPB entries per row: 64 entries up to 8 tokens, 48 / 24 beyond
  unsigned epre[2][kPre];
  if (NBUF != 0) {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int jb = rr == 0 ? j0 : j1, je = rr == 0 ? j1 : j2;
#pragma unroll
      for (int u = 0; u < kPre; ++u) {
        const int j = jb + u * EPB + lane / TS;
        epre[rr][u] = j < je ? __ldg(p.cv + j) : 0u;   // value 0, column 0
      }
    }
  }
  // ---- from here on x is read
  pdl_wait();
  // NBUF == 0: copy of all activations into the chunk buffers, by the whole CTA: token row by token row, piece pc of a
  // row goes to chunk pc / 128, place xs_piece(pc % 128, m) (few instructions per piece: this runs in every CTA)
  auto stage_all = [&]() {
    const int ppr = p.K >> 3;   // 16-byte pieces per token row
    const unsigned base = (unsigned)__cvta_generic_to_shared(sm_x);
    for (int m = 0; m < p.M; ++m) {
      const uint16_t* src = p.x + (size_t)m * p.K;
      const unsigned dst0 = base + (unsigned)(m * kRowPitch + ((m & 1) << 1)) * 16u;
      for (int pc = tid; pc < ppr; pc += kThreads) {
        const int c = pc >> 7, q = pc & (kChunkPieces - 1);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (unsigned)(c * buf_pieces + q + (q >> 3)) * 16u),
                     "l"(src + pc * 8));
      }
    }
  };
  // ring mode: copy of the activations of this warp's step c (group warp + 8 c) into its buffer c % NBUF
  constexpr int kBufs = NBUF == 0 ? 1 : NBUF;
  const int tile_pieces = p.M * kTilePitch;
  uint4* wtile = sm_x + warp * kBufs * tile_pieces;
  // lane L copies piece L & 15 of the token rows (L >> 4), (L >> 4) + 2, ...: constant strides, three
  // instructions per 16-byte piece
  const int st_m0 = lane >> 4, st_pc = lane & 15;
  const unsigned st_dst0 = (unsigned)__cvta_generic_to_shared(wtile);
  const uint16_t* st_src0 = p.x + (size_t)st_m0 * p.K + (size_t)warp * 128 + st_pc * 8;
  auto stage_tile = [&](int c) {
    if (c < nsteps) {
      const uint16_t* src = st_src0 + (size_t)c * (kWarps * 128);
      const unsigned dst = st_dst0 + (unsigned)((c % kBufs) * tile_pieces) * 16u;
      for (int m = st_m0; m < p.M; m += 2) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (unsigned)tile_piece(st_pc, m) * 16u),
                     "l"(src));
        src += 2 * (size_t)p.K;
      }
    }
  };
  if (NBUF == 0) {
    stage_all();
  } else {
    stage_tile(0);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");   // also carries the scale / zero-point tables
  if (NBUF != 0) {   // the tiles of the following steps, one group each
#pragma unroll
    for (int c = 1; c + 1 < kBufs; ++c) {
      stage_tile(c);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }

  // outlier payload of the two owned rows.  With everything staged (NBUF == 0) entry lane + 32 e of a
  // row is loaded into cv[row][e] now (up to 96 per row; all ones = no entry) and meets the staged
  // activations after the loop; in ring mode the entries are read after the loop.
  unsigned cv[2][kOutSlots];
  if (NBUF == 0) {
    j0 = __shfl_sync(0xFFFFFFFFu, rp, 0);
    j1 = __shfl_sync(0xFFFFFFFFu, rp, 1);
    j2 = __shfl_sync(0xFFFFFFFFu, rp, 2);
#pragma unroll
    for (int e = 0; e < kOutSlots; ++e) {
      const int ja = j0 + lane + 32 * e, jb = j1 + lane + 32 * e;
      cv[0][e] = ja < j1 ? __ldcs(p.cv + ja) : 0xFFFFFFFFu;
      cv[1][e] = jb < j2 ? __ldcs(p.cv + jb) : 0xFFFFFFFFu;
    }
  }

  if (NBUF != 0) {
    // ring mode: the outliers are done now, while the first codes are still on their way.  The
    // activations come from the token-major copy xt[K][TP] (one short contiguous read per entry).
    // All reads for the entries requested above are issued before any is used; longer rows continue
    // with two batches of entries in flight.
    const uint16_t* xt = TP == 1 ? p.x : p.xt;
    const int part = lane % TS;
    auto xt_load = [&](unsigned ent) {
      const uint16_t* src = xt + (size_t)(ent & 0xFFFFu) * TP + part * VT;
      if (VT == 8) return __ldg(reinterpret_cast<const uint4*>(src));
      if (VT == 4) { const uint2 q = __ldg(reinterpret_cast<const uint2*>(src)); return make_uint4(q.x, q.y, 0, 0); }
      return make_uint4(__ldg(src), 0, 0, 0);
    };
    uint4 xpre[2][kPre];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr)
#pragma unroll
      for (int u = 0; u < kPre; ++u) xpre[rr][u] = xt_load(epre[rr][u]);
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int jb = rr == 0 ? j0 : j1, je = rr == 0 ? j1 : j2;
      float v[VT];
#pragma unroll
      for (int i = 0; i < VT; ++i) v[i] = 0.f;
      auto add = [&](unsigned ent, const uint4& xq) {
        const float wv = __half2float(__ushort_as_half((unsigned short)(ent >> 16)));
        const unsigned w4[4] = {xq.x, xq.y, xq.z, xq.w};
#pragma unroll
        for (int i = 0; i < VT; ++i)
          v[i] = fmaf(wv, act_to_float<BF16>((uint16_t)(w4[i >> 1] >> (16 * (i & 1)))), v[i]);
      };
#pragma unroll
      for (int u = 0; u < kPre; ++u) add(epre[rr][u], xpre[rr][u]);
      for (int jj = jb + kPre * EPB; jj < je; jj += 2 * EPB) {
        unsigned e[2];
        uint4 xq[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int j = jj + u * EPB + lane / TS;
          e[u] = j < je ? __ldg(p.cv + j) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) xq[u] = xt_load(e[u]);
#pragma unroll
        for (int u = 0; u < 2; ++u) add(e[u], xq[u]);
      }
      reduce_tokens<VT, TS>(v, lane);
      constexpr int LPV = 32 / VT;   // lanes per value after the halving stages
      const int tok = part * VT + lane / LPV;
      if ((lane % LPV) / TS == 0) sm_out[(2 * warp + rr) * TP + tok] = v[0];
    }
  }
  asm volatile("cp.async.wait_group %0;" ::"n"(NBUF == 0 ? 0 : NBUF - 2) : "memory");   // tables (and first tile) landed
  __syncthreads();

  // lane constants inside a chunk buffer: this lane's 64-byte segment of group `warp` for token gid
  // of every token block (lanes without a token read the zero page), the scale tables, the x sums
  // (ring mode: the four pieces of the segment sit in one aligned block of the permuted row, in the order i ^ xcx)
  int xoff[NB], xcx[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    const int m = G64 ? nb * 4 + (gid & 3) : nb * 8 + gid;
    const bool live = m < p.M && (!G64 || (gid >> 2) == (t >> 1));   // groups of 64: the other group's columns read as zero
    xoff[nb] = !live ? -1 : (NBUF == 0 ? xs_piece(warp * 16 + t * 4, m) : m * kTilePitch + ((t ^ ((m >> 1) & 1)) << 2));
    xcx[nb] = (NBUF == 0 || !live) ? 0 : ((t >> 1) ^ ((m & 1) << 1));
  }
  // scale | zero-point << 16 of row gid, group `warp` (groups of 64: the lane's own half of step `warp`)
  const uint32_t* tp = sm_tab + (G64 ? 2 * warp + (t >> 1) : warp) * kRows + gid;
  const int xsum_off = (NBUF == 0 ? xs_piece(warp * 16 + (lane >> 1), 0) : ((lane >> 1) ^ (lane >> 4))) * 2 + (lane & 1);   // 8-byte units, token 0

  float yacc[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int i = 0; i < 4; ++i) yacc[nb][i] = 0.f;

  // one chunk: stage the next one, this warp's group step (register slot D = c % kDepth), the owned
  // rows' outliers of the chunk, then the hand-over barrier
  // `checked` = false promises c < nsteps (no branch, so that neighbouring steps can be interleaved);
  // xsum_in carries the single token's group sum when the caller has already reduced it
  auto do_chunk = [&](const int c, auto slot, auto checked_t, const float xsum_in) {
    constexpr int d = decltype(slot)::value;
    constexpr bool checked = decltype(checked_t)::value;
    if (NBUF != 0) {   // next step's activations on their way, this step's landed and visible to the warp
      __syncwarp();
      stage_tile(c + kBufs - 1);
      asm volatile("cp.async.commit_group;\ncp.async.wait_group %0;" ::"n"(NBUF == 0 ? 0 : NBUF - 1) : "memory");
      __syncwarp();
    }
    const uint4* buf = NBUF == 0 ? sm_x + c * buf_pieces : wtile + (c % kBufs) * tile_pieces;
    if (!checked || c < nsteps) {
      unsigned xr[NB][16];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        const uint4* seg = xoff[nb] >= 0 ? buf + xoff[nb] : reinterpret_cast<const uint4*>(smem_raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 v = seg[i ^ xcx[nb]];
          xr[nb][4 * i] = v.x; xr[nb][4 * i + 1] = v.y; xr[nb][4 * i + 2] = v.z; xr[nb][4 * i + 3] = v.w;
        }
      }
      // (s 2^24, s z) on the raw path, (s, magic | z) on the subtract path
      float2 ta, tb;
      {
        const unsigned sza = tp[0], szb = tp[8];
        tp += (G64 ? 2 * kWarps : kWarps) * kRows;
        const float sa = __half2float(__ushort_as_half((unsigned short)sza));
        const float sb = __half2float(__ushort_as_half((unsigned short)szb));
        const unsigned za = sza >> 16, zb = szb >> 16;
        if (BF16) {
          ta = make_float2(sa, __uint_as_float(0x43004300u | (za * 0x00010001u)));
          tb = make_float2(sb, __uint_as_float(0x43004300u | (zb * 0x00010001u)));
        } else {
          ta = make_float2(sa * 16777216.f, sa * (float)za);
          tb = make_float2(sb * 16777216.f, sb * (float)zb);
        }
      }
      float2 xg2[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) xg2[nb] = make_float2(0.f, 0.f);
      if (!BF16 && !ONES && TP != 1) {   // group sums of tokens 2t, 2t+1 of every token block
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          xg2[nb] = __ldg(reinterpret_cast<const float2*>(p.xg + (size_t)(warp + kWarps * c) * TP + nb * 8 + 2 * t));
      }
      float xsum1 = xsum_in;
      if (!BF16 && !ONES && TP == 1 && checked) {   // one token: sum_k x_k of the group, lane L adding columns 4L..4L+3
        const uint2 h4 = reinterpret_cast<const uint2*>(buf)[xsum_off];
        const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h4.x));
        const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h4.y));
        xsum1 = (f0.x + f0.y) + (f1.x + f1.y);
#pragma unroll
        for (int o = G64 ? 8 : 16; o > 0; o >>= 1) xsum1 += __shfl_xor_sync(0xFFFFFFFFu, xsum1, o);
        if (G64) xsum1 = __shfl_sync(0xFFFFFFFFu, xsum1, (t >> 1) << 4);   // lanes 0-15 summed the first group, 16-31 the second
      }
      typename StepAcc<BITS, NB, BF16>::type acc = {};
      unsigned qa[BITS], qb[BITS];
#pragma unroll
      for (int i = 0; i < BITS; ++i) {
        qa[i] = wa[d][i];
        qb[i] = wb[d][i];
      }
      if (BF16) {
        step_sub<BITS, NB>(qa, qb, __float_as_uint(ta.y), __float_as_uint(tb.y), xr, reinterpret_cast<AccSub<NB>&>(acc));
      } else if (BITS == 4) {
        step_raw4<NB, ONES>(reinterpret_cast<const unsigned(&)[4]>(qa), reinterpret_cast<const unsigned(&)[4]>(qb), xr,
                            reinterpret_cast<AccRaw4<NB>&>(acc));
      } else {
        step_raw3<NB, ONES>(reinterpret_cast<const unsigned(&)[3]>(qa), reinterpret_cast<const unsigned(&)[3]>(qb), xr,
                            reinterpret_cast<AccRaw3<NB>&>(acc));
      }
      // refill the slot with the group kDepth steps ahead
      const bool refill = c + kDepth < nsteps;
      load_run_if<BITS>(p.codes, oa + kDepth * kStepWords, wa[d], refill);
      load_run_if<BITS>(p.codes, ob + kDepth * kStepWords, wb[d], refill);
      oa += kStepWords;
      ob += kStepWords;
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 tt = i < 2 ? ta : tb;
          if (BF16) {
            yacc[nb][i] = fmaf(tt.x, reinterpret_cast<AccSub<NB>&>(acc).c[nb][i], yacc[nb][i]);
          } else if (BITS == 4) {
            AccRaw4<NB>& a4 = reinterpret_cast<AccRaw4<NB>&>(acc);
            const float code_sum = fmaf(a4.c4[nb][i], 0.0625f, a4.c0[nb][i]);  // units of 2^-24
            const float xsum = ONES ? a4.xs[nb][i & 1]
                                    : (TP == 1 ? ((i & 1) == 0 && (G64 ? (t & 1) == 0 : t == 0) ? xsum1 : 0.f) : ((i & 1) ? xg2[nb].y : xg2[nb].x));
            yacc[nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xsum, yacc[nb][i]));
          } else {
            AccRaw3<NB>& a3 = reinterpret_cast<AccRaw3<NB>&>(acc);
            const float code_sum = fmaf(a3.c6[nb][i], 0.015625f, fmaf(a3.c3[nb][i], 0.125f, a3.c0[nb][i]));
            const float xsum = ONES ? a3.xs[nb][i & 1]
                                    : (TP == 1 ? ((i & 1) == 0 && (G64 ? (t & 1) == 0 : t == 0) ? xsum1 : 0.f) : ((i & 1) ? xg2[nb].y : xg2[nb].x));
            yacc[nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xsum, yacc[nb][i]));
          }
        }
      }
    }

  };
  using std::integral_constant;
  for (int c0 = 0; c0 < nchunks; c0 += kDepth) {
    if (c0 + kDepth <= nsteps) {
      // four full steps of this warp: branch-free, the single token's four group sums reduced together
      float xs4[kDepth] = {0.f, 0.f, 0.f, 0.f};
      if (!BF16 && !ONES && TP == 1) {
#pragma unroll
        for (int d = 0; d < kDepth; ++d) {
          const uint4* buf = NBUF == 0 ? sm_x + (c0 + d) * buf_pieces : wtile + ((c0 + d) % kBufs) * tile_pieces;
          if (NBUF == 0) {
            const uint2 h4 = reinterpret_cast<const uint2*>(buf)[xsum_off];
            const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h4.x));
            const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h4.y));
            xs4[d] = (f0.x + f0.y) + (f1.x + f1.y);
          }
        }
        if (NBUF == 0) {
#pragma unroll
          for (int o = G64 ? 8 : 16; o > 0; o >>= 1)
#pragma unroll
            for (int d = 0; d < kDepth; ++d) xs4[d] += __shfl_xor_sync(0xFFFFFFFFu, xs4[d], o);
          if (G64) {
#pragma unroll
            for (int d = 0; d < kDepth; ++d) xs4[d] = __shfl_sync(0xFFFFFFFFu, xs4[d], (t >> 1) << 4);
          }
        }
      }
      if (NBUF == 0) {
        do_chunk(c0, integral_constant<int, 0>{}, integral_constant<bool, false>{}, xs4[0]);
        do_chunk(c0 + 1, integral_constant<int, 1>{}, integral_constant<bool, false>{}, xs4[1]);
        do_chunk(c0 + 2, integral_constant<int, 2>{}, integral_constant<bool, false>{}, xs4[2]);
        do_chunk(c0 + 3, integral_constant<int, 3>{}, integral_constant<bool, false>{}, xs4[3]);
        continue;
      }
    }
    // general path (a partial block of steps, or ring mode where the tile of a single token is not yet
    // there when the block starts)
    do_chunk(c0, integral_constant<int, 0>{}, integral_constant<bool, true>{}, 0.f);
    if (c0 + 1 < nchunks) do_chunk(c0 + 1, integral_constant<int, 1>{}, integral_constant<bool, true>{}, 0.f);
    if (c0 + 2 < nchunks) do_chunk(c0 + 2, integral_constant<int, 2>{}, integral_constant<bool, true>{}, 0.f);
    if (c0 + 3 < nchunks) do_chunk(c0 + 3, integral_constant<int, 3>{}, integral_constant<bool, true>{}, 0.f);
  }
  static_assert(kDepth == 4, "the chunk loop is written out for four register slots");

  // partial sums of the 8 warps: sm_red[warp][nb][row][token]
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    float* r = sm_red + (warp * NB + nb) * 128;
    *reinterpret_cast<float2*>(r + gid * 8 + 2 * t) = make_float2(yacc[nb][0], yacc[nb][1]);
    *reinterpret_cast<float2*>(r + (gid + 8) * 8 + 2 * t) = make_float2(yacc[nb][2], yacc[nb][3]);
  }
  // CSR outliers of the two owned rows
  if (NBUF == 0) {
    // every chunk is still in shared memory: lane = entry, every token per lane, one transposing
    // reduction per row; entries beyond the 96 held in registers (rare) read x from global memory
    const uint16_t* xs16 = reinterpret_cast<const uint16_t*>(sm_x);
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int lr = 2 * warp + rr;
      const int jb = rr == 0 ? j0 : j1, je = rr == 0 ? j1 : j2;
      float v[TP];
#pragma unroll
      for (int m = 0; m < TP; ++m) v[m] = 0.f;
      if (je > jb) {
        const int ne = min(kOutSlots, (je - jb + 31) >> 5);   // warp-uniform
#pragma unroll
        for (int e = 0; e < kOutSlots; ++e) {
          if (e < ne && cv[rr][e] != 0xFFFFFFFFu) {
            const float wv = __half2float(__ushort_as_half((unsigned short)(cv[rr][e] >> 16)));
            const unsigned col = cv[rr][e] & 0xFFFFu;
            const int base = (int)(col >> 10) * buf_pieces;            // chunk = col / 1024
            const int pc = (int)((col & 1023u) >> 3), sub = (int)(col & 7u);
#pragma unroll
            for (int m = 0; m < TP; ++m)
              if (TP == 1 || m < p.M)
                v[m] = fmaf(wv, act_to_float<BF16>(xs16[((base + xs_piece(pc, m)) << 3) + sub]), v[m]);
          }
        }
        for (int j = jb + 32 * kOutSlots + lane; j < je; j += 32) {
          const unsigned e = __ldg(p.cv + j);
          const float wv = __half2float(__ushort_as_half((unsigned short)(e >> 16)));
#pragma unroll
          for (int m = 0; m < TP; ++m)
            if (TP == 1 || m < p.M)
              v[m] = fmaf(wv, act_to_float<BF16>(__ldg(p.x + (size_t)m * p.K + (e & 0xFFFFu))), v[m]);
        }
      }
      reduce_tokens<TP, 1>(v, lane);
      constexpr int LPT = 32 / TP;   // lanes per token after the reduction
      if ((lane & (LPT - 1)) == 0) sm_out[lr * TP + lane / LPT] = v[0];
    }
  }
  __syncthreads();

  // final sum and store: o -> (token, local row), rows fastest
  for (int o = tid; o < kRows * p.M; o += kThreads) {
    const int lr = o & 15, m = o >> 4;
    const int row = r0 + lr;
    if (row < p.N) {
      const int nb = G64 ? m >> 2 : m >> 3, tk = G64 ? m & 3 : m & 7;
      float v = sm_out[lr * TP + m];
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        v += sm_red[(w * NB + nb) * 128 + lr * 8 + tk];
        if (G64) v += sm_red[(w * NB + nb) * 128 + lr * 8 + tk + 4];   // the token's second group of every step
      }
      store_y(p.y, p.yd, (long long)m * p.N + row, v);
    }
  }
}

// One CTA per group of 128 columns: xt[col][token] = x[token][col] for token < M (zero beyond), TP tokens
// per column, and xg[group][token] = sum of x[token][col] over the group's columns (FP32).
template <int TP, bool BF16>
__global__ void __launch_bounds__(128) tokens_to_columns(const uint16_t* __restrict__ x, uint16_t* __restrict__ xt,
                                                         float* __restrict__ xg, int M, int K) {
  __shared__ float red[4][TP];
  const int col = blockIdx.x * 128 + threadIdx.x;
  uint16_t v[TP];
#pragma unroll
  for (int m = 0; m < TP; ++m) v[m] = m < M ? __ldg(x + (size_t)m * K + col) : (uint16_t)0;
  if (TP % 8 == 0) {
#pragma unroll
    for (int q = 0; q < TP / 8; ++q) {
      uint4 o;
      o.x = v[8 * q] | ((unsigned)v[8 * q + 1] << 16);     o.y = v[8 * q + 2] | ((unsigned)v[8 * q + 3] << 16);
      o.z = v[8 * q + 4] | ((unsigned)v[8 * q + 5] << 16); o.w = v[8 * q + 6] | ((unsigned)v[8 * q + 7] << 16);
      reinterpret_cast<uint4*>(xt + (size_t)col * TP)[q] = o;
    }
  } else {
#pragma unroll
    for (int m = 0; m < TP; ++m) xt[(size_t)col * TP + m] = v[m];
  }
#pragma unroll
  for (int m = 0; m < TP; ++m) {
    float f = act_to_float<BF16>(v[m]);
    for (int o = 16; o > 0; o >>= 1) f += __shfl_xor_sync(0xFFFFFFFFu, f, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5][m] = f;
  }
  __syncthreads();
  if (threadIdx.x < TP)
    xg[(size_t)blockIdx.x * TP + threadIdx.x] =
        (red[0][threadIdx.x] + red[1][threadIdx.x]) + (red[2][threadIdx.x] + red[3][threadIdx.x]);
}

constexpr size_t kStageAllLimit = 72 * 1024;   // stage every chunk up front when it fits in this much
constexpr size_t kStageAllLimitSmallGrid = 80 * 1024;   // the same for grids of at most two CTAs per SM

template <int BITS, int TP, bool BF16, int NBUF, bool G64>
cudaError_t launch(const MultiArgs& a, cudaStream_t stream) {
  constexpr int NB = TokenBlocks<TP, G64>::value;
  const int ngroups = a.K / 128;
  const int nchunks = (ngroups + kChunkGroups - 1) / kChunkGroups;
  const size_t smem = 64 + (size_t)kRows * (G64 ? 2 * ngroups : ngroups) * 4 + (size_t)kWarps * NB * 128 * 4 + (size_t)kRows * TP * 4 +
                      (NBUF == 0 ? (size_t)nchunks * a.M * kRowPitch : (size_t)kWarps * NBUF * a.M * kTilePitch) * 16;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<BITS, TP, BF16, NBUF, G64>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)a.first_block[a.count]);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_kernel<BITS, TP, BF16, NBUF, G64>, a);
}

// shared memory of a CTA with a ring of `bufs` activation tiles per warp
template <int TP, bool G64>
size_t ring_smem(int K, int M, int bufs) {
  constexpr int NB = TokenBlocks<TP, G64>::value;
  return 64 + (size_t)kRows * (K / (G64 ? 64 : 128)) * 4 + (size_t)kWarps * NB * 128 * 4 + (size_t)kRows * TP * 4 +
         (size_t)kWarps * bufs * M * kTilePitch * 16;
}
constexpr size_t kSmemPerCta = 227 * 1024;

// RING = ring depth used when the activations do not fit up front (one buffer less when the tables of a very wide
// layer leave no room for it)
template <int BITS, int TP, bool BF16, int RING, bool G64>
cudaError_t launch_buf(const MultiArgs& a, cudaStream_t stream) {
  const int nchunks = (a.K / 128 + kChunkGroups - 1) / kChunkGroups;
  // staging everything up front costs shared memory, hence resident CTAs: beyond kStageAllLimit only two fit on an
  // SM, which pays off as long as the whole grid is resident at that rate
  const size_t lim = a.first_block[a.count] <= 2 * a.sm_count ? kStageAllLimitSmallGrid : kStageAllLimit;
  if (TP <= 8 && (size_t)nchunks * a.M * kRowPitch * 16 <= lim) return launch<BITS, TP, BF16, 0, G64>(a, stream);
  if (ring_smem<TP, G64>(a.K, a.M, 2) > kSmemPerCta) return cudaErrorInvalidConfiguration;   // nothing launched yet
  if (TP > 1) {   // ring mode gathers the outliers' activations from a token-major copy
    if (!a.xt || !a.xg) return cudaErrorInvalidValue;
    tokens_to_columns<TP, BF16><<<a.K / 128, 128, 0, stream>>>(a.x, const_cast<uint16_t*>(a.xt), const_cast<float*>(a.xg), a.M, a.K);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (RING > 2 && ring_smem<TP, G64>(a.K, a.M, RING) > kSmemPerCta) return launch<BITS, TP, BF16, 2, G64>(a, stream);
  return launch<BITS, TP, BF16, RING, G64>(a, stream);
}

template <int BITS, bool BF16>
cudaError_t launch_tp(const MultiArgs& a, cudaStream_t stream) {
  if (a.M == 1) return launch_buf<BITS, 1, BF16, 2, false>(a, stream);
  if (a.M <= 4) return launch_buf<BITS, 4, BF16, 2, false>(a, stream);
  if (a.M <= 8) return launch_buf<BITS, 8, BF16, 2, false>(a, stream);
  if (a.M <= 16) return launch_buf<BITS, 16, BF16, 3, false>(a, stream);
  return launch_buf<BITS, 32, BF16, 3, false>(a, stream);
}

// groups of 64: up to 16 tokens (blocks of 4)
template <int BITS, bool BF16>
cudaError_t launch_tp64(const MultiArgs& a, cudaStream_t stream) {
  if (a.M == 1) return launch_buf<BITS, 1, BF16, 2, true>(a, stream);
  if (a.M <= 4) return launch_buf<BITS, 4, BF16, 2, true>(a, stream);
  if (a.M <= 8) return launch_buf<BITS, 8, BF16, 2, true>(a, stream);
  return launch_buf<BITS, 16, BF16, 3, true>(a, stream);
}

}  // namespace

// Decode launcher for `count` layers that read the same x: group size 128 (M <= 32) or 64 (M <= 8; M <= 16 for
// layers up to kMaxWeights64Wide weights), K <= 65536, same K and bit
// width in every layer.  Returns GWQ_ERR_UNSUPPORTED for anything else (nothing has been launched then).
// The scratch for the token-major copy of x is the first layer's.
gwq_status gwq_launch_decode_multi(const gwq_packed* const* P, int count, const void* x, gwq_dtype xd, int M,
                                   void* const* y, gwq_dtype yd, cudaStream_t stream) {
  if (count < 1 || count > kMaxLayers || M > 32) return GWQ_ERR_UNSUPPORTED;
  const bool g64 = P[0]->group == 64;
  if (g64 && (M > kMaxTokens64 || P[0]->K % 128 != 0)) return GWQ_ERR_UNSUPPORTED;   // a warp step is 128 columns
  for (int i = 0; i < count; ++i) {
    const gwq_priv* pvi = static_cast<const gwq_priv*>(P[i]->priv);
    if ((P[i]->group != 128 && P[i]->group != 64) || P[i]->group != P[0]->group || !pvi->cv || !pvi->sz_t || P[i]->K != P[0]->K || P[i]->bits != P[0]->bits) return GWQ_ERR_UNSUPPORTED;
  }
  if (g64 && M > 8)
    for (int i = 0; i < count; ++i)
      if ((long long)P[i]->N * P[i]->K > kMaxWeights64Wide) return GWQ_ERR_UNSUPPORTED;
  gwq_priv* pv = static_cast<gwq_priv*>(P[0]->priv);
  MultiArgs a;
  a.xt = nullptr;
  a.xg = nullptr;
  const int K = P[0]->K;
  if (M > 1) {   // scratch for the token-major copy and the group sums (used when x is not staged up front)
    const size_t need = (size_t)K * 32 * 2 + (size_t)(K / 128) * 32 * 4;
    if (pv->xt_bytes < need) {
      if (cudaStreamSynchronize(stream) != cudaSuccess) return GWQ_ERR_CUDA;
      if (pv->xt) cudaFree(pv->xt);
      pv->xt = nullptr;
      pv->xt_bytes = 0;
      if (cudaMalloc(&pv->xt, need) != cudaSuccess) {
        (void)cudaGetLastError();
        return GWQ_ERR_ALLOC;
      }
      pv->xt_bytes = need;
    }
    a.xt = static_cast<const uint16_t*>(pv->xt);
    a.xg = reinterpret_cast<const float*>(static_cast<const char*>(pv->xt) + (size_t)K * 32 * 2);
  }
  int blocks = 0;
  for (int i = 0; i < kMaxLayers; ++i) {
    const gwq_packed* Pi = P[i < count ? i : 0];
    a.layer[i].codes = Pi->codes; a.layer[i].szt = static_cast<const gwq_priv*>(Pi->priv)->sz_t;
    a.layer[i].row_ptr = Pi->S->row_ptr; a.layer[i].cv = static_cast<const gwq_priv*>(Pi->priv)->cv;
    a.layer[i].y = y[i < count ? i : 0]; a.layer[i].N = Pi->N;
    a.first_block[i] = blocks;
    if (i < count) blocks += (Pi->N + kRows - 1) / kRows;
  }
  a.first_block[kMaxLayers] = blocks;
  for (int i = count; i < kMaxLayers; ++i) a.first_block[i] = blocks;
  a.count = count;
  a.sm_count = pv->sm_count > 0 ? pv->sm_count : 148;
  a.x = static_cast<const uint16_t*>(x); a.yd = yd; a.K = K; a.M = M;
  cudaError_t e;
  if (g64) {
    if (P[0]->bits == 4) e = (xd == GWQ_BF16) ? launch_tp64<4, true>(a, stream) : launch_tp64<4, false>(a, stream);
    else e = (xd == GWQ_BF16) ? launch_tp64<3, true>(a, stream) : launch_tp64<3, false>(a, stream);
  } else if (P[0]->bits == 4) e = (xd == GWQ_BF16) ? launch_tp<4, true>(a, stream) : launch_tp<4, false>(a, stream);
  else e = (xd == GWQ_BF16) ? launch_tp<3, true>(a, stream) : launch_tp<3, false>(a, stream);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return e == cudaErrorInvalidConfiguration ? GWQ_ERR_UNSUPPORTED : GWQ_ERR_CUDA;   // too wide for shared memory
  }
  return GWQ_OK;
}

// Decode launcher: group size 128 with M <= 32 or 64 with M <= 8 (16 for layers of moderate size), K <= 65536.
// Groups of 64 with more tokens go to the tensor-core kernel, other shapes to the general kernel.
gwq_status gwq_launch_decode(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y, gwq_dtype yd,
                             cudaStream_t stream) {
  const gwq_status st = gwq_launch_decode_multi(&P, 1, x, xd, M, &y, yd, stream);
  if (st != GWQ_ERR_UNSUPPORTED) return st;
  // groups of 64 beyond the tokens the streaming kernel takes: the tensor-core kernel with its smallest token tile
  if (P->group == 64 && M > 8) return gwq_launch_prefill(P, x, xd, M, y, yd, stream);
  return gwq_launch_simt(P, x, xd, M, y, yd, stream);
}
