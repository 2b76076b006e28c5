// Decode path (M <= 32) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w"): bandwidth-bound.
//
// One CTA owns 16 RT output rows (RT = 1 or 2 m16 tiles); its 8 warps split K by quantization group
// (128 columns).  Per group a warp streams the packed codes of its rows straight from global memory
// into registers (each lane: one run of 32 columns for rows g and g+8 of every tile), masks them into
// 16-bit floating-point integers and multiplies them with the activations on the tensor
// cores (mma.sync m16n8k16: the 16 weight rows are the A operand, 8 tokens the B operand,
// FP32 accumulators).  The B fragments and the sums of x of a group are fetched once per step and
// serve every tile.  Scale and zero-point are applied once per group to the
// accumulator, y += s (sum x q) - s z (sum x), so no scaled weight is ever rounded:
//  * fp16 activations: the raw code bits are used as fp16 subnormals q 2^-24 (one shift
//    and one mask per pair of codes) and sum x comes from a second MMA whose A operand is
//    all ones (one token: from shuffles);
//  * bf16 activations: (bits | magic) - (z | magic) gives q - z exactly (one more packed
//    subtract per pair), no second MMA.
// The pair-interleaved packed order makes both operands natural: pair h of a lane's run
// holds columns (2h, 2h+1), the same pair as 32-bit word h of its activation segment.
// Activations are staged in shared memory: all of x up front when it is small, else per-warp tiles in
// a cp.async ring.  The CSR outliers of a row are added by the warp that owns the row.  After the K
// loop the warps' partial sums meet in shared memory and y is stored.  The kernel is launched with
// programmatic stream serialization: its weight prefetch may overlap the previous kernel, everything
// that touches x or y comes after griddepcontrol.wait.
#pragma once

#include <type_traits>

#include "common.cuh"

namespace gwq_decode {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxLayers = GWQ_MULTI_MAX;

// One launch may serve several layers that read the same activations (sibling projections): the grid is the
// concatenation of the layers' row blocks, layer l owning the blocks [first_block[l], first_block[l + 1]).
struct LayerArgs {
  const uint32_t* codes;
  const uint32_t* szt;   // [K / group][N]: scale (fp16 bits) | zero-point << 16
  const int32_t* row_ptr;
  const uint32_t* cv;    // per outlier: fp16 value << 16 | column
  void* y;
  int N;
};
struct MultiArgs {
  LayerArgs layer[kMaxLayers];
  int first_block[kMaxLayers + 1];
  int count;
  int sm_count;
  const uint16_t* x;
  const uint16_t* xt;  // [K][TP] copy of x (ring mode with more than one token), else null
  const float* xg;     // [K/128][TP] sums of x over each group of columns (same mode), else null
  gwq_dtype yd;
  int K, M;
  int cvcap;           // outlier entries per owned row that are prefetched into shared memory (x staged up front)
};

// What a launch needs besides the arguments: chosen on the host (see plan() in linear_decode.cu).
struct Variant {
  int tp;      // tokens rounded up to 1, 4, 8, 16 or 32
  int nbuf;    // 0: all of x staged up front; 2, 3: per-warp ring of that many tiles
  int rt;      // m16 tiles per CTA (rows = 16 rt)
  int deep;    // 1: eight groups of codes in flight per warp instead of four (one tile, up to 8 tokens; two CTAs per SM)
  int gs;      // scale groups per 128-column step: 1 (groups of 128), 2 (64), 4 (32), 8 (16)
};

size_t smem_bytes(const Variant& v, int K, int M, int cvcap);

// Implemented once per (bit width, activation type) in a translation unit of its own.
cudaError_t launch_w4_f16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w4_bf16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w3_f16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w3_bf16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w8_f16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w8_bf16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w2_f16(const Variant& v, const MultiArgs& a, cudaStream_t stream);
cudaError_t launch_w2_bf16(const Variant& v, const MultiArgs& a, cudaStream_t stream);

constexpr int kChunkGroups = kWarps;                 // groups per chunk
constexpr int kChunkPieces = kChunkGroups * 16;      // 16-byte pieces per token row per chunk
constexpr int kRowPitch = kChunkPieces + kChunkPieces / 8 + 4;   // pieces, with padding
constexpr int kTilePitch = 16;   // pieces per token row of a warp tile: no padding, the pieces of a row are permuted

// token blocks of 8 / gs tokens (an MMA has 8 columns: tokens x groups of the step)
__host__ __device__ constexpr int token_blocks(int tp, int gs) { return tp * gs <= 8 ? 1 : tp * gs / 8; }

}  // namespace gwq_decode

#ifdef GWQ_DECODE_KERNEL_IMPL

namespace gwq_decode {
namespace {

template <bool BF16, bool ZERO>
__device__ __forceinline__ void mma16816(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
  // ZERO: the accumulator starts at 0 (no register has to be cleared for it)
  if (ZERO) {
    if (BF16) {
      asm volatile(
          "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
          : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
          : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
    } else {
      asm volatile(
          "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
          : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
          : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
    }
  } else if (BF16) {
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
__device__ __forceinline__ unsigned sub_zero_bf16(unsigned qm, unsigned zm) {
  __nv_bfloat162 r = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&qm), *reinterpret_cast<__nv_bfloat162*>(&zm));
  return *reinterpret_cast<unsigned*>(&r);
}

// ---------------------------------------------------------------------------------------------
// One group step of a warp for one m16 tile: 8 (x NB) weight MMAs for the 16 rows x 128 columns whose
// packed words are qa (row g) and qb (row g + 8) of this lane, against the activation words
// xr[nb][0..15] (word h = columns 2h, 2h+1 of the lane's run).  The accumulators start at zero.
//
// Raw variant (fp16 activations).  The masked code bits are used directly as fp16 subnormals:
// a code at mantissa bit position p is the number q 2^(p-24).  Integer instructions are the
// scarce resource of this kernel (half-rate pipe), so codes are masked where a shift or two per
// word has put them, not moved one by one; the positions that occur (0 and 4 for 4 bits,
// 0, 3 and 6 for 3 bits) each get their own accumulator, merged with the right power of two in
// the group epilogue.
template <int NB>
struct AccRaw4 {
  float c0[NB][4], c4[NB][4];
};
template <int NB>
struct AccRaw3 {
  float c0[NB][4], c3[NB][4], c6[NB][4];
};
template <int NB>
struct AccSub {
  float c[NB][4];
};

#define GWQ_ONES 0x3C003C00u

template <int NB>
__device__ __forceinline__ void step_raw4(const unsigned (&qa)[4], const unsigned (&qb)[4],
                                          const unsigned (&xr)[NB][16], AccRaw4<NB>& acc) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // pairs 4i, 4i+1 end at position 0 and pairs 4i+2, 4i+3 at position 4, so that the two k-halves of an MMA are
    // neighbouring words of the activation segment (one 64-bit register pair of the 128-bit load)
    const unsigned ta4 = qa[i] >> 4, tb4 = qb[i] >> 4, ta8 = qa[i] >> 8, tb8 = qb[i] >> 8;
    const unsigned a00 = qa[i] & 0x000F000Fu, b00 = qb[i] & 0x000F000Fu;  // pair 4i   (position 0)
    const unsigned a01 = ta4 & 0x000F000Fu, b01 = tb4 & 0x000F000Fu;      // pair 4i+1 (position 0)
    const unsigned a02 = ta4 & 0x00F000F0u, b02 = tb4 & 0x00F000F0u;      // pair 4i+2 (position 4)
    const unsigned a03 = ta8 & 0x00F000F0u, b03 = tb8 & 0x00F000F0u;      // pair 4i+3 (position 4)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      if (i == 0) {
        mma16816<false, true>(acc.c0[nb], a00, b00, a01, b01, xr[nb][4 * i], xr[nb][4 * i + 1]);
        mma16816<false, true>(acc.c4[nb], a02, b02, a03, b03, xr[nb][4 * i + 2], xr[nb][4 * i + 3]);
      } else {
        mma16816<false, false>(acc.c0[nb], a00, b00, a01, b01, xr[nb][4 * i], xr[nb][4 * i + 1]);
        mma16816<false, false>(acc.c4[nb], a02, b02, a03, b03, xr[nb][4 * i + 2], xr[nb][4 * i + 3]);
      }
    }
  }
}

template <int NB>
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
#define GWQ_M3(Z, ACC, H1, H2) mma16816<false, Z>(ACC[nb], a[H1], b[H1], a[H2], b[H2], xr[nb][H1], xr[nb][H2]);
    GWQ_M3(true, acc.c0, 0, 3) GWQ_M3(false, acc.c0, 5, 8) GWQ_M3(false, acc.c0, 10, 13)
    GWQ_M3(true, acc.c3, 1, 4) GWQ_M3(false, acc.c3, 6, 9) GWQ_M3(false, acc.c3, 11, 14)
    GWQ_M3(true, acc.c6, 2, 7) GWQ_M3(false, acc.c6, 12, 15)
#undef GWQ_M3
  }
}

// 8-bit codes: pair 2i is the low byte of both halves of word i, pair 2i+1 the high byte (one shift, two masks per
// word); codes up to 255 are still fp16 subnormals q 2^-24.  One position, one accumulator.
template <int NB>
struct AccRaw8 {
  float c0[NB][4];
};
template <int NB>
__device__ __forceinline__ void step_raw8(const unsigned (&qa)[8], const unsigned (&qb)[8],
                                          const unsigned (&xr)[NB][16], AccRaw8<NB>& acc) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const unsigned a0 = qa[i] & 0x00FF00FFu, b0 = qb[i] & 0x00FF00FFu;
    const unsigned a1 = (qa[i] >> 8) & 0x00FF00FFu, b1 = (qb[i] >> 8) & 0x00FF00FFu;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      if (i == 0) mma16816<false, true>(acc.c0[nb], a0, b0, a1, b1, xr[nb][2 * i], xr[nb][2 * i + 1]);
      else mma16816<false, false>(acc.c0[nb], a0, b0, a1, b1, xr[nb][2 * i], xr[nb][2 * i + 1]);
    }
  }
}

// 2-bit codes: word i holds pairs 8i .. 8i+7, pair 8i+p at bits 2p of both halves.  Three shifts (by 4, 8, 12) leave
// the even pairs at position 0 and the odd ones at position 2: two accumulators, merged with 1/4 in the epilogue.
template <int NB>
struct AccRaw2 {
  float c0[NB][4], c2[NB][4];
};
template <int NB>
__device__ __forceinline__ void step_raw2(const unsigned (&qa)[2], const unsigned (&qb)[2],
                                          const unsigned (&xr)[NB][16], AccRaw2<NB>& acc) {
#pragma unroll
  for (int i = 0; i < 2; ++i) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {   // pairs 8i + 4u .. 8i + 4u + 3
      const unsigned ta = qa[i] >> (8 * u), tb = qb[i] >> (8 * u), ua = ta >> 4, ub = tb >> 4;
      const unsigned a0 = ta & 0x00030003u, b0 = tb & 0x00030003u;   // pair 8i+4u   (position 0)
      const unsigned a1 = ta & 0x000C000Cu, b1 = tb & 0x000C000Cu;   // pair 8i+4u+1 (position 2)
      const unsigned a2 = ua & 0x00030003u, b2 = ub & 0x00030003u;   // pair 8i+4u+2 (position 0)
      const unsigned a3 = ua & 0x000C000Cu, b3 = ub & 0x000C000Cu;   // pair 8i+4u+3 (position 2)
      const int h = 8 * i + 4 * u;
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        if (i == 0 && u == 0) {
          mma16816<false, true>(acc.c0[nb], a0, b0, a2, b2, xr[nb][h], xr[nb][h + 2]);
          mma16816<false, true>(acc.c2[nb], a1, b1, a3, b3, xr[nb][h + 1], xr[nb][h + 3]);
        } else {
          mma16816<false, false>(acc.c0[nb], a0, b0, a2, b2, xr[nb][h], xr[nb][h + 2]);
          mma16816<false, false>(acc.c2[nb], a1, b1, a3, b3, xr[nb][h + 1], xr[nb][h + 3]);
        }
      }
    }
  }
}

// sum_k x_k of the step's columns for every token of the block, through an A operand of all ones
template <int NB>
__device__ __forceinline__ void step_ones(const unsigned (&xr)[NB][16], float (&xs)[NB][4]) {
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    mma16816<false, true>(xs[nb], GWQ_ONES, GWQ_ONES, GWQ_ONES, GWQ_ONES, xr[nb][0], xr[nb][1]);
#pragma unroll
    for (int h = 1; h < 8; ++h)
      mma16816<false, false>(xs[nb], GWQ_ONES, GWQ_ONES, GWQ_ONES, GWQ_ONES, xr[nb][2 * h], xr[nb][2 * h + 1]);
  }
}

// Subtract variant (bf16 activations): (bits | magic) - (z | magic) = q - z exactly in bf16; one
// accumulator, no ones operand.  zma / zmb hold magic | z in both halves.
// (zma[h], zmb[h]: for pairs 8 h .. 8 h + 7 of the run; the two differ only with groups of 16 columns)
template <int BITS, int NB>
__device__ __forceinline__ void step_sub(const unsigned (&qa)[BITS], const unsigned (&qb)[BITS], const unsigned (&zma)[2],
                                         const unsigned (&zmb)[2], const unsigned (&xr)[NB][16], AccSub<NB>& acc) {
  constexpr unsigned MAGIC = 0x43004300u;  // bf16 128.0: ulp = 1
  unsigned a[16], b[16];
  if (BITS == 8) {
    // codes up to 255 do not fit under the bf16 magic number: q - z is taken in fp16 (magic 1024, exact) and
    // converted, exactly, to bf16 (|q - z| <= 255 has 8 significant bits).  zma / zmb hold the fp16 magic | z here.
#pragma unroll
    for (int h = 0; h < 16; ++h) {
      const unsigned va = ((qa[(h >> 1) % BITS] >> (8 * (h & 1))) & 0x00FF00FFu) | 0x64006400u;
      const unsigned vb = ((qb[(h >> 1) % BITS] >> (8 * (h & 1))) & 0x00FF00FFu) | 0x64006400u;
      const float2 fa = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&va),
                                               *reinterpret_cast<const __half2*>(&zma[h >> 3])));
      const float2 fb = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&vb),
                                               *reinterpret_cast<const __half2*>(&zmb[h >> 3])));
      const __nv_bfloat162 ca = __floats2bfloat162_rn(fa.x, fa.y), cb = __floats2bfloat162_rn(fb.x, fb.y);
      a[h] = *reinterpret_cast<const unsigned*>(&ca);
      b[h] = *reinterpret_cast<const unsigned*>(&cb);
    }
  } else if (BITS == 2) {
#pragma unroll
    for (int h = 0; h < 16; ++h) {
      a[h] = sub_zero_bf16(((qa[(h >> 3) % BITS] >> (2 * (h & 7))) & 0x00030003u) | MAGIC, zma[h >> 3]);
      b[h] = sub_zero_bf16(((qb[(h >> 3) % BITS] >> (2 * (h & 7))) & 0x00030003u) | MAGIC, zmb[h >> 3]);
    }
  } else if (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        a[4 * i + j] = sub_zero_bf16(((qa[i % BITS] >> (4 * j)) & 0x000F000Fu) | MAGIC, zma[i >> 1]);
        b[4 * i + j] = sub_zero_bf16(((qb[i % BITS] >> (4 * j)) & 0x000F000Fu) | MAGIC, zmb[i >> 1]);
      }
  } else {
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
      for (int p = 0; p < 5; ++p) {
        a[5 * i + p] = sub_zero_bf16(((qa[i % BITS] >> (3 * p)) & 0x00070007u) | MAGIC, zma[(5 * i + p) >> 3]);
        b[5 * i + p] = sub_zero_bf16(((qb[i % BITS] >> (3 * p)) & 0x00070007u) | MAGIC, zmb[(5 * i + p) >> 3]);
      }
    const unsigned la = ((qa[0] >> 15) & 0x00010001u) | ((qa[1 % BITS] >> 14) & 0x00020002u) |
                        ((qa[BITS - 1] >> 13) & 0x00040004u);
    const unsigned lb = ((qb[0] >> 15) & 0x00010001u) | ((qb[1 % BITS] >> 14) & 0x00020002u) |
                        ((qb[BITS - 1] >> 13) & 0x00040004u);
    a[15] = sub_zero_bf16(la | MAGIC, zma[1]);
    b[15] = sub_zero_bf16(lb | MAGIC, zmb[1]);
  }
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    mma16816<true, true>(acc.c[nb], a[0], b[0], a[1], b[1], xr[nb][0], xr[nb][1]);
#pragma unroll
    for (int m8 = 1; m8 < 8; ++m8)
      mma16816<true, false>(acc.c[nb], a[2 * m8], b[2 * m8], a[2 * m8 + 1], b[2 * m8 + 1], xr[nb][2 * m8],
                            xr[nb][2 * m8 + 1]);
  }
}

template <int BITS>
__device__ __forceinline__ void load_run(const uint32_t* __restrict__ base, unsigned off, unsigned (&w)[BITS]) {
  const uint32_t* p = base + off;
  if (BITS == 4) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));  // streamed once: evict first
    w[0] = v.x; w[1 % BITS] = v.y; w[2 % BITS] = v.z; w[BITS - 1] = v.w;
  } else if (BITS == 8) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p)), u = __ldcs(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = v.x; w[1 % BITS] = v.y; w[2 % BITS] = v.z; w[3 % BITS] = v.w;
    w[4 % BITS] = u.x; w[5 % BITS] = u.y; w[6 % BITS] = u.z; w[7 % BITS] = u.w;
  } else if (BITS == 2) {
    const uint2 v = __ldcs(reinterpret_cast<const uint2*>(p));
    w[0] = v.x; w[BITS - 1] = v.y;
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
  if constexpr (BITS == 4) {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %5, 0;\n @q ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];\n}\n"
        : "+r"(w[0]), "+r"(w[1 % BITS]), "+r"(w[2 % BITS]), "+r"(w[BITS - 1])
        : "l"(p), "r"((int)pred));
  } else if constexpr (BITS == 8) {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %9, 0;\n @q ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%8];\n"
        " @q ld.global.cs.v4.u32 {%4,%5,%6,%7}, [%8+16];\n}\n"
        : "+r"(w[0]), "+r"(w[1 % BITS]), "+r"(w[2 % BITS]), "+r"(w[3 % BITS]), "+r"(w[4 % BITS]), "+r"(w[5 % BITS]),
          "+r"(w[6 % BITS]), "+r"(w[7 % BITS])
        : "l"(p), "r"((int)pred));
  } else if constexpr (BITS == 2) {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %3, 0;\n @q ld.global.cs.v2.u32 {%0,%1}, [%2];\n}\n"
        : "+r"(w[0]), "+r"(w[BITS - 1])
        : "l"(p), "r"((int)pred));
  } else {
    asm volatile(
        "{\n .reg .pred q;\n setp.ne.b32 q, %4, 0;\n @q ld.global.cs.u32 %0, [%3];\n @q ld.global.cs.u32 %1, [%3+4];\n"
        " @q ld.global.cs.u32 %2, [%3+8];\n}\n"
        : "+r"(w[0]), "+r"(w[1 % BITS]), "+r"(w[2 % BITS])
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

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// Activations staged up front are laid out chunk by chunk: one chunk is 8 groups (1024 columns), one group
// per warp.  16-byte piece c of token row m sits at piece c + (c >> 3) + 2 (m & 1) of its
// row (one pad piece per 128 bytes, odd rows shifted by two): the 64-byte segments of the four lanes
// of a quad and of two neighbouring token rows then fall into all eight 16-byte bank groups.
__device__ __forceinline__ int xs_piece(int c, int m) { return m * kRowPitch + c + (c >> 3) + ((m & 1) << 1); }
// piece p (16 bytes) of token row m of a warp tile: the XOR keeps the four lanes of a quad and four neighbouring
// token rows in different 16-byte bank groups
__device__ __forceinline__ int tile_piece(int pc, int m) { return m * kTilePitch + (pc ^ (pc >> 3) ^ ((m & 3) << 1)); }

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
template <int NB> struct StepAcc<8, NB, false> { using type = AccRaw8<NB>; };
template <int NB> struct StepAcc<2, NB, false> { using type = AccRaw2<NB>; };
template <int BITS, int NB> struct StepAcc<BITS, NB, true> { using type = AccSub<NB>; };

// resident CTAs the register budget is cut for
__host__ __device__ constexpr int min_blocks(int nb, int rt, bool deep) {
  return deep ? 2 : (rt == 1 ? (nb == 1 ? 3 : (nb == 2 ? 2 : 1)) : (nb == 1 ? 2 : 1));
}

template <class F, int... I>
__device__ __forceinline__ void unroll_slots(F&& f, std::integer_sequence<int, I...>) {
  (f(std::integral_constant<int, I>{}), ...);
}

// TP = tokens rounded up to 1, 4, 8, 16 or 32.
// NBUF = 0: the activations of all chunks are staged up front by the whole CTA (small M K).
// NBUF = 2, 3: every warp keeps a private ring of NBUF buffers with the activations of its own group only
//           (M x 128 columns), copied one step ahead with cp.async; no CTA barrier in the K loop.
// G64: groups of 64 columns.  A warp step still covers 128 columns, i.e. two groups: the runs of lanes t = 0, 1 belong
// to the first, those of t = 2, 3 to the second.  An MMA sums over all four lanes, so the two groups are kept apart on
// the token side: a token block holds 4 tokens, output column n < 4 is token n with the activations of the second
// group replaced by zeros (lanes t >= 2 read the zero page), column n >= 4 is token n - 4 with those of the first
// group replaced by zeros.  Accumulator columns 2t, 2t+1 of lane t then belong to the lane's own group (t >> 1), whose
// scale and zero-point it applies; the two halves of a token meet in the final sum.  With more than one token the sums
// of x come from the all-ones MMA (which sees the same zeros); a single token's are reduced over half a warp each.
// TP <= 16 there.
// GS = 4, 8 (groups of 32, 16 columns) continue the scheme: a block holds 8 / GS tokens, column n is token n % (8 / GS)
// restricted to group n / (8 / GS) of the step.  A lane's run of 32 columns is one group of 32 (its accumulator columns
// 2t, 2t+1 are two tokens of that group), or two groups of 16 (pairs 0..7 and 8..15 of the run: column 2t is the first,
// 2t+1 the second, one token per block; the two halves of the B fragment come from different places and the lane
// applies two scales).  The sums of x come from the all-ones MMA.  Activations staged up front only.
// RT: m16 tiles (16 rows each) of the CTA; every warp step loads the B fragments once and runs all RT tiles on them.
// DEEP: eight groups of codes in flight per warp (grids that leave an SM at most two CTAs: fewer warps have to keep
// as many bytes in flight).
template <int BITS, int TP, bool BF16, int NBUF, int GS, int RT, bool DEEP>
__global__ void __launch_bounds__(kThreads, min_blocks(token_blocks(TP, GS), RT, DEEP))
decode_kernel(const MultiArgs ma) {
  constexpr int R = 16 * RT;                       // rows of the CTA
  // groups of codes in flight per warp and tile (about the same bytes whatever the code width)
  constexpr int D = (DEEP ? 8 : (RT == 1 ? 4 : 2)) * (BITS == 2 ? 2 : 1) / (BITS == 8 ? 2 : 1);
  constexpr bool G64 = GS == 2;
  constexpr int TB = 8 / GS;                       // tokens of a block
  constexpr int NB = token_blocks(TP, GS);         // token blocks of the MMA
  static_assert(GS < 4 || (NBUF == 0 && RT == 1 && !DEEP), "small groups: staged activations, one tile");
  constexpr int WPR = BITS;                        // words per run of 32 columns
  // raw path: sum_k x_k of a group from shared memory (one token), from the table that comes with the
  // token-major copy (ring mode), else from a second MMA with an all-ones A operand
  constexpr bool ONES = !BF16 && ((TP != 1 && (GS > 1 || NBUF == 0)) || GS > 2);
  constexpr int OWN = 2 * RT;                      // rows whose outliers a warp adds

  // the layer this CTA works for and its row block inside that layer
  const uint32_t* codes; const uint32_t* szt; const int32_t* row_ptr; const uint32_t* cvp; void* yout; int N;
  int blk = blockIdx.x;
  {
    int l = 0;
#pragma unroll
    for (int i = 1; i < kMaxLayers; ++i)
      if (i < ma.count && (int)blockIdx.x >= ma.first_block[i]) l = i;
    codes = ma.layer[0].codes; szt = ma.layer[0].szt; row_ptr = ma.layer[0].row_ptr; cvp = ma.layer[0].cv;
    yout = ma.layer[0].y; N = ma.layer[0].N;
#pragma unroll
    for (int i = 1; i < kMaxLayers; ++i) {
      if (i == l) {
        codes = ma.layer[i].codes; szt = ma.layer[i].szt; row_ptr = ma.layer[i].row_ptr; cvp = ma.layer[i].cv;
        yout = ma.layer[i].y; N = ma.layer[i].N;
        blk = (int)blockIdx.x - ma.first_block[i];
      }
    }
  }
  const int K = ma.K, M = ma.M;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int ngroups = K >> 7;               // warp steps of 128 columns in a row
  const int ntab = GS * ngroups;   // scale / zero-point entries in a row
  // shared: zero page 64 B | scale and zero-point table [ntab][R] u32 | red [kWarps][RT][NB][128] f32 |
  //         outl [R][TP] f32 | outlier entries [kWarps][OWN][cvcap] u32 (x staged up front only) | x buffers
  // (the table is group-major: the eight rows a load instruction asks for are eight neighbouring words, no bank
  // conflicts however wide the layer is)
  uint32_t* sm_tab = reinterpret_cast<uint32_t*>(smem_raw + 64);
  float* sm_red = reinterpret_cast<float*>(sm_tab + R * ntab);
  float* sm_out = sm_red + kWarps * RT * NB * 128;
  uint32_t* sm_cv = reinterpret_cast<uint32_t*>(sm_out + R * TP);
  const int kCvCap = ma.cvcap;
  uint4* sm_x = reinterpret_cast<uint4*>(sm_cv + (NBUF == 0 ? kWarps * OWN * kCvCap : 0));
  const int buf_pieces = M * kRowPitch;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, t = lane & 3;
  const int r0 = blk * R;
  const unsigned row_words = (unsigned)(K >> 5) * WPR;
  constexpr unsigned kStepWords = kWarps * 4 * WPR;  // codes of 8 groups
  unsigned oa[RT], ob[RT];                           // group `warp`, this lane's run, rows g / g + 8 of every tile
#pragma unroll
  for (int rt = 0; rt < RT; ++rt) {
    const int ra = min(r0 + 16 * rt + gid, N - 1), rb = min(r0 + 16 * rt + gid + 8, N - 1);
    oa[rt] = (unsigned)ra * row_words + (unsigned)(warp * 4 + t) * WPR;
    ob[rt] = (unsigned)rb * row_words + (unsigned)(warp * 4 + t) * WPR;
  }
  const int nsteps = (ngroups - warp + kWarps - 1) / kWarps;  // this warp's groups: warp, warp + 8, ...
  const int nchunks = (ngroups + kChunkGroups - 1) / kChunkGroups;

  pdl_launch_dependents();

  // ---- everything that does not depend on the previous kernel: all loads are issued before any is awaited
  // CSR extents of the OWN rows this warp owns (rows OWN warp .. OWN warp + OWN - 1 of the CTA)
  int rp = 0;
  if (lane <= OWN) rp = __ldg(row_ptr + min(r0 + OWN * warp + lane, N));
  {
    // scales and zero-points of the R rows: 4 R contiguous bytes per group of the group-major table
    const int rows_here = min(R, N - r0);
    if (rows_here == R && (N & 3) == 0) {
      const unsigned dst0 = (unsigned)__cvta_generic_to_shared(sm_tab);
      for (int c = tid; c < (R / 4) * ntab; c += kThreads) {   // piece c: rows 4 (c % (R/4)) .. + 3 of group c / (R/4)
        const uint32_t* src = szt + (size_t)(c / (R / 4)) * N + r0 + 4 * (c % (R / 4));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (unsigned)c * 16u), "l"(src));
      }
    } else {   // partial last CTA, or rows that do not start on 16-byte boundaries: rows past N read as scale 0
      for (int i = tid; i < R * ntab; i += kThreads) {
        const int r = i % R, g = i / R;
        sm_tab[i] = r < rows_here ? __ldg(szt + (size_t)g * N + r0 + r) : 0u;
      }
    }
  }
  unsigned wa[RT][D][BITS], wb[RT][D][BITS];
#pragma unroll
  for (int d = 0; d < D; ++d) {
    if (d < nsteps) {
#pragma unroll
      for (int rt = 0; rt < RT; ++rt) {
        load_run<BITS>(codes, oa[rt] + d * kStepWords, wa[rt][d]);
        load_run<BITS>(codes, ob[rt] + d * kStepWords, wb[rt][d]);
      }
    }
  }
  if (tid < 16) reinterpret_cast<unsigned*>(smem_raw)[tid] = 0u;

  // CSR extents of the owned rows: jr[i] .. jr[i + 1] are the entries of owned row i
  int jr[OWN + 1];
  if (NBUF != 0) {
#pragma unroll
    for (int i = 0; i <= OWN; ++i) jr[i] = __shfl_sync(0xFFFFFFFFu, rp, i);
  }
  constexpr int VT = TP < 8 ? TP : 8, TS = TP / VT, EPB = 32 / TS;
  constexpr int kPre = TP <= 8 ? 2 : 3;   // batches of EPB entries per row: 64 entries up to 8 tokens, 48 / 24 beyond
  unsigned epre[2][kPre];
  if (NBUF != 0) {
    // ring mode (lane = (entry, group of VT tokens)): the first kPre batches of outlier entries of the first two owned
    // rows are requested before the wait on the previous kernel, they are weights
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
#pragma unroll
      for (int u = 0; u < kPre; ++u) {
        const int j = jr[rr] + u * EPB + lane / TS;
        epre[rr][u] = j < jr[rr + 1] ? __ldg(cvp + j) : 0u;   // value 0, column 0
      }
    }
  }
  // ---- from here on x is read
  pdl_wait();
  // NBUF == 0: copy of all activations into the chunk buffers, by the whole CTA: token row by token row, piece pc of a
  // row goes to chunk pc / 128, place xs_piece(pc % 128, m) (few instructions per piece: this runs in every CTA)
  auto stage_all = [&]() {
    const int ppr = K >> 3;   // 16-byte pieces per token row
    const unsigned base = (unsigned)__cvta_generic_to_shared(sm_x);
    for (int m = 0; m < M; ++m) {
      const uint16_t* src = ma.x + (size_t)m * K;
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
  const int tile_pieces = M * kTilePitch;
  uint4* wtile = sm_x + warp * kBufs * tile_pieces;
  // lane L copies piece L & 15 of the token rows (L >> 4), (L >> 4) + 2, ...  The place of a piece inside its row
  // (tile_piece) takes two values only, 64 bytes apart, for the rows m and m + 2 (they differ in (m & 3) << 1), and the
  // rows are a fixed number of bytes apart: the copies of a step cost an address each.  (Unrolled this way for 4 and 16
  // tokens; with 8 tokens, and with 3-bit codes at 16, the plain loop measured faster: registers.)
  constexpr bool kUnrolledCopies = TP == 4 || (TP == 16 && BITS == 4);
  const int st_m0 = lane >> 4, st_pc = lane & 15;
  const unsigned st_dst0 = (unsigned)__cvta_generic_to_shared(wtile);
  const unsigned st_place = (unsigned)(tile_piece(st_pc, st_m0) - st_m0 * kTilePitch) * 16u;
  const uint16_t* st_src0 = ma.x + (size_t)st_m0 * K + (size_t)warp * 128 + st_pc * 8;
  auto stage_tile = [&](int c) {
    if (c < nsteps) {
      const uint16_t* src = st_src0 + (size_t)c * (kWarps * 128);
      if constexpr (kUnrolledCopies) {
        const unsigned dst = st_dst0 + (unsigned)((c % kBufs) * tile_pieces + st_m0 * kTilePitch) * 16u;
        const unsigned d0 = dst + st_place, d1 = dst + (st_place ^ 64u);
#pragma unroll
        for (int j = 0; j < (TP + 1) / 2; ++j) {   // row st_m0 + 2 j
          if (st_m0 + 2 * j < M)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(((j & 1) ? d1 : d0) + (unsigned)(2 * j * kTilePitch * 16)),
                         "l"(src));
          src += 2 * (size_t)K;
        }
      } else {
        const unsigned dst = st_dst0 + (unsigned)((c % kBufs) * tile_pieces) * 16u;
        for (int m = st_m0; m < M; m += 2) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (unsigned)tile_piece(st_pc, m) * 16u),
                       "l"(src));
          src += 2 * (size_t)K;
        }
      }
    }
  };
  if (NBUF == 0) {
    stage_all();
  } else {
    stage_tile(0);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");   // also carries the scale / zero-point tables
  if (NBUF == 0) {
    // everything staged: the outlier entries of the owned rows (up to cvcap each) are copied into shared memory in a
    // group of their own (their addresses need the row pointers, a second trip to memory that nothing else waits
    // for); they meet the staged activations after the K loop
#pragma unroll
    for (int i = 0; i <= OWN; ++i) jr[i] = __shfl_sync(0xFFFFFFFFu, rp, i);
    const unsigned dst0 = (unsigned)__cvta_generic_to_shared(sm_cv + warp * OWN * kCvCap);
#pragma unroll
    for (int rr = 0; rr < OWN; ++rr) {
      const int n = min(jr[rr + 1] - jr[rr], kCvCap);
      for (int e = lane; e < n; e += 32)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst0 + (unsigned)(rr * kCvCap + e) * 4u),
                     "l"(cvp + jr[rr] + e));
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  if (NBUF != 0) {   // the tiles of the following steps, one group each
#pragma unroll
    for (int c = 1; c + 1 < kBufs; ++c) {
      stage_tile(c);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }

  if (NBUF != 0) {
    // ring mode: the outliers are done now, while the first codes are still on their way.  The
    // activations come from the token-major copy xt[K][TP] (one short contiguous read per entry).
    // All reads for the entries requested above are issued before any is used; longer rows (and the
    // owned rows after the first two) continue with two batches of entries in flight.
    const uint16_t* xt = TP == 1 ? ma.x : ma.xt;
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
    for (int rr = 0; rr < OWN; ++rr) {
      const int jb = jr[rr], je = jr[rr + 1];
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
      if (rr < 2) {
#pragma unroll
        for (int u = 0; u < kPre; ++u) add(epre[rr][u], xpre[rr][u]);
      }
      for (int jj = jb + (rr < 2 ? kPre * EPB : 0); jj < je; jj += 2 * EPB) {
        unsigned e[2];
        uint4 xq[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int j = jj + u * EPB + lane / TS;
          e[u] = j < je ? __ldg(cvp + j) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) xq[u] = xt_load(e[u]);
#pragma unroll
        for (int u = 0; u < 2; ++u) add(e[u], xq[u]);
      }
      reduce_tokens<VT, TS>(v, lane);
      constexpr int LPV = 32 / VT;   // lanes per value after the halving stages
      const int tok = part * VT + lane / LPV;
      if ((lane % LPV) / TS == 0) sm_out[(OWN * warp + rr) * TP + tok] = v[0];
    }
  }
  asm volatile("cp.async.wait_group %0;" ::"n"(NBUF == 0 ? 1 : NBUF - 2) : "memory");   // tables and x (or first tile) landed
  __syncthreads();

  // lane constants inside a chunk buffer: this lane's 64-byte segment of group `warp` for token gid
  // of every token block (lanes without a token read the zero page), the scale tables, the x sums
  // (ring mode: the four pieces of the segment sit in one aligned block of the permuted row, in the order i ^ xcx)
  int xoff[NB][2], xcx[NB];   // [0]: pairs 0..7 of the run, [1]: pairs 8..15 (they differ only with groups of 16)
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    const int m = nb * TB + (gid % TB);
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      // the column's group must be the group of the lane's (half) run: the other groups' columns read as zero
      const bool live = m < M && (GS == 8 ? gid == 2 * t + hh : (gid / TB) == (t * GS) / 4);
      xoff[nb][hh] = !live ? -1 : (NBUF == 0 ? xs_piece(warp * 16 + t * 4, m) : m * kTilePitch + ((t ^ ((m >> 1) & 1)) << 2));
    }
    xcx[nb] = (NBUF == 0 || xoff[nb][0] < 0) ? 0 : ((t >> 1) ^ ((m & 1) << 1));
  }
  // scale | zero-point << 16 of row gid of tile 0, first group of the lane's run in step `warp`
  const uint32_t* tp = sm_tab + (GS * warp + (GS == 8 ? 2 * t : (t * GS) / 4)) * R + gid;
  const int xsum_off = (NBUF == 0 ? xs_piece(warp * 16 + (lane >> 1), 0) : ((lane >> 1) ^ (lane >> 4))) * 2 + (lane & 1);   // 8-byte units, token 0

  float yacc[RT][NB][4];
#pragma unroll
  for (int rt = 0; rt < RT; ++rt)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int i = 0; i < 4; ++i) yacc[rt][nb][i] = 0.f;

  // one step of this warp (group warp + 8 c, register slot d = c % D): the next tile on its way (ring mode), the
  // B fragments and the group's sums of x once, then every tile: MMAs, refill of its slot, scale and zero-point
  auto do_step = [&](const int c, auto slot) {
    constexpr int d = decltype(slot)::value;
    if (NBUF != 0) {   // next step's activations on their way, this step's landed and visible to the warp
      __syncwarp();
      stage_tile(c + kBufs - 1);
      asm volatile("cp.async.commit_group;\ncp.async.wait_group %0;" ::"n"(NBUF == 0 ? 0 : NBUF - 1) : "memory");
      __syncwarp();
    }
    const uint4* buf = NBUF == 0 ? sm_x + c * buf_pieces : wtile + (c % kBufs) * tile_pieces;
    unsigned xr[NB][16];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      const uint4* seg0 = xoff[nb][0] >= 0 ? buf + xoff[nb][0] : reinterpret_cast<const uint4*>(smem_raw);
      const uint4* seg1 = GS == 8 ? (xoff[nb][1] >= 0 ? buf + xoff[nb][1] : reinterpret_cast<const uint4*>(smem_raw)) : seg0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 v = (i < 2 ? seg0 : seg1)[i ^ xcx[nb]];
        xr[nb][4 * i] = v.x; xr[nb][4 * i + 1] = v.y; xr[nb][4 * i + 2] = v.z; xr[nb][4 * i + 3] = v.w;
      }
    }
    // sums of x over the group's columns: per accumulator column (tokens 2t, 2t+1 of every block)
    float xs[NB][4];
    if (ONES) {
      step_ones<NB>(xr, xs);
    } else if (!BF16 && TP != 1) {   // from the table that comes with the token-major copy
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        const float2 g2 = __ldg(reinterpret_cast<const float2*>(ma.xg + (size_t)(warp + kWarps * c) * TP + nb * 8 + 2 * t));
        xs[nb][0] = g2.x; xs[nb][1] = g2.y;
      }
    } else if (!BF16 && GS <= 2) {   // one token: lane L adds columns 4L..4L+3, then the lanes of the group are summed
      const uint2 h4 = reinterpret_cast<const uint2*>(buf)[xsum_off];
      const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h4.x));
      const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h4.y));
      float xsum1 = (f0.x + f0.y) + (f1.x + f1.y);
#pragma unroll
      for (int o = G64 ? 8 : 16; o > 0; o >>= 1) xsum1 += __shfl_xor_sync(0xFFFFFFFFu, xsum1, o);
      if (G64) xsum1 = __shfl_sync(0xFFFFFFFFu, xsum1, (t >> 1) << 4);   // lanes 0-15 summed the first group, 16-31 the second
      xs[0][0] = (G64 ? (t & 1) == 0 : t == 0) ? xsum1 : 0.f;   // only column 0 (2: groups of 64) carries the token
      xs[0][1] = 0.f;
    }
    const bool refill = c + D < nsteps;
#pragma unroll
    for (int rt = 0; rt < RT; ++rt) {
      // (s 2^24, s z) on the raw path, (s, magic | z) on the subtract path
      float2 ta[2], tb[2];   // per accumulator column parity (two groups of 16 per lane), else both the same
#pragma unroll
      for (int e = 0; e < (GS == 8 ? 2 : 1); ++e) {
        const unsigned sza = tp[16 * rt + e * R], szb = tp[16 * rt + 8 + e * R];
        const float sa = __half2float(__ushort_as_half((unsigned short)sza));
        const float sb = __half2float(__ushort_as_half((unsigned short)szb));
        const unsigned za = sza >> 16, zb = szb >> 16;
        if (BF16) {
          constexpr unsigned kZeroMagic = BITS == 8 ? 0x64006400u : 0x43004300u;   // see step_sub
          ta[e] = make_float2(sa, __uint_as_float(kZeroMagic | (za * 0x00010001u)));
          tb[e] = make_float2(sb, __uint_as_float(kZeroMagic | (zb * 0x00010001u)));
        } else {
          ta[e] = make_float2(sa * 16777216.f, sa * (float)za);
          tb[e] = make_float2(sb * 16777216.f, sb * (float)zb);
        }
      }
      if (GS != 8) { ta[1] = ta[0]; tb[1] = tb[0]; }
      typename StepAcc<BITS, NB, BF16>::type acc;
      if constexpr (BF16) {
        const unsigned zma[2] = {__float_as_uint(ta[0].y), __float_as_uint(ta[1].y)};
        const unsigned zmb[2] = {__float_as_uint(tb[0].y), __float_as_uint(tb[1].y)};
        step_sub<BITS, NB>(wa[rt][d], wb[rt][d], zma, zmb, xr, acc);
      } else if constexpr (BITS == 4) {
        step_raw4<NB>(wa[rt][d], wb[rt][d], xr, acc);
      } else if constexpr (BITS == 8) {
        step_raw8<NB>(wa[rt][d], wb[rt][d], xr, acc);
      } else if constexpr (BITS == 2) {
        step_raw2<NB>(wa[rt][d], wb[rt][d], xr, acc);
      } else {
        step_raw3<NB>(wa[rt][d], wb[rt][d], xr, acc);
      }
      // refill the slot with the group D steps ahead
      load_run_if<BITS>(codes, oa[rt] + D * kStepWords, wa[rt][d], refill);
      load_run_if<BITS>(codes, ob[rt] + D * kStepWords, wb[rt][d], refill);
      oa[rt] += kStepWords;
      ob[rt] += kStepWords;
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (TP == 1 && GS < 8 && (i & 1)) continue;   // a single token lives in the even accumulator columns
          const float2 tt = i < 2 ? ta[i & 1] : tb[i & 1];
          if constexpr (BF16) {
            yacc[rt][nb][i] = fmaf(tt.x, acc.c[nb][i], yacc[rt][nb][i]);
          } else if constexpr (BITS == 4) {
            const float code_sum = fmaf(acc.c4[nb][i], 0.0625f, acc.c0[nb][i]);  // units of 2^-24
            yacc[rt][nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xs[nb][i & 1], yacc[rt][nb][i]));
          } else if constexpr (BITS == 8) {
            yacc[rt][nb][i] = fmaf(tt.x, acc.c0[nb][i], fmaf(-tt.y, xs[nb][i & 1], yacc[rt][nb][i]));
          } else if constexpr (BITS == 2) {
            const float code_sum = fmaf(acc.c2[nb][i], 0.25f, acc.c0[nb][i]);
            yacc[rt][nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xs[nb][i & 1], yacc[rt][nb][i]));
          } else {
            const float code_sum = fmaf(acc.c6[nb][i], 0.015625f, fmaf(acc.c3[nb][i], 0.125f, acc.c0[nb][i]));
            yacc[rt][nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xs[nb][i & 1], yacc[rt][nb][i]));
          }
        }
      }
    }
    tp += GS * kWarps * R;
  };
  for (int c0 = 0; c0 < nsteps; c0 += D)   // the register slot of a step is a compile-time constant
    unroll_slots([&](auto slot) { if (c0 + decltype(slot)::value < nsteps) do_step(c0 + decltype(slot)::value, slot); },
                 std::make_integer_sequence<int, D>{});

  if (NBUF == 0) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // this warp's outlier entries have landed
    __syncwarp();
    // CSR outliers of the owned rows: lane = entry, every token per lane,
    // one transposing reduction per row; the entries come from shared memory (those beyond cvcap, rare, from global
    // memory), the activations from the staged copy
    const uint16_t* xs16 = reinterpret_cast<const uint16_t*>(sm_x);
    const uint32_t* mycv = sm_cv + warp * OWN * kCvCap;
#pragma unroll
    for (int rr = 0; rr < OWN; ++rr) {
      const int jb = jr[rr], je = jr[rr + 1];
      float v[TP];
#pragma unroll
      for (int m = 0; m < TP; ++m) v[m] = 0.f;
      for (int e0 = lane; e0 < je - jb; e0 += 32) {
        const unsigned e = e0 < kCvCap ? mycv[rr * kCvCap + e0] : __ldg(cvp + jb + e0);
        const float wv = __half2float(__ushort_as_half((unsigned short)(e >> 16)));
        const unsigned col = e & 0xFFFFu;
        const int base = (int)(col >> 10) * buf_pieces;            // chunk = col / 1024
        const int pc = (int)((col & 1023u) >> 3), sub = (int)(col & 7u);
#pragma unroll
        for (int m = 0; m < TP; ++m)
          if (TP == 1 || m < M)
            v[m] = fmaf(wv, act_to_float<BF16>(xs16[((base + xs_piece(pc, m)) << 3) + sub]), v[m]);
      }
      reduce_tokens<TP, 1>(v, lane);
      constexpr int LPT = 32 / TP;   // lanes per token after the reduction
      if ((lane & (LPT - 1)) == 0) sm_out[(OWN * warp + rr) * TP + lane / LPT] = v[0];
    }
  }

  // partial sums of the 8 warps: sm_red[warp][tile][nb][row][token]
#pragma unroll
  for (int rt = 0; rt < RT; ++rt)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      float* r = sm_red + ((warp * RT + rt) * NB + nb) * 128;
      *reinterpret_cast<float2*>(r + gid * 8 + 2 * t) = make_float2(yacc[rt][nb][0], yacc[rt][nb][1]);
      *reinterpret_cast<float2*>(r + (gid + 8) * 8 + 2 * t) = make_float2(yacc[rt][nb][2], yacc[rt][nb][3]);
    }
  __syncthreads();

  // final sum and store: o -> (token, local row), rows fastest
  for (int o = tid; o < R * M; o += kThreads) {
    const int lr = o % R, m = o / R;
    const int row = r0 + lr;
    if (row < N) {
      const int rt = lr >> 4, l16 = lr & 15;
      const int nb = m / TB, tk = m % TB;
      float v = sm_out[lr * TP + m];
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float* r = sm_red + ((w * RT + rt) * NB + nb) * 128 + l16 * 8 + tk;
#pragma unroll
        for (int g = 0; g < GS; ++g) v += r[TB * g];   // the token's column in every group of the step
      }
      store_y(yout, ma.yd, (long long)m * N + row, v);
    }
  }
}

template <int BITS, int TP, bool BF16, int NBUF, int GS, int RT, bool DEEP = false>
cudaError_t launch(const Variant& v, const MultiArgs& a, cudaStream_t stream) {
  const size_t smem = smem_bytes(v, a.K, a.M, a.cvcap);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<BITS, TP, BF16, NBUF, GS, RT, DEEP>,
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
  return cudaLaunchKernelEx(&cfg, decode_kernel<BITS, TP, BF16, NBUF, GS, RT, DEEP>, a);
}

// the variants that exist: x staged up front for up to 8 tokens, rings of two tiles up to 8 tokens and of three beyond
// (two when shared memory is short); two m16 tiles per CTA, or eight groups of codes in flight, up to 8 tokens with
// groups of 128; groups of 64 up to 16 tokens; groups of 32 up to 4 tokens and of 16 for one token, staged only
template <int BITS, bool BF16, int TP, int GS>
cudaError_t launch_tp(const Variant& v, const MultiArgs& a, cudaStream_t stream) {
  if constexpr (GS >= 4) {
    if (v.nbuf == 0 && v.rt == 1 && !v.deep) return launch<BITS, TP, BF16, 0, GS, 1>(v, a, stream);
    return cudaErrorInvalidValue;
  } else {
    if (v.nbuf == 0) {
      if constexpr (TP <= 8) {
        constexpr bool kWide = BITS == 3 || BITS == 4;   // two tiles per CTA and the deep variant: these widths only
        if (v.rt == 2) {
          if constexpr (GS == 1 && kWide) return launch<BITS, TP, BF16, 0, GS, 2>(v, a, stream);
          return cudaErrorInvalidValue;
        }
        if constexpr (GS == 1 && kWide) {
          if (v.deep) return launch<BITS, TP, BF16, 0, GS, 1, true>(v, a, stream);
        }
        return launch<BITS, TP, BF16, 0, GS, 1>(v, a, stream);
      }
      return cudaErrorInvalidValue;
    }
    constexpr bool kWide = BITS == 3 || BITS == 4;
    if (v.rt == 2) {
      if constexpr (GS == 1 && TP <= 8 && kWide) {
        if (v.nbuf == 2) return launch<BITS, TP, BF16, 2, GS, 2>(v, a, stream);
      }
      return cudaErrorInvalidValue;
    }
    if constexpr (GS == 1 && TP <= 8 && kWide) {
      if (v.deep && v.nbuf == 2) return launch<BITS, TP, BF16, 2, GS, 1, true>(v, a, stream);
    }
    if (v.nbuf == 2) return launch<BITS, TP, BF16, 2, GS, 1>(v, a, stream);
    if constexpr (TP >= 16) return launch<BITS, TP, BF16, 3, GS, 1>(v, a, stream);
    return cudaErrorInvalidValue;
  }
}

template <int BITS, bool BF16>
cudaError_t launch_any(const Variant& v, const MultiArgs& a, cudaStream_t stream) {
  if (v.gs == 8) return v.tp == 1 ? launch_tp<BITS, BF16, 1, 8>(v, a, stream) : cudaErrorInvalidValue;
  if (v.gs == 4) {
    if (v.tp == 1) return launch_tp<BITS, BF16, 1, 4>(v, a, stream);
    if (v.tp == 4) return launch_tp<BITS, BF16, 4, 4>(v, a, stream);
    return cudaErrorInvalidValue;
  }
  if (v.gs == 2) {
    switch (v.tp) {
      case 1: return launch_tp<BITS, BF16, 1, 2>(v, a, stream);
      case 4: return launch_tp<BITS, BF16, 4, 2>(v, a, stream);
      case 8: return launch_tp<BITS, BF16, 8, 2>(v, a, stream);
      case 16: return launch_tp<BITS, BF16, 16, 2>(v, a, stream);
    }
    return cudaErrorInvalidValue;
  }
  switch (v.tp) {
    case 1: return launch_tp<BITS, BF16, 1, 1>(v, a, stream);
    case 4: return launch_tp<BITS, BF16, 4, 1>(v, a, stream);
    case 8: return launch_tp<BITS, BF16, 8, 1>(v, a, stream);
    case 16: return launch_tp<BITS, BF16, 16, 1>(v, a, stream);
    case 32: return launch_tp<BITS, BF16, 32, 1>(v, a, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace
}  // namespace gwq_decode

#endif  // GWQ_DECODE_KERNEL_IMPL
