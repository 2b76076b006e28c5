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
// Activations are staged once per CTA in shared memory (XOR-swizzled 16-byte chunks)
// when they fit, else read through L1.  After the K loop the warps' partial sums meet in
// shared memory, the CSR outliers of a row are added by the warp that owns it, and y is
// stored.  The kernel is launched with programmatic stream serialization: its weight
// prefetch may overlap the previous kernel, everything that touches x or y comes after
// griddepcontrol.wait.
#include "common.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kRows = 16;   // rows per CTA (one m16 tile)
constexpr int kDepth = 4;   // groups of codes in flight per warp

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
  const uint16_t* scales;
  const uint8_t* zeros;
  const int32_t* row_ptr;
  const uint32_t* cv;  // per outlier: fp16 value << 16 | column
  const uint16_t* x;
  void* y;
  gwq_dtype yd;
  int N, K, M;
};

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Sum TP per-lane values over the 32 lanes with TP - 1 + log2(32 / TP) shuffles: every
// stage halves the values a lane keeps.  Afterwards lane L holds the total of value
// L / (32 / TP) in v[0].
template <int TP>
__device__ __forceinline__ void reduce_across_lanes(float (&v)[TP], int lane) {
  int n = TP;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    if (n > 1) {
      const int half = n >> 1;
      const bool up = (lane & o) != 0;
#pragma unroll
      for (int i = 0; i < (TP > 1 ? TP / 2 : 1); ++i) {
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


constexpr int kOutSlots = 3;  // outlier entries per lane held in registers (96 per row); the rest is looped

// Staged activations: 16-byte chunk c of token row m lives at chunk c + (c >> 3) + 2 (m & 1) of
// its row (one pad chunk per 128 bytes, odd rows shifted by two chunks), so that the 64-byte
// segments of the four lanes of a quad and of two neighbouring token rows fall into all eight
// 16-byte bank groups.  Row pitch in chunks:
__host__ __device__ inline int xs_pitch_chunks(int K) { return (K >> 3) + (K >> 6) + 4; }
__device__ __forceinline__ int xs_chunk(int c, int m, int pitch) { return m * pitch + c + (c >> 3) + ((m & 1) << 1); }

template <int BITS, int NB, bool BF16>
struct StepAcc;
template <int NB> struct StepAcc<4, NB, false> { using type = AccRaw4<NB>; };
template <int NB> struct StepAcc<3, NB, false> { using type = AccRaw3<NB>; };
template <int BITS, int NB> struct StepAcc<BITS, NB, true> { using type = AccSub<NB>; };

// TP = tokens rounded up to 1, 4, 8, 16 or 32.  XS: activations staged in shared memory.  Group size 128.
template <int BITS, int TP, bool BF16, bool XS>
__global__ void __launch_bounds__(kThreads, TP <= 8 ? 3 : (TP == 16 ? 2 : 1)) decode_kernel(const DecodeArgs p) {
  constexpr int NB = TP <= 8 ? 1 : TP / 8;  // 8-token blocks
  constexpr int WPR = BITS;                  // words per run of 32 columns
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int ngroups = p.K >> 7;
  constexpr bool ONES = !BF16 && !(TP == 1 && XS);  // raw path: sum_k x_k by MMA unless one staged token
  // shared: zero page 64 B | scales [16][ngroups] f16 | zeros [16][ngroups] u8 | red [kWarps][NB][16][8] f32 |
  //         outl [16][TP] f32 | x (XS)
  uint16_t* sm_s = reinterpret_cast<uint16_t*>(smem_raw + 64);
  uint8_t* sm_z = reinterpret_cast<uint8_t*>(sm_s + kRows * ngroups);
  float* sm_red = reinterpret_cast<float*>(sm_z + kRows * ngroups);
  float* sm_out = sm_red + kWarps * NB * 128;
  uint4* sm_x = reinterpret_cast<uint4*>(sm_out + kRows * TP);
  const int pitch = xs_pitch_chunks(p.K);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, t = lane & 3;
  const int r0 = blockIdx.x * kRows;
  const int ra = min(r0 + gid, p.N - 1), rb = min(r0 + gid + 8, p.N - 1);
  const unsigned row_words = (unsigned)(p.K >> 5) * WPR;
  constexpr unsigned kStepWords = kWarps * 4 * WPR;  // codes of 8 groups
  unsigned oa = (unsigned)ra * row_words + (unsigned)(warp * 4 + t) * WPR;  // group `warp`, this lane's run
  unsigned ob = (unsigned)rb * row_words + (unsigned)(warp * 4 + t) * WPR;
  const int nsteps = (ngroups - warp + kWarps - 1) / kWarps;  // groups warp, warp+8, ...

  pdl_launch_dependents();

  // ---- everything that does not depend on the previous kernel: all loads are issued before any is awaited
  // CSR extents of the two rows this warp owns (rows 2 warp and 2 warp + 1 of the CTA)
  int rp = 0;
  if (lane < 3) rp = __ldg(p.row_ptr + min(r0 + 2 * warp + lane, p.N));
  {
    // scales and zero-points of the 16 rows: two contiguous, 16-byte aligned ranges
    const int rows_here = min(kRows, p.N - r0);
    const char* gs = reinterpret_cast<const char*>(p.scales + (size_t)r0 * ngroups);
    const char* gz = reinterpret_cast<const char*>(p.zeros + (size_t)r0 * ngroups);
    if (rows_here == kRows) {
      for (int c = tid; c < 3 * ngroups; c += kThreads) {   // 32 ng + 16 ng bytes = 3 ng chunks
        const bool is_s = c < 2 * ngroups;
        const char* src = is_s ? gs + c * 16 : gz + (c - 2 * ngroups) * 16;
        const unsigned dst = (unsigned)__cvta_generic_to_shared(reinterpret_cast<char*>(sm_s) + c * 16);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src));
      }
    } else {   // last, partial CTA: rows past N read as scale 0
      for (int i = tid; i < kRows * ngroups; i += kThreads) {
        const bool live = i < rows_here * ngroups;
        sm_s[i] = live ? p.scales[(size_t)r0 * ngroups + i] : (uint16_t)0;
        sm_z[i] = live ? p.zeros[(size_t)r0 * ngroups + i] : (uint8_t)0;
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

  // ---- from here on x is read
  pdl_wait();
  if (XS) {
    const int chunks_per_row = p.K >> 3;
    for (int m = 0; m < p.M; ++m) {
      for (int c = tid; c < chunks_per_row; c += kThreads) {
        const unsigned dst = (unsigned)__cvta_generic_to_shared(sm_x + xs_chunk(c, m, pitch));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p.x + (size_t)m * p.K + c * 8));
      }
    }
  }
  // outlier payload of the two owned rows (needs the row extents: the one load awaited here)
  const int j0 = __shfl_sync(0xFFFFFFFFu, rp, 0), j1 = __shfl_sync(0xFFFFFFFFu, rp, 1),
            j2 = __shfl_sync(0xFFFFFFFFu, rp, 2);
  unsigned cv[2][kOutSlots];
#pragma unroll
  for (int e = 0; e < kOutSlots; ++e) {
    const int ja = j0 + lane + 32 * e, jb = j1 + lane + 32 * e;
    cv[0][e] = ja < j1 ? __ldcs(p.cv + ja) : 0u;  // value 0 contributes nothing
    cv[1][e] = jb < j2 ? __ldcs(p.cv + jb) : 0u;
  }
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // this lane's activation segment (64 bytes per group) for token gid of every token block;
  // lanes without a token read the zero page and never advance
  const uint4* xp[NB];
  int xstep[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    const int m = nb * 8 + gid;
    if (XS) {
      const bool live = m < p.M;
      xp[nb] = live ? sm_x + xs_chunk(warp * 16 + t * 4, m, pitch) : reinterpret_cast<const uint4*>(smem_raw);
      xstep[nb] = live ? kWarps * 18 : 0;  // 8 groups ahead: 8 * (16 + 2 pad) chunks
    } else {
      const int mm = min(m, p.M - 1);
      xp[nb] = reinterpret_cast<const uint4*>(p.x + (size_t)mm * p.K) + warp * 16 + t * 4;
      xstep[nb] = kWarps * 16;
    }
  }
  const uint16_t* sp = sm_s + gid * ngroups + warp;   // scale / zero-point of row gid, group `warp`
  const uint8_t* zp = sm_z + gid * ngroups + warp;
  const int hi_row = 8 * ngroups;
  // single staged token: its group sums come from shared memory, lane L adding columns 4L..4L+3
  const uint2* xsum_p = reinterpret_cast<const uint2*>(sm_x + xs_chunk(warp * 16 + (lane >> 1), 0, pitch)) + (lane & 1);

  float yacc[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int i = 0; i < 4; ++i) yacc[nb][i] = 0.f;

  for (int s0 = 0; s0 < nsteps; s0 += kDepth) {
#pragma unroll
    for (int d = 0; d < kDepth; ++d) {
      if (s0 + d < nsteps) {
        unsigned xr[NB][16];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 v = XS ? xp[nb][i] : __ldg(xp[nb] + i);
            if (!XS && nb * 8 + gid >= p.M) v = make_uint4(0, 0, 0, 0);  // token rows past M contribute nothing
            xr[nb][4 * i] = v.x; xr[nb][4 * i + 1] = v.y; xr[nb][4 * i + 2] = v.z; xr[nb][4 * i + 3] = v.w;
          }
          xp[nb] += xstep[nb];
        }
        // (s 2^24, s z) on the raw path, (s, magic | z) on the subtract path
        float2 ta, tb;
        {
          const float sa = __half2float(__ushort_as_half(sp[0])), sb = __half2float(__ushort_as_half(sp[hi_row]));
          const unsigned za = zp[0], zb = zp[hi_row];
          sp += kWarps;
          zp += kWarps;
          if (BF16) {
            ta = make_float2(sa, __uint_as_float(0x43004300u | (za * 0x00010001u)));
            tb = make_float2(sb, __uint_as_float(0x43004300u | (zb * 0x00010001u)));
          } else {
            ta = make_float2(sa * 16777216.f, sa * (float)za);
            tb = make_float2(sb * 16777216.f, sb * (float)zb);
          }
        }
        float xsum1 = 0.f;
        if (!BF16 && !ONES) {
          const uint2 h4 = *xsum_p;
          xsum_p += kWarps * 18 * 2;
          const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h4.x));
          const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h4.y));
          xsum1 = (f0.x + f0.y) + (f1.x + f1.y);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) xsum1 += __shfl_xor_sync(0xFFFFFFFFu, xsum1, o);
        }
        typename StepAcc<BITS, NB, BF16>::type acc = {};
        if (BF16) {
          step_sub<BITS, NB>(wa[d], wb[d], __float_as_uint(ta.y), __float_as_uint(tb.y), xr,
                             reinterpret_cast<AccSub<NB>&>(acc));
        } else if (BITS == 4) {
          step_raw4<NB, ONES>(reinterpret_cast<const unsigned(&)[4]>(wa[d]), reinterpret_cast<const unsigned(&)[4]>(wb[d]), xr,
                        reinterpret_cast<AccRaw4<NB>&>(acc));
        } else {
          step_raw3<NB, ONES>(reinterpret_cast<const unsigned(&)[3]>(wa[d]), reinterpret_cast<const unsigned(&)[3]>(wb[d]), xr,
                        reinterpret_cast<AccRaw3<NB>&>(acc));
        }
        // refill this slot with the group kDepth steps ahead (its registers are dead now)
        if (s0 + d + kDepth < nsteps) {
          load_run<BITS>(p.codes, oa + kDepth * kStepWords, wa[d]);
          load_run<BITS>(p.codes, ob + kDepth * kStepWords, wb[d]);
        }
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
              const float code_sum = fmaf(a4.c4[nb][i], 0.0625f, a4.c0[nb][i]);         // units of 2^-24
              const float xsum = ONES ? a4.xs[nb][i & 1] : ((i & 1) == 0 && t == 0 ? xsum1 : 0.f);  // token 0 only
              yacc[nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xsum, yacc[nb][i]));
            } else {
              AccRaw3<NB>& a3 = reinterpret_cast<AccRaw3<NB>&>(acc);
              const float code_sum = fmaf(a3.c6[nb][i], 0.015625f, fmaf(a3.c3[nb][i], 0.125f, a3.c0[nb][i]));
              const float xsum = ONES ? a3.xs[nb][i & 1] : ((i & 1) == 0 && t == 0 ? xsum1 : 0.f);  // token 0 only
              yacc[nb][i] = fmaf(tt.x, code_sum, fmaf(-tt.y, xsum, yacc[nb][i]));
            }
          }
        }
      }
    }
  }

  // partial sums of the 8 warps: sm_red[warp][nb][row][token]
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    float* r = sm_red + (warp * NB + nb) * 128;
    *reinterpret_cast<float2*>(r + gid * 8 + 2 * t) = make_float2(yacc[nb][0], yacc[nb][1]);
    *reinterpret_cast<float2*>(r + (gid + 8) * 8 + 2 * t) = make_float2(yacc[nb][2], yacc[nb][3]);
  }

  // CSR outliers of the two owned rows: lane = entry, every token per lane, then one
  // transposing reduction over the lanes
  auto x_at = [&](int m, unsigned col) -> float {
    if (XS) {
      const uint16_t* xs16 = reinterpret_cast<const uint16_t*>(sm_x);
      return act_to_float<BF16>(xs16[(xs_chunk((int)(col >> 3), m, pitch) << 3) + (col & 7)]);
    }
    return act_to_float<BF16>(__ldg(p.x + (size_t)m * p.K + col));
  };
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int lr = 2 * warp + rr;
    const int jb = rr == 0 ? j0 : j1, je = rr == 0 ? j1 : j2;
    float v[TP];
#pragma unroll
    for (int m = 0; m < TP; ++m) v[m] = 0.f;
    if (r0 + lr < p.N && je > jb) {
      const int ne = min(kOutSlots, (je - jb + 31) >> 5);  // warp-uniform
#pragma unroll
      for (int e = 0; e < kOutSlots; ++e) {
        if (e < ne) {
          const float wv = __half2float(__ushort_as_half((unsigned short)(cv[rr][e] >> 16)));
          const unsigned col = cv[rr][e] & 0xFFFFu;
#pragma unroll
          for (int m = 0; m < TP; ++m)
            if (TP == 1 || m < p.M) v[m] = fmaf(wv, x_at(m, col), v[m]);
        }
      }
      for (int j = jb + 32 * kOutSlots + lane; j < je; j += 32) {  // rows with more than 96 outliers
        const unsigned e = __ldg(p.cv + j);
        const float wv = __half2float(__ushort_as_half((unsigned short)(e >> 16)));
#pragma unroll
        for (int m = 0; m < TP; ++m)
          if (TP == 1 || m < p.M) v[m] = fmaf(wv, x_at(m, e & 0xFFFFu), v[m]);
      }
    }
    reduce_across_lanes<TP>(v, lane);
    constexpr int LPT = 32 / TP;  // lanes per token after the reduction
    if ((lane & (LPT - 1)) == 0) sm_out[lr * TP + lane / LPT] = v[0];
  }
  __syncthreads();

  // final sum and store: o -> (token, local row), rows fastest
  for (int o = tid; o < kRows * p.M; o += kThreads) {
    const int lr = o & 15, m = o >> 4;
    const int row = r0 + lr;
    if (row < p.N) {
      const int nb = m >> 3, tk = m & 7;
      float v = sm_out[lr * TP + m];
#pragma unroll
      for (int w = 0; w < kWarps; ++w) v += sm_red[(w * NB + nb) * 128 + lr * 8 + tk];
      store_y(p.y, p.yd, (long long)m * p.N + row, v);
    }
  }
}

constexpr size_t kXStageLimit = 72 * 1024;  // activations above this are read through L1 instead

template <int BITS, int TP, bool BF16, bool XS>
cudaError_t launch(const DecodeArgs& a, cudaStream_t stream) {
  constexpr int NB = TP <= 8 ? 1 : TP / 8;
  const int ngroups = a.K / 128;
  const size_t smem = 64 + (size_t)kRows * ngroups * 3 + (size_t)kWarps * NB * 128 * 4 + (size_t)kRows * TP * 4 +
                      (XS ? (size_t)a.M * xs_pitch_chunks(a.K) * 16 : 0);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<BITS, TP, BF16, XS>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((a.N + kRows - 1) / kRows));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_kernel<BITS, TP, BF16, XS>, a);
}

template <int BITS, bool BF16, bool XS>
cudaError_t launch_tp(const DecodeArgs& a, cudaStream_t stream) {
  if (a.M == 1) return launch<BITS, 1, BF16, XS>(a, stream);
  if (a.M <= 4) return launch<BITS, 4, BF16, XS>(a, stream);
  if (a.M <= 8) return launch<BITS, 8, BF16, XS>(a, stream);
  if (a.M <= 16) return launch<BITS, 16, BF16, XS>(a, stream);
  return launch<BITS, 32, BF16, XS>(a, stream);
}

template <int BITS, bool BF16>
cudaError_t launch_xs(const DecodeArgs& a, cudaStream_t stream) {
  if ((size_t)a.M * xs_pitch_chunks(a.K) * 16 <= kXStageLimit) return launch_tp<BITS, BF16, true>(a, stream);
  return launch_tp<BITS, BF16, false>(a, stream);
}

}  // namespace

// Decode launcher: group size 128, M <= 32, K <= 65536.  Other shapes go to the general kernel.
gwq_status gwq_launch_decode(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y, gwq_dtype yd,
                             cudaStream_t stream) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  if (P->group != 128 || M > 32 || !pv->cv) return gwq_launch_simt(P, x, xd, M, y, yd, stream);
  DecodeArgs a;
  a.codes = P->codes; a.scales = P->scales; a.zeros = P->zeros;
  a.row_ptr = P->S->row_ptr; a.cv = pv->cv;
  a.x = static_cast<const uint16_t*>(x); a.y = y; a.yd = yd;
  a.N = P->N; a.K = P->K; a.M = M;
  cudaError_t e;
  if (P->bits == 4) e = (xd == GWQ_BF16) ? launch_xs<4, true>(a, stream) : launch_xs<4, false>(a, stream);
  else e = (xd == GWQ_BF16) ? launch_xs<3, true>(a, stream) : launch_xs<3, false>(a, stream);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  return GWQ_OK;
}
