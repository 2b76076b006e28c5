// Host side of the decode path (M <= 32) of y = x (s (q - z) + S)^T (Section 3.2, Eq. "w"): choice of the
// kernel variant, the token-major copy of the activations that the variants with more than 8 tokens gather
// the outliers' activations from, and the launch.  The kernels are in decode_kernel.cuh.
#include "decode_kernel.cuh"

namespace gwq_decode {

size_t smem_bytes(const Variant& v, int K, int M, int cvcap) {
  const int R = 16 * v.rt, NB = token_blocks(v.tp, v.gs);
  const int ngroups = K / 128, nchunks = (ngroups + kChunkGroups - 1) / kChunkGroups;
  const size_t fixed = 64 + (size_t)R * (v.gs * ngroups) * 4 + (size_t)kWarps * v.rt * NB * 128 * 4 +
                       (size_t)R * v.tp * 4;
  if (v.nbuf != 0) return fixed + (size_t)kWarps * v.nbuf * M * kTilePitch * 16;
  return fixed + (size_t)kWarps * 2 * v.rt * cvcap * 4 + (size_t)nchunks * M * kRowPitch * 16;
}

}  // namespace gwq_decode

namespace {
using namespace gwq_decode;

template <bool BF16>
__device__ __forceinline__ float act_to_float(uint16_t b) {
  if (BF16) return __uint_as_float((unsigned)b << 16);
  return __half2float(__ushort_as_half(b));
}

// One CTA per group of 128 columns: xt[col][token] = x[token][col] for token < M (zero beyond), TP tokens
// per column, and xg[group][token] = sum of x[token][col] over the group's columns (FP32).
template <int TP, bool BF16>
__global__ void __launch_bounds__(128) tokens_to_columns(const uint16_t* __restrict__ x, uint16_t* __restrict__ xt,
                                                         float* __restrict__ xg, int M, int K) {
  __shared__ float red[4][TP];
  // launched with programmatic stream serialization: the product that follows may start fetching its weights now;
  // x may still be being written by the kernel before this one
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
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


constexpr int kMaxTokens64 = 16;  // groups of 64: tokens one launch takes
// Groups of 64 with 9 to 16 tokens need four token blocks (184 to 229 registers, one CTA per SM): faster than the
// tensor-core kernel's 32-token tile up to about this many weights (measured: 59.8 against 84.8 us on 8192 x 8192,
// 184.5 against 163.1 us on 28672 x 8192), slower beyond.
constexpr long long kMaxWeights64Wide = 160LL * 1000 * 1000;
constexpr size_t kSmemPerCta = 227 * 1024;
// Staging all of x up front costs shared memory, hence resident CTAs: the limits keep three CTAs of one tile (two of
// two tiles) on an SM; grids of at most two CTAs per SM may take a little more.
constexpr size_t kStageAllLimit = 72 * 1024;
constexpr size_t kStageAllLimitSmallGrid = 80 * 1024;
constexpr size_t kStageAllLimitTwoTiles = 96 * 1024;
#ifndef GWQ_TUNE_RT
#define GWQ_TUNE_RT 0   // 1 / 2 force the tiles per CTA (tuning builds); 0: chosen from the grid size
#endif

// The variant for `count` layers that read the same x, or false when the streaming kernel has none: group size
// 128 (M <= 32) or 64 (M <= 8; M <= 16 for layers up to kMaxWeights64Wide weights), K <= 65536 and a multiple of
// 128, same K, group size and bit width in every layer, shared memory for at least a ring of two tiles.
bool plan(const gwq_packed* const* P, int count, int M, Variant* v, int* cvcap) {
  if (count < 1 || count > kMaxLayers || M < 1 || M > 32) return false;
  const int group = P[0]->group;
  if (group != 128 && group != 64 && group != 32 && group != 16) return false;
  const bool g64 = group == 64;
  const int gs = 128 / group;
  if (gs >= 4 && M > (gs == 4 ? 4 : 1)) return false;   // small groups: the token blocks shrink with the group
  const int K = P[0]->K;
  if (K % 128 != 0) return false;   // a warp step is 128 columns
  if (g64 && M > kMaxTokens64) return false;
  long long rows = 0, nnz = 0;
  for (int i = 0; i < count; ++i) {
    const gwq_priv* pvi = static_cast<const gwq_priv*>(P[i]->priv);
    if (P[i]->group != group || !pvi->cv || !pvi->sz_t ||
        P[i]->K != K || P[i]->bits != P[0]->bits)
      return false;
    if (g64 && M > 8 && (long long)P[i]->N * K > kMaxWeights64Wide) return false;
    rows += P[i]->N;
    nnz += P[i]->S->nnz;
  }
  const gwq_priv* pv = static_cast<const gwq_priv*>(P[0]->priv);
  const int sms = pv->sm_count > 0 ? pv->sm_count : 148;
  v->gs = gs;
  v->tp = M == 1 ? 1 : (M <= 4 ? 4 : (M <= 8 ? 8 : (M <= 16 ? 16 : 32)));
  // Two tiles per CTA (up to 8 tokens, groups of 128) halve the per-row cost of everything a CTA does once, but an SM
  // holds two such CTAs instead of three: they are taken where they turn a grid of more than one wave into a single one
  long long blocks1 = 0, blocks2 = 0;
  for (int i = 0; i < count; ++i) {
    blocks1 += (P[i]->N + 15) / 16;
    blocks2 += (P[i]->N + 31) / 32;
  }
  const bool wide = P[0]->bits == 3 || P[0]->bits == 4;   // two tiles per CTA and the deep variant exist for these widths
  v->rt = (wide && gs == 1 && v->tp <= 8 && blocks1 > 3LL * sms && blocks2 <= 2LL * sms) ? 2 : 1;
  if (GWQ_TUNE_RT == 1 || (GWQ_TUNE_RT == 2 && wide && gs == 1 && v->tp <= 8)) v->rt = GWQ_TUNE_RT;
  long long blocks = 0;
  for (int i = 0; i < count; ++i) blocks += (P[i]->N + 16 * v->rt - 1) / (16 * v->rt);
  // a grid that leaves an SM two CTAs at most anyway: twice the codes in flight per warp (more registers, which then
  // cost no occupancy)
  v->deep = (wide && v->rt == 1 && gs == 1 && v->tp <= 8 && blocks <= 2LL * sms) ? 1 : 0;
#ifdef GWQ_TUNE_DEEP
  v->deep = (wide && v->rt == 1 && gs == 1 && v->tp <= 8) ? GWQ_TUNE_DEEP : 0;
#endif
  const int nchunks = (K / 128 + kChunkGroups - 1) / kChunkGroups;
  const size_t lim = v->rt == 2 ? kStageAllLimitTwoTiles : (blocks <= 2LL * sms ? kStageAllLimitSmallGrid : kStageAllLimit);
  // outlier entries per row kept in shared memory: one and a half times the average row, in steps of 32
  long long cap = rows > 0 ? (3 * nnz / (2 * rows) + 47) / 32 * 32 : 32;
  *cvcap = (int)(cap < 32 ? 32 : (cap > 512 ? 512 : cap));
  v->nbuf = 0;
  if (v->tp <= 8 && (size_t)nchunks * M * kRowPitch * 16 <= lim &&
      smem_bytes(*v, K, M, *cvcap) <= kSmemPerCta)
    return true;
  if (gs >= 4) return false;                // small groups: staged activations only
  if (v->tp > 1 && !pv->xt) return false;   // ring mode gathers the outliers' activations from a token-major copy
  v->nbuf = v->tp <= 8 ? 2 : 3;
  if (v->nbuf == 3 && smem_bytes(*v, K, M, *cvcap) > kSmemPerCta) v->nbuf = 2;
  if (smem_bytes(*v, K, M, *cvcap) > kSmemPerCta && v->rt == 2) {   // the tables of a very wide layer: one tile per CTA
    v->rt = 1;
    v->nbuf = v->tp <= 8 ? 2 : 3;
    if (v->nbuf == 3 && smem_bytes(*v, K, M, *cvcap) > kSmemPerCta) v->nbuf = 2;
  }
  return smem_bytes(*v, K, M, *cvcap) <= kSmemPerCta;
}

}  // namespace

size_t gwq_decode_scratch_bytes(int K) { return (size_t)K * 32 * 2 + (size_t)(K / 128) * 32 * 4; }

bool gwq_decode_takes(const gwq_packed* P, int M) {
  Variant v;
  int cvcap;
  return plan(&P, 1, M, &v, &cvcap);
}

// Decode launcher for `count` layers that read the same x.  Returns GWQ_ERR_UNSUPPORTED where the streaming kernel
// has no variant (nothing has been launched then).  The scratch for the token-major copy of x is the first layer's.
gwq_status gwq_launch_decode_multi(const gwq_packed* const* P, int count, const void* x, gwq_dtype xd, int M,
                                   void* const* y, gwq_dtype yd, cudaStream_t stream) {
  Variant v;
  MultiArgs a;
  if (!plan(P, count, M, &v, &a.cvcap)) return GWQ_ERR_UNSUPPORTED;
  const gwq_priv* pv = static_cast<const gwq_priv*>(P[0]->priv);
  const int K = P[0]->K;
  a.xt = nullptr;
  a.xg = nullptr;
  int blocks = 0;
  for (int i = 0; i < kMaxLayers; ++i) {
    const gwq_packed* Pi = P[i < count ? i : 0];
    a.layer[i].codes = Pi->codes; a.layer[i].szt = static_cast<const gwq_priv*>(Pi->priv)->sz_t;
    a.layer[i].row_ptr = Pi->S->row_ptr; a.layer[i].cv = static_cast<const gwq_priv*>(Pi->priv)->cv;
    a.layer[i].y = y[i < count ? i : 0]; a.layer[i].N = Pi->N;
    a.first_block[i] = blocks;
    if (i < count) blocks += (Pi->N + 16 * v.rt - 1) / (16 * v.rt);
  }
  a.first_block[kMaxLayers] = blocks;
  for (int i = count; i < kMaxLayers; ++i) a.first_block[i] = blocks;
  a.count = count;
  a.sm_count = pv->sm_count > 0 ? pv->sm_count : 148;
  a.x = static_cast<const uint16_t*>(x); a.yd = yd; a.K = K; a.M = M;
  if (v.nbuf != 0 && v.tp > 1) {   // token-major copy of x and its group sums, once for all layers
    uint16_t* xt = static_cast<uint16_t*>(pv->xt);
    float* xg = reinterpret_cast<float*>(static_cast<char*>(pv->xt) + (size_t)K * 32 * 2);
    const bool bf = xd == GWQ_BF16;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(K / 128));
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t pe = cudaSuccess;
    switch (v.tp) {
#define GWQ_T2C(TP)                                                                                   \
  case TP:                                                                                            \
    pe = bf ? cudaLaunchKernelEx(&cfg, tokens_to_columns<TP, true>, a.x, xt, xg, M, K)               \
            : cudaLaunchKernelEx(&cfg, tokens_to_columns<TP, false>, a.x, xt, xg, M, K);             \
    break;
      GWQ_T2C(4) GWQ_T2C(8) GWQ_T2C(16) GWQ_T2C(32)
#undef GWQ_T2C
    }
    if (pe != cudaSuccess) {
      (void)cudaGetLastError();
      return GWQ_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return GWQ_ERR_CUDA;
    a.xt = xt;
    a.xg = xg;
  }
  cudaError_t e;
  const bool bf = xd == GWQ_BF16;
  switch (P[0]->bits) {
    case 4: e = bf ? launch_w4_bf16(v, a, stream) : launch_w4_f16(v, a, stream); break;
    case 3: e = bf ? launch_w3_bf16(v, a, stream) : launch_w3_f16(v, a, stream); break;
    case 8: e = bf ? launch_w8_bf16(v, a, stream) : launch_w8_f16(v, a, stream); break;
    case 2: e = bf ? launch_w2_bf16(v, a, stream) : launch_w2_f16(v, a, stream); break;
    default: return GWQ_ERR_UNSUPPORTED;
  }
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  return GWQ_OK;
}

// One layer.  GWQ_ERR_UNSUPPORTED: the caller takes the tensor-core or the general kernel.
gwq_status gwq_launch_decode(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y, gwq_dtype yd,
                             cudaStream_t stream) {
  return gwq_launch_decode_multi(&P, 1, x, xd, M, &y, yd, stream);
}
