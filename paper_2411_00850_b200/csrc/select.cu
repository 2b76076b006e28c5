// Outlier location: exact top-k of |G| per weight matrix (Section 3.2, Eq. "o").
//
// The rank key of an entry is the bit pattern of |g| (31 bits); equal keys are
// taken in ascending flat index.  The threshold key is found with a three-pass
// most-significant-digit radix select (11 + 10 + 10 bits); the rows are then
// counted, scanned and emitted as CSR in column order, so the result is
// deterministic and independent of the launch shape.
#include <math.h>

#include <new>

#include "common.cuh"

namespace {

constexpr int kBins = 2048;
constexpr int kThreads = 256;

struct SelState {
  unsigned int prefix;       // key bits decided so far
  unsigned int prefix_mask;  // which key bits are decided
  unsigned int k_rem;        // entries still to take among keys matching the prefix
  unsigned int pad;
};

__device__ __forceinline__ unsigned int abs_key(unsigned int bits) { return bits & 0x7FFFFFFFu; }

// Start of a selection: clears the histogram and the state words and sets the count to take (a kernel
// argument, so nothing is copied from host memory that the caller might reuse).
__global__ void __launch_bounds__(kThreads) sel_init_kernel(unsigned int* __restrict__ scratch, unsigned int k_out) {
  for (int i = threadIdx.x; i < kBins + 4; i += kThreads) scratch[i] = 0u;
  __syncthreads();
  if (threadIdx.x == 0) reinterpret_cast<SelState*>(scratch + kBins)->k_rem = k_out;
}

// Histogram of one radix digit over the keys that match the decided prefix.
__global__ void __launch_bounds__(kThreads) sel_hist_kernel(const uint4* __restrict__ G4, long long n4,
                                                            const SelState* __restrict__ st,
                                                            unsigned int* __restrict__ hist, int shift,
                                                            int nbits) {
  __shared__ unsigned int sh[kBins];
  for (int i = threadIdx.x; i < kBins; i += kThreads) sh[i] = 0;
  __syncthreads();
  const unsigned int prefix = st->prefix, pmask = st->prefix_mask;
  const unsigned int dmask = (1u << nbits) - 1u;
  const long long stride = (long long)gridDim.x * kThreads;
  for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n4; i += stride) {
    const uint4 v = __ldg(G4 + i);
    const unsigned int k0 = abs_key(v.x), k1 = abs_key(v.y), k2 = abs_key(v.z), k3 = abs_key(v.w);
    if ((k0 & pmask) == prefix) atomicAdd(&sh[(k0 >> shift) & dmask], 1u);
    if ((k1 & pmask) == prefix) atomicAdd(&sh[(k1 >> shift) & dmask], 1u);
    if ((k2 & pmask) == prefix) atomicAdd(&sh[(k2 >> shift) & dmask], 1u);
    if ((k3 & pmask) == prefix) atomicAdd(&sh[(k3 >> shift) & dmask], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kBins; i += kThreads)
    if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// Picks the digit that holds the k_rem-th largest key, updates the state and clears
// the histogram for the next pass.  One block of 1024 threads.
__global__ void __launch_bounds__(1024) sel_find_kernel(SelState* st, unsigned int* hist, int shift,
                                                        int nbits) {
  __shared__ unsigned int h[kBins];
  __shared__ unsigned int suf[2][kBins + 1];
  const int t = threadIdx.x;
  for (int i = t; i < kBins; i += 1024) {
    h[i] = hist[i];
    hist[i] = 0;
    suf[0][i] = h[i];
  }
  __syncthreads();
  // inclusive suffix sums: suf[d] = sum_{j >= d} h[j]
  int cur = 0;
  for (int off = 1; off < kBins; off <<= 1) {
    for (int i = t; i < kBins; i += 1024)
      suf[cur ^ 1][i] = suf[cur][i] + ((i + off < kBins) ? suf[cur][i + off] : 0u);
    cur ^= 1;
    __syncthreads();
  }
  const unsigned int k = st->k_rem;
  const int nb = 1 << nbits;
  __syncthreads();
  for (int d = t; d < nb; d += 1024) {
    const unsigned int ge = suf[cur][d];
    const unsigned int gt = (d + 1 < kBins) ? suf[cur][d + 1] : 0u;
    if (ge >= k && gt < k) {  // unique: implies h[d] > 0
      st->k_rem = k - gt;
      st->prefix |= (unsigned int)d << shift;
      st->prefix_mask |= ((1u << nbits) - 1u) << shift;
    }
  }
}

__device__ __forceinline__ unsigned int block_sum(unsigned int v, unsigned int* sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned int total = 0;
  for (int w = 0; w < kThreads / 32; ++w) total += sh[w];
  __syncthreads();
  return total;
}

// Per row: entries above the threshold key, and entries equal to it.
__global__ void __launch_bounds__(kThreads) sel_rowcount_kernel(const uint4* __restrict__ G4, int K4,
                                                                const SelState* __restrict__ st,
                                                                unsigned int* __restrict__ n_gt,
                                                                unsigned int* __restrict__ n_tie) {
  __shared__ unsigned int sh[kThreads / 32];
  const unsigned int thr = st->prefix;
  const uint4* row = G4 + (long long)blockIdx.x * K4;
  unsigned int gt = 0, tie = 0;
  for (int i = threadIdx.x; i < K4; i += kThreads) {
    const uint4 v = __ldg(row + i);
    const unsigned int k0 = abs_key(v.x), k1 = abs_key(v.y), k2 = abs_key(v.z), k3 = abs_key(v.w);
    gt += (k0 > thr) + (k1 > thr) + (k2 > thr) + (k3 > thr);
    tie += (k0 == thr) + (k1 == thr) + (k2 == thr) + (k3 == thr);
  }
  gt = block_sum(gt, sh);
  tie = block_sum(tie, sh);
  if (threadIdx.x == 0) {
    n_gt[blockIdx.x] = gt;
    n_tie[blockIdx.x] = tie;
  }
}

// Exclusive scan over 1024 per-thread partial sums (one block of 1024 threads).
__device__ __forceinline__ unsigned int block_excl_scan_1024(unsigned int v, unsigned int* sh,
                                                             unsigned int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int inc = v;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += u;
  }
  if (lane == 31) sh[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned int w = sh[lane];
    unsigned int winc = w;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int u = __shfl_up_sync(0xFFFFFFFFu, winc, o);
      if (lane >= o) winc += u;
    }
    sh[lane] = winc - w;
    if (lane == 31) sh[32] = winc;
  }
  __syncthreads();
  const unsigned int res = sh[warp] + inc - v;
  *total = sh[32];
  __syncthreads();
  return res;
}

// Row order decides which ties are kept: the first k_rem ties in flat-index order.
// Writes take[row] (ties kept in that row) and the CSR row pointers.
__global__ void __launch_bounds__(1024) sel_rowscan_kernel(int N, const SelState* __restrict__ st,
                                                           const unsigned int* __restrict__ n_gt,
                                                           const unsigned int* __restrict__ n_tie,
                                                           unsigned int* __restrict__ take,
                                                           int32_t* __restrict__ row_ptr) {
  __shared__ unsigned int sh[33];
  const int chunk = (N + 1023) / 1024;
  const int r0 = min(N, (int)threadIdx.x * chunk), r1 = min(N, r0 + chunk);
  const unsigned int k_ties = st->k_rem;
  unsigned int tsum = 0;
  for (int r = r0; r < r1; ++r) tsum += n_tie[r];
  unsigned int total;
  unsigned int tpre = block_excl_scan_1024(tsum, sh, &total);
  unsigned int csum = 0;
  for (int r = r0; r < r1; ++r) {
    const unsigned int nt = n_tie[r];
    const unsigned int left = (tpre < k_ties) ? (k_ties - tpre) : 0u;
    const unsigned int tk = min(nt, left);
    take[r] = tk;
    csum += n_gt[r] + tk;
    tpre += nt;
  }
  unsigned int cpre = block_excl_scan_1024(csum, sh, &total);
  for (int r = r0; r < r1; ++r) {
    row_ptr[r] = (int32_t)cpre;
    cpre += n_gt[r] + take[r];
  }
  if (threadIdx.x == 0) row_ptr[N] = (int32_t)total;
}

// Emits the CSR rows in column order, one warp per row: every entry above the threshold, and the first
// take[row] entries equal to it.  A lane reads four consecutive columns (one 16-byte load, four loads in flight);
// a 128-column slice without a candidate costs one ballot, the others a warp scan of the per-lane counts.
constexpr int kEmitUnroll = 4;
__global__ void __launch_bounds__(kThreads) sel_emit_kernel(const uint4* __restrict__ G4,
                                                            const uint16_t* __restrict__ W, int N, int K,
                                                            const SelState* __restrict__ st,
                                                            const unsigned int* __restrict__ take,
                                                            const int32_t* __restrict__ row_ptr,
                                                            int32_t* __restrict__ col_idx,
                                                            uint16_t* __restrict__ val) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  if (row >= N) return;
  const int begin = row_ptr[row];
  if (row_ptr[row + 1] == begin) return;   // the whole warp leaves
  const unsigned int thr = st->prefix;
  const unsigned int tk = take[row];
  const int n4 = K >> 2;
  const uint4* g = G4 + (long long)row * n4;
  const uint16_t* w = W + (long long)row * K;
  unsigned int run_gt = 0, run_tie = 0;
  for (int c0 = 0; c0 < n4; c0 += 32 * kEmitUnroll) {
    uint4 v[kEmitUnroll];
#pragma unroll
    for (int u = 0; u < kEmitUnroll; ++u) {
      const int idx = c0 + u * 32 + lane;
      v[u] = idx < n4 ? __ldg(g + idx) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < kEmitUnroll; ++u) {
      const int idx = c0 + u * 32 + lane;
      const bool valid = idx < n4;
      const unsigned int k4[4] = {abs_key(v[u].x), abs_key(v[u].y), abs_key(v[u].z), abs_key(v[u].w)};
      unsigned int mg = 0, mt = 0;   // this lane's four columns: above / equal to the threshold
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        mg |= (valid && k4[e] > thr) ? (1u << e) : 0u;
        mt |= (valid && k4[e] == thr) ? (1u << e) : 0u;
      }
      if (__ballot_sync(0xFFFFFFFFu, (mg | mt) != 0u) == 0u) continue;
      const unsigned int mine = (unsigned int)__popc(mg) | ((unsigned int)__popc(mt) << 16);
      unsigned int scan = mine;   // inclusive scan over the lanes of both counts (at most 128 each)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, scan, o);
        if (lane >= o) scan += up;
      }
      const unsigned int total = __shfl_sync(0xFFFFFFFFu, scan, 31);
      unsigned int gt_before = run_gt + ((scan - mine) & 0xFFFFu), tie_before = run_tie + ((scan - mine) >> 16);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool is_gt = (mg >> e) & 1u, is_tie = (mt >> e) & 1u;
        if (is_gt || (is_tie && tie_before < tk)) {
          const unsigned int pos = gt_before + min(tie_before, tk);
          const int col = idx * 4 + e;
          col_idx[begin + pos] = col;
          val[begin + pos] = w[col];
        }
        gt_before += is_gt ? 1u : 0u;
        tie_before += is_tie ? 1u : 0u;
      }
      run_gt += total & 0xFFFFu;
      run_tie += total >> 16;
    }
  }
}

}  // namespace

// Scratch (32-bit words): histogram [kBins], state [4], n_gt [N], n_tie [N], take [N].
size_t gwq_select_scratch_words(int N) { return (size_t)kBins + 4 + 3 * (size_t)N; }

// Runs the selection into caller-provided outputs and scratch.  k_out >= 1.
cudaError_t gwq_select_run(const uint16_t* W, const float* G, int N, int K, unsigned int k_out,
                           int32_t* row_ptr, int32_t* col_idx, uint16_t* val, unsigned int* scratch,
                           int sm_count, cudaStream_t stream) {
  unsigned int* hist = scratch;
  SelState* st = reinterpret_cast<SelState*>(scratch + kBins);
  unsigned int* n_gt = scratch + kBins + 4;
  unsigned int* n_tie = n_gt + N;
  unsigned int* take = n_tie + N;
  const long long numel = (long long)N * K;
  const long long n4 = numel / 4;
  sel_init_kernel<<<1, kThreads, 0, stream>>>(scratch, k_out);
  long long want = (n4 + kThreads - 1) / kThreads;
  const int grid = (int)(want < (long long)sm_count * 8 ? (want > 0 ? want : 1) : (long long)sm_count * 8);
  const int shifts[3] = {20, 10, 0}, nbits[3] = {11, 10, 10};
  for (int p = 0; p < 3; ++p) {
    sel_hist_kernel<<<grid, kThreads, 0, stream>>>(reinterpret_cast<const uint4*>(G), n4, st, hist,
                                                   shifts[p], nbits[p]);
    sel_find_kernel<<<1, 1024, 0, stream>>>(st, hist, shifts[p], nbits[p]);
  }
  sel_rowcount_kernel<<<N, kThreads, 0, stream>>>(reinterpret_cast<const uint4*>(G), K / 4, st, n_gt, n_tie);
  sel_rowscan_kernel<<<1, 1024, 0, stream>>>(N, st, n_gt, n_tie, take, row_ptr);
  sel_emit_kernel<<<(N + kThreads / 32 - 1) / (kThreads / 32), kThreads, 0, stream>>>(
      reinterpret_cast<const uint4*>(G), W, N, K, st, take, row_ptr, col_idx, val);
  return cudaGetLastError();
}

extern "C" gwq_status gwq_select_outliers(const uint16_t* W, const float* G, int32_t N, int32_t K,
                                          double frac, gwq_outliers** out, void* stream_) {
  if (out) *out = nullptr;
  if (!W || !G || !out || N <= 0 || K <= 0) return GWQ_ERR_INVALID_ARG;
  if (!(frac >= 0.0 && frac <= 1.0)) return GWQ_ERR_INVALID_ARG;
  if (!gwq_aligned16(W) || !gwq_aligned16(G)) return GWQ_ERR_INVALID_ARG;
  const long long numel = (long long)N * K;
  if (numel >= (1LL << 31)) return GWQ_ERR_INVALID_ARG;
  if (K % 32 != 0) return GWQ_ERR_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  double kd = ceil(frac * (double)numel);
  if (kd < 0) kd = 0;
  if (kd > (double)numel) kd = (double)numel;
  const long long k_out = (long long)kd;

  gwq_status st = GWQ_OK;
  unsigned int* scratch = nullptr;
  gwq_outliers* S = new (std::nothrow) gwq_outliers();
  if (!S) return GWQ_ERR_ALLOC;
  S->tag = GWQ_TAG_OUTLIERS;
  S->N = N;
  S->K = K;
  S->nnz = k_out;
  S->row_ptr = nullptr;
  S->col_idx = nullptr;
  S->val = nullptr;
  int dev = 0, sms = 0;
  GWQ_CUDA_TRY(cudaGetDevice(&dev));
  GWQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  GWQ_CUDA_TRY(cudaMalloc(&S->row_ptr, ((size_t)N + 1) * sizeof(int32_t)));
  GWQ_CUDA_TRY(cudaMalloc(&S->col_idx, (size_t)(k_out > 0 ? k_out : 1) * sizeof(int32_t)));
  GWQ_CUDA_TRY(cudaMalloc(&S->val, (size_t)(k_out > 0 ? k_out : 1) * sizeof(uint16_t) + 16));
  if (k_out == 0) {
    GWQ_CUDA_TRY(cudaMemsetAsync(S->row_ptr, 0, ((size_t)N + 1) * sizeof(int32_t), stream));
  } else {
    GWQ_CUDA_TRY(cudaMalloc(&scratch, gwq_select_scratch_words(N) * sizeof(unsigned int)));
    GWQ_CUDA_TRY(gwq_select_run(W, G, N, K, (unsigned int)k_out, S->row_ptr, S->col_idx, S->val, scratch,
                                sms, stream));
  }
  GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  if (scratch) cudaFree(scratch);
  *out = S;
  return GWQ_OK;
fail:
  if (scratch) cudaFree(scratch);
  if (S->row_ptr) cudaFree(S->row_ptr);
  if (S->col_idx) cudaFree(S->col_idx);
  if (S->val) cudaFree(S->val);
  delete S;
  return st;
}


namespace {
__global__ void rebase_row_ptr_kernel(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int n, int32_t base) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[i] - base;
}
}  // namespace

extern "C" gwq_status gwq_outliers_rows(const gwq_outliers* S, int32_t row0, int32_t row1, gwq_outliers** out,
                                        void* stream_) {
  if (out) *out = nullptr;
  if (!S || !out || S->tag != GWQ_TAG_OUTLIERS || row0 < 0 || row1 > S->N || row0 >= row1) return GWQ_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  gwq_status st = GWQ_OK;
  int32_t ends[2] = {0, 0};
  gwq_outliers* R = new (std::nothrow) gwq_outliers();
  if (!R) return GWQ_ERR_ALLOC;
  R->tag = GWQ_TAG_OUTLIERS;
  R->N = row1 - row0;
  R->K = S->K;
  R->nnz = 0;
  R->row_ptr = nullptr;
  R->col_idx = nullptr;
  R->val = nullptr;
  GWQ_CUDA_TRY(cudaMemcpyAsync(&ends[0], S->row_ptr + row0, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  GWQ_CUDA_TRY(cudaMemcpyAsync(&ends[1], S->row_ptr + row1, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
  GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  R->nnz = ends[1] - ends[0];
  GWQ_CUDA_TRY(cudaMalloc(&R->row_ptr, ((size_t)R->N + 1) * sizeof(int32_t)));
  GWQ_CUDA_TRY(cudaMalloc(&R->col_idx, (size_t)(R->nnz > 0 ? R->nnz : 1) * sizeof(int32_t)));
  GWQ_CUDA_TRY(cudaMalloc(&R->val, (size_t)(R->nnz > 0 ? R->nnz : 1) * sizeof(uint16_t) + 16));
  rebase_row_ptr_kernel<<<(R->N + 1 + 255) / 256, 256, 0, stream>>>(S->row_ptr + row0, R->row_ptr, R->N + 1, ends[0]);
  GWQ_CUDA_TRY(cudaGetLastError());
  if (R->nnz > 0) {
    GWQ_CUDA_TRY(cudaMemcpyAsync(R->col_idx, S->col_idx + ends[0], (size_t)R->nnz * sizeof(int32_t), cudaMemcpyDeviceToDevice, stream));
    GWQ_CUDA_TRY(cudaMemcpyAsync(R->val, S->val + ends[0], (size_t)R->nnz * sizeof(uint16_t), cudaMemcpyDeviceToDevice, stream));
  }
  GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  *out = R;
  return GWQ_OK;
fail:
  if (R->row_ptr) cudaFree(R->row_ptr);
  if (R->col_idx) cudaFree(R->col_idx);
  if (R->val) cudaFree(R->val);
  delete R;
  return st;
}
