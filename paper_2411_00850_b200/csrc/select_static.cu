// Outlier selection for callers that must not allocate device memory.
//
// Same kernels as gwq_select_outliers, but the work area (radix histogram, select
// state, per-row counters) lives in a fixed array inside the library image instead of
// coming from cudaMalloc, and the CSR arrays are supplied by the caller.
#include <math.h>

#include <mutex>

#include "common.cuh"

// Implemented next to the selection kernels.
size_t gwq_select_scratch_words(int N);
cudaError_t gwq_select_run(const uint16_t* W, const float* G, int N, int K, unsigned int k_out,
                           int32_t* row_ptr, int32_t* col_idx, uint16_t* val, unsigned int* scratch,
                           int sm_count, cudaStream_t stream);

#define GWQ_STATIC_MAX_ROWS 32768
#define GWQ_STATIC_SCRATCH_WORDS (2048 + 4 + 3 * GWQ_STATIC_MAX_ROWS)

// 401 424 bytes (392 KiB) of device memory, held by every GPU that loads this library until
// the process exits.  Shared by all calls: its contents are whatever the last call left.
static __device__ __align__(256) unsigned int g_select_scratch[GWQ_STATIC_SCRATCH_WORDS];

namespace {
constexpr int kMaxDevices = 64;
unsigned int* g_scratch_addr[kMaxDevices] = {nullptr};
int g_sm_count[kMaxDevices] = {0};
gwq_status g_lookup_status[kMaxDevices] = {GWQ_OK};
std::once_flag g_lookup_once[kMaxDevices];

// The symbol's name is only a host-side handle; the kernels need its device address,
// which differs per GPU.  Looked up once per device, with that device current; host
// threads that make their first call at the same time wait for the one lookup.
gwq_status scratch_for_current_device(unsigned int** ptr, int* sms) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GWQ_ERR_CUDA;
  std::call_once(g_lookup_once[dev], [dev]() {
    void* p = nullptr;
    int n = 0;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      (void)cudaGetLastError();
      g_lookup_status[dev] = GWQ_ERR_CUDA;
      return;
    }
    g_sm_count[dev] = n;
    g_scratch_addr[dev] = static_cast<unsigned int*>(p);
  });
  if (g_lookup_status[dev] != GWQ_OK) return g_lookup_status[dev];
  *ptr = g_scratch_addr[dev];
  *sms = g_sm_count[dev];
  return GWQ_OK;
}
}  // namespace

extern "C" gwq_status gwq_select_outliers_static(const uint16_t* W, const float* G, int32_t N, int32_t K,
                                                 double frac, int32_t* row_ptr, int32_t* col_idx,
                                                 uint16_t* val, int64_t capacity, int64_t* nnz_host,
                                                 void* stream_) {
  if (nnz_host) *nnz_host = 0;
  if (!W || !G || !row_ptr || !col_idx || !val || !nnz_host || N <= 0 || K <= 0) return GWQ_ERR_INVALID_ARG;
  if (!(frac >= 0.0 && frac <= 1.0)) return GWQ_ERR_INVALID_ARG;
  if (!gwq_aligned16(W) || !gwq_aligned16(G)) return GWQ_ERR_INVALID_ARG;
  const long long numel = (long long)N * K;
  if (numel >= (1LL << 31)) return GWQ_ERR_INVALID_ARG;
  if (K % 32 != 0) return GWQ_ERR_UNSUPPORTED;
  if (N > GWQ_STATIC_MAX_ROWS || gwq_select_scratch_words(N) > (size_t)GWQ_STATIC_SCRATCH_WORDS)
    return GWQ_ERR_UNSUPPORTED;  // more rows than the fixed work area can count
  double kd = ceil(frac * (double)numel);
  if (kd < 0) kd = 0;
  if (kd > (double)numel) kd = (double)numel;
  const long long k_out = (long long)kd;
  if (capacity < k_out) {  // caller's col_idx / val are too short: report the size they need
    *nnz_host = k_out;
    return GWQ_ERR_INVALID_ARG;
  }

  unsigned int* scratch = nullptr;
  int sms = 0;
  gwq_status st = scratch_for_current_device(&scratch, &sms);
  if (st != GWQ_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (k_out == 0) {
    if (cudaMemsetAsync(row_ptr, 0, ((size_t)N + 1) * sizeof(int32_t), stream) != cudaSuccess) return GWQ_ERR_CUDA;
  } else {
    // gwq_select_run clears the histogram and the state words itself; the per-row
    // counters are fully overwritten before they are read.
    if (gwq_select_run(W, G, N, K, (unsigned int)k_out, row_ptr, col_idx, val, scratch, sms, stream) != cudaSuccess) {
      (void)cudaGetLastError();
      return GWQ_ERR_CUDA;
    }
  }
  if (cudaStreamSynchronize(stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  *nnz_host = k_out;
  return GWQ_OK;
}
