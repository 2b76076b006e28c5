// Mean of the gradients of several calibration samples (Section 4.3, "Effect on Number of
// Calibration": the outliers are located on the gradient mean).  One pass over all samples; the
// arithmetic is fixed so that the result is reproducible bit for bit: FP32 additions in sample order
// (round to nearest), then one FP32 division by the count.
#include "common.cuh"

namespace {

constexpr int kMaxSamples = GWQ_GRAD_SAMPLES_MAX;

struct MeanArgs {
  const float* g[kMaxSamples];
  int count;
};

__global__ void __launch_bounds__(256) gradient_mean_kernel(const MeanArgs a, float* __restrict__ out, long long numel) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  const float n = (float)a.count;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < numel; i += stride) {
    float acc = __ldcs(a.g[0] + i);
#pragma unroll
    for (int s = 1; s < kMaxSamples; ++s)
      if (s < a.count) acc = __fadd_rn(acc, __ldcs(a.g[s] + i));
    out[i] = __fdiv_rn(acc, n);
  }
}

}  // namespace

extern "C" gwq_status gwq_gradient_mean(const float* const* G_list, int32_t count, int64_t numel, float* G_mean,
                                        void* stream_) {
  if (!G_list || !G_mean || count < 1 || count > kMaxSamples || numel <= 0) return GWQ_ERR_INVALID_ARG;
  MeanArgs a;
  for (int s = 0; s < kMaxSamples; ++s) {
    a.g[s] = G_list[s < count ? s : 0];
    if (!a.g[s]) return GWQ_ERR_INVALID_ARG;
  }
  a.count = count;
  long long blocks = (numel + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  gradient_mean_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream_)>>>(a, G_mean, numel);
  return cudaGetLastError() == cudaSuccess ? GWQ_OK : GWQ_ERR_CUDA;
}
