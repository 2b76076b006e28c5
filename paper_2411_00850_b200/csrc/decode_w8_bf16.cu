// Decode kernels for 8-bit codes and bf16 activations (one translation unit per combination keeps the
// build parallel).
#define GWQ_DECODE_KERNEL_IMPL
#include "decode_kernel.cuh"

namespace gwq_decode {
cudaError_t launch_w8_bf16(const Variant& v, const MultiArgs& a, cudaStream_t stream) {
  return launch_any<8, true>(v, a, stream);
}
}  // namespace gwq_decode
