// Measurement aid for the benchmark (no part of the method and no part of the library's interface): one launch
// that only READS a list of device arrays and does no arithmetic on them.  Given the arrays a forward product
// reads of a packed layer at one token (codes, scales, zero-points, CSR row pointers, 4 bytes per outlier), its
// duration is the floor of any one-launch-per-layer product on this device (launch, ramp-up and drain included),
// which is what the decode timings are set beside.  Built as a shared library of its own.
#include <cuda_runtime.h>
#include <cstdint>

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeUnroll = 8;
constexpr int kMaxArrays = 8;

struct ProbeArgs {
  const uint4* base[kMaxArrays];
  unsigned long long count[kMaxArrays];   // 16-byte items
  int arrays;
  unsigned* sink;
  unsigned never;   // a value the folded words are compared with (run-time argument, so the loads stay)
};

__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const ProbeArgs p) {
  unsigned acc = 0;
  const unsigned long long nthreads = (unsigned long long)gridDim.x * kProbeThreads;
  const unsigned long long t0 = (unsigned long long)blockIdx.x * kProbeThreads + threadIdx.x;
  for (int a = 0; a < p.arrays; ++a) {
    const uint4* __restrict__ b = p.base[a];
    const unsigned long long n = p.count[a];
    for (unsigned long long i = t0; i < n; i += nthreads * kProbeUnroll) {
      uint4 v[kProbeUnroll];
#pragma unroll
      for (int u = 0; u < kProbeUnroll; ++u) {
        const unsigned long long j = i + (unsigned long long)u * nthreads;
        v[u] = j < n ? __ldcs(b + j) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kProbeUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
  }
  // keeps the loads alive: the store needs the folded words
  if (acc == p.never) p.sink[0] = acc;
}

}  // namespace

// Reads bytes[i] / 16 whole 16-byte items from base[i] (device pointers, 16-byte aligned; base and bytes are
// host arrays of `arrays` <= 8 entries), asynchronously on `stream`, with `ctas_per_sm` x the device's SM count
// blocks.  sink: one device word the kernel may write.  Returns the bytes one launch reads, or -1 on a bad
// argument or a failed launch.
extern "C" long long bench_read_probe(const void* const* base, const unsigned long long* bytes, int arrays,
                                      void* sink, int blocks, void* stream) {
  if (!base || !bytes || arrays < 1 || arrays > kMaxArrays || !sink || blocks < 1) return -1;
  ProbeArgs a{};
  long long total = 0;
  for (int i = 0; i < arrays; ++i) {
    if (!base[i] || (reinterpret_cast<uintptr_t>(base[i]) & 15)) return -1;
    a.base[i] = static_cast<const uint4*>(base[i]);
    a.count[i] = bytes[i] / 16;
    total += (long long)a.count[i] * 16;
  }
  a.arrays = arrays;
  a.sink = static_cast<unsigned*>(sink);
  a.never = 0x9E3779B9u;
  read_probe_kernel<<<blocks, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? total : -1;
}
