// Shared host/device helpers of the GWQ library (internal; not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gwq.h"

#define GWQ_TAG_OUTLIERS 0x4F515747u /* "GWQO" */
#define GWQ_TAG_PACKED 0x50515747u   /* "GWQP" */

// Needs a local `gwq_status st` and a label `fail`.
#define GWQ_CUDA_TRY(expr)                                                    \
  do {                                                                        \
    cudaError_t e__ = (expr);                                                 \
    if (e__ != cudaSuccess) {                                                 \
      (void)cudaGetLastError();                                               \
      st = (e__ == cudaErrorMemoryAllocation) ? GWQ_ERR_ALLOC : GWQ_ERR_CUDA; \
      goto fail;                                                              \
    }                                                                         \
  } while (0)

// Kernel-private part of a packed layer.
struct gwq_priv {
  uint32_t* cv;          // per outlier: fp16 value << 16 | column (NULL when K > 65536)
  void* x_stage;         // staging for gwq_linear_host
  void* y_stage;
  size_t x_stage_bytes;
  size_t y_stage_bytes;
  uint32_t* sz_t;        // [K/group][N]: scale fp16 bits | zero-point << 16 (tensor-core path)
  void* ws_stage;        // scratch for gwq_linear_host where the product needs some
  size_t ws_stage_bytes;
  void* xt;              // token-major copy [K][32] of the activations and their group sums (decode path with more
  size_t xt_bytes;       // than 8 tokens); created by gwq_pack
  uint32_t* ob;          // outliers ordered by block of 128 rows x 128 columns: row << 23 | column << 16 | fp16 value
  int32_t* ob_ptr;       // [blocks + 1] extents of the blocks in ob (block = tile * (K / 128) + column block)
  void* ob_scratch;      // counters while gwq_pack builds ob
  int32_t* dev_status;   // device status word written by bounded waits
  int sm_count;
  long long wait_cycles; // SM cycles a bounded device-side wait may spin (gwq_set_wait_limit)
};

#define GWQ_DEFAULT_WAIT_CYCLES (1000LL * 1000LL * 1000LL)

static inline bool gwq_aligned16(const void* p) {
  return (reinterpret_cast<uintptr_t>(p) & 15u) == 0;
}

// Kernel launchers implemented in the other translation units.
gwq_status gwq_launch_simt(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y,
                           gwq_dtype yd, cudaStream_t stream);
gwq_status gwq_launch_decode(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y,
                             gwq_dtype yd, cudaStream_t stream);
gwq_status gwq_launch_decode_multi(const gwq_packed* const* P, int count, const void* x, gwq_dtype xd, int M,
                                   void* const* y, gwq_dtype yd, cudaStream_t stream);
gwq_status gwq_launch_prefill(const gwq_packed* P, const void* x, gwq_dtype xd, int M, void* y,
                              gwq_dtype yd, void* ws, size_t ws_bytes, cudaStream_t stream);
size_t gwq_prefill_workspace_bytes(const gwq_packed* P, gwq_dtype xd, int M);
bool gwq_skinny_takes(const gwq_packed* P, gwq_dtype xd, int M);
size_t gwq_skinny_workspace_bytes(const gwq_packed* P, int M);
gwq_status gwq_launch_skinny(const gwq_packed* P, const void* x, int M, void* y, gwq_dtype yd, void* ws, size_t ws_bytes,
                             cudaStream_t stream);
bool gwq_decode_takes(const gwq_packed* P, int M);   // the streaming kernel has a variant for (P, M)
size_t gwq_decode_scratch_bytes(int K);              // bytes of gwq_priv::xt
