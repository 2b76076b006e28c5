// Entry points that are not kernels of their own: dispatch of the forward product,
// the host-buffer variant, object release and status names.
#include "common.cuh"

#ifndef GWQ_DECODE_MAX_M
#define GWQ_DECODE_MAX_M 32   // up to here the streaming mma.sync kernel; above, the tcgen05 kernel
#endif

static size_t dtype_bytes(gwq_dtype d) { return d == GWQ_F32 ? 4 : 2; }

// 17 to 32 tokens that the tcgen05 streaming kernel does not take (bf16 activations, or no workspace): the mma.sync
// kernel needs four token blocks there (one CTA of 8 warps per SM, 8 KB of activations copied per KB of codes), so
// the tensor-core kernel's 32-token tile is faster as soon as its 128-row tiles keep at least half of the SMs busy
// (measured, 4 bit, M = 32: 44 against 52 us on 11008 x 4096 and 161 against 215 us on 28672 x 8192; 84 against 70 us
// on 8192 x 8192, whose 64 tiles leave most SMs idle).
static bool prefers_tensor_core(const gwq_packed* P, int M) {
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  const int sms = pv->sm_count > 0 ? pv->sm_count : 148;
  return M > 16 && M <= GWQ_DECODE_MAX_M && P->group == 128 && 2 * ((P->N + 127) / 128) >= sms && P->K % 64 == 0 &&
         pv->cv && pv->sz_t;
}

#ifndef GWQ_TUNE_SKINNY_MIN_M
// fewest tokens that go to the tcgen05 streaming kernel when a workspace is given: its cost per step hardly depends on
// the token count, the mma.sync kernel's grows with it; measured cross-over between 16 and 17 tokens (4 bit, 16 tokens:
// 37 against 35 us on 8192 x 8192, 31 against 25 us on 11008 x 4096; 32 tokens: 37 against 70 us, 31 against 44 us)
#define GWQ_TUNE_SKINNY_MIN_M 17
#endif

static bool wants_skinny(const gwq_packed* P, gwq_dtype xd, int M) {
  return M >= GWQ_TUNE_SKINNY_MIN_M && M <= GWQ_DECODE_MAX_M && gwq_skinny_takes(P, xd, M);
}

extern "C" size_t gwq_linear_workspace_bytes(const gwq_packed* P, gwq_dtype xd, int32_t M) {
  if (!P || P->tag != GWQ_TAG_PACKED || !P->priv || M <= 0) return 0;
  if (wants_skinny(P, xd, M)) return gwq_skinny_workspace_bytes(P, M);
  if (M <= GWQ_DECODE_MAX_M && !prefers_tensor_core(P, M) && gwq_decode_takes(P, M)) return 0;
  return gwq_prefill_workspace_bytes(P, xd, M);
}

extern "C" gwq_status gwq_linear_ws(const gwq_packed* P, const void* x, gwq_dtype xd, int32_t M, void* y,
                                    gwq_dtype yd, void* ws, size_t ws_bytes, void* stream_) {
  if (!P || P->tag != GWQ_TAG_PACKED || !P->S || !P->priv || !x || !y || M <= 0) return GWQ_ERR_INVALID_ARG;
  if (xd != GWQ_F16 && xd != GWQ_BF16) return GWQ_ERR_UNSUPPORTED;
  if (yd != GWQ_F16 && yd != GWQ_BF16 && yd != GWQ_F32) return GWQ_ERR_INVALID_ARG;
  if (!gwq_aligned16(x) || !gwq_aligned16(y)) return GWQ_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // with a workspace, 17 to 32 fp16 tokens take the tcgen05 streaming kernel; without one the other kernels serve them
  if (wants_skinny(P, xd, M) && ws && ws_bytes >= gwq_skinny_workspace_bytes(P, M))
    return gwq_launch_skinny(P, x, M, y, yd, ws, ws_bytes, stream);
  if (M <= GWQ_DECODE_MAX_M && !prefers_tensor_core(P, M)) {
    const gwq_status st = gwq_launch_decode(P, x, xd, M, y, yd, stream);
    if (st != GWQ_ERR_UNSUPPORTED) return st;   // shapes the streaming kernel does not take: the tensor-core kernel
  }
  return gwq_launch_prefill(P, x, xd, M, y, yd, ws, ws_bytes, stream);
}

extern "C" gwq_status gwq_linear(const gwq_packed* P, const void* x, gwq_dtype xd, int32_t M, void* y,
                                 gwq_dtype yd, void* stream_) {
  return gwq_linear_ws(P, x, xd, M, y, yd, nullptr, 0, stream_);
}

extern "C" gwq_status gwq_linear_multi(const gwq_packed* const* P, int32_t count, const void* x, gwq_dtype xd,
                                       int32_t M, void* const* y, gwq_dtype yd, void* stream_) {
  if (!P || !y || !x || count < 1 || count > GWQ_MULTI_MAX || M <= 0) return GWQ_ERR_INVALID_ARG;
  if (xd != GWQ_F16 && xd != GWQ_BF16) return GWQ_ERR_UNSUPPORTED;
  if (yd != GWQ_F16 && yd != GWQ_BF16 && yd != GWQ_F32) return GWQ_ERR_INVALID_ARG;
  if (!gwq_aligned16(x)) return GWQ_ERR_INVALID_ARG;
  for (int i = 0; i < count; ++i) {
    if (!P[i] || P[i]->tag != GWQ_TAG_PACKED || !P[i]->S || !P[i]->priv || !y[i] || !gwq_aligned16(y[i]))
      return GWQ_ERR_INVALID_ARG;
    if (P[i]->K != P[0]->K) return GWQ_ERR_INVALID_ARG;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  bool fused = M <= GWQ_DECODE_MAX_M;
  for (int i = 0; i < count; ++i) fused = fused && !prefers_tensor_core(P[i], M);   // same kernels as gwq_linear
  if (fused) {
    const gwq_status st = gwq_launch_decode_multi(P, count, x, xd, M, y, yd, stream);
    if (st != GWQ_ERR_UNSUPPORTED) return st;
  }
  for (int i = 0; i < count; ++i) {
    const gwq_status st = gwq_linear(P[i], x, xd, M, y[i], yd, stream_);
    if (st != GWQ_OK) return st;
  }
  return GWQ_OK;
}

static gwq_status linear_host(gwq_packed* P, const void* x_host, gwq_dtype xd, int32_t M, void* y_host, gwq_dtype yd,
                              void* stream_, bool synchronise) {
  if (!P || P->tag != GWQ_TAG_PACKED || !P->priv || !x_host || !y_host || M <= 0) return GWQ_ERR_INVALID_ARG;
  if (xd != GWQ_F16 && xd != GWQ_BF16) return GWQ_ERR_UNSUPPORTED;
  if (yd != GWQ_F16 && yd != GWQ_BF16 && yd != GWQ_F32) return GWQ_ERR_INVALID_ARG;
  gwq_priv* pv = static_cast<gwq_priv*>(P->priv);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const size_t xb = (size_t)M * P->K * dtype_bytes(xd), yb = (size_t)M * P->N * dtype_bytes(yd);
  gwq_status st = GWQ_OK;
  if (pv->x_stage_bytes < xb) {
    GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
    if (pv->x_stage) cudaFree(pv->x_stage);
    pv->x_stage = nullptr;
    pv->x_stage_bytes = 0;
    GWQ_CUDA_TRY(cudaMalloc(&pv->x_stage, xb));
    pv->x_stage_bytes = xb;
  }
  if (pv->y_stage_bytes < yb) {
    GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
    if (pv->y_stage) cudaFree(pv->y_stage);
    pv->y_stage = nullptr;
    pv->y_stage_bytes = 0;
    GWQ_CUDA_TRY(cudaMalloc(&pv->y_stage, yb));
    pv->y_stage_bytes = yb;
  }
  {
    const size_t wb = gwq_linear_workspace_bytes(P, xd, M);
    if (pv->ws_stage_bytes < wb) {
      GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
      if (pv->ws_stage) cudaFree(pv->ws_stage);
      pv->ws_stage = nullptr;
      pv->ws_stage_bytes = 0;
      GWQ_CUDA_TRY(cudaMalloc(&pv->ws_stage, wb));
      pv->ws_stage_bytes = wb;
    }
  }
  GWQ_CUDA_TRY(cudaMemcpyAsync(pv->x_stage, x_host, xb, cudaMemcpyHostToDevice, stream));
  st = gwq_linear_ws(P, pv->x_stage, xd, M, pv->y_stage, yd, pv->ws_stage, pv->ws_stage_bytes, stream);
  if (st != GWQ_OK) return st;
  GWQ_CUDA_TRY(cudaMemcpyAsync(y_host, pv->y_stage, yb, cudaMemcpyDeviceToHost, stream));
  if (synchronise) GWQ_CUDA_TRY(cudaStreamSynchronize(stream));
  return GWQ_OK;
fail:
  return st;
}

extern "C" gwq_status gwq_linear_host(gwq_packed* P, const void* x_host, gwq_dtype xd, int32_t M,
                                      void* y_host, gwq_dtype yd, void* stream_) {
  return linear_host(P, x_host, xd, M, y_host, yd, stream_, true);
}

extern "C" gwq_status gwq_linear_host_async(gwq_packed* P, const void* x_host, gwq_dtype xd, int32_t M,
                                            void* y_host, gwq_dtype yd, void* stream_) {
  return linear_host(P, x_host, xd, M, y_host, yd, stream_, false);
}

extern "C" gwq_status gwq_device_status(const gwq_packed* P, void* stream_) {
  if (!P || P->tag != GWQ_TAG_PACKED || !P->priv) return GWQ_ERR_INVALID_ARG;
  const gwq_priv* pv = static_cast<const gwq_priv*>(P->priv);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, pv->dev_status, sizeof(h), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return GWQ_ERR_CUDA;
  }
  if (h != 0) (void)cudaMemsetAsync(pv->dev_status, 0, sizeof(int32_t), stream);
  return (gwq_status)h;
}

extern "C" gwq_status gwq_set_wait_limit(gwq_packed* P, int64_t cycles) {
  if (!P || P->tag != GWQ_TAG_PACKED || !P->priv) return GWQ_ERR_INVALID_ARG;
  static_cast<gwq_priv*>(P->priv)->wait_cycles = cycles < 0 ? GWQ_DEFAULT_WAIT_CYCLES : (long long)cycles;
  return GWQ_OK;
}

static void free_outliers(gwq_outliers* S) {
  if (!S) return;
  if (S->row_ptr) cudaFree(S->row_ptr);
  if (S->col_idx) cudaFree(S->col_idx);
  if (S->val) cudaFree(S->val);
  S->tag = 0;
  delete S;
}

extern "C" void gwq_free(void* obj) {
  if (!obj) return;
  const uint32_t tag = *static_cast<const uint32_t*>(obj);
  if (tag == GWQ_TAG_OUTLIERS) {
    free_outliers(static_cast<gwq_outliers*>(obj));
  } else if (tag == GWQ_TAG_PACKED) {
    gwq_packed* P = static_cast<gwq_packed*>(obj);
    if (P->codes) cudaFree(P->codes);
    if (P->scales) cudaFree(P->scales);
    if (P->zeros) cudaFree(P->zeros);
    free_outliers(P->S);
    gwq_priv* pv = static_cast<gwq_priv*>(P->priv);
    if (pv) {
      if (pv->cv) cudaFree(pv->cv);
      if (pv->x_stage) cudaFree(pv->x_stage);
      if (pv->y_stage) cudaFree(pv->y_stage);
      if (pv->ws_stage) cudaFree(pv->ws_stage);
      if (pv->xt) cudaFree(pv->xt);
      if (pv->ob) cudaFree(pv->ob);
      if (pv->ob_ptr) cudaFree(pv->ob_ptr);
      if (pv->sz_t) cudaFree(pv->sz_t);
      if (pv->dev_status) cudaFree(pv->dev_status);
      delete pv;
    }
    P->tag = 0;
    delete P;
  }
}

extern "C" const char* gwq_status_string(gwq_status s) {
  switch (s) {
    case GWQ_OK: return "GWQ_OK";
    case GWQ_ERR_INVALID_ARG: return "GWQ_ERR_INVALID_ARG";
    case GWQ_ERR_UNSUPPORTED: return "GWQ_ERR_UNSUPPORTED";
    case GWQ_ERR_ALLOC: return "GWQ_ERR_ALLOC";
    case GWQ_ERR_NONFINITE: return "GWQ_ERR_NONFINITE";
    case GWQ_ERR_TIMEOUT: return "GWQ_ERR_TIMEOUT";
    case GWQ_ERR_CUDA: return "GWQ_ERR_CUDA";
    case GWQ_ERR_WORKSPACE: return "GWQ_ERR_WORKSPACE";
  }
  return "GWQ_ERR_UNKNOWN";
}
