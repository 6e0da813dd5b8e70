// Handle, allocator plumbing, status strings.
#include "common.cuh"

#include <new>

namespace comet {

static void *default_alloc(void *, size_t bytes, void *) {
  void *p = nullptr;
  if (cudaMalloc(&p, bytes ? bytes : 1) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return p;
}
static void default_free(void *, void *p, void *) { if (p) cudaFree(p); }

comet_status_t cuda_fail(Context *ctx, cudaError_t e) {
  if (ctx) { ctx->last_cuda_error = (int)e; ctx->counters_dirty = true; }
  cudaGetLastError();   // clear the sticky-less error state
  return COMET_ERR_CUDA;
}

void *ctx_alloc(Context *ctx, size_t bytes, cudaStream_t stream) {
  return ctx->allocator.alloc(ctx->allocator.ctx, bytes ? bytes : 1, (void *)stream);
}
void ctx_free(Context *ctx, void *p, cudaStream_t stream) {
  if (p) ctx->allocator.free(ctx->allocator.ctx, p, (void *)stream);
}

// The scratch and the device counters (words 32..35 of d_status, which the kernels that use them leave at zero)
// belong to one call at a time. Two things could break that silently and are made safe here, where every
// contraction passes: a call on ANOTHER stream than the handle's previous call waits for that stream first (its
// kernels may still be using both), and after any failed CUDA call the counters are cleared before the next use
// (a kernel that did not run to its end may not have put them back).
static void ctx_enter(Context *ctx, cudaStream_t stream) {
  if (ctx->has_last_stream && ctx->last_stream != stream) cudaStreamSynchronize(ctx->last_stream);
  ctx->last_stream = stream;
  ctx->has_last_stream = true;
  if (ctx->counters_dirty && ctx->d_status) {
    if (cudaMemsetAsync(ctx->d_status + 32, 0, 4 * sizeof(int32_t), stream) == cudaSuccess) ctx->counters_dirty = false;
    else cudaGetLastError();
  }
}

void *scratch_get(Context *ctx, size_t bytes, cudaStream_t stream) {
  ctx_enter(ctx, stream);
  if (bytes <= ctx->scratch_bytes && ctx->scratch) return ctx->scratch;
  if (ctx->scratch) {
    // work queued on the stream may still read the old buffer
    cudaStreamSynchronize(stream);
    ctx_free(ctx, ctx->scratch, stream);
    ctx->scratch = nullptr;
    ctx->scratch_bytes = 0;
  }
  size_t want = align_up(bytes + bytes / 4, 1 << 20);
  ctx->scratch = ctx_alloc(ctx, want, stream);
  if (!ctx->scratch) return nullptr;
  ctx->scratch_bytes = want;
  return ctx->scratch;
}

}  // namespace comet

using comet::Context;

extern "C" comet_status_t comet_create(comet_handle_t *handle, const comet_allocator_t *allocator) {
  if (!handle) return COMET_ERR_INVALID_ARG;
  *handle = nullptr;
  if (allocator && (!allocator->alloc || !allocator->free)) return COMET_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return COMET_ERR_CUDA; }
  Context *ctx = new (std::nothrow) Context();
  if (!ctx) return COMET_ERR_ALLOC;
  ctx->user_allocator = allocator != nullptr;
  if (allocator) ctx->allocator = *allocator;
  else ctx->allocator = comet_allocator_t{comet::default_alloc, comet::default_free, nullptr};
  ctx->device = dev;
  ctx->last_cuda_error = 0;
  ctx->has_last_stream = false;
  ctx->last_stream = nullptr;
  ctx->counters_dirty = false;
  ctx->has_copy_streams = false;
  ctx->launches = 0;
  ctx->scratch = nullptr;
  ctx->scratch_bytes = 0;
  ctx->h_pinned = nullptr;
  ctx->d_status = nullptr;
  if (cudaMallocHost((void **)&ctx->h_pinned, 64 * sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc((void **)&ctx->d_status, 64 * sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
    delete ctx;
    return COMET_ERR_CUDA;
  }
  // words 32.. hold counters that kernels leave at zero when they finish (see contract_scalar.cu)
  if (cudaMemset(ctx->d_status, 0, 64 * sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    cudaFreeHost(ctx->h_pinned);
    cudaFree(ctx->d_status);
    delete ctx;
    return COMET_ERR_CUDA;
  }
  *handle = reinterpret_cast<comet_handle_t>(ctx);
  return COMET_OK;
}

extern "C" comet_status_t comet_destroy(comet_handle_t handle) {
  if (!handle) return COMET_OK;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaDeviceSynchronize();
  comet::host_streams_destroy(ctx);
  if (ctx->scratch) comet::ctx_free(ctx, ctx->scratch, nullptr);
  if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
  if (ctx->d_status) cudaFree(ctx->d_status);
  delete ctx;
  return COMET_OK;
}

extern "C" int comet_last_cuda_error(comet_handle_t handle) {
  return handle ? reinterpret_cast<Context *>(handle)->last_cuda_error : 0;
}

extern "C" int64_t comet_kernel_launches(comet_handle_t handle) {
  return handle ? reinterpret_cast<Context *>(handle)->launches : 0;
}

extern "C" const char *comet_status_string(comet_status_t s) {
  switch (s) {
    case COMET_OK: return "ok";
    case COMET_ERR_INVALID_ARG: return "invalid argument";
    case COMET_ERR_UNSUPPORTED_FORMAT: return "unsupported level-attribute combination or dtype";
    case COMET_ERR_COORD_OUT_OF_RANGE: return "coordinate out of range";
    case COMET_ERR_DUPLICATE_COORD: return "duplicate coordinate";
    case COMET_ERR_INDEX_OVERFLOW: return "size does not fit int32 indices";
    case COMET_ERR_ALLOC: return "device allocation failed";
    case COMET_ERR_CUDA: return "CUDA runtime error";
    case COMET_ERR_WORKSPACE: return "workspace too small";
    case COMET_ERR_MISALIGNED: return "misaligned pointer";
    case COMET_ERR_INVALID_TENSOR: return "tensor arrays violate the level invariants";
  }
  return "unknown status";
}
