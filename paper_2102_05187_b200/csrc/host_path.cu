// comet_spmm_from_host: the whole SpMM path (the conversion of the COO input, then the SpMM definition of the
// Sparse Tensor Operations subsection) from HOST buffers in one call, with the transfers overlapped.
//
// The bus is the bound of this path (config 2: 852 MB in, 537 MB out, 2.7 ms of kernels), and it carries both
// directions at once. C_{:, c} depends on B_{:, c} only, so B and C are cut into column chunks of 256 bytes per
// row (strided copies of that width run at the bus's full rate; 64-byte ones at half of it):
//
//   stream of the call   COO in | pack ............ | SpMM chunk 0 | SpMM chunk 1 | ...
//   inbound stream              | B chunk 0 | B chunk 1 | ...
//   outbound stream                          | C chunk 0 ........ | C chunk 1 ........ | ...
//
// so that the result starts to leave while the rest of B is still arriving. On the device a chunk of B and of C
// is a packed matrix of its own (leading dimension = its width). Host buffers should be pinned (page-locked);
// with pageable memory the copies are staged by the driver and nothing overlaps.
#include "common.cuh"
#include "kernels.cuh"

#include <stdlib.h>
#include <string.h>

namespace comet {

static comet_status_t host_streams(Context *ctx) {
  if (ctx->has_copy_streams) return COMET_OK;
  COMET_CUDA_TRY(ctx, cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking));
  COMET_CUDA_TRY(ctx, cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking));
  for (int i = 0; i < kCopyEvents; ++i) COMET_CUDA_TRY(ctx, cudaEventCreateWithFlags(&ctx->copy_event[i], cudaEventDisableTiming));
  ctx->has_copy_streams = true;
  return COMET_OK;
}

void host_streams_destroy(Context *ctx) {
  if (!ctx->has_copy_streams) return;
  cudaStreamDestroy(ctx->copy_in);
  cudaStreamDestroy(ctx->copy_out);
  for (int i = 0; i < kCopyEvents; ++i) cudaEventDestroy(ctx->copy_event[i]);
  ctx->has_copy_streams = false;
}

}  // namespace comet

using comet::Context;

extern "C" comet_status_t comet_spmm_from_host(comet_handle_t handle, const int64_t *h_dims, int64_t nnz,
                                               const int32_t *h_row, const int32_t *h_col, const void *h_val,
                                               comet_dtype_t dtype, const void *h_B, int64_t ldb, int64_t R, void *h_C,
                                               int64_t ldc, void *stream) {
  if (!handle || !h_dims || nnz < 0 || R < 1 || ldb < R || ldc < R) return COMET_ERR_INVALID_ARG;
  if (dtype != COMET_F64 && dtype != COMET_F32) return COMET_ERR_UNSUPPORTED_FORMAT;
  const int64_t rows = h_dims[0], cols = h_dims[1];
  if (rows < 0 || cols < 0) return COMET_ERR_INVALID_ARG;
  if (nnz > 0 && (!h_row || !h_col || !h_val)) return COMET_ERR_INVALID_ARG;
  if ((cols > 0 && !h_B) || (rows > 0 && !h_C)) return COMET_ERR_INVALID_ARG;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  const size_t elt = dtype == COMET_F32 ? 4 : 8;
  comet_status_t st = comet::host_streams(ctx);
  if (st != COMET_OK) return st;

  // column chunks of `chunk_bytes` per row (COMET_HOST_CHUNK_BYTES; 0 = one chunk), at most kCopyChunks of them
  int64_t chunk_bytes = 256;
  if (const char *e = getenv("COMET_HOST_CHUNK_BYTES")) chunk_bytes = atoll(e);
  int64_t width = chunk_bytes > 0 ? chunk_bytes / (int64_t)elt : R;
  if (width < 1 || width > R) width = R;
  if (comet::ceil_div(R, width) > comet::kCopyChunks) width = comet::ceil_div(R, (int64_t)comet::kCopyChunks);
  const int chunks = (int)comet::ceil_div(R, width);

  int32_t *d_row = nullptr, *d_col = nullptr;
  void *d_val = nullptr, *d_B = nullptr, *d_C = nullptr;
  comet_sptensor_t A;
  memset(&A, 0, sizeof(A));
  bool packed = false;
  auto release = [&]() {
    if (packed) comet_sptensor_free(handle, &A, stream);
    comet::ctx_free(ctx, d_row, s); comet::ctx_free(ctx, d_col, s); comet::ctx_free(ctx, d_val, s);
    comet::ctx_free(ctx, d_B, s); comet::ctx_free(ctx, d_C, s);
  };
  auto fail = [&](comet_status_t code) {
    // nothing of this call may still be running on the copy streams when the buffers go back
    cudaStreamSynchronize(ctx->copy_in); cudaStreamSynchronize(ctx->copy_out); cudaStreamSynchronize(s);
    release();
    return code;
  };
#define HOST_TRY(expr)                                              \
  do {                                                              \
    cudaError_t e__ = (expr);                                       \
    if (e__ != cudaSuccess) return fail(comet::cuda_fail(ctx, e__)); \
  } while (0)

  d_row = (int32_t *)comet::ctx_alloc(ctx, (size_t)(nnz > 0 ? nnz : 1) * 4, s);
  d_col = (int32_t *)comet::ctx_alloc(ctx, (size_t)(nnz > 0 ? nnz : 1) * 4, s);
  d_val = comet::ctx_alloc(ctx, (size_t)(nnz > 0 ? nnz : 1) * elt, s);
  d_B = comet::ctx_alloc(ctx, (size_t)(cols * R > 0 ? cols * R : 1) * elt, s);
  d_C = comet::ctx_alloc(ctx, (size_t)(rows * R > 0 ? rows * R : 1) * elt, s);
  if (!d_row || !d_col || !d_val || !d_B || !d_C) return fail(COMET_ERR_ALLOC);

  cudaEvent_t *ev = ctx->copy_event;                 // [0] COO in; [1 + c] chunk c of B in; [1 + chunks + c] chunk c of C ready
  if (nnz > 0) {
    HOST_TRY(cudaMemcpyAsync(d_row, h_row, (size_t)nnz * 4, cudaMemcpyHostToDevice, s));
    HOST_TRY(cudaMemcpyAsync(d_col, h_col, (size_t)nnz * 4, cudaMemcpyHostToDevice, s));
    HOST_TRY(cudaMemcpyAsync(d_val, h_val, (size_t)nnz * elt, cudaMemcpyHostToDevice, s));
  }
  HOST_TRY(cudaEventRecord(ev[0], s));
  HOST_TRY(cudaStreamWaitEvent(ctx->copy_in, ev[0], 0));       // the bus serves the COO entries first: the packing needs them
  for (int c = 0; c < chunks; ++c) {
    const int64_t c0 = (int64_t)c * width, w = c0 + width <= R ? width : R - c0;
    if (cols > 0)
      HOST_TRY(cudaMemcpy2DAsync((char *)d_B + (size_t)cols * c0 * elt, (size_t)w * elt, (const char *)h_B + (size_t)c0 * elt,
                                 (size_t)ldb * elt, (size_t)w * elt, (size_t)cols, cudaMemcpyHostToDevice, ctx->copy_in));
    HOST_TRY(cudaEventRecord(ev[1 + c], ctx->copy_in));
  }

  const int32_t mode_order[2] = {0, 1}, attr[2] = {COMET_D, COMET_CU};
  const int32_t *coo[2] = {d_row, d_col};
  st = comet_pack(handle, 2, h_dims, nnz, coo, d_val, dtype, mode_order, attr, stream, &A);
  if (st != COMET_OK) return fail(st);
  packed = true;

  for (int c = 0; c < chunks; ++c) {
    const int64_t c0 = (int64_t)c * width, w = c0 + width <= R ? width : R - c0;
    HOST_TRY(cudaStreamWaitEvent(s, ev[1 + c], 0));
    st = comet_spmm(handle, &A, (const char *)d_B + (size_t)cols * c0 * elt, w, w, (char *)d_C + (size_t)rows * c0 * elt, w, stream);
    if (st != COMET_OK) return fail(st);
    HOST_TRY(cudaEventRecord(ev[1 + chunks + c], s));
    HOST_TRY(cudaStreamWaitEvent(ctx->copy_out, ev[1 + chunks + c], 0));
    if (rows > 0)
      HOST_TRY(cudaMemcpy2DAsync((char *)h_C + (size_t)c0 * elt, (size_t)ldc * elt, (const char *)d_C + (size_t)rows * c0 * elt,
                                 (size_t)w * elt, (size_t)w * elt, (size_t)rows, cudaMemcpyDeviceToHost, ctx->copy_out));
  }
  HOST_TRY(cudaEventRecord(ev[1 + 2 * chunks], ctx->copy_out));
  HOST_TRY(cudaStreamWaitEvent(s, ev[1 + 2 * chunks], 0));
  HOST_TRY(cudaStreamSynchronize(s));                          // the result has landed in h_C
#undef HOST_TRY
  release();
  return COMET_OK;
}
