// comet_reorder: the reordering pre-pass (Data Reordering section). The paper sorts one dimension per
// iteration lexicographically by the coordinates of its entries in the other dimensions, and all dimensions
// in turn, so that the entries gather around the diagonal; it gives no further detail. The reading built
// here keeps the FIRST element of every index's sorted entry list:
//
//   one step for mode m:  key(x) = the smallest tuple (current numbers of the other modes' coordinates, in
//                         increasing mode order) over the entries whose mode-m index is x, +infinity when x
//                         has no entry; the indices of mode m are re-numbered in ascending key order, ties
//                         (and empty indices) in the order of their current numbers
//   one iteration:        a step for mode 0, then mode 1, ...
//
// Per step: one pass over the entries (a 64-bit atomic minimum per entry into the key of its index), one
// stable radix sort of dims[m] (key, current number) pairs, one pass that composes the new numbering with
// the old one. Integer work throughout; the result is bit-exact against the CPU oracle.
#include "common.cuh"
#include "kernels.cuh"

namespace comet {

struct ReorderModes {
  const int32_t *crd[COMET_MAX_ORDER];   // original coordinates, one array per mode
  const int32_t *label[COMET_MAX_ORDER]; // current number of every original index
  int64_t dim[COMET_MAX_ORDER];
  int order;
};

__global__ void iota_kernel(int32_t *p, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = (int32_t)i;
}

// `inf` = one more than the largest tuple: the key of an index without entries
__global__ void reorder_init_keys_kernel(uint64_t *keys, uint32_t *ids, int64_t n, uint64_t inf) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) { keys[i] = inf; ids[i] = (uint32_t)i; }
}

// keys[current number of the entry's mode-m index] = min(that, tuple of the other modes' current numbers)
template <int ORDER>
__global__ void reorder_min_keys_kernel(ReorderModes r, int m, int64_t nnz, unsigned long long *__restrict__ keys) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= nnz) return;
  unsigned long long tup = 0;
#pragma unroll
  for (int o = 0; o < ORDER; ++o)
    if (o != m) tup = tup * (unsigned long long)r.dim[o] + (unsigned long long)__ldg(r.label[o] + __ldg(r.crd[o] + e));
  atomicMin(keys + __ldg(r.label[m] + __ldg(r.crd[m] + e)), tup);
}

// sorted_ids[i] = the current number that becomes i; renumber[current] = i
__global__ void reorder_rank_kernel(const uint32_t *__restrict__ sorted_ids, int64_t n, int32_t *__restrict__ renumber) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) renumber[sorted_ids[i]] = (int32_t)i;
}

__global__ void reorder_compose_kernel(int32_t *__restrict__ label, int64_t n, const int32_t *__restrict__ renumber) {
  const int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (x < n) label[x] = renumber[label[x]];
}

__global__ void reorder_range_kernel(const int32_t *__restrict__ crd, int64_t nnz, int64_t dim, int32_t *status) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e < nnz) {
    const int32_t c = crd[e];
    if (c < 0 || (int64_t)c >= dim) atomicOr(status, 1);
  }
}

}  // namespace comet

using namespace comet;

extern "C" comet_status_t comet_reorder(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                                        const int32_t *const *h_coo_crd, int32_t iterations,
                                        int32_t *const *h_new_label, void *stream) {
  if (!handle || !h_dims || !h_coo_crd || !h_new_label || nnz < 0 || iterations < 0) return COMET_ERR_INVALID_ARG;
  if (order < 2 || order > COMET_MAX_ORDER) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (nnz > 2147483647ll - 1024) return COMET_ERR_INDEX_OVERFLOW;
  int64_t max_dim = 0;
  for (int m = 0; m < order; ++m) {
    if (h_dims[m] < 0 || !h_new_label[m] || (nnz > 0 && !h_coo_crd[m])) return COMET_ERR_INVALID_ARG;
    if (h_dims[m] > 2147483646ll) return COMET_ERR_INDEX_OVERFLOW;
    if (h_dims[m] > max_dim) max_dim = h_dims[m];
  }
  // span[m] = number of distinct tuples of the other modes' numbers = the key that stands for +infinity
  uint64_t span[COMET_MAX_ORDER];
  for (int m = 0; m < order; ++m) {
    long double prod = 1.0L;
    for (int o = 0; o < order; ++o) if (o != m) prod *= (long double)(h_dims[o] > 0 ? h_dims[o] : 1);
    if (prod >= 9.2e18L) return COMET_ERR_INDEX_OVERFLOW;
    span[m] = 1;
    for (int o = 0; o < order; ++o) if (o != m) span[m] *= (uint64_t)(h_dims[o] > 0 ? h_dims[o] : 1);
  }
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;

  ReorderModes r{};
  r.order = order;
  for (int m = 0; m < order; ++m) {
    r.crd[m] = h_coo_crd[m];
    r.label[m] = h_new_label[m];
    r.dim[m] = h_dims[m];
    if (h_dims[m] > 0) {
      iota_kernel<<<(unsigned)ceil_div(h_dims[m], 256), 256, 0, s>>>(h_new_label[m], h_dims[m]);
      COMET_LAUNCH_CHECK(ctx);
    }
  }
  if (nnz == 0 || iterations == 0) return COMET_OK;

  // coordinates are checked once (a bad one would index outside the label arrays)
  COMET_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, 16 * sizeof(int32_t), s));
  for (int m = 0; m < order; ++m) {
    reorder_range_kernel<<<(unsigned)ceil_div(nnz, 256), 256, 0, s>>>(h_coo_crd[m], nnz, h_dims[m], ctx->d_status);
    COMET_LAUNCH_CHECK(ctx);
  }
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  if (ctx->h_pinned[0]) return COMET_ERR_COORD_OUT_OF_RANGE;

  const int64_t table_words = radix_sort_table_words(max_dim);
  void *blocks[7] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  uint64_t *ka = (uint64_t *)(blocks[0] = ctx_alloc(ctx, (size_t)(max_dim + 1) * 8, s));
  uint64_t *kb = (uint64_t *)(blocks[1] = ctx_alloc(ctx, (size_t)(max_dim + 1) * 8, s));
  uint32_t *pa = (uint32_t *)(blocks[2] = ctx_alloc(ctx, (size_t)(max_dim + 1) * 4, s));
  uint32_t *pb = (uint32_t *)(blocks[3] = ctx_alloc(ctx, (size_t)(max_dim + 1) * 4, s));
  uint32_t *table = (uint32_t *)(blocks[4] = ctx_alloc(ctx, (size_t)table_words * 4, s));
  uint32_t *scan_tmp = (uint32_t *)(blocks[5] = ctx_alloc(ctx, (size_t)scan_tmp_words(table_words) * 4, s));
  int32_t *renumber = (int32_t *)(blocks[6] = ctx_alloc(ctx, (size_t)(max_dim + 1) * 4, s));
  comet_status_t st = COMET_OK;
  for (int b = 0; b < 7; ++b) if (!blocks[b]) st = COMET_ERR_ALLOC;

  for (int it = 0; it < iterations && st == COMET_OK; ++it) {
    for (int m = 0; m < order && st == COMET_OK; ++m) {
      const int64_t d = h_dims[m];
      if (d == 0) continue;
      int bits = 1;                                    // key bits in use: values 0 .. span[m]
      while (bits < 64 && (span[m] >> bits) != 0) ++bits;
      reorder_init_keys_kernel<<<(unsigned)ceil_div(d, 256), 256, 0, s>>>(ka, pa, d, span[m]);
      if (order == 2) reorder_min_keys_kernel<2><<<(unsigned)ceil_div(nnz, 256), 256, 0, s>>>(r, m, nnz, (unsigned long long *)ka);
      else if (order == 3) reorder_min_keys_kernel<3><<<(unsigned)ceil_div(nnz, 256), 256, 0, s>>>(r, m, nnz, (unsigned long long *)ka);
      else reorder_min_keys_kernel<4><<<(unsigned)ceil_div(nnz, 256), 256, 0, s>>>(r, m, nnz, (unsigned long long *)ka);
      ctx->launches += 2;
      cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) { st = cuda_fail(ctx, e); break; }
      st = radix_sort_pairs(ctx, ka, kb, pa, pb, d, bits, table, scan_tmp, s);
      if (st != COMET_OK) break;
      reorder_rank_kernel<<<(unsigned)ceil_div(d, 256), 256, 0, s>>>(pa, d, renumber);
      reorder_compose_kernel<<<(unsigned)ceil_div(d, 256), 256, 0, s>>>(h_new_label[m], d, renumber);
      ctx->launches += 2;
      e = cudaGetLastError();
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
    }
  }
  for (int b = 0; b < 7; ++b) if (blocks[b]) ctx_free(ctx, blocks[b], s);
  return st;
}
