// ELLPACK, which the paper's Tensor Storage Format section names among the formats that the four level
// attributes compose. The paper does not spell the composition out; the reading built here: a matrix with at most
// K entries per row is THREE levels [D, D, S] -- the rows (dense), K slots per row (dense; this level stores no
// tensor mode, the descriptor lists it as a third "mode" of extent K), and one singleton coordinate per slot, the
// entry's column. Row i's entries fill its first slots in ascending column order; unused slots hold column -1 and
// value 0. K is the longest row.
//
// Packing goes through the CSR packing (sort, row positions) and spreads the rows over the slots. The products
// (SpMV and SpMM definitions of the Sparse Tensor Operations subsection) walk the slots of a row and skip the
// padding; every output element is written by exactly one thread or warp, in a fixed order (deterministic).
#include "common.cuh"
#include "kernels.cuh"

namespace comet {

__global__ void ell_longest_row_kernel(const int32_t *__restrict__ pos, int64_t rows, int32_t *__restrict__ longest) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int32_t len = i < rows ? pos[i + 1] - pos[i] : 0;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) len = max(len, __shfl_xor_sync(0xffffffffu, len, d));
  if ((threadIdx.x & 31) == 0 && len > 0) atomicMax(longest, len);
}

template <class T>
__global__ void ell_fill_kernel(const int32_t *__restrict__ pos, const int32_t *__restrict__ crd, const T *__restrict__ val,
                                int64_t rows, int64_t K, int32_t *__restrict__ ell_crd, T *__restrict__ ell_val) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= rows * K) return;
  const int64_t i = p / K, k = p - i * K;
  const int64_t at = (int64_t)pos[i] + k;
  const bool stored = at < pos[i + 1];
  ell_crd[p] = stored ? crd[at] : -1;
  ell_val[p] = stored ? val[at] : (T)0;
}

// y_i: a warp per row; lane l adds the slots l, l + 32, ... in order, the lanes are then added as a fixed tree.
template <class T>
__global__ void __launch_bounds__(kBlockThreads) ell_spmv_kernel(const int32_t *__restrict__ crd, const T *__restrict__ val,
                                                                 int64_t rows, int64_t K, const T *__restrict__ x,
                                                                 T *__restrict__ y) {
  const int lane = threadIdx.x & 31;
  const int64_t i = ((int64_t)blockIdx.x * kBlockThreads + threadIdx.x) >> 5;
  if (i >= rows) return;
  double sum = 0.0;
  for (int64_t k = lane; k < K; k += 32) {
    const int32_t c = __ldcs(crd + i * K + k);
    if (c >= 0) sum = fma((double)__ldcs(val + i * K + k), (double)__ldg(x + c), sum);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
  if (lane == 0) y[i] = (T)sum;
}

// C_ir: a thread per (row, column); the threads of a row read the same slot (a broadcast) and consecutive
// columns of the gathered row of B.
template <class T>
__global__ void __launch_bounds__(kBlockThreads) ell_spmm_kernel(const int32_t *__restrict__ crd, const T *__restrict__ val,
                                                                 int64_t rows, int64_t K, const T *__restrict__ B, int64_t ldb,
                                                                 int64_t R, T *__restrict__ C, int64_t ldc) {
  const int64_t idx = (int64_t)blockIdx.x * kBlockThreads + threadIdx.x;
  if (idx >= rows * R) return;
  const int64_t i = idx / R, r = idx - i * R;
  double sum = 0.0;
  for (int64_t k = 0; k < K; ++k) {
    const int32_t c = __ldg(crd + i * K + k);
    if (c < 0) break;                                        // the padding is at the end of a row
    sum = fma((double)__ldg(val + i * K + k), (double)__ldg(B + (int64_t)c * ldb + r), sum);
  }
  C[i * ldc + r] = (T)sum;
}

// csr -> out (both descriptors are the caller's; out's arrays are allocated into `owner`). Synchronises once.
comet_status_t ell_from_csr(Context *ctx, const comet_sptensor_t *csr, void *owner, comet_sptensor_t *out, cudaStream_t s) {
  const int64_t rows = csr->dims[csr->mode_order[0]];
  int32_t *d_longest = ctx->d_status + 8;
  COMET_CUDA_TRY(ctx, cudaMemsetAsync(d_longest, 0, 4, s));
  if (rows > 0 && csr->nnz > 0) {
    ell_longest_row_kernel<<<(unsigned)ceil_div(rows, 256), 256, 0, s>>>(csr->pos[1], rows, d_longest);
    COMET_LAUNCH_CHECK(ctx);
  }
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, d_longest, 4, cudaMemcpyDeviceToHost, s));
  COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  const int64_t K = ctx->h_pinned[0];
  if (rows * K > 2147483647ll - 1024) return COMET_ERR_INDEX_OVERFLOW;
  const size_t elt = csr->dtype == COMET_F32 ? 4 : 8;

  memset(out, 0, sizeof(*out));
  out->order = 3;
  out->dtype = csr->dtype;
  out->dims[0] = csr->dims[0]; out->dims[1] = csr->dims[1]; out->dims[2] = K;
  out->mode_order[0] = csr->mode_order[0]; out->mode_order[1] = 2; out->mode_order[2] = csr->mode_order[1];
  out->attr[0] = COMET_D; out->attr[1] = COMET_D; out->attr[2] = COMET_S;
  out->nnz = rows * K;                                       // stored positions, padding included
  out->pos_len[0] = 1; out->pos_len[1] = 1; out->crd_len[2] = rows * K;
  out->pos[0] = (int32_t *)owner_alloc(ctx, owner, 4, s);
  out->pos[1] = (int32_t *)owner_alloc(ctx, owner, 4, s);
  out->crd[2] = (int32_t *)owner_alloc(ctx, owner, (size_t)(rows * K > 0 ? rows * K : 1) * 4, s);
  out->val = owner_alloc(ctx, owner, (size_t)(rows * K > 0 ? rows * K : 1) * elt, s);
  if (!out->pos[0] || !out->pos[1] || !out->crd[2] || !out->val) return COMET_ERR_ALLOC;
  const int32_t h_rows = (int32_t)rows, h_K = (int32_t)K;
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(out->pos[0], &h_rows, 4, cudaMemcpyHostToDevice, s));
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(out->pos[1], &h_K, 4, cudaMemcpyHostToDevice, s));
  if (rows * K > 0) {
    const unsigned blocks = (unsigned)ceil_div(rows * K, 256);
    if (csr->dtype == COMET_F32)
      ell_fill_kernel<float><<<blocks, 256, 0, s>>>(csr->pos[1], csr->crd[1], (const float *)csr->val, rows, K, out->crd[2], (float *)out->val);
    else
      ell_fill_kernel<double><<<blocks, 256, 0, s>>>(csr->pos[1], csr->crd[1], (const double *)csr->val, rows, K, out->crd[2], (double *)out->val);
    COMET_LAUNCH_CHECK(ctx);
  }
  COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));            // the two host words above must outlive their copies
  return COMET_OK;
}

bool is_ellpack(const comet_sptensor_t *A) {
  return A && A->order == 3 && A->attr[0] == COMET_D && A->attr[1] == COMET_D && A->attr[2] == COMET_S && A->mode_order[1] == 2 &&
         A->mode_order[0] + A->mode_order[2] == 1;
}

comet_status_t ell_check(const comet_sptensor_t *A) {
  if (A->dtype != COMET_F64 && A->dtype != COMET_F32) return COMET_ERR_UNSUPPORTED_FORMAT;
  const int64_t rows = A->dims[A->mode_order[0]], K = A->dims[2];
  if (rows < 0 || K < 0 || A->nnz != rows * K) return COMET_ERR_INVALID_ARG;
  if (A->nnz > 0 && (!A->crd[2] || !A->val)) return COMET_ERR_INVALID_ARG;
  return COMET_OK;
}

comet_status_t ell_spmv(Context *ctx, const comet_sptensor_t *A, const void *x, void *y, cudaStream_t s) {
  const int64_t rows = A->dims[A->mode_order[0]], K = A->dims[2];
  if (rows == 0) return COMET_OK;
  const unsigned blocks = (unsigned)ceil_div(rows * 32, kBlockThreads);
  if (A->dtype == COMET_F32)
    ell_spmv_kernel<float><<<blocks, kBlockThreads, 0, s>>>(A->crd[2], (const float *)A->val, rows, K, (const float *)x, (float *)y);
  else
    ell_spmv_kernel<double><<<blocks, kBlockThreads, 0, s>>>(A->crd[2], (const double *)A->val, rows, K, (const double *)x, (double *)y);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

comet_status_t ell_spmm(Context *ctx, const comet_sptensor_t *A, const void *B, int64_t ldb, int64_t R, void *C, int64_t ldc,
                        cudaStream_t s) {
  const int64_t rows = A->dims[A->mode_order[0]], K = A->dims[2];
  if (rows == 0 || R == 0) return COMET_OK;
  const unsigned blocks = (unsigned)ceil_div(rows * R, kBlockThreads);
  if (A->dtype == COMET_F32)
    ell_spmm_kernel<float><<<blocks, kBlockThreads, 0, s>>>(A->crd[2], (const float *)A->val, rows, K, (const float *)B, ldb, R, (float *)C, ldc);
  else
    ell_spmm_kernel<double><<<blocks, kBlockThreads, 0, s>>>(A->crd[2], (const double *)A->val, rows, K, (const double *)B, ldb, R, (double *)C, ldc);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

}  // namespace comet
