// extern "C" entry points for the contractions: descriptor checks, dispatch on the level attributes
// (the role Table 1 of the paper plays for its loop generator), symbolic output construction.
#include "common.cuh"
#include "kernels.cuh"

#include <string.h>

#include <new>

using namespace comet;

namespace {

constexpr int64_t kIndexLimit = 2147483646;   // sizes must be < 2^31 - 1

bool is_fmt(const comet_sptensor_t *t, int order, int a0, int a1, int a2 = -1) {
  if (t->order != order) return false;
  if (t->attr[0] != a0 || t->attr[1] != a1) return false;
  return order < 3 || t->attr[2] == a2;
}

comet_status_t check_tensor(const comet_sptensor_t *t, int order) {
  if (!t) return COMET_ERR_INVALID_ARG;
  if (t->order != order) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (t->dtype != COMET_F64 && t->dtype != COMET_F32) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (t->nnz < 0) return COMET_ERR_INVALID_ARG;
  if (t->nnz > kIndexLimit) return COMET_ERR_INDEX_OVERFLOW;
  bool seen[COMET_MAX_ORDER] = {false, false, false, false};
  for (int l = 0; l < order; ++l) {
    const int m = t->mode_order[l];
    if (m < 0 || m >= order || seen[m]) return COMET_ERR_INVALID_ARG;
    seen[m] = true;
    if (t->dims[l] < 0) return COMET_ERR_INVALID_ARG;
    if (t->dims[l] > kIndexLimit) return COMET_ERR_INDEX_OVERFLOW;
    const int a = t->attr[l];
    if (a < COMET_D || a > COMET_S) return COMET_ERR_INVALID_ARG;
    if ((a == COMET_CU || a == COMET_CN) && !t->pos[l]) return COMET_ERR_INVALID_ARG;
    if (a != COMET_D && t->crd_len[l] > 0 && !t->crd[l]) return COMET_ERR_INVALID_ARG;
  }
  if (t->nnz > 0 && !t->val) return COMET_ERR_INVALID_ARG;
  return COMET_OK;
}

// Dense operands and outputs carry the tensor's value type and must be aligned to one element of it.
size_t elem_size(int dtype) { return dtype == COMET_F32 ? 4 : 8; }
bool misaligned(const void *p, int dtype) { return (reinterpret_cast<uintptr_t>(p) & (elem_size(dtype) - 1)) != 0; }

struct Owner {           // bookkeeping of a library-owned tensor: the blocks to release
  int count;
  void *blocks[2 * COMET_MAX_ORDER + 1];
};

void *owned_alloc(Context *ctx, Owner *o, size_t bytes, cudaStream_t stream) {
  void *p = ctx_alloc(ctx, bytes, stream);
  if (p) o->blocks[o->count++] = p;
  return p;
}

void release(Context *ctx, Owner *o, cudaStream_t stream) {
  if (!o) return;
  for (int b = 0; b < o->count; ++b) ctx_free(ctx, o->blocks[b], stream);
  delete o;
}

// pos of a CSR output from a compressed root level: out[i] = pos1[#stored root coordinates < i]
__global__ void expand_root_pos_kernel(const int32_t *__restrict__ crd0, const int32_t *__restrict__ pos1, int64_t S,
                                       int64_t rows, int32_t *__restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i > rows) return;
  int64_t lo = 0, hi = S;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)crd0[mid] < i) lo = mid + 1; else hi = mid;
  }
  out[i] = pos1[lo];
}

__global__ void set_word_kernel(int32_t *p, int32_t v) { *p = v; }
__global__ void set_two_words_kernel(int32_t *p, int32_t v0, int32_t v1) { p[0] = v0; p[1] = v1; }

// Coordinates of every fiber of a 3-level CSF structure: out0[f] = crd0[slice that holds f], out1[f] = crd1[f]
// (the slice is the last one whose first fiber is at or before f).
__global__ void fiber_coords_kernel(const int32_t *__restrict__ pos1, const int32_t *__restrict__ crd0,
                                    const int32_t *__restrict__ crd1, int64_t S, int64_t F, int32_t *__restrict__ out0,
                                    int32_t *__restrict__ out1) {
  const int64_t f = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= F) return;
  int64_t lo = 0, hi = S;
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(pos1 + mid) <= f) lo = mid; else hi = mid;
  }
  out0[f] = __ldg(crd0 + lo);
  out1[f] = __ldg(crd1 + f);
}

// CSR pos of a sorted COO matrix: pos[i] = number of entries whose root coordinate is below i
__global__ void coo_row_pos_kernel(const int32_t *__restrict__ crd0, int64_t n, int64_t rows, int32_t *__restrict__ pos) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i > rows) return;
  int64_t lo = 0, hi = n;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(crd0 + mid) < i) lo = mid + 1; else hi = mid;
  }
  pos[i] = (int32_t)lo;
}

// [CN,S] matrices go through the CSR kernels: the row structure the compressed level would store is
// rebuilt from the sorted root coordinates into scratch that sits in front of the kernels' own scratch.
comet_status_t coo_rows(Context *ctx, const comet_sptensor_t *A, int64_t rows, cudaStream_t s, int32_t **pos_out) {
  int32_t *pos = (int32_t *)ctx_alloc(ctx, (size_t)(rows + 1) * sizeof(int32_t), s);
  if (!pos) return COMET_ERR_ALLOC;
  coo_row_pos_kernel<<<(unsigned)ceil_div(rows + 1, 256), 256, 0, s>>>(A->crd[0], A->nnz, rows, pos);
  ctx->launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { ctx_free(ctx, pos, s); return cuda_fail(ctx, e); }
  *pos_out = pos;
  return COMET_OK;
}

}  // namespace

namespace comet {
void *owner_new() { Owner *o = new (std::nothrow) Owner(); if (o) o->count = 0; return o; }
void *owner_alloc(Context *ctx, void *owner, size_t bytes, cudaStream_t stream) {
  return owned_alloc(ctx, static_cast<Owner *>(owner), bytes, stream);
}
void owner_release(Context *ctx, void *owner, cudaStream_t stream) { release(ctx, static_cast<Owner *>(owner), stream); }
}  // namespace comet

extern "C" comet_status_t comet_sptensor_free(comet_handle_t handle, comet_sptensor_t *t, void *stream) {
  if (!handle || !t) return COMET_ERR_INVALID_ARG;
  Context *ctx = reinterpret_cast<Context *>(handle);
  if (t->owner) release(ctx, static_cast<Owner *>(t->owner), (cudaStream_t)stream);
  memset(t, 0, sizeof(*t));
  return COMET_OK;
}

// ------------------------------------------------------------------------------------------ SpMV / SpMM
extern "C" comet_status_t comet_spmv(comet_handle_t handle, const comet_sptensor_t *A, const void *x, void *y,
                                     void *stream) {
  if (!handle || !x || !y) return COMET_ERR_INVALID_ARG;
  if (is_ellpack(A)) {
    const comet_status_t es = ell_check(A);
    if (es != COMET_OK) return es;
    if (misaligned(x, A->dtype) || misaligned(y, A->dtype)) return COMET_ERR_MISALIGNED;
    return ell_spmv(reinterpret_cast<Context *>(handle), A, x, y, (cudaStream_t)stream);
  }
  comet_status_t st = check_tensor(A, 2);
  if (st != COMET_OK) return st;
  if (misaligned(x, A->dtype) || misaligned(y, A->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  const int64_t rows = A->dims[A->mode_order[0]];
  if (is_fmt(A, 2, COMET_D, COMET_CU))
    return seg_dot(ctx, A->dtype, A->pos[1] + 1, A->crd[1], A->val, rows, A->nnz, x, A->dims[A->mode_order[1]], y, nullptr,
                   rows, s);
  if (is_fmt(A, 2, COMET_CU, COMET_CU))
    return seg_dot(ctx, A->dtype, A->pos[1] + 1, A->crd[1], A->val, A->crd_len[0], A->nnz, x, A->dims[A->mode_order[1]], y,
                   A->crd[0], rows, s);
  if (is_fmt(A, 2, COMET_CN, COMET_S)) {
    int32_t *pos = nullptr;
    st = coo_rows(ctx, A, rows, s, &pos);
    if (st != COMET_OK) return st;
    st = seg_dot(ctx, A->dtype, pos + 1, A->crd[1], A->val, rows, A->nnz, x, A->dims[A->mode_order[1]], y, nullptr, rows, s);
    ctx_free(ctx, pos, s);          // stream-ordered allocators release after the queued work
    return st;
  }
  return COMET_ERR_UNSUPPORTED_FORMAT;
}

extern "C" comet_status_t comet_spmm(comet_handle_t handle, const comet_sptensor_t *A, const void *B, int64_t R,
                                     int64_t ldb, void *C, int64_t ldc, void *stream) {
  if (!handle || !B || !C || R < 1 || ldb < R || ldc < R) return COMET_ERR_INVALID_ARG;
  if (is_ellpack(A)) {
    const comet_status_t es = ell_check(A);
    if (es != COMET_OK) return es;
    if (misaligned(B, A->dtype) || misaligned(C, A->dtype)) return COMET_ERR_MISALIGNED;
    return ell_spmm(reinterpret_cast<Context *>(handle), A, B, ldb, R, C, ldc, (cudaStream_t)stream);
  }
  comet_status_t st = check_tensor(A, 2);
  if (st != COMET_OK) return st;
  if (misaligned(B, A->dtype) || misaligned(C, A->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  const int64_t rows = A->dims[A->mode_order[0]];
  if (is_fmt(A, 2, COMET_D, COMET_CU))
    return seg_gather(ctx, A->dtype, A->pos[1] + 1, A->crd[1], A->val, rows, A->nnz, B, ldb, R, C, ldc, nullptr, rows,
                      A->dims[A->mode_order[1]], s);
  if (is_fmt(A, 2, COMET_CU, COMET_CU)) {
    if (A->crd_len[0] == 0) return zero_rows(ctx, C, A->dtype, rows, R, ldc, s);
    return seg_gather(ctx, A->dtype, A->pos[1] + 1, A->crd[1], A->val, A->crd_len[0], A->nnz, B, ldb, R, C, ldc, A->crd[0],
                      rows, 0, s);
  }
  if (is_fmt(A, 2, COMET_CN, COMET_S)) {
    int32_t *pos = nullptr;
    st = coo_rows(ctx, A, rows, s, &pos);
    if (st != COMET_OK) return st;
    st = seg_gather(ctx, A->dtype, pos + 1, A->crd[1], A->val, rows, A->nnz, B, ldb, R, C, ldc, nullptr, rows,
                    A->dims[A->mode_order[1]], s);
    ctx_free(ctx, pos, s);
    return st;
  }
  return COMET_ERR_UNSUPPORTED_FORMAT;
}

// ------------------------------------------------------------------------------------------ TTV / TTM
// TTV / TTM take 3-order tensors in CSF or sorted COO and 4-order tensors in CSF ([CU,CU,CU,CU]); the
// contracted mode must be stored last. The kernels only see the last level (where each fiber of the level
// above ends, the leaf coordinates, the values), so the order only matters for the result's structure.
static comet_status_t check_last_mode(const comet_sptensor_t *X, int32_t mode) {
  if (!X) return COMET_ERR_INVALID_ARG;
  if (X->order != 3 && X->order != 4) return COMET_ERR_UNSUPPORTED_FORMAT;
  comet_status_t st = check_tensor(X, X->order);
  if (st != COMET_OK) return st;
  if (mode < 0 || mode >= X->order) return COMET_ERR_INVALID_ARG;
  bool csf = true;
  for (int l = 0; l < X->order; ++l) csf = csf && X->attr[l] == COMET_CU;
  const bool coo4 = X->order == 4 && X->attr[0] == COMET_CN && X->attr[1] == COMET_S && X->attr[2] == COMET_S && X->attr[3] == COMET_S;
  if (!csf && !coo4 && !is_fmt(X, 3, COMET_CN, COMET_S, COMET_S)) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (X->mode_order[X->order - 1] != mode) return COMET_ERR_UNSUPPORTED_FORMAT;   // re-pack with the contracted mode last
  return COMET_OK;
}

// ---- sorted COO [CN,S,S] as input of TTV / TTM -------------------------------------------------------
// The kernels want the fibers of the two leading modes: where each fiber ends in the entry list, and
// the (slice, fiber) coordinates of the result's structure. A sorted COO tensor has them implicitly: a
// fiber starts where (crd0, crd1) changes, a slice where crd0 changes. The symbolic call derives the two
// upper CSF levels from those head flags (flags -> two exclusive scans -> one read of the counts ->
// compaction); the leaf level is the COO tensor's own third coordinate array and values, untouched.
__global__ void coo_heads_kernel(const int32_t *__restrict__ c0, const int32_t *__restrict__ c1, int64_t n,
                                 uint32_t *__restrict__ fiber_head, uint32_t *__restrict__ slice_head) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n) return;
  const bool s = p == 0 || c0[p] != c0[p - 1];
  fiber_head[p] = (s || c1[p] != c1[p - 1]) ? 1u : 0u;
  slice_head[p] = s ? 1u : 0u;
}

// fiber_rank / slice_rank: exclusive scans of the head flags (rank of the fiber / slice an entry opens)
__global__ void coo_levels_kernel(const int32_t *__restrict__ c0, const int32_t *__restrict__ c1, int64_t n,
                                  const uint32_t *__restrict__ fiber_rank, const uint32_t *__restrict__ slice_rank,
                                  int64_t S, int64_t F, int32_t *__restrict__ pos0, int32_t *__restrict__ crd0,
                                  int32_t *__restrict__ pos1, int32_t *__restrict__ crd1, int32_t *__restrict__ pos2) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p == 0) { pos0[0] = 0; pos0[1] = (int32_t)S; pos1[S] = (int32_t)F; pos2[F] = (int32_t)n; }
  if (p >= n) return;
  const bool s = p == 0 || c0[p] != c0[p - 1];
  if (s || c1[p] != c1[p - 1]) {
    const uint32_t f = fiber_rank[p];
    crd1[f] = c1[p];
    pos2[f] = (int32_t)p;
    if (s) {
      const uint32_t sl = slice_rank[p];
      crd0[sl] = c0[p];
      pos1[sl] = (int32_t)f;
    }
  }
}

struct CooAsCsf {
  comet_sptensor_t t;       // CSF-shaped view: derived upper levels + the COO tensor's leaf arrays
  int32_t *pos2;            // fiber boundaries (F + 1); handed to the result, which the numeric call reads
  void *temps[6];           // the upper levels of the view: pos0, crd0, pos1, crd1 (and pos2, crd2 for order 4)
};

static void coo_view_release(Context *ctx, CooAsCsf *v, bool keep_pos2, cudaStream_t s) {
  for (int i = 0; i < 6; ++i) if (v->temps[i]) ctx_free(ctx, v->temps[i], s);
  if (!keep_pos2 && v->pos2) ctx_free(ctx, v->pos2, s);
}

// 4-order sorted COO [CN,S,S,S]: the three upper CSF levels come from the packing itself (the entries are sorted
// once more, which a symbolic call can afford); the leaf level stays the COO tensor's own last coordinate array
// and values, whose order is the packed order.
static comet_status_t coo4_as_csf(Context *ctx, const comet_sptensor_t *X, cudaStream_t s, CooAsCsf *v) {
  memset(v, 0, sizeof(*v));
  const int32_t *by_mode[4];
  for (int l = 0; l < 4; ++l) by_mode[X->mode_order[l]] = X->crd[l];
  const int32_t attr[4] = {COMET_CU, COMET_CU, COMET_CU, COMET_CU};
  comet_sptensor_t P;
  comet_status_t st = comet_pack(reinterpret_cast<comet_handle_t>(ctx), 4, X->dims, X->nnz, by_mode, X->val,
                                 (comet_dtype_t)X->dtype, X->mode_order, attr, (void *)s, &P);
  if (st != COMET_OK) return st;
  // take the level arrays over from the packed tensor; its leaf coordinates and values are not needed
  Owner *po = static_cast<Owner *>(P.owner);
  for (int b = 0; b < po->count; ++b)
    if (po->blocks[b] == (void *)P.crd[3] || po->blocks[b] == P.val) ctx_free(ctx, po->blocks[b], s);
  delete po;
  v->temps[0] = P.pos[0]; v->temps[1] = P.crd[0]; v->temps[2] = P.pos[1]; v->temps[3] = P.crd[1];
  v->temps[4] = P.pos[2]; v->temps[5] = P.crd[2];
  v->pos2 = P.pos[3];
  v->t = P;
  v->t.owner = nullptr;
  v->t.crd[3] = X->crd[3]; v->t.crd_len[3] = X->nnz;
  v->t.val = X->val; v->t.nnz = X->nnz;
  return COMET_OK;
}

static comet_status_t coo_as_csf(Context *ctx, const comet_sptensor_t *X, cudaStream_t s, CooAsCsf *v) {
  if (X->order == 4) return coo4_as_csf(ctx, X, s, v);
  memset(v, 0, sizeof(*v));
  const int64_t n = X->nnz;
  int64_t S = 0, F = 0;
  uint32_t *fiber_rank = nullptr, *slice_rank = nullptr, *tmp = nullptr;
  comet_status_t st = COMET_OK;
  if (n > 0) {
    fiber_rank = (uint32_t *)ctx_alloc(ctx, (size_t)n * 4, s);
    slice_rank = (uint32_t *)ctx_alloc(ctx, (size_t)n * 4, s);
    tmp = (uint32_t *)ctx_alloc(ctx, (size_t)scan_tmp_words(n) * 4, s);
    if (!fiber_rank || !slice_rank || !tmp) st = COMET_ERR_ALLOC;
    uint32_t *d_counts = reinterpret_cast<uint32_t *>(ctx->d_status) + 8;
    if (st == COMET_OK) {
      coo_heads_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, s>>>(X->crd[0], X->crd[1], n, fiber_rank, slice_rank);
      ctx->launches += 1;
      st = exclusive_scan(ctx, fiber_rank, fiber_rank, n, tmp, d_counts, s);
    }
    if (st == COMET_OK) st = exclusive_scan(ctx, slice_rank, slice_rank, n, tmp, d_counts + 1, s);
    if (st == COMET_OK) {
      cudaError_t e = cudaMemcpyAsync(ctx->h_pinned, d_counts, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
      if (e == cudaSuccess) e = cudaStreamSynchronize(s);
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
      F = reinterpret_cast<uint32_t *>(ctx->h_pinned)[0];
      S = reinterpret_cast<uint32_t *>(ctx->h_pinned)[1];
    }
  }
  int32_t *pos0 = nullptr, *crd0 = nullptr, *pos1 = nullptr, *crd1 = nullptr;
  if (st == COMET_OK) {
    v->temps[0] = pos0 = (int32_t *)ctx_alloc(ctx, 2 * 4, s);
    v->temps[1] = crd0 = (int32_t *)ctx_alloc(ctx, (size_t)(S > 0 ? S : 1) * 4, s);
    v->temps[2] = pos1 = (int32_t *)ctx_alloc(ctx, (size_t)(S + 1) * 4, s);
    v->temps[3] = crd1 = (int32_t *)ctx_alloc(ctx, (size_t)(F > 0 ? F : 1) * 4, s);
    v->pos2 = (int32_t *)ctx_alloc(ctx, (size_t)(F + 1) * 4, s);
    if (!pos0 || !crd0 || !pos1 || !crd1 || !v->pos2) st = COMET_ERR_ALLOC;
  }
  if (st == COMET_OK) {
    coo_levels_kernel<<<(unsigned)ceil_div(n > 0 ? n : 1, 256), 256, 0, s>>>(X->crd[0], X->crd[1], n, fiber_rank,
                                                                           slice_rank, S, F, pos0, crd0, pos1, crd1,
                                                                           v->pos2);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) st = cuda_fail(ctx, e);
  }
  if (fiber_rank) ctx_free(ctx, fiber_rank, s);
  if (slice_rank) ctx_free(ctx, slice_rank, s);
  if (tmp) ctx_free(ctx, tmp, s);
  if (st != COMET_OK) { coo_view_release(ctx, v, false, s); memset(v, 0, sizeof(*v)); return st; }
  comet_sptensor_t *t = &v->t;
  *t = *X;
  t->owner = nullptr;
  t->attr[0] = t->attr[1] = t->attr[2] = COMET_CU;
  t->pos[0] = pos0; t->pos_len[0] = 2; t->crd[0] = crd0; t->crd_len[0] = S;
  t->pos[1] = pos1; t->pos_len[1] = S + 1; t->crd[1] = crd1; t->crd_len[1] = F;
  t->pos[2] = v->pos2; t->pos_len[2] = F + 1;          // crd[2], crd_len[2], val, nnz stay the COO tensor's
  return COMET_OK;
}

// The fiber boundaries of a COO input travel with the result: level slot `slot` of Y (beyond Y's own
// levels) holds pos2, owned by Y. The numeric call finds them there.
static void stash_fiber_pos(comet_sptensor_t *Y, Owner *o, int slot, CooAsCsf *v) {
  o->blocks[o->count++] = v->pos2;
  if (slot < COMET_MAX_ORDER) {
    Y->pos[slot] = v->pos2;
    Y->pos_len[slot] = v->t.pos_len[v->t.order - 1];
  } else {                               // all four pos slots are Y's own (4-order TTM): the dense last level has no crd
    Y->crd[COMET_MAX_ORDER - 1] = v->pos2;
    Y->crd_len[COMET_MAX_ORDER - 1] = v->t.pos_len[v->t.order - 1];
  }
}
static const int32_t *stashed_fiber_pos(const comet_sptensor_t *Y, int slot, int64_t *len) {
  if (slot < COMET_MAX_ORDER) { *len = Y->pos_len[slot]; return Y->pos[slot]; }
  *len = Y->crd_len[COMET_MAX_ORDER - 1];
  return Y->crd[COMET_MAX_ORDER - 1];
}

// Copies X's upper levels (all but the last) into the same levels of Y, device to device.
static comet_status_t copy_upper_levels(Context *ctx, const comet_sptensor_t *X, comet_sptensor_t *Y, Owner *o,
                                        cudaStream_t s) {
  for (int l = 0; l < X->order - 1; ++l) {
    Y->pos_len[l] = X->pos_len[l];
    Y->crd_len[l] = X->crd_len[l];
    Y->pos[l] = (int32_t *)owned_alloc(ctx, o, (size_t)X->pos_len[l] * 4, s);
    Y->crd[l] = (int32_t *)owned_alloc(ctx, o, (size_t)X->crd_len[l] * 4, s);
    if (!Y->pos[l] || !Y->crd[l]) return COMET_ERR_ALLOC;
    if (X->pos_len[l])
      COMET_CUDA_TRY(ctx, cudaMemcpyAsync(Y->pos[l], X->pos[l], (size_t)X->pos_len[l] * 4, cudaMemcpyDeviceToDevice, s));
    if (X->crd_len[l])
      COMET_CUDA_TRY(ctx, cudaMemcpyAsync(Y->crd[l], X->crd[l], (size_t)X->crd_len[l] * 4, cudaMemcpyDeviceToDevice, s));
  }
  return COMET_OK;
}

extern "C" comet_status_t comet_ttv_symbolic(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                             const int32_t *h_out_attr, void *stream, comet_sptensor_t *Y) {
  if (!handle || !Y || !h_out_attr) return COMET_ERR_INVALID_ARG;
  comet_status_t st = check_last_mode(X, mode);
  if (st != COMET_OK) return st;
  const int out_order = X->order - 1;
  const bool csr = out_order == 2 && h_out_attr[0] == COMET_D && h_out_attr[1] == COMET_CU;
  bool dcsr = true;                       // every level compressed: DCSR (3-order input) or CSF (4-order input)
  for (int l = 0; l < out_order; ++l) dcsr = dcsr && h_out_attr[l] == COMET_CU;
  if (!csr && !dcsr) return COMET_ERR_UNSUPPORTED_FORMAT;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  memset(Y, 0, sizeof(*Y));
  CooAsCsf view;
  const bool from_coo = X->attr[0] == COMET_CN;
  if (from_coo) {
    st = coo_as_csf(ctx, X, s, &view);
    if (st != COMET_OK) return st;
    X = &view.t;
  }
  Owner *o = static_cast<Owner *>(owner_new());
  if (!o) { if (from_coo) coo_view_release(ctx, &view, false, s); return COMET_ERR_ALLOC; }
  const int64_t S = X->crd_len[0], F = X->crd_len[out_order - 1];
  const int64_t rows = X->dims[X->mode_order[0]];
  Y->order = out_order;
  Y->dtype = X->dtype;
  for (int l = 0; l < out_order; ++l) {       // the kept modes, renumbered in storage order
    Y->dims[l] = X->dims[X->mode_order[l]];
    Y->mode_order[l] = l;
    Y->attr[l] = h_out_attr[l];
  }
  Y->nnz = F;
  st = COMET_OK;
  if (dcsr) {
    st = copy_upper_levels(ctx, X, Y, o, s);
  } else {
    Y->pos_len[0] = 1; Y->crd_len[0] = 0; Y->pos_len[1] = rows + 1; Y->crd_len[1] = F;
    Y->pos[0] = (int32_t *)owned_alloc(ctx, o, 4, s);
    Y->pos[1] = (int32_t *)owned_alloc(ctx, o, (size_t)(rows + 1) * 4, s);
    Y->crd[1] = (int32_t *)owned_alloc(ctx, o, (size_t)F * 4, s);
    if (!Y->pos[0] || !Y->pos[1] || !Y->crd[1]) st = COMET_ERR_ALLOC;
    if (st == COMET_OK) {
      set_word_kernel<<<1, 1, 0, s>>>(Y->pos[0], (int32_t)rows);
      expand_root_pos_kernel<<<(unsigned)ceil_div(rows + 1, 256), 256, 0, s>>>(X->crd[0], X->pos[1], S, rows, Y->pos[1]);
      ctx->launches += 2;
      cudaError_t e = cudaGetLastError();
      if (e == cudaSuccess && F)
        e = cudaMemcpyAsync(Y->crd[1], X->crd[1], (size_t)F * 4, cudaMemcpyDeviceToDevice, s);
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
    }
  }
  if (st == COMET_OK) {
    Y->val = owned_alloc(ctx, o, (size_t)F * elem_size(X->dtype), s);
    if (!Y->val) st = COMET_ERR_ALLOC;
  }
  if (from_coo) {
    if (st == COMET_OK) stash_fiber_pos(Y, o, out_order, &view);
    coo_view_release(ctx, &view, st == COMET_OK, s);
  }
  if (st != COMET_OK) { release(ctx, o, s); memset(Y, 0, sizeof(*Y)); return st; }
  Y->owner = o;
  return COMET_OK;
}

extern "C" comet_status_t comet_ttv(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, const void *v,
                                    comet_sptensor_t *Y, void *stream) {
  if (!handle || !v || !Y) return COMET_ERR_INVALID_ARG;
  comet_status_t st = check_last_mode(X, mode);
  if (st != COMET_OK) return st;
  // fibers: X's level-2 pos for CSF; for COO the boundaries that the symbolic call left in Y's spare slot
  const bool from_coo = X->attr[0] == COMET_CN;
  const int last = X->order - 1;
  int64_t stashed = 0;
  const int32_t *fiber_pos = from_coo ? stashed_fiber_pos(Y, last, &stashed) : X->pos[last];
  const int64_t F = from_coo ? stashed - 1 : X->crd_len[last - 1];
  if (!fiber_pos || F < 0) return COMET_ERR_INVALID_ARG;
  if (Y->order != last || Y->nnz != F || (Y->nnz > 0 && !Y->val)) return COMET_ERR_INVALID_ARG;
  if (Y->dtype != X->dtype) return COMET_ERR_INVALID_ARG;
  if (misaligned(v, X->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  return seg_dot(ctx, X->dtype, fiber_pos + 1, X->crd[last], X->val, F, X->nnz, v, X->dims[mode], Y->val, nullptr, F,
                 (cudaStream_t)stream);
}

extern "C" comet_status_t comet_ttm_symbolic(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                             int64_t R, void *stream, comet_sptensor_t *Y) {
  return comet_ttm_symbolic_ex(handle, X, mode, R, nullptr, stream, Y);
}

extern "C" comet_status_t comet_ttm_symbolic_ex(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                                int64_t R, const int32_t *h_out_attr, void *stream,
                                                comet_sptensor_t *Y) {
  if (!handle || !Y || R < 1) return COMET_ERR_INVALID_ARG;
  if (R > kIndexLimit) return COMET_ERR_INDEX_OVERFLOW;
  comet_status_t st = check_last_mode(X, mode);
  if (st != COMET_OK) return st;
  // result format: compressed upper levels + dense last level (default), or, for 3-order inputs, the
  // mode-generic form [CN,S,D]: one coordinate pair per stored fiber + dense last level
  bool generic = false;
  if (h_out_attr) {
    bool semi = h_out_attr[X->order - 1] == COMET_D;
    for (int l = 0; l + 1 < X->order; ++l) semi = semi && h_out_attr[l] == COMET_CU;
    generic = X->order == 3 && h_out_attr[0] == COMET_CN && h_out_attr[1] == COMET_S && h_out_attr[2] == COMET_D;
    if (!semi && !generic) return COMET_ERR_UNSUPPORTED_FORMAT;
  }
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  memset(Y, 0, sizeof(*Y));
  CooAsCsf view;
  const bool from_coo = X->attr[0] == COMET_CN;
  if (from_coo) {
    st = coo_as_csf(ctx, X, s, &view);
    if (st != COMET_OK) return st;
    X = &view.t;
  }
  Owner *o = static_cast<Owner *>(owner_new());
  if (!o) { if (from_coo) coo_view_release(ctx, &view, false, s); return COMET_ERR_ALLOC; }
  const int last = X->order - 1;
  const int64_t F = X->crd_len[last - 1];
  Y->order = X->order;
  Y->dtype = X->dtype;
  for (int m = 0; m < X->order; ++m) { Y->dims[m] = X->dims[m]; Y->mode_order[m] = X->mode_order[m]; }
  Y->dims[mode] = R;                      // mode n is replaced by r in place
  for (int l = 0; l < last; ++l) Y->attr[l] = COMET_CU;
  Y->attr[last] = COMET_D;
  Y->nnz = F * R;
  if (generic) {
    Y->attr[0] = COMET_CN; Y->attr[1] = COMET_S;
    Y->pos_len[0] = 2; Y->crd_len[0] = F; Y->crd_len[1] = F;
    Y->pos[0] = (int32_t *)owned_alloc(ctx, o, 8, s);
    Y->crd[0] = (int32_t *)owned_alloc(ctx, o, (size_t)(F > 0 ? F : 1) * 4, s);
    Y->crd[1] = (int32_t *)owned_alloc(ctx, o, (size_t)(F > 0 ? F : 1) * 4, s);
    if (!Y->pos[0] || !Y->crd[0] || !Y->crd[1]) st = COMET_ERR_ALLOC;
    else {
      set_two_words_kernel<<<1, 1, 0, s>>>(Y->pos[0], 0, (int32_t)F);
      if (F > 0)
        fiber_coords_kernel<<<(unsigned)ceil_div(F, 256), 256, 0, s>>>(X->pos[1], X->crd[0], X->crd[1], X->crd_len[0], F,
                                                                      Y->crd[0], Y->crd[1]);
      ctx->launches += F > 0 ? 2 : 1;
      cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
    }
  } else {
    st = copy_upper_levels(ctx, X, Y, o, s);
  }
  if (st == COMET_OK) {
    Y->pos_len[last] = 1;
    Y->pos[last] = (int32_t *)owned_alloc(ctx, o, 4, s);
    Y->val = owned_alloc(ctx, o, (size_t)F * R * elem_size(X->dtype), s);
    if (!Y->pos[last] || !Y->val) st = COMET_ERR_ALLOC;
    else {
      set_word_kernel<<<1, 1, 0, s>>>(Y->pos[last], (int32_t)R);
      ctx->launches += 1;
      cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
    }
  }
  if (from_coo) {
    if (st == COMET_OK) stash_fiber_pos(Y, o, X->order, &view);
    coo_view_release(ctx, &view, st == COMET_OK, s);
  }
  if (st != COMET_OK) { release(ctx, o, s); memset(Y, 0, sizeof(*Y)); return st; }
  Y->owner = o;
  return COMET_OK;
}

extern "C" comet_status_t comet_ttm(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, const void *U,
                                    int64_t R, int64_t ldu, comet_sptensor_t *Y, void *stream) {
  if (!handle || !U || !Y || R < 1 || ldu < R) return COMET_ERR_INVALID_ARG;
  comet_status_t st = check_last_mode(X, mode);
  if (st != COMET_OK) return st;
  const bool from_coo = X->attr[0] == COMET_CN;
  const int last = X->order - 1;
  int64_t stashed = 0;
  const int32_t *fiber_pos = from_coo ? stashed_fiber_pos(Y, X->order, &stashed) : X->pos[last];
  const int64_t F = from_coo ? stashed - 1 : X->crd_len[last - 1];
  if (!fiber_pos || F < 0) return COMET_ERR_INVALID_ARG;
  if (Y->order != X->order || Y->nnz != F * R || (Y->nnz > 0 && !Y->val)) return COMET_ERR_INVALID_ARG;
  if (Y->dtype != X->dtype) return COMET_ERR_INVALID_ARG;
  if (misaligned(U, X->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  return seg_gather(ctx, X->dtype, fiber_pos + 1, X->crd[last], X->val, F, X->nnz, U, ldu, R, Y->val, R, nullptr, F, 0,
                    (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------ element-wise
extern "C" comet_status_t comet_elementwise_mul(comet_handle_t handle, const comet_sptensor_t *A, const void *B,
                                                const int64_t *h_strides, void *out_val, void *stream) {
  if (!handle || !A || !h_strides) return COMET_ERR_INVALID_ARG;
  comet_status_t st;
  int modes = A->order;
  if (is_ellpack(A)) {
    st = ell_check(A);
    modes = 2;
  } else {
    st = check_tensor(A, A->order);
  }
  if (st != COMET_OK) return st;
  if (A->nnz > 0 && (!B || !out_val)) return COMET_ERR_INVALID_ARG;
  if (misaligned(B, A->dtype) || misaligned(out_val, A->dtype)) return COMET_ERR_MISALIGNED;
  for (int m = 0; m < modes; ++m)
    if (h_strides[m] < 0) return COMET_ERR_INVALID_ARG;
  return elementwise_mul(reinterpret_cast<Context *>(handle), A, B, h_strides, out_val, (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------ MTTKRP
// 4-order tensors: COO [CN,S,S,S] or CSF [CU,CU,CU,CU], any output mode, atomic accumulation throughout.
static comet_status_t mttkrp_order4(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                    const void *const *h_factors, const int64_t *h_ld, int64_t R, void *out,
                                    int64_t ldo, void *stream) {
  comet_status_t st = check_tensor(X, 4);
  if (st != COMET_OK) return st;
  if (mode < 0 || mode > 3) return COMET_ERR_INVALID_ARG;
  bool coo = X->attr[0] == COMET_CN, csf = X->attr[0] == COMET_CU;
  for (int l = 1; l < 4; ++l) { coo = coo && X->attr[l] == COMET_S; csf = csf && X->attr[l] == COMET_CU; }
  if (!coo && !csf) return COMET_ERR_UNSUPPORTED_FORMAT;
  int level = 0;
  while (X->mode_order[level] != mode) ++level;
  int other[3], n = 0;                                 // the three other levels, in storage order
  for (int l = 0; l < 4; ++l) if (l != level) other[n++] = l;
  const void *F[3];
  int64_t ld[3];
  for (int q = 0; q < 3; ++q) {
    const int m = X->mode_order[other[q]];
    if (!h_factors[m] || h_ld[m] < R) return COMET_ERR_INVALID_ARG;
    if (misaligned(h_factors[m], X->dtype)) return COMET_ERR_MISALIGNED;
    if (h_ld[m] >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;
    F[q] = h_factors[m];
    ld[q] = h_ld[m];
  }
  if (misaligned(out, X->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  const int64_t rows = X->dims[mode];
  if (coo) {
    const int32_t *crd[4] = {X->crd[level], X->crd[other[0]], X->crd[other[1]], X->crd[other[2]]};
    return mttkrp_scatter4(ctx, X->dtype, -1, nullptr, nullptr, nullptr, crd, X->val, 0, 0, 0, X->nnz, rows, F[0], ld[0],
                           F[1], ld[1], F[2], ld[2], R, out, ldo, (cudaStream_t)stream);
  }
  const int32_t *crd[4] = {X->crd[0], X->crd[1], X->crd[2], X->crd[3]};
  return mttkrp_scatter4(ctx, X->dtype, level, X->pos[1], X->pos[2], X->pos[3], crd, X->val, X->crd_len[0], X->crd_len[1],
                         X->crd_len[2], X->nnz, rows, F[0], ld[0], F[1], ld[1], F[2], ld[2], R, out, ldo,
                         (cudaStream_t)stream);
}

extern "C" comet_status_t comet_mttkrp(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                       const void *const *h_factors, const int64_t *h_ld, int64_t R, void *out,
                                       int64_t ldo, void *stream) {
  if (!handle || !h_factors || !h_ld || !out || R < 1 || ldo < R) return COMET_ERR_INVALID_ARG;
  if (X && X->order == 4) return mttkrp_order4(handle, X, mode, h_factors, h_ld, R, out, ldo, stream);
  comet_status_t st = check_tensor(X, 3);
  if (st != COMET_OK) return st;
  if (mode < 0 || mode > 2) return COMET_ERR_INVALID_ARG;
  const bool coo = is_fmt(X, 3, COMET_CN, COMET_S, COMET_S), csf = is_fmt(X, 3, COMET_CU, COMET_CU, COMET_CU);
  if (!coo && !csf) return COMET_ERR_UNSUPPORTED_FORMAT;
  int level = 0;                                     // the level that stores the output mode
  while (X->mode_order[level] != mode) ++level;
  const int la = level == 0 ? 1 : 0, lb = level == 2 ? 1 : 2;      // the two other levels, in storage order
  const int m1 = X->mode_order[la], m2 = X->mode_order[lb];
  if (!h_factors[m1] || !h_factors[m2] || h_ld[m1] < R || h_ld[m2] < R) return COMET_ERR_INVALID_ARG;
  if (misaligned(h_factors[m1], X->dtype) || misaligned(h_factors[m2], X->dtype) || misaligned(out, X->dtype)) return COMET_ERR_MISALIGNED;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  const int64_t rows = X->dims[mode];
  const void *P = h_factors[m1], *Q = h_factors[m2];
  if (level > 0) {
    // output mode below the root: atomic accumulation on the tensor as stored
    if (h_ld[m1] >= (1ll << 28) || h_ld[m2] >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;
    if (coo)
      return mttkrp_scatter(ctx, X->dtype, 0, nullptr, X->crd[level], X->crd[la], nullptr, X->crd[lb], X->val, 0, 0,
                            X->nnz, rows, X->dims[m1], X->dims[m2], P, h_ld[m1], Q, h_ld[m2], R, out, ldo, s);
    if (level == 1) {                    // the tiled walker with atomic adds per fiber, where its shapes apply
      const comet_status_t ws = mttkrp_csf_level1(ctx, X->dtype, X->pos[1], X->crd[0], X->crd[1], X->pos[2], X->crd[2], X->val,
                                                  X->crd_len[0], X->crd_len[1], X->nnz, rows, P, h_ld[m1], Q, h_ld[m2], R, out,
                                                  ldo, s);
      if (ws != COMET_ERR_UNSUPPORTED_FORMAT) return ws;
    }
    return mttkrp_scatter(ctx, X->dtype, level, X->pos[1], X->crd[0], X->crd[1], X->pos[2], X->crd[2], X->val,
                          X->crd_len[0], X->crd_len[1], X->nnz, rows, X->dims[m1], X->dims[m2], P, h_ld[m1], Q, h_ld[m2], R,
                          out, ldo, s);
  }
  if (coo)
    return mttkrp_coo(ctx, X->dtype, X->crd[0], X->crd[1], X->crd[2], X->val, X->nnz, rows, P, h_ld[m1], Q, h_ld[m2], R, out,
                      ldo, s);
  if (csf)
    return mttkrp_csf(ctx, X->dtype, X->pos[1], X->crd[0], X->crd[1], X->pos[2], X->crd[2], X->val, X->crd_len[0],
                      X->crd_len[1], X->nnz, rows, P, h_ld[m1], Q, h_ld[m2], R, out, ldo, s);
  return COMET_ERR_UNSUPPORTED_FORMAT;
}
