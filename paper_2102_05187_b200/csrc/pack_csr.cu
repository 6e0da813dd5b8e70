// COO -> CSR ([D,CU], 2 levels) without the full sort. The dense root level makes the row structure a
// histogram: count the rows, scan, drop every entry into its row in any order, then sort inside each row
// by column. The entries are distinct, so the sorted order is unique and the result is, bit for bit, what
// the generic radix path produces; rows of every length class are sorted by a kernel sized for them:
//   1..32 entries     a warp per row, bitonic network over registers (shuffles)
//   33..2048          a CTA per row, bitonic network in shared memory (padded to the next power of two)
//   2049..12288       a CTA per row, stable 8-bit LSD radix sort in shared memory over the column bits
//   longer            not handled here: the caller falls back to the generic path
// An entry travels as one 16-byte record (column, value), so the scattered write is one access per entry
// and no value is gathered afterwards. Equal columns inside a row are duplicates and are reported.
#include "common.cuh"
#include "kernels.cuh"

#include <string.h>

namespace comet {

constexpr int kCsrShortMax = 32;
constexpr int kCsrMidMax = 2048;
constexpr int kCsrLongMax = 12288;
constexpr int kCsrLongThreads = 1024;

enum { kCsrRange = 0, kCsrDuplicate = 1, kCsrTooLong = 2, kCsrMidCount = 4, kCsrLongCount = 5 };   // status words

template <class V> struct CsrRec;                 // 16 bytes: the column and the value of an entry
template <> struct __align__(16) CsrRec<double> { int32_t col; int32_t pad; double val; };
template <> struct __align__(16) CsrRec<float> { int32_t col; int32_t pad; float val; float pad2; };

__global__ void csr_count_kernel(const int32_t *__restrict__ row, const int32_t *__restrict__ col, int64_t n,
                                 int64_t rows, int64_t cols, uint32_t *__restrict__ cnt, int32_t *__restrict__ status) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n) return;
  const int32_t r = __ldcs(row + p), c = __ldcs(col + p);
  if (r < 0 || (int64_t)r >= rows || c < 0 || (int64_t)c >= cols) { atomicOr(status + kCsrRange, 1); return; }
  atomicAdd(cnt + r, 1u);
}

// Entries with a coordinate out of range were not counted and are skipped here too (the call then fails, but
// nothing may be indexed outside the arrays before the host learns of it).
template <class V>
__global__ void csr_scatter_kernel(const int32_t *__restrict__ row, const int32_t *__restrict__ col,
                                   const V *__restrict__ val, int64_t n, int64_t rows, int64_t cols,
                                   const uint32_t *__restrict__ pos, uint32_t *__restrict__ cursor,
                                   CsrRec<V> *__restrict__ rec) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n) return;
  const int32_t r = __ldcs(row + p), c = __ldcs(col + p);
  if (r < 0 || (int64_t)r >= rows || c < 0 || (int64_t)c >= cols) return;
  const uint32_t slot = pos[r] + atomicAdd(cursor + r, 1u);
  CsrRec<V> e{};
  e.col = c;
  e.val = __ldcs(val + p);
  rec[slot] = e;
}

// A warp per row: rows of up to 32 entries are sorted here; longer ones are put on the list of their class.
template <class V>
__global__ void __launch_bounds__(256) csr_sort_short_kernel(const CsrRec<V> *__restrict__ rec,
                                                             const uint32_t *__restrict__ pos, int64_t rows,
                                                             int32_t *__restrict__ crd, V *__restrict__ val,
                                                             uint32_t *__restrict__ list_mid, uint32_t *__restrict__ list_long,
                                                             int32_t *__restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (r >= rows) return;
  const uint32_t p0 = pos[r], len = pos[r + 1] - p0;
  if (len == 0) return;
  if (len > kCsrShortMax) {
    if (lane == 0) {
      if (len > kCsrLongMax) atomicOr(status + kCsrTooLong, 1);
      else if (len > kCsrMidMax) list_long[atomicAdd(reinterpret_cast<unsigned int *>(status + kCsrLongCount), 1u)] = (uint32_t)r;
      else list_mid[atomicAdd(reinterpret_cast<unsigned int *>(status + kCsrMidCount), 1u)] = (uint32_t)r;
    }
    return;
  }
  int32_t c = 0x7fffffff;
  V v = (V)0;
  if (lane < (int)len) { const CsrRec<V> e = rec[p0 + lane]; c = e.col; v = e.val; }
#pragma unroll
  for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      const int32_t oc = __shfl_xor_sync(0xffffffffu, c, j);
      const V ov = __shfl_xor_sync(0xffffffffu, v, j);
      const bool up = ((lane & k) == 0) == ((lane & j) == 0);     // this lane keeps the smaller of the pair
      if ((oc < c) == up && oc != c) { c = oc; v = ov; }
    }
  }
  const int32_t prev = __shfl_up_sync(0xffffffffu, c, 1);
  if (lane > 0 && lane < (int)len && prev == c) atomicOr(status + kCsrDuplicate, 1);
  if (lane < (int)len) { crd[p0 + lane] = c; val[p0 + lane] = v; }
}

// A CTA per row of 33..2048 entries (rows come from the list): bitonic network in shared memory.
template <class V>
__global__ void __launch_bounds__(256) csr_sort_mid_kernel(const CsrRec<V> *__restrict__ rec,
                                                           const uint32_t *__restrict__ pos,
                                                           const uint32_t *__restrict__ list, const int32_t *status,
                                                           int32_t *__restrict__ crd, V *__restrict__ val,
                                                           int32_t *status_out) {
  __shared__ int32_t s_col[kCsrMidMax];
  __shared__ V s_val[kCsrMidMax];
  const uint32_t count = (uint32_t)status[kCsrMidCount];
  for (uint32_t q = blockIdx.x; q < count; q += gridDim.x) {
    const uint32_t r = list[q];
    const uint32_t p0 = pos[r], len = pos[r + 1] - p0;
    uint32_t P = 64;
    while (P < len) P <<= 1;
    for (uint32_t t = threadIdx.x; t < P; t += blockDim.x) {
      if (t < len) { const CsrRec<V> e = rec[p0 + t]; s_col[t] = e.col; s_val[t] = e.val; }
      else { s_col[t] = 0x7fffffff; s_val[t] = (V)0; }
    }
    __syncthreads();
    for (uint32_t k = 2; k <= P; k <<= 1) {
      for (uint32_t j = k >> 1; j > 0; j >>= 1) {
        for (uint32_t t = threadIdx.x; t < P / 2; t += blockDim.x) {
          const uint32_t lo = 2 * t - (t & (j - 1));             // the pair (lo, lo + j)
          const uint32_t hi = lo + j;
          const bool asc = (lo & k) == 0;
          const int32_t a = s_col[lo], b = s_col[hi];
          if ((a > b) == asc && a != b) {
            s_col[lo] = b; s_col[hi] = a;
            const V va = s_val[lo]; s_val[lo] = s_val[hi]; s_val[hi] = va;
          }
        }
        __syncthreads();
      }
    }
    for (uint32_t t = threadIdx.x; t < len; t += blockDim.x) {
      const int32_t c = s_col[t];
      if (t > 0 && s_col[t - 1] == c) atomicOr(status_out + kCsrDuplicate, 1);
      crd[p0 + t] = c;
      val[p0 + t] = s_val[t];
    }
    __syncthreads();
  }
}

// A CTA per row of 2049..12288 entries: stable LSD radix sort of (column, position in the row) in shared memory,
// 8 bits per pass over the column bits; the values are then fetched through the sorted positions (the row is a
// contiguous, recently written stretch of the record array).
template <class V>
__global__ void __launch_bounds__(kCsrLongThreads, 1) csr_sort_long_kernel(
    const CsrRec<V> *__restrict__ rec, const uint32_t *__restrict__ pos, const uint32_t *__restrict__ list,
    const int32_t *status, int col_bits, int32_t *__restrict__ crd, V *__restrict__ val, int32_t *status_out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t *buf_a = reinterpret_cast<uint64_t *>(smem_raw);              // (column << 32) | position in the row
  uint64_t *buf_b = buf_a + kCsrLongMax;
  uint32_t *s_hist = reinterpret_cast<uint32_t *>(buf_b + kCsrLongMax);  // 256 digit counts, then running offsets
  uint32_t *s_wcnt = s_hist + 256;                                       // [32 warps][256] per-warp digit counts of a chunk
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t count = (uint32_t)status[kCsrLongCount];
  for (uint32_t q = blockIdx.x; q < count; q += gridDim.x) {
    const uint32_t r = list[q];
    const uint32_t p0 = pos[r], len = pos[r + 1] - p0;
    for (uint32_t t = tid; t < len; t += kCsrLongThreads)
      buf_a[t] = ((uint64_t)(uint32_t)rec[p0 + t].col << 32) | t;
    __syncthreads();
    uint64_t *in = buf_a, *out = buf_b;
    for (int shift = 0; shift < col_bits; shift += 8) {
      if (tid < 256) s_hist[tid] = 0;
      __syncthreads();
      for (uint32_t t = tid; t < len; t += kCsrLongThreads) atomicAdd(&s_hist[(uint32_t)(in[t] >> (32 + shift)) & 255u], 1u);
      __syncthreads();
      if (warp == 0) {                                                   // exclusive scan of the 256 counts by one warp
        uint32_t v[8], sum = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) { v[k] = s_hist[lane * 8 + k]; sum += v[k]; }
        uint32_t inc = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) { const uint32_t o = __shfl_up_sync(0xffffffffu, inc, off); if (lane >= off) inc += o; }
        uint32_t run = inc - sum;
#pragma unroll
        for (int k = 0; k < 8; ++k) { s_hist[lane * 8 + k] = run; run += v[k]; }
      }
      __syncthreads();
      // stable scatter, 1024 entries at a time in row order: rank inside the warp by matching digits, warps in order
      for (uint32_t base = 0; base < len; base += kCsrLongThreads) {
        for (int k = tid; k < 32 * 256; k += kCsrLongThreads) s_wcnt[k] = 0;
        __syncthreads();
        const uint32_t t = base + tid;
        const bool live = t < len;
        const uint64_t key = live ? in[t] : ~0ull;
        const uint32_t d = live ? (uint32_t)(key >> (32 + shift)) & 255u : 256u;   // 256: matches only other idle lanes
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
        if (live && rank == 0) s_wcnt[warp * 256 + d] = __popc(peers);
        __syncthreads();
        if (tid < 256) {                                                 // digit `tid`: offsets of the warps' groups
          uint32_t run = s_hist[tid];
          for (int w = 0; w < 32; ++w) { const uint32_t c = s_wcnt[w * 256 + tid]; s_wcnt[w * 256 + tid] = run; run += c; }
          s_hist[tid] = run;                                             // the next chunk continues behind this one
        }
        __syncthreads();
        if (live) out[s_wcnt[warp * 256 + d] + rank] = key;
        __syncthreads();
      }
      uint64_t *sw = in; in = out; out = sw;
    }
    for (uint32_t t = tid; t < len; t += kCsrLongThreads) {
      const uint64_t key = in[t];
      const int32_t c = (int32_t)(key >> 32);
      if (t > 0 && (int32_t)(in[t - 1] >> 32) == c) atomicOr(status_out + kCsrDuplicate, 1);
      crd[p0 + t] = c;
      val[p0 + t] = rec[p0 + (uint32_t)key].val;
    }
    __syncthreads();
  }
}

template <class V>
static comet_status_t pack_csr_typed(Context *ctx, const int32_t *row, const int32_t *col, const V *val, int64_t n,
                                     int64_t rows, int64_t cols, int32_t *pos_out, int32_t *crd_out, V *val_out,
                                     int *fallback, cudaStream_t s) {
  *fallback = 0;
  uint32_t *pos = reinterpret_cast<uint32_t *>(pos_out);
  void *blocks[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  uint32_t *cursor = (uint32_t *)(blocks[0] = ctx_alloc(ctx, (size_t)(rows + 1) * 4, s));
  CsrRec<V> *rec = (CsrRec<V> *)(blocks[1] = ctx_alloc(ctx, (size_t)(n > 0 ? n : 1) * sizeof(CsrRec<V>), s));
  uint32_t *scan_tmp = (uint32_t *)(blocks[2] = ctx_alloc(ctx, (size_t)scan_tmp_words(rows + 1) * 4, s));
  uint32_t *list_mid = (uint32_t *)(blocks[3] = ctx_alloc(ctx, (size_t)(n / (kCsrShortMax + 1) + 1) * 4, s));
  uint32_t *list_long = (uint32_t *)(blocks[4] = ctx_alloc(ctx, (size_t)(n / (kCsrMidMax + 1) + 1) * 4, s));
  comet_status_t st = COMET_OK;
  for (int b = 0; b < 5; ++b) if (!blocks[b]) st = COMET_ERR_ALLOC;
  auto done = [&](comet_status_t r) { for (int b = 0; b < 5; ++b) if (blocks[b]) ctx_free(ctx, blocks[b], s); return r; };
  if (st != COMET_OK) return done(st);

  cudaError_t e = cudaMemsetAsync(ctx->d_status, 0, 16 * sizeof(int32_t), s);
  if (e == cudaSuccess) e = cudaMemsetAsync(pos, 0, (size_t)(rows + 1) * 4, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(cursor, 0, (size_t)(rows + 1) * 4, s);
  if (e != cudaSuccess) return done(cuda_fail(ctx, e));
  const unsigned gn = (unsigned)ceil_div(n > 0 ? n : 1, 256);
  if (n > 0) {
    csr_count_kernel<<<gn, 256, 0, s>>>(row, col, n, rows, cols, pos, ctx->d_status);
    ctx->launches += 1;
  }
  st = exclusive_scan(ctx, pos, pos, rows + 1, scan_tmp, nullptr, s);
  if (st != COMET_OK) return done(st);
  if (n > 0) {
    csr_scatter_kernel<V><<<gn, 256, 0, s>>>(row, col, val, n, rows, cols, pos, cursor, rec);
    csr_sort_short_kernel<V><<<(unsigned)ceil_div(rows * 32, 256), 256, 0, s>>>(rec, pos, rows, crd_out, val_out, list_mid,
                                                                              list_long, ctx->d_status);
    csr_sort_mid_kernel<V><<<kSmCount * 8, 256, 0, s>>>(rec, pos, list_mid, ctx->d_status, crd_out, val_out, ctx->d_status);
    int col_bits = 1;
    while (col_bits < 31 && (1ll << col_bits) < cols) ++col_bits;
    const size_t smem = (size_t)kCsrLongMax * 16 + 256 * 4 + 32 * 256 * 4;
    auto kernel = csr_sort_long_kernel<V>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return done(cuda_fail(ctx, e));
    kernel<<<kSmCount, kCsrLongThreads, smem, s>>>(rec, pos, list_long, ctx->d_status, col_bits, crd_out, val_out, ctx->d_status);
    ctx->launches += 4;
    e = cudaGetLastError();
    if (e != cudaSuccess) return done(cuda_fail(ctx, e));
  }
  e = cudaMemcpyAsync(ctx->h_pinned, ctx->d_status, 16 * sizeof(int32_t), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return done(cuda_fail(ctx, e));
  if (ctx->h_pinned[kCsrRange]) return done(COMET_ERR_COORD_OUT_OF_RANGE);
  if (ctx->h_pinned[kCsrTooLong]) { *fallback = 1; return done(COMET_OK); }
  if (ctx->h_pinned[kCsrDuplicate]) return done(COMET_ERR_DUPLICATE_COORD);
  return done(COMET_OK);
}

// Fills pos_out (rows + 1), crd_out (n), val_out (n). *fallback = 1 (with COMET_OK) when a row is longer than this
// path sorts: the caller then runs the generic path, which overwrites everything written here.
comet_status_t pack_csr_fast(Context *ctx, int dtype, const int32_t *row, const int32_t *col, const void *val, int64_t n,
                             int64_t rows, int64_t cols, int32_t *pos_out, int32_t *crd_out, void *val_out,
                             int *fallback, cudaStream_t s) {
  if (dtype == COMET_F32)
    return pack_csr_typed<float>(ctx, row, col, (const float *)val, n, rows, cols, pos_out, crd_out, (float *)val_out,
                                 fallback, s);
  return pack_csr_typed<double>(ctx, row, col, (const double *)val, n, rows, cols, pos_out, crd_out, (double *)val_out,
                                fallback, s);
}

}  // namespace comet
