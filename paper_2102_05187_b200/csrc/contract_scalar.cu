// Segment dot products with a dense vector operand: SpMV and TTV (the SpMV / SpTTV definitions of the
// paper's Sparse Tensor Operations subsection): y[s] = sum over leaf entries p of segment s of
// val[p] * x[crd[p]], where a segment is a CSR row (SpMV) or a CSF fiber (TTV).
//
// These are pure streaming kernels (12 bytes per leaf entry, the vector stays in L1/L2), so the leaf
// arrays must be read with fully coalesced loads whatever the segment lengths are. Each CTA takes a
// fixed number of items of the merge list (segment-end markers interleaved with leaf positions):
//   1. two threads locate the tile on the merge path (binary search over the segment ends);
//   2. the CTA loads its leaf entries coalesced, multiplies by the gathered vector element and parks
//      the products in shared memory, with the tile's segment ends beside them;
//   3. every thread walks IPT consecutive merge items out of shared memory, writes the segments that
//      end inside its span, and a segmented block scan (keyed by segment) supplies the part of its
//      first segment that earlier threads summed;
//   4. the partial sum of the segment the tile stops in goes to a carry slot that a second small
//      kernel adds in tile order. No atomics: results are bit-reproducible.
#include "common.cuh"
#include "kernels.cuh"

#include <mutex>

namespace comet {

struct SegDotArgs {
  const int32_t *seg_end;
  const int32_t *crd;
  const double *val;
  int64_t M, N;
  const double *x;
  double *y;
  const int32_t *out_row;   // NULL: segment s -> y[s]; else y[out_row[s]] (y pre-zeroed by the launcher)
  int64_t num_tiles;
  double *carry_val;
  int32_t *carry_seg;
};

template <int THREADS, int IPT>
__global__ void __launch_bounds__(THREADS) seg_dot_kernel(const SegDotArgs a) {
  constexpr int TILE = THREADS * IPT;
  constexpr int WARPS = THREADS / 32;
  __shared__ int32_t s_end[TILE + 1];
  __shared__ double s_prod[TILE];
  __shared__ int64_t s_split[2];
  __shared__ int32_t s_wkey[WARPS];
  __shared__ double s_wval[WARPS];

  const int tid = threadIdx.x;
  const int64_t tile = blockIdx.x;
  const int64_t total = a.M + a.N;
  const int64_t d0 = tile * TILE;
  const int64_t d1 = (d0 + TILE < total) ? d0 + TILE : total;
  if (tid < 2) s_split[tid] = merge_path_segments(a.seg_end, a.M, a.N, tid ? d1 : d0);
  __syncthreads();
  const int64_t i0 = s_split[0], i1 = s_split[1];
  const int64_t j0 = d0 - i0, j1 = d1 - i1;
  const int rows = (int)(i1 - i0);       // segment-end markers inside the tile
  const int nnz = (int)(j1 - j0);        // leaf entries inside the tile

  for (int t = tid; t < rows; t += THREADS) s_end[t] = (int32_t)((int64_t)__ldg(a.seg_end + i0 + t) - j0);
  for (int t = tid; t < nnz; t += THREADS) {
    const int32_t c = ld_stream(a.crd + j0 + t);
    const double v = ld_stream(a.val + j0 + t);
    s_prod[t] = v * __ldg(a.x + c);
  }
  __syncthreads();

  // thread-level split of the tile's merge list
  const int items = rows + nnz;
  const int t0 = (tid * IPT < items) ? tid * IPT : items;
  const int t1 = (t0 + IPT < items) ? t0 + IPT : items;
  int lo = t0 > nnz ? t0 - nnz : 0;
  int hi = t0 < rows ? t0 : rows;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (s_end[mid] + mid < t0) lo = mid + 1; else hi = mid;
  }
  int i = lo, j = t0 - lo;

  double running = 0.0;
  bool have_first = false;
  int first_row = 0;
  double first_val = 0.0;
  for (int it = t0; it < t1; ++it) {
    if (i < rows && j >= s_end[i]) {     // next item is the end marker of segment i
      if (!have_first) {
        have_first = true;
        first_row = i;
        first_val = running;             // completed once the earlier threads' part is known
      } else {
        const int64_t s = i0 + i;
        a.y[a.out_row ? (int64_t)__ldg(a.out_row + s) : s] = running;
      }
      running = 0.0;
      ++i;
    } else {
      running += s_prod[j];
      ++j;
    }
  }

  // Inclusive segmented scan over threads of (segment the thread stopped in, its open partial sum).
  // Keys are non-decreasing, so "same key at distance off" implies the same key in between.
  const int lane = tid & 31, warp = tid >> 5;
  int key = i;
  double sum = running;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int k2 = __shfl_up_sync(0xffffffffu, key, off);
    const double v2 = __shfl_up_sync(0xffffffffu, sum, off);
    if (lane >= off && k2 == key) sum += v2;
  }
  if (lane == 31) { s_wkey[warp] = key; s_wval[warp] = sum; }
  __syncthreads();
  if (warp == 0) {
    int wk = lane < WARPS ? s_wkey[lane] : 0x7fffffff;
    double wv = lane < WARPS ? s_wval[lane] : 0.0;
#pragma unroll
    for (int off = 1; off < WARPS; off <<= 1) {
      const int k2 = __shfl_up_sync(0xffffffffu, wk, off);
      const double v2 = __shfl_up_sync(0xffffffffu, wv, off);
      if (lane >= off && k2 == wk) wv += v2;
    }
    if (lane < WARPS) s_wval[lane] = wv;
  }
  __syncthreads();
  if (warp > 0 && s_wkey[warp - 1] == key) sum += s_wval[warp - 1];
  // what the threads before this one hold for the segment this thread started in
  int prev_key = __shfl_up_sync(0xffffffffu, key, 1);
  double prev_sum = __shfl_up_sync(0xffffffffu, sum, 1);
  if (lane == 0) {
    prev_key = warp > 0 ? s_wkey[warp - 1] : -1;
    prev_sum = warp > 0 ? s_wval[warp - 1] : 0.0;
  }
  if (have_first) {
    const double carry_in = (tid > 0 && prev_key == first_row) ? prev_sum : 0.0;
    const int64_t s = i0 + first_row;
    a.y[a.out_row ? (int64_t)__ldg(a.out_row + s) : s] = first_val + carry_in;
  }
  if (tid == THREADS - 1) {
    // key == rows here: the segment the tile stops in
    a.carry_seg[tile] = (i1 < a.M) ? (int32_t)i1 : -1;
    a.carry_val[tile] = sum;
  }
}

template <int THREADS, int IPT>
static comet_status_t launch_dot(Context *ctx, SegDotArgs a, cudaStream_t stream) {
  const int64_t total = a.M + a.N;
  a.num_tiles = ceil_div(total, (int64_t)THREADS * IPT);
  const size_t val_bytes = align_up((size_t)a.num_tiles * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  seg_dot_kernel<THREADS, IPT><<<(unsigned)a.num_tiles, THREADS, 0, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
  if (a.num_tiles > 1) {
    carry_fixup_kernel<<<(unsigned)ceil_div(a.num_tiles, 256), 256, 0, stream>>>(
        a.carry_val, a.carry_seg, a.num_tiles, 1, 1, a.y, 1, a.out_row);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}

comet_status_t seg_dot(Context *ctx, const int32_t *seg_end, const int32_t *crd, const double *val, int64_t M,
                       int64_t N, const double *x, double *y, const int32_t *out_row, int64_t out_rows,
                       cudaStream_t stream) {
  if (out_row) {
    comet_status_t st = zero_rows(ctx, y, out_rows, 1, 1, stream);
    if (st != COMET_OK) return st;
  }
  if (M == 0) return COMET_OK;
  SegDotArgs a{};
  a.seg_end = seg_end; a.crd = crd; a.val = val; a.M = M; a.N = N; a.x = x; a.y = y; a.out_row = out_row;
  // Small problems: short tiles so that the grid still covers the 148 SMs.
  if (M + N < (int64_t)kSmCount * 2048 * 2) return launch_dot<128, 4>(ctx, a, stream);
  return launch_dot<256, 8>(ctx, a, stream);
}

}  // namespace comet

// ------------------------------------------------------------------------------------------------
// comet_spmv_static: CSR SpMV for callers that must not allocate device memory.
//
// The regular entry point takes its carry slots (one double and one int32 per tile) from the handle's
// scratch, which the handle obtains from an allocator. This variant keeps those slots in a fixed
// array that is part of the library image, so the call reaches no allocator at all and needs no
// handle. The price: a hard upper limit on the problem size and one array shared by every call.
namespace {

constexpr int kStaticThreads = 256;
constexpr int kStaticIpt = 8;
constexpr int64_t kStaticMaxTiles = 65536;                                   // tiles of 2048 merge items
constexpr int64_t kStaticMaxItems = kStaticMaxTiles * kStaticThreads * kStaticIpt;   // rows + nnz <= 134,217,728
constexpr size_t kStaticValBytes = (size_t)kStaticMaxTiles * sizeof(double);
constexpr size_t kStaticBytes = kStaticValBytes + (size_t)kStaticMaxTiles * sizeof(int32_t);   // 768 KiB

// Lives in every GPU that loads the library, from load until the process exits. In HOST code this
// name is only a stand-in for the symbol: the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_spmv_static_scratch[kStaticBytes];

constexpr int kStaticMaxDevices = 64;
void *g_static_scratch_addr[kStaticMaxDevices];   // per device, filled by the first call on that device
std::mutex g_static_mutex;

// Device address of the static scratch on the CURRENT device (looked up once per device).
comet_status_t static_scratch_address(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) { cudaGetLastError(); return COMET_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_scratch_addr[dev]) {
    void *p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_spmv_static_scratch);
    if (e != cudaSuccess || !p) { cudaGetLastError(); return COMET_ERR_CUDA; }
    g_static_scratch_addr[dev] = p;
  }
  *out = g_static_scratch_addr[dev];
  return COMET_OK;
}

}  // namespace

extern "C" comet_status_t comet_spmv_static(const comet_sptensor_t *A, const void *x, void *y, void *stream) {
  using namespace comet;
  if (!A || !x || !y) return COMET_ERR_INVALID_ARG;
  if (A->order != 2 || A->dtype != COMET_F64) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (A->attr[0] != COMET_D || A->attr[1] != COMET_CU) return COMET_ERR_UNSUPPORTED_FORMAT;
  const int m0 = A->mode_order[0], m1 = A->mode_order[1];
  if (!((m0 == 0 && m1 == 1) || (m0 == 1 && m1 == 0))) return COMET_ERR_INVALID_ARG;
  const int64_t M = A->dims[m0], N = A->nnz;
  if (M < 0 || N < 0 || !A->pos[1] || A->pos_len[1] != M + 1 || (N > 0 && (!A->crd[1] || !A->val)))
    return COMET_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 7) || (reinterpret_cast<uintptr_t>(y) & 7)) return COMET_ERR_MISALIGNED;
  if (M + N > kStaticMaxItems) return COMET_ERR_WORKSPACE;      // beyond the fixed scratch: use comet_spmv
  if (M == 0) return COMET_OK;

  void *scratch = nullptr;
  const comet_status_t st = static_scratch_address(&scratch);
  if (st != COMET_OK) return st;

  SegDotArgs a{};
  a.seg_end = A->pos[1] + 1; a.crd = A->crd[1]; a.val = (const double *)A->val;
  a.M = M; a.N = N; a.x = (const double *)x; a.y = (double *)y; a.out_row = nullptr;
  a.num_tiles = ceil_div(M + N, (int64_t)kStaticThreads * kStaticIpt);
  a.carry_val = (double *)scratch;                               // every tile writes its slot before the
  a.carry_seg = (int32_t *)((char *)scratch + kStaticValBytes);  // fix-up reads it: nothing to clear
  cudaStream_t s = (cudaStream_t)stream;
  seg_dot_kernel<kStaticThreads, kStaticIpt><<<(unsigned)a.num_tiles, kStaticThreads, 0, s>>>(a);
  if (a.num_tiles > 1)
    carry_fixup_kernel<<<(unsigned)ceil_div(a.num_tiles, 256), 256, 0, s>>>(a.carry_val, a.carry_seg, a.num_tiles, 1, 1,
                                                                            a.y, 1, nullptr);
  if (cudaGetLastError() != cudaSuccess) return COMET_ERR_CUDA;
  return COMET_OK;
}
