// MTTKRP for an output mode that is NOT stored first (levels 1 and 2 of a 3-level tensor), on the
// tensor as it is: nothing is re-packed or permuted.
//
// With the output mode below the root the terms of one output row are spread over the whole tensor
// (the entries are sorted by the root mode first), so no tile owns a row. The terms are therefore
// added into the output with floating-point atomic adds. Two consequences, both stated in the header:
// the summation order is not fixed (results agree from run to run only up to rounding, unlike every
// other kernel of the library), and the output is zero-filled first. Sums are kept in double: for
// fp32 tensors the atomics go to a double scratch matrix that is rounded into the output at the end.
//
// CSF [CU,CU,CU], coordinates (i, j, k) at levels 0..2, A / B = the factors of the two other modes:
//   level 1:  out[j, :] += (sum over the fiber's entries of val * B[k, :]) * A[i, :]     one add per fiber
//   level 2:  out[k, :] += val * (A[i, :] * B[j, :])                                     one add per entry
// COO [CN,S,S]:  out[c_out, :] += val * A[c_a, :] * B[c_b, :]                            one add per entry
//
// A worker is G lanes (G = the power of two covering min(R, 32) columns); it owns a few consecutive
// fibers (CSF) or entries (COO), finds its slice once by binary search in the level-1 pos array and
// then advances it. Lanes of a worker touch consecutive columns, so row reads and atomic adds are
// one contiguous request per worker.
#include "common.cuh"
#include "kernels.cuh"

#include <stdlib.h>

namespace comet {

struct ScatterArgs {
  const int32_t *pos1, *crd0, *crd1, *pos2, *crd2;   // CSF levels (COO: crd0/crd1/crd2 = out / a / b coordinates)
  const void *val;
  int64_t S, F, N;
  const void *A, *B;
  int64_t lda, ldb;
  double *acc;                                         // rows x R sums, leading dimension ldacc
  int64_t ldacc;
  int32_t R;
  int32_t per_worker;                                  // fibers (CSF) or entries (COO) per worker
};

constexpr int kScatterThreads = 256;

template <class T, int LEVEL, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_csf_scatter_kernel(const ScatterArgs a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t f0 = worker * a.per_worker;
  if (f0 >= a.F) return;
  const int64_t f1 = f0 + a.per_worker < a.F ? f0 + a.per_worker : a.F;
  // the slice of fiber f0: the largest s with pos1[s] <= f0 (pos1[0] = 0 and pos1[S] = F > f0 bracket it)
  int64_t lo = 0, hi = a.S;
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(a.pos1 + mid) <= f0) lo = mid; else hi = mid;
  }
  int64_t s = lo;
  int64_t s_end = __ldg(a.pos1 + s + 1);
  for (int64_t f = f0; f < f1; ++f) {
    while (f >= s_end && s + 1 < a.S) { ++s; s_end = __ldg(a.pos1 + s + 1); }
    const int64_t i = __ldg(a.crd0 + s), j = __ldg(a.crd1 + f);
    const int64_t p0 = __ldg(a.pos2 + f), p1 = __ldg(a.pos2 + f + 1);
    for (int c = g; c < a.R; c += G) {
      if (LEVEL == 1) {
        double t = 0.0;
        for (int64_t p = p0; p < p1; ++p)
          t += (double)ld_stream(val + p) * (double)__ldg(B + (int64_t)__ldg(a.crd2 + p) * a.ldb + c);
        atomicAdd(a.acc + j * a.ldacc + c, t * (double)__ldg(A + i * a.lda + c));
      } else {
        const double w = (double)__ldg(A + i * a.lda + c) * (double)__ldg(B + j * a.ldb + c);
        for (int64_t p = p0; p < p1; ++p)
          atomicAdd(a.acc + (int64_t)__ldg(a.crd2 + p) * a.ldacc + c, (double)ld_stream(val + p) * w);
      }
    }
  }
}

template <class T, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_coo_scatter_kernel(const ScatterArgs a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t p0 = worker * a.per_worker;
  const int64_t p1 = p0 + a.per_worker < a.N ? p0 + a.per_worker : a.N;
  for (int64_t p = p0; p < p1; ++p) {
    const int64_t ro = __ldg(a.crd0 + p), ia = __ldg(a.crd1 + p), ib = __ldg(a.crd2 + p);
    const double v = (double)ld_stream(val + p);
    for (int c = g; c < a.R; c += G)
      atomicAdd(a.acc + ro * a.ldacc + c, v * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c));
  }
}

// ------------------------------------------------------------------------------- popular output rows
// Atomic adds to ONE address retire one after the other in L2 (measured on B200: 0.12 G row adds per second
// into a single 256-byte row against 18 G/s into rows drawn uniformly), so an output mode whose coordinates are
// drawn with very unequal frequencies is bound by its most popular rows. The leaf-mode kernel below therefore
// keeps the most popular output rows in shared memory: a sample of the leaf coordinates is counted, the rows
// that were seen most often get a slot each (as many as fit), every CTA adds their terms into its own copy and
// adds that copy into the output once, at the end. Which rows are chosen changes the speed only, not the sums.
constexpr int kHotThreads = 512;
constexpr int kHotCtas = 2;                        // CTAs per SM
// Entries per warp and step; the warps draw chunk numbers from a counter. Dealt out round-robin instead, the last
// round is only partly filled: 100 M entries over 9,472 warps take 42 rounds of 256 (2 % idle) but 3 rounds of
// 4,096 where 2.6 would do (measured, round-robin: 6.70 / 6.76 / 7.88 ms with 256 / 1,024 / 4,096 entries; with the
// counter 6.43 / 6.44 / 6.45 ms with 256 / 512 / 1,024).
constexpr int kHotChunk = 256;
// Shared memory per CTA for the popular rows: 256 rows of 32 columns. Measured on config 5 (leaf frequencies
// (k + 100)^-1.5 over 200,000 rows): 32 rows 16.6 ms, 128 rows 6.75 to 8.9 ms depending on where the output
// matrix happened to be allocated (the next few hundred rows still collide in L2), 256 rows 6.87 ms wherever it
// was, 384 rows 7.16 ms (an add in shared memory is a compare-and-swap loop of about a dozen instructions, an
// add in L2 one instruction: past the rows that L2 serialises, more slots cost more than they save).
constexpr size_t kHotBytes = 64 * 1024;
constexpr int64_t kHotMaxRows = 1ll << 24;         // two 32-bit words per output row are allocated for the call
constexpr int64_t kHotSamples = 1ll << 22;

__global__ void sample_rows_kernel(const int32_t *__restrict__ crd, int64_t n, int64_t stride, int32_t *__restrict__ counts) {
  const int64_t p = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * stride;
  if (p < n) atomicAdd(counts + __ldg(crd + p), 1);
}

// Which rows get a slot: a histogram of the sampled counts over bins of 1/16 octave (counts within 6 % of each
// other share a bin), the lowest bin that at most `slots` rows reach, and a slot for every row that reaches it
// (slot numbers in the order the rows arrive; should the top bin alone hold more rows than slots, the first
// `slots` of them are taken).
constexpr int kCountBins = 512;

__device__ __forceinline__ int count_bin(int32_t c) {         // c >= 1; monotone in c
  const int e = 31 - __clz(c);
  const int m = e >= 4 ? (c >> (e - 4)) & 15 : (c << (4 - e)) & 15;
  return e * 16 + m;
}

__global__ void __launch_bounds__(256) count_histogram_kernel(const int32_t *__restrict__ counts, int64_t rows,
                                                              int32_t *__restrict__ bins) {
  __shared__ int32_t s_bins[kCountBins];
  for (int b = threadIdx.x; b < kCountBins; b += 256) s_bins[b] = 0;
  __syncthreads();
  for (int64_t r = (int64_t)blockIdx.x * 256 + threadIdx.x; r < rows; r += (int64_t)gridDim.x * 256) {
    const int32_t c = __ldg(counts + r);
    if (c > 0) atomicAdd(&s_bins[count_bin(c)], 1);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kCountBins; b += 256)
    if (s_bins[b]) atomicAdd(bins + b, s_bins[b]);
}

// *threshold = the lowest bin t such that at most `slots` rows have a count in bin t or above
__global__ void pick_threshold_kernel(const int32_t *__restrict__ bins, int32_t slots, int32_t *__restrict__ threshold) {
  __shared__ int32_t s_bins[kCountBins];
  for (int b = threadIdx.x; b < kCountBins; b += blockDim.x) s_bins[b] = bins[b];
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = kCountBins - 1;
    int64_t reach = s_bins[t];
    while (t > 0 && reach + s_bins[t - 1] <= slots) { --t; reach += s_bins[t]; }
    *threshold = t;
  }
}

__global__ void assign_slots_kernel(const int32_t *__restrict__ counts, int64_t rows, const int32_t *__restrict__ threshold,
                                    int32_t slots, int32_t *__restrict__ hot_slot, int32_t *__restrict__ hot_rows,
                                    int32_t *__restrict__ n_hot) {
  const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  int32_t slot = -1;
  const int32_t c = counts[r];
  if (c > 0 && count_bin(c) >= *threshold) {
    slot = atomicAdd(n_hot, 1);
    if (slot < slots) hot_rows[slot] = (int32_t)r; else slot = -1;
  }
  hot_slot[r] = slot;
}

// fiber_root[f] = the root coordinate of the slice that holds fiber f (a warp per slice).
__global__ void fiber_root_kernel(const int32_t *__restrict__ pos1, const int32_t *__restrict__ crd0, int64_t S,
                                  int32_t *__restrict__ fiber_root) {
  const int64_t s = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (s >= S) return;
  const int32_t i = __ldg(crd0 + s);
  for (int64_t f = (int64_t)__ldg(pos1 + s) + (threadIdx.x & 31); f < (int64_t)__ldg(pos1 + s + 1); f += 32) fiber_root[f] = i;
}

// CSF with the output mode at the leaf level, out[k, :] += val * (A[i, :] * B[j, :]), or (COO) a sorted coordinate
// list with the output mode anywhere but first: one row add per entry; rows with a slot are added in shared memory. A warp takes kHotChunk consecutive ENTRIES per step. Its lanes first work
// entry-parallel: each reads one entry's coordinate, value and slot and finds the entry's fiber in a window of 32
// fiber ends held one per lane (so the loads of 32 entries are in flight together, whatever the fiber lengths);
// then the lanes are the columns (R > 32: several sweeps) and the 32 entries are handed round with shuffles.
template <class T, bool COO>
__global__ void __launch_bounds__(kHotThreads, kHotCtas) mttkrp_csf_leaf_hot_kernel(const ScatterArgs a,
                                                                                   const int32_t *__restrict__ fiber_root,
                                                                                   const int32_t *__restrict__ hot_slot,
                                                                                   const int32_t *__restrict__ hot_rows,
                                                                                   const int32_t *__restrict__ n_hot, int32_t slots,
                                                                                   unsigned long long *__restrict__ next_chunk) {
  extern __shared__ double s_acc[];                // slots x R
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B);
  const int used = *n_hot < slots ? *n_hot : slots;
  for (int x = threadIdx.x; x < used * a.R; x += kHotThreads) s_acc[x] = 0.0;
  __syncthreads();
  const unsigned full = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  const int64_t chunks = (a.N + kHotChunk - 1) / kHotChunk;
  while (true) {                                   // chunks are handed out as the warps ask: no partly filled last round
    unsigned long long ticket = 0;
    if (lane == 0) ticket = atomicAdd(next_chunk, 1ull);
    const int64_t chunk = (int64_t)__shfl_sync(full, ticket, 0);
    if (chunk >= chunks) break;
    const int64_t p0 = chunk * kHotChunk;
    const int64_t p1 = p0 + kHotChunk < a.N ? p0 + kHotChunk : a.N;
    int64_t fw = 0;                                // CSF: the window of fibers fw .. fw + 31, one per lane
    int32_t w_end = 0x7fffffff, w_i = 0, w_j = 0;
    if constexpr (!COO) {
      int64_t lo = 0, hi = a.F;                    // the fiber of entry p0: the largest f with pos2[f] <= p0
      while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)__ldg(a.pos2 + mid) <= p0) lo = mid; else hi = mid;
      }
      fw = lo;
      w_end = fw + lane < a.F ? __ldg(a.pos2 + fw + lane + 1) : 0x7fffffff;
      w_i = fw + lane < a.F ? __ldg(fiber_root + fw + lane) : 0;
      w_j = fw + lane < a.F ? __ldg(a.crd1 + fw + lane) : 0;
    }
    for (int64_t pb = p0; pb < p1; pb += 32) {
      const int cnt = p1 - pb < 32 ? (int)(p1 - pb) : 32;
      const int32_t p = (int32_t)pb + lane;
      // the output coordinate: the leaf's (CSF) or the one listed first (COO: crd0 / crd1 / crd2 = output, A's, B's)
      const int32_t kk = lane < cnt ? __ldg((COO ? a.crd0 : a.crd2) + p) : 0;
      const double vv = lane < cnt ? (double)ld_stream(val + p) : 0.0;
      const int32_t qq = lane < cnt ? __ldg(hot_slot + kk) : -1;
      uint32_t row_a = 0, row_b = 0;               // element offsets of this entry's rows of A and B (32 bits: the host checks the sizes)
      if constexpr (COO) {
        if (lane < cnt) {
          row_a = (uint32_t)__ldg(a.crd1 + p) * (uint32_t)a.lda;
          row_b = (uint32_t)__ldg(a.crd2 + p) * (uint32_t)a.ldb;
        }
      } else {
        bool found = lane >= cnt;
        while (true) {                             // this entry's fiber: the ends at or below p, counted over the window
          int u = 0;                               // binary search over the 32 sorted ends, held one per lane
#pragma unroll
          for (int step = 16; step > 0; step >>= 1)
            if (__shfl_sync(full, w_end, u + step - 1) <= p) u += step;
          if (__shfl_sync(full, w_end, 31) <= p && u == 31) u = 32;
          const int32_t ci = __shfl_sync(full, w_i, u & 31), cj = __shfl_sync(full, w_j, u & 31);
          if (!found && u < 32) { row_a = (uint32_t)ci * (uint32_t)a.lda; row_b = (uint32_t)cj * (uint32_t)a.ldb; found = true; }
          if (__all_sync(full, found)) break;
          fw += 32;                                // entries beyond the window's last fiber: next window
          w_end = fw + lane < a.F ? __ldg(a.pos2 + fw + lane + 1) : 0x7fffffff;
          w_i = fw + lane < a.F ? __ldg(fiber_root + fw + lane) : 0;
          w_j = fw + lane < a.F ? __ldg(a.crd1 + fw + lane) : 0;
        }
      }
      // where the entry's term goes: a slot's row in shared memory (bit 31 set) or the output row's element offset
      const uint32_t dest = qq >= 0 ? 0x80000000u | (uint32_t)(qq * a.R) : (uint32_t)kk * (uint32_t)a.ldacc;
      for (int c0 = 0; c0 < a.R; c0 += 32) {
        const int c = c0 + lane;
        const bool inb = c < a.R;
#pragma unroll 4
        for (int e = 0; e < cnt; ++e) {            // the rows of consecutive entries of a fiber come from L1
          const uint32_t d = __shfl_sync(full, dest, e);
          const uint32_t ra = __shfl_sync(full, row_a, e), rb = __shfl_sync(full, row_b, e);
          const double v = __shfl_sync(full, vv, e);
          if (inb) {
            const double t = v * ((double)__ldg(A + (ra + c)) * (double)__ldg(B + (rb + c)));
            if (d & 0x80000000u) atomicAdd(&s_acc[(d & 0x7fffffffu) + c], t);
            else atomicAdd(a.acc + (d + c), t);
          }
        }
      }
    }
  }
  __syncthreads();
  for (int x = threadIdx.x; x < used * a.R; x += kHotThreads) {
    const double v = s_acc[x];
    const int q = x / a.R;
    if (v != 0.0) atomicAdd(a.acc + (int64_t)__ldg(hot_rows + q) * a.ldacc + (x - q * a.R), v);
  }
}

// The per-entry product (CSF leaf mode, or any non-root mode of a COO tensor) with the popular rows in shared
// memory; *done = 0 when the shape is not this path's (the caller then runs the general kernel).
template <class T>
static comet_status_t entries_hot(Context *ctx, const ScatterArgs &a, bool coo, int64_t rows, int64_t a_rows, int64_t b_rows,
                                  int *done, cudaStream_t stream) {
  *done = 0;
  const char *force = getenv("COMET_MTTKRP_HOT_ROWS");      // tests: "1" takes this path on any size, "0" never
  if (force && force[0] == '0') return COMET_OK;
  const bool forced = force && force[0] == '1';
  if (rows < 1 || rows > kHotMaxRows || a.R > 4096) return COMET_OK;
  if (!forced && (a.R < 16 || a.N < (1ll << 20))) return COMET_OK;
  // the kernel indexes the three matrices with 32-bit element offsets
  if (rows * a.ldacc + a.R >= (1ll << 31) || a_rows * a.lda + a.R >= (1ll << 31) || b_rows * a.ldb + a.R >= (1ll << 31)) return COMET_OK;
  int64_t slots = (int64_t)(kHotBytes / ((size_t)a.R * sizeof(double)));
  if (slots > rows) slots = rows;
  if (slots < 1) return COMET_OK;
  const int32_t *out_crd = coo ? a.crd0 : a.crd2;
  // counts[rows] | bins[kCountBins] | slots in use | threshold | chunk counter (64 bits, 8-byte aligned): one block,
  // zero-filled at once
  const int64_t words = align_up((size_t)(rows + kCountBins + 2), 2) + 2;
  int32_t *counts = (int32_t *)ctx_alloc(ctx, (size_t)words * 4, stream);
  int32_t *hot_slot = (int32_t *)ctx_alloc(ctx, (size_t)rows * 4, stream);
  int32_t *hot_rows = (int32_t *)ctx_alloc(ctx, (size_t)slots * 4, stream);
  int32_t *fiber_root = coo ? nullptr : (int32_t *)ctx_alloc(ctx, (size_t)a.F * 4, stream);
  comet_status_t st = (counts && hot_slot && hot_rows && (coo || fiber_root)) ? COMET_OK : COMET_ERR_ALLOC;
  if (st == COMET_OK) {
    cudaError_t e = cudaMemsetAsync(counts, 0, (size_t)words * 4, stream);
    if (e != cudaSuccess) st = cuda_fail(ctx, e);
  }
  if (st == COMET_OK) {
    int32_t *bins = counts + rows, *n_hot = bins + kCountBins, *threshold = n_hot + 1;
    const int64_t stride = a.N > kHotSamples ? a.N / kHotSamples : 1;
    const int64_t samples = ceil_div(a.N, stride);
    sample_rows_kernel<<<(unsigned)ceil_div(samples, 256), 256, 0, stream>>>(out_crd, a.N, stride, counts);
    const int64_t hist_ctas = ceil_div(rows, 256) < 2 * kSmCount ? ceil_div(rows, 256) : 2 * kSmCount;
    count_histogram_kernel<<<(unsigned)hist_ctas, 256, 0, stream>>>(counts, rows, bins);
    pick_threshold_kernel<<<1, 256, 0, stream>>>(bins, (int32_t)slots, threshold);
    assign_slots_kernel<<<(unsigned)ceil_div(rows, 256), 256, 0, stream>>>(counts, rows, threshold, (int32_t)slots, hot_slot, hot_rows, n_hot);
    ctx->launches += 4;
    if (!coo) {
      fiber_root_kernel<<<(unsigned)ceil_div(a.S * 32, 256), 256, 0, stream>>>(a.pos1, a.crd0, a.S, fiber_root);
      ctx->launches += 1;
    }
    auto kernel = coo ? mttkrp_csf_leaf_hot_kernel<T, true> : mttkrp_csf_leaf_hot_kernel<T, false>;
    const size_t smem = (size_t)slots * a.R * sizeof(double);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) st = cuda_fail(ctx, e);
    if (st == COMET_OK) {
      kernel<<<kHotCtas * kSmCount, kHotThreads, smem, stream>>>(a, fiber_root, hot_slot, hot_rows, n_hot, (int32_t)slots,
                                                                 reinterpret_cast<unsigned long long *>(counts + words - 2));
      ctx->launches += 1;
      e = cudaGetLastError();
      if (e != cudaSuccess) st = cuda_fail(ctx, e);
      else *done = 1;
    }
  }
  if (fiber_root) ctx_free(ctx, fiber_root, stream);
  if (counts) ctx_free(ctx, counts, stream);
  if (hot_slot) ctx_free(ctx, hot_slot, stream);
  if (hot_rows) ctx_free(ctx, hot_rows, stream);
  return st;
}

__global__ void zero_acc_kernel(double *__restrict__ acc, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) acc[i] = 0.0;
}

// out[r, c] = (float)acc[r, c]: the one rounding of an fp32 result
__global__ void round_acc_kernel(const double *__restrict__ acc, int64_t rows, int32_t R, float *__restrict__ out,
                                 int64_t ldo) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t r = i / R;
  if (r < rows) out[r * ldo + (i - r * R)] = (float)acc[i];
}

template <class T, int G>
static void launch_scatter(int kind, const ScatterArgs &a, int64_t units, cudaStream_t stream) {
  const int64_t workers = ceil_div(units, a.per_worker);
  const unsigned blocks = (unsigned)ceil_div(workers * G, kScatterThreads);
  if (kind == 0) mttkrp_coo_scatter_kernel<T, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 1) mttkrp_csf_scatter_kernel<T, 1, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else mttkrp_csf_scatter_kernel<T, 2, G><<<blocks, kScatterThreads, 0, stream>>>(a);
}

template <class T>
static void launch_scatter_width(int kind, const ScatterArgs &a, int64_t units, cudaStream_t stream) {
  if (a.R > 16) launch_scatter<T, 32>(kind, a, units, stream);
  else if (a.R > 8) launch_scatter<T, 16>(kind, a, units, stream);
  else if (a.R > 4) launch_scatter<T, 8>(kind, a, units, stream);
  else if (a.R > 2) launch_scatter<T, 4>(kind, a, units, stream);
  else if (a.R > 1) launch_scatter<T, 2>(kind, a, units, stream);
  else launch_scatter<T, 1>(kind, a, units, stream);
}

// kind 0: COO (crd0 = output-mode coordinates, crd1 / crd2 = coordinates of A's / B's modes);
// kind 1 / 2: CSF with the output mode at level 1 / 2.
comet_status_t mttkrp_scatter(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *crd0,
                              const int32_t *crd1, const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S,
                              int64_t F, int64_t N, int64_t rows, int64_t a_rows, int64_t b_rows, const void *A,
                              int64_t lda, const void *B, int64_t ldb, int64_t R, void *out, int64_t ldo,
                              cudaStream_t stream) {
  if (R > 2147483647ll) return COMET_ERR_INDEX_OVERFLOW;
  ScatterArgs a{};
  a.pos1 = pos1; a.crd0 = crd0; a.crd1 = crd1; a.pos2 = pos2; a.crd2 = crd2; a.val = val;
  a.S = S; a.F = F; a.N = N; a.A = A; a.lda = lda; a.B = B; a.ldb = ldb; a.R = (int32_t)R;
  if (dtype == COMET_F32) {
    if (rows == 0) return COMET_OK;
    const int64_t n = rows * R;
    a.acc = (double *)scratch_get(ctx, (size_t)n * sizeof(double), stream);
    if (!a.acc) return COMET_ERR_ALLOC;
    a.ldacc = R;
    zero_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, n);
    COMET_LAUNCH_CHECK(ctx);
  } else {
    comet_status_t st = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
    if (st != COMET_OK) return st;
    a.acc = (double *)out;
    a.ldacc = ldo;
  }
  if (N > 0) {
    int done = 0;
    if (kind == 2 || kind == 0) {                   // one add per entry: the popular output rows go to shared memory
      comet_status_t st = dtype == COMET_F32 ? entries_hot<float>(ctx, a, kind == 0, rows, a_rows, b_rows, &done, stream)
                                              : entries_hot<double>(ctx, a, kind == 0, rows, a_rows, b_rows, &done, stream);
      if (st != COMET_OK) return st;
    }
    if (!done) {
      a.per_worker = kind == 0 ? 16 : 8;
      const int64_t units = kind == 0 ? N : F;
      if (dtype == COMET_F32) launch_scatter_width<float>(kind, a, units, stream);
      else launch_scatter_width<double>(kind, a, units, stream);
      COMET_LAUNCH_CHECK(ctx);
    }
  }
  if (dtype == COMET_F32) {
    const int64_t n = rows * R;
    round_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, rows, (int32_t)R, (float *)out, ldo);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}


// ------------------------------------------------------------------------------------------- 4-order tensors
// The same accumulation for tensors of four modes, every output mode (the mode stored first included: there
// is no tiled kernel for 4-order tensors). CSF [CU,CU,CU,CU], coordinates (c0, c1, c2, c3) at levels 0..3; a
// worker owns a few consecutive level-2 fibers and tracks the level-1 fiber and the slice that hold them.
//   output at level 3:   out[c3, :] += val * (A[c0, :] * B[c1, :] * C[c2, :])                 one add per entry
//   output at level < 3: out[c_L, :] += (sum over the fiber of val * C[c3, :]) * A[.] * B[.]   one add per fiber
// (A, B, C = the factors of the three other levels in storage order.) COO [CN,S,S,S]: one add per entry.
struct Scatter4Args {
  const int32_t *pos1, *pos2, *pos3, *crd[4];   // COO: crd[0] = output coordinates, crd[1..3] = those of A, B, C
  const void *val;
  int64_t S, F1, F2, N;
  const void *A, *B, *C;
  int64_t lda, ldb, ldc;
  double *acc;
  int64_t ldacc;
  int32_t R;
  int32_t per_worker;
};

__device__ __forceinline__ int64_t last_at_or_below(const int32_t *pos, int64_t n, int64_t x) {
  int64_t lo = 0, hi = n;                       // pos[0] = 0 <= x < pos[n]: the largest index with pos[index] <= x
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(pos + mid) <= x) lo = mid; else hi = mid;
  }
  return lo;
}

template <class T, int LEVEL, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_csf4_scatter_kernel(const Scatter4Args a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B), *const Cf = static_cast<const T *>(a.C);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t f0 = worker * a.per_worker;
  if (f0 >= a.F2) return;
  const int64_t f1 = f0 + a.per_worker < a.F2 ? f0 + a.per_worker : a.F2;
  int64_t u = last_at_or_below(a.pos2, a.F1, f0);          // level-1 fiber that holds level-2 fiber f0
  int64_t s = last_at_or_below(a.pos1, a.S, u);            // slice that holds it
  int64_t u_end = __ldg(a.pos2 + u + 1), s_end = __ldg(a.pos1 + s + 1);
  for (int64_t f = f0; f < f1; ++f) {
    while (f >= u_end && u + 1 < a.F1) { ++u; u_end = __ldg(a.pos2 + u + 1); }
    while (u >= s_end && s + 1 < a.S) { ++s; s_end = __ldg(a.pos1 + s + 1); }
    const int64_t c0 = __ldg(a.crd[0] + s), c1 = __ldg(a.crd[1] + u), c2 = __ldg(a.crd[2] + f);
    const int64_t p0 = __ldg(a.pos3 + f), p1 = __ldg(a.pos3 + f + 1);
    // the upper coordinates that index A and B (and C when the output is the leaf), and the output's
    const int64_t ia = LEVEL == 0 ? c1 : c0;
    const int64_t ib = LEVEL <= 1 ? c2 : c1;
    const int64_t io = LEVEL == 0 ? c0 : (LEVEL == 1 ? c1 : c2);
    for (int c = g; c < a.R; c += G) {
      if (LEVEL == 3) {
        const double w = (double)__ldg(A + c0 * a.lda + c) * (double)__ldg(B + c1 * a.ldb + c) *
                         (double)__ldg(Cf + c2 * a.ldc + c);
        for (int64_t p = p0; p < p1; ++p)
          atomicAdd(a.acc + (int64_t)__ldg(a.crd[3] + p) * a.ldacc + c, (double)ld_stream(val + p) * w);
      } else {
        double t = 0.0;
        for (int64_t p = p0; p < p1; ++p)
          t += (double)ld_stream(val + p) * (double)__ldg(Cf + (int64_t)__ldg(a.crd[3] + p) * a.ldc + c);
        atomicAdd(a.acc + io * a.ldacc + c, t * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c));
      }
    }
  }
}

template <class T, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_coo4_scatter_kernel(const Scatter4Args a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B), *const Cf = static_cast<const T *>(a.C);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t p0 = worker * a.per_worker;
  const int64_t p1 = p0 + a.per_worker < a.N ? p0 + a.per_worker : a.N;
  for (int64_t p = p0; p < p1; ++p) {
    const int64_t ro = __ldg(a.crd[0] + p), ia = __ldg(a.crd[1] + p), ib = __ldg(a.crd[2] + p), ic = __ldg(a.crd[3] + p);
    const double v = (double)ld_stream(val + p);
    for (int c = g; c < a.R; c += G)
      atomicAdd(a.acc + ro * a.ldacc + c, v * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c) *
                                              (double)__ldg(Cf + ic * a.ldc + c));
  }
}

template <class T, int G>
static void launch_scatter4(int kind, const Scatter4Args &a, int64_t units, cudaStream_t stream) {
  const int64_t workers = ceil_div(units, a.per_worker);
  const unsigned blocks = (unsigned)ceil_div(workers * G, kScatterThreads);
  if (kind < 0) mttkrp_coo4_scatter_kernel<T, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 0) mttkrp_csf4_scatter_kernel<T, 0, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 1) mttkrp_csf4_scatter_kernel<T, 1, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 2) mttkrp_csf4_scatter_kernel<T, 2, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else mttkrp_csf4_scatter_kernel<T, 3, G><<<blocks, kScatterThreads, 0, stream>>>(a);
}

template <class T>
static void launch_scatter4_width(int kind, const Scatter4Args &a, int64_t units, cudaStream_t stream) {
  if (a.R > 16) launch_scatter4<T, 32>(kind, a, units, stream);
  else if (a.R > 8) launch_scatter4<T, 16>(kind, a, units, stream);
  else if (a.R > 4) launch_scatter4<T, 8>(kind, a, units, stream);
  else if (a.R > 2) launch_scatter4<T, 4>(kind, a, units, stream);
  else if (a.R > 1) launch_scatter4<T, 2>(kind, a, units, stream);
  else launch_scatter4<T, 1>(kind, a, units, stream);
}

// kind -1: COO (crd[0] = output-mode coordinates, crd[1..3] = coordinates of A's, B's, C's modes);
// kind 0..3: CSF with the output mode at that level (crd = the four levels' coordinate arrays).
comet_status_t mttkrp_scatter4(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *pos2,
                               const int32_t *pos3, const int32_t *const *crd, const void *val, int64_t S, int64_t F1,
                               int64_t F2, int64_t N, int64_t rows, const void *A, int64_t lda, const void *B,
                               int64_t ldb, const void *C, int64_t ldc, int64_t R, void *out, int64_t ldo,
                               cudaStream_t stream) {
  if (R > 2147483647ll) return COMET_ERR_INDEX_OVERFLOW;
  Scatter4Args a{};
  a.pos1 = pos1; a.pos2 = pos2; a.pos3 = pos3; a.val = val;
  for (int l = 0; l < 4; ++l) a.crd[l] = crd[l];
  a.S = S; a.F1 = F1; a.F2 = F2; a.N = N;
  a.A = A; a.lda = lda; a.B = B; a.ldb = ldb; a.C = C; a.ldc = ldc; a.R = (int32_t)R;
  if (dtype == COMET_F32) {
    if (rows == 0) return COMET_OK;
    const int64_t n = rows * R;
    a.acc = (double *)scratch_get(ctx, (size_t)n * sizeof(double), stream);
    if (!a.acc) return COMET_ERR_ALLOC;
    a.ldacc = R;
    zero_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, n);
    COMET_LAUNCH_CHECK(ctx);
  } else {
    comet_status_t st = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
    if (st != COMET_OK) return st;
    a.acc = (double *)out;
    a.ldacc = ldo;
  }
  if (N > 0) {
    a.per_worker = kind < 0 ? 16 : 8;
    const int64_t units = kind < 0 ? N : F2;
    if (dtype == COMET_F32) launch_scatter4_width<float>(kind, a, units, stream);
    else launch_scatter4_width<double>(kind, a, units, stream);
    COMET_LAUNCH_CHECK(ctx);
  }
  if (dtype == COMET_F32) {
    const int64_t n = rows * R;
    round_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, rows, (int32_t)R, (float *)out, ldo);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}

}  // namespace comet
