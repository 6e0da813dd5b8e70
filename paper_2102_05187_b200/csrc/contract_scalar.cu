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

#include <string.h>

#include <mutex>

namespace comet {

struct SegDotArgs {
  const int32_t *seg_end;
  const int32_t *crd;
  const void *val;          // values, vector and output are T (double or float); sums are kept in double
  int64_t M, N;
  const void *x;
  void *y;
  const int32_t *out_row;   // NULL: segment s -> y[s]; else y[out_row[s]] (y pre-zeroed by the launcher)
  int64_t num_tiles;
  double *carry_val;
  int32_t *carry_seg;
  unsigned int *ctas_done;  // tile kernel only, may be NULL: counter (zero between calls) that lets the CTA which
                            // finishes last add the carries itself, so that a small problem is ONE launch
};

struct BlockBarrier {
  __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
struct NamedBarrier {          // a barrier over `count` threads of the CTA (a "virtual CTA")
  int id, count;
  __device__ __forceinline__ void operator()() const { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
};

// Steps 3 and 4 for a tile whose products and (tile-relative) segment ends are staged in shared memory.
// `tid` is the thread's index among the THREADS threads that share the tile and the barrier.
template <class T, int THREADS, int IPT, class Bar>
__device__ __forceinline__ void walk_staged_tile(const SegDotArgs &a, const int32_t *s_end, const double *s_prod,
                                                 int32_t *s_wkey, double *s_wval, int tid, int rows, int nnz,
                                                 int64_t i0, int64_t i1, int64_t tile, Bar bar) {
  constexpr int WARPS = THREADS / 32;
  T *const y = static_cast<T *>(a.y);
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
        y[a.out_row ? (int64_t)__ldg(a.out_row + s) : s] = (T)running;
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
  bar();
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
  bar();
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
    y[a.out_row ? (int64_t)__ldg(a.out_row + s) : s] = (T)(first_val + carry_in);
  }
  if (tid == THREADS - 1) {
    // key == rows here: the segment the tile stops in
    a.carry_seg[tile] = (i1 < a.M) ? (int32_t)i1 : -1;
    a.carry_val[tile] = sum;
  }
}

template <class T, int THREADS, int IPT>
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
  if (tid < 64) {          // warps 0 and 1 locate the two ends of the tile, 32 probes per round each
    const int64_t split = merge_path_segments_coop<32>(a.seg_end, a.M, a.N, tid < 32 ? d0 : d1, tid & 31, 0xffffffffu);
    if ((tid & 31) == 0) s_split[tid >> 5] = split;
  }
  __syncthreads();
  const int64_t i0 = s_split[0], i1 = s_split[1];
  const int64_t j0 = d0 - i0, j1 = d1 - i1;
  const int rows = (int)(i1 - i0);       // segment-end markers inside the tile
  const int nnz = (int)(j1 - j0);        // leaf entries inside the tile
  const T *const val = static_cast<const T *>(a.val), *const x = static_cast<const T *>(a.x);

  // Load phase, fully unrolled (a tile holds at most IPT entries and IPT markers per thread): all of a
  // thread's coordinate/value loads are issued before the first dependent vector gather, and all
  // gathers before the first product, so a thread has up to 3*IPT loads in flight instead of one.
  {
    int32_t c[IPT], e[IPT];
    double v[IPT];
#pragma unroll
    for (int k = 0; k < IPT; ++k) {
      const int t = tid + k * THREADS;
      c[k] = 0; v[k] = 0.0; e[k] = 0;
      if (t < nnz) { c[k] = ld_stream(a.crd + j0 + t); v[k] = (double)ld_stream(val + j0 + t); }
      if (t < rows) e[k] = __ldg(a.seg_end + i0 + t);
    }
#pragma unroll
    for (int k = 0; k < IPT; ++k) {
      const int t = tid + k * THREADS;
      if (t < nnz) v[k] *= (double)__ldg(x + c[k]);
    }
#pragma unroll
    for (int k = 0; k < IPT; ++k) {
      const int t = tid + k * THREADS;
      if (t < nnz) s_prod[t] = v[k];
      if (t < rows) s_end[t] = (int32_t)((int64_t)e[k] - j0);
    }
  }
  __syncthreads();

  walk_staged_tile<T, THREADS, IPT>(a, s_end, s_prod, s_wkey, s_wval, tid, rows, nnz, i0, i1, tile, BlockBarrier());

  if (a.ctas_done == nullptr) return;
  // Single-launch mode (few tiles): no CTA waits for another; each counts itself done, and the one that finds
  // all others already counted adds the carries (their writers fenced before counting) and zeroes the counter.
  __shared__ bool s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(a.ctas_done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  T *const y = static_cast<T *>(a.y);
  for (int64_t t0 = tid; t0 < a.num_tiles; t0 += THREADS) {
    const int32_t seg = __ldcg(a.carry_seg + t0);                      // written by other SMs: read past this SM's L1
    if (seg < 0) continue;
    if (t0 > 0 && __ldcg(a.carry_seg + t0 - 1) == seg) continue;        // the first tile of a run adds the whole run
    double sum = 0.0;
    for (int64_t t = t0; t < a.num_tiles && __ldcg(a.carry_seg + t) == seg; ++t) sum += __ldcg(a.carry_val + t);
    const int64_t row = a.out_row ? (int64_t)a.out_row[seg] : (int64_t)seg;
    y[row] = (T)((double)__ldcg(y + row) + sum);
  }
  if (tid == 0) *a.ctas_done = 0u;
}

// ------------------------------------------------------------------------------------------------
// The resident-vector variant: when the dense vector fits in shared memory beside the tile staging
// (x up to ~21,000 doubles), the random 8-byte gathers x[crd] are served from shared memory instead of
// L2, whose sector-request rate otherwise bounds the kernel (measured on TTV: 589 us with L2 gathers,
// 188 us with the gather removed). One persistent CTA per SM holds x and runs VC "virtual CTAs" of
// THREADS threads, each walking its own sequence of tiles with its own staging and named barrier.
// A virtual CTA keeps the next tile's leaf loads in flight (registers) while it walks the current
// one, and reads its tile boundaries from a table a small partition kernel wrote, two tiles ahead.

// splits[b] = segment-end markers among the first b * tile_items merge items, one warp per boundary
__global__ void tile_split_kernel(const int32_t *__restrict__ seg_end, int64_t M, int64_t N, int32_t tile_items,
                                  int64_t num_tiles, int32_t *__restrict__ splits) {
  const int64_t b = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (b > num_tiles) return;
  const int64_t total = M + N;
  const int64_t diag = b * tile_items < total ? b * tile_items : total;
  const int64_t split = merge_path_segments_coop<32>(seg_end, M, N, diag, threadIdx.x & 31, 0xffffffffu);
  if ((threadIdx.x & 31) == 0) splits[b] = (int32_t)split;
}

template <int THREADS, int IPT> struct ResidentLayout {
  static constexpr int TILE = THREADS * IPT;
  static constexpr int WARPS = THREADS / 32;
  static constexpr int kProdBytes = TILE * 8;
  static constexpr int kEndBytes = (TILE + 4) * 4;
  static constexpr int kScanBytes = WARPS * 16;
  static constexpr int kStageBytes = kProdBytes + kEndBytes + kScanBytes;    // multiple of 16
};

template <class T, int VC, int THREADS, int IPT>
__global__ void __launch_bounds__(VC *THREADS, 1)
seg_dot_resident_kernel(const SegDotArgs a, const int32_t *__restrict__ splits, int64_t x_len, int32_t x_bytes_padded) {
  using RL = ResidentLayout<THREADS, IPT>;
  constexpr int TILE = RL::TILE;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T *s_x = reinterpret_cast<T *>(smem_raw);
  const T *const val = static_cast<const T *>(a.val), *const x = static_cast<const T *>(a.x);
  for (int64_t i = threadIdx.x; i < x_len; i += VC * THREADS) s_x[i] = __ldg(x + i);
  __syncthreads();

  const int vc = threadIdx.x / THREADS, tid = threadIdx.x % THREADS;
  unsigned char *stage = smem_raw + x_bytes_padded + vc * RL::kStageBytes;
  double *s_prod = reinterpret_cast<double *>(stage);
  int32_t *s_end = reinterpret_cast<int32_t *>(stage + RL::kProdBytes);
  double *s_wval = reinterpret_cast<double *>(stage + RL::kProdBytes + RL::kEndBytes);
  int32_t *s_wkey = reinterpret_cast<int32_t *>(stage + RL::kProdBytes + RL::kEndBytes + RL::WARPS * 8);
  const NamedBarrier bar{1 + vc, THREADS};

  const int64_t total = a.M + a.N;
  const int64_t stride = (int64_t)gridDim.x * VC;
  int64_t t = (int64_t)blockIdx.x * VC + vc;

  // registers of the tile in flight
  int32_t c[IPT], e[IPT];
  double v[IPT];
  int64_t f_i0 = 0, f_i1 = 0, f_j0 = 0;
  int f_rows = 0, f_nnz = 0;
  // boundaries of the tile after it
  int32_t n_i0 = 0, n_i1 = 0;

  auto fetch = [&](int64_t tile, int32_t i0, int32_t i1) {     // issue the leaf loads of `tile`
    const int64_t d0 = tile * TILE;
    const int64_t d1 = (d0 + TILE < total) ? d0 + TILE : total;
    f_i0 = i0; f_i1 = i1; f_j0 = d0 - i0;
    f_rows = i1 - i0;
    f_nnz = (int)((d1 - i1) - f_j0);
#pragma unroll
    for (int k = 0; k < IPT; ++k) {
      const int tt = tid + k * THREADS;
      c[k] = 0; v[k] = 0.0; e[k] = 0;
      if (tt < f_nnz) { c[k] = ld_stream(a.crd + f_j0 + tt); v[k] = (double)ld_stream(val + f_j0 + tt); }
      if (tt < f_rows) e[k] = __ldg(a.seg_end + f_i0 + tt);
    }
  };

  if (t < a.num_tiles) fetch(t, __ldg(splits + t), __ldg(splits + t + 1));
  if (t + stride < a.num_tiles) { n_i0 = __ldg(splits + t + stride); n_i1 = __ldg(splits + t + stride + 1); }

  for (; t < a.num_tiles; t += stride) {
    // publish the fetched tile: products (vector element from shared memory) and tile-relative segment ends
    const int rows = f_rows, nnz = f_nnz;
    const int64_t i0 = f_i0, i1 = f_i1, j0 = f_j0;
#pragma unroll
    for (int k = 0; k < IPT; ++k) {
      const int tt = tid + k * THREADS;
      if (tt < nnz) s_prod[tt] = v[k] * (double)s_x[c[k]];
      if (tt < rows) s_end[tt] = (int32_t)((int64_t)e[k] - j0);
    }
    // the next tile's loads fly while this one is walked; its successor's boundaries follow
    if (t + stride < a.num_tiles) fetch(t + stride, n_i0, n_i1);
    if (t + 2 * stride < a.num_tiles) { n_i0 = __ldg(splits + t + 2 * stride); n_i1 = __ldg(splits + t + 2 * stride + 1); }
    bar();
    walk_staged_tile<T, THREADS, IPT>(a, s_end, s_prod, s_wkey, s_wval, tid, rows, nnz, i0, i1, t, bar);
    bar();                                               // the staging area may be overwritten
  }
}

// ------------------------------------------------------------------------------------------------
// The warp-stream variant: every warp owns a span of consecutive leaf entries and walks it 32 entries
// per step with fully coalesced loads; nothing is staged in shared memory except (optionally) the dense
// vector. Lanes accumulate private partial sums while no segment ends inside a step -- one DADD per 32
// entries, which is where the long fibers of a power-law tensor spend their time -- and only a step in
// which a segment ends pays for a segmented warp scan (shuffles) and the stores. The warp keeps the ends
// of the next 32 segments in registers (one per lane) and finds the ends that fall into a step with one
// REDUX.OR; a lane that owns a closing segment fetches that segment's sum from the lane holding its last
// entry. Segments are closed by the span that holds their last entry; the open partial of a span goes to
// a carry slot as in the other kernels (deterministic, no atomics).
template <class T, bool XSMEM>
__global__ void __launch_bounds__(1024, 1)
seg_dot_stream_kernel(const SegDotArgs a, int64_t x_len, int32_t span, unsigned long long *next_tile) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const T *s_x = reinterpret_cast<const T *>(smem_raw);
  const T *const val = static_cast<const T *>(a.val), *const x = static_cast<const T *>(a.x);
  T *const y = static_cast<T *>(a.y);
  if (XSMEM) {
    T *w = reinterpret_cast<T *>(smem_raw);
    for (int64_t i = threadIdx.x; i < x_len; i += blockDim.x) w[i] = __ldg(x + i);
    __syncthreads();
  }
  const unsigned full = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  auto xval = [&](int32_t c) -> double { return XSMEM ? (double)s_x[c] : (double)__ldg(x + c); };
  auto warp_sum = [&](double v) -> double {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(full, v, off);
    return v;
  };

  // Spans are handed out dynamically (one atomic per span): spans full of short segments take several times
  // longer than spans inside one long segment, and a static assignment leaves warps idle at the end.
  while (true) {
    int64_t tile = 0;
    if (lane == 0) tile = atomicAdd(next_tile, 1ull);
    tile = __shfl_sync(full, tile, 0);
    if (tile >= a.num_tiles) break;
    const int32_t w0 = (int32_t)(tile * span);
    const int32_t w1 = (int64_t)w0 + span < a.N ? w0 + span : (int32_t)a.N;
    const bool whole = w1 - w0 == span;                  // span is a multiple of 128: no bounds checks inside

    // open segment: the first one whose end lies beyond w0 (segments ending at w0 closed in the previous span)
    int64_t lo = 0, hi = a.M;
    while (lo < hi) {
      const int64_t stride = (hi - lo + 31) / 32;
      const int64_t q = lo + (int64_t)lane * stride + stride - 1;
      const bool inside = q < hi && __ldg(a.seg_end + q) <= w0;
      const int fullr = __popc(__ballot_sync(full, inside));
      lo += (int64_t)fullr * stride;
      const int64_t cap = lo + stride - 1;
      if (cap < hi) hi = cap;
    }
    int64_t s = lo;
    if (tile == 0)                                       // leading empty segments (end == 0) belong to nobody else
      for (int64_t q = lane; q < s; q += 32) y[a.out_row ? (int64_t)__ldg(a.out_row + q) : q] = (T)0;

    int32_t ew = (s + lane < a.M) ? __ldg(a.seg_end + s + lane) : 0x7fffffff;   // ends of the next 32 segments
    int32_t last_end = w0;                               // end of the most recently closed segment
    double run = 0.0;                                    // this lane's share of the open segment's sum

    for (int32_t j0 = w0; j0 < w1; j0 += 128) {          // four steps per round: their loads are issued together
      int32_t c[4];
      double v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int32_t jj = j0 + u * 32 + lane;
        c[u] = 0; v[u] = 0.0;
        if (whole || jj < w1) { c[u] = ld_stream(a.crd + jj); v[u] = (double)ld_stream(val + jj); }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int32_t j = j0 + u * 32;
        if (!whole && j >= w1) break;
        const double p = (whole || j + lane < w1) ? v[u] * xval(c[u]) : 0.0;
        const int32_t top = (whole || j + 32 < w1) ? j + 32 : w1;   // segments with an end in (j, top] close in this step
        if (!__any_sync(full, ew <= top)) { run += p; continue; }

        // every end that falls into this step, as a bit per position (more than the 32 cached ends may)
        unsigned endbits = __reduce_or_sync(full, ew <= top ? 1u << (ew - j - 1) : 0u);
        if (__all_sync(full, ew <= top)) {
          for (int64_t more = s + 32;; more += 32) {
            const int32_t e2 = (more + lane < a.M) ? __ldg(a.seg_end + more + lane) : 0x7fffffff;
            endbits |= __reduce_or_sync(full, e2 <= top ? 1u << (e2 - j - 1) : 0u);
            if (!__all_sync(full, e2 <= top)) break;
          }
        }
        // inclusive segmented scan of p; a new sub-sum starts after every end position
        const unsigned heads = (endbits << 1) | 1u;
        const int dist = lane - (31 - __clz(heads & (0xffffffffu >> (31 - lane))));   // entries since the sub-sum started
        double sc = p;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const double t = __shfl_up_sync(full, sc, off);
          if (off <= dist) sc += t;
        }
        const int firstb = __ffs(endbits) - 1, lastb = 31 - __clz(endbits);
        const double tot = warp_sum(run);                // what earlier steps hold for the segment closed first
        run = lane > lastb ? p : 0.0;                    // entries behind the last end open the next segment

        while (true) {                                   // emit: each lane owns the segment whose end it caches
          const bool closing = ew <= top;
          const unsigned cm = __ballot_sync(full, closing);
          if (cm == 0) break;
          const int src = closing ? ew - j - 1 : 0;
          double segsum = __shfl_sync(full, sc, src);
          int32_t prev = __shfl_up_sync(full, ew, 1);
          if (lane == 0) prev = last_end;
          if (closing) {
            if (ew == prev) segsum = 0.0;                // an empty segment: its end repeats its predecessor's
            else if (src == firstb) segsum += tot;
            const int64_t seg = s + lane;
            y[a.out_row ? (int64_t)__ldg(a.out_row + seg) : seg] = (T)segsum;
          }
          const int k = __popc(cm);                      // closing lanes are a prefix: ends are sorted
          last_end = __shfl_sync(full, ew, k - 1);
          s += k;
          ew = (s + lane < a.M) ? __ldg(a.seg_end + s + lane) : 0x7fffffff;
        }
      }
    }
    const double open = warp_sum(run);
    if (lane == 0) {
      a.carry_seg[tile] = s < a.M ? (int32_t)s : -1;
      a.carry_val[tile] = open;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// The same walk with 64 entries per step: lane l owns entries 2l and 2l+1 of the step (one 8-byte and one
// 16-byte load per step and lane), so a step that contains a segment end -- the expensive kind: segmented
// scan, warp sum of the private partials, stores -- pays for 64 entries instead of 32. Inside a lane the
// pair is summed before the scan unless a segment ends between its two entries; a lane then contributes a
// "tail" (the sub-sum still open at its second entry, which the lane-level scan extends) and, if a segment
// ends at its first entry, a "head" sum (its first product plus the tail of the lane before it).
#ifndef COMET_STREAM2_STEPS
#define COMET_STREAM2_STEPS 3      // 64-entry steps whose loads are issued together (4 spills registers)
#endif
template <class T> struct Pair2;
template <> struct Pair2<double> {
  static __device__ __forceinline__ void load(const double *p, double &a, double &b) {
    const double2 t = __ldcs(reinterpret_cast<const double2 *>(p));
    a = t.x; b = t.y;
  }
};
template <> struct Pair2<float> {
  static __device__ __forceinline__ void load(const float *p, double &a, double &b) {
    const float2 t = __ldcs(reinterpret_cast<const float2 *>(p));
    a = (double)t.x; b = (double)t.y;
  }
};

template <class T, bool XSMEM>
__global__ void __launch_bounds__(1024, 1)
seg_dot_stream2_kernel(const SegDotArgs a, int64_t x_len, int32_t span, unsigned long long *next_tile,
                       unsigned int *ctas_done) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const T *s_x = reinterpret_cast<const T *>(smem_raw);
  const T *const val = static_cast<const T *>(a.val), *const x = static_cast<const T *>(a.x);
  T *const y = static_cast<T *>(a.y);
  if (XSMEM) {
    T *w = reinterpret_cast<T *>(smem_raw);
    for (int64_t i = threadIdx.x; i < x_len; i += blockDim.x) w[i] = __ldg(x + i);
    __syncthreads();
  }
  const unsigned full = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  auto xval = [&](int32_t c) -> double { return XSMEM ? (double)s_x[c] : (double)__ldg(x + c); };
  auto warp_sum = [&](double v) -> double {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(full, v, off);
    return v;
  };

  while (true) {
    int64_t tile = 0;
    if (lane == 0) tile = atomicAdd(next_tile, 1ull);
    tile = __shfl_sync(full, tile, 0);
    if (tile >= a.num_tiles) break;
    const int32_t w0 = (int32_t)(tile * span);
    const int32_t w1 = (int64_t)w0 + span < a.N ? w0 + span : (int32_t)a.N;
    const bool whole = w1 - w0 == span && span % (64 * COMET_STREAM2_STEPS) == 0;   // full rounds only: no bounds checks inside

    int64_t lo = 0, hi = a.M;                            // open segment: the first one whose end lies beyond w0
    while (lo < hi) {
      const int64_t stride = (hi - lo + 31) / 32;
      const int64_t q = lo + (int64_t)lane * stride + stride - 1;
      const bool inside = q < hi && __ldg(a.seg_end + q) <= w0;
      const int fullr = __popc(__ballot_sync(full, inside));
      lo += (int64_t)fullr * stride;
      const int64_t cap = lo + stride - 1;
      if (cap < hi) hi = cap;
    }
    int64_t s = lo;
    if (tile == 0)
      for (int64_t q = lane; q < s; q += 32) y[a.out_row ? (int64_t)__ldg(a.out_row + q) : q] = (T)0;

    // ends of the next 32 segments, and of the 32 after them: closing k segments shifts the window by k with
    // shuffles, and the load that refills the far half is not waited for until the shift after
    int32_t ew = (s + lane < a.M) ? __ldg(a.seg_end + s + lane) : 0x7fffffff;
    int32_t ew2 = (s + 32 + lane < a.M) ? __ldg(a.seg_end + s + 32 + lane) : 0x7fffffff;
    int32_t last_end = w0;
    double run = 0.0;

    for (int32_t j0 = w0; j0 < w1; j0 += 64 * COMET_STREAM2_STEPS) {   // the loads of a round's steps are issued together
      int32_t c[COMET_STREAM2_STEPS][2];
      double v[COMET_STREAM2_STEPS][2];
#pragma unroll
      for (int u = 0; u < COMET_STREAM2_STEPS; ++u) {
        const int32_t jj = j0 + u * 64 + 2 * lane;
        if (whole) {
          const int2 cc = __ldcs(reinterpret_cast<const int2 *>(a.crd + jj));
          c[u][0] = cc.x; c[u][1] = cc.y;
          Pair2<T>::load(val + jj, v[u][0], v[u][1]);
        } else {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            c[u][h] = 0; v[u][h] = 0.0;
            if (jj + h < w1) { c[u][h] = ld_stream(a.crd + jj + h); v[u][h] = (double)ld_stream(val + jj + h); }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < COMET_STREAM2_STEPS; ++u) {
        const int32_t j = j0 + u * 64;
        if (!whole && j >= w1) break;
        const int32_t q0 = j + 2 * lane;
        const double p0 = (whole || q0 < w1) ? v[u][0] * xval(c[u][0]) : 0.0;
        const double p1 = (whole || q0 + 1 < w1) ? v[u][1] * xval(c[u][1]) : 0.0;
        const int32_t top = (whole || j + 64 < w1) ? j + 64 : w1;   // segments with an end in (j, top] close in this step
        if (!__any_sync(full, ew <= top)) { run += p0 + p1; continue; }

        // every end that falls into this step, as one bit per entry position (64 of them)
        unsigned elo, ehi;
        {
          const bool closing = ew <= top;
          const int b = ew - j - 1;
          elo = __reduce_or_sync(full, (closing && b < 32) ? 1u << b : 0u);
          ehi = __reduce_or_sync(full, (closing && b >= 32) ? 1u << (b - 32) : 0u);
          if (__all_sync(full, closing)) {
            for (int64_t more = s + 32;; more += 32) {
              const int32_t e2 = (more + lane < a.M) ? __ldg(a.seg_end + more + lane) : 0x7fffffff;
              const bool c2 = e2 <= top;
              const int b2 = e2 - j - 1;
              elo |= __reduce_or_sync(full, (c2 && b2 < 32) ? 1u << b2 : 0u);
              ehi |= __reduce_or_sync(full, (c2 && b2 >= 32) ? 1u << (b2 - 32) : 0u);
              if (!__all_sync(full, c2)) break;
            }
          }
        }
        const unsigned long long endbits = (unsigned long long)elo | ((unsigned long long)ehi << 32);
        const bool e0 = (endbits >> (2 * lane)) & 1ull, e1 = (endbits >> (2 * lane + 1)) & 1ull;
        const unsigned E0 = __ballot_sync(full, e0), E1 = __ballot_sync(full, e1);
        // lane-level scan of the tails: a lane starts a fresh sub-sum when a segment ends at its first entry
        // or at the second entry of the lane before it
        const unsigned heads = E0 | (E1 << 1) | 1u;
        const int dist = lane - (31 - __clz(heads & (0xffffffffu >> (31 - lane))));
        double sc = e0 ? p1 : p0 + p1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const double t = __shfl_up_sync(full, sc, off);
          if (off <= dist) sc += t;
        }
        // sum of the segment that ends at this lane's FIRST entry: that product plus what the lane before left open
        const double before = __shfl_up_sync(full, sc, 1);
        const double hd = p0 + ((lane > 0 && !((E1 >> (lane - 1)) & 1u)) ? before : 0.0);
        const int firstb = elo ? __ffs(elo) - 1 : 32 + __ffs(ehi) - 1;
        const int lastb = ehi ? 63 - __clz(ehi) : 31 - __clz(elo);
        const double tot = warp_sum(run);                // what earlier steps hold for the segment closed first
        run = (2 * lane > lastb ? p0 : 0.0) + (2 * lane + 1 > lastb ? p1 : 0.0);   // entries behind the last end

        while (true) {                                   // emit: each lane owns the segment whose end it caches
          const bool closing = ew <= top;
          const unsigned cm = __ballot_sync(full, closing);
          const int b = closing ? ew - j - 1 : 0;
          const double tail = __shfl_sync(full, sc, b >> 1), head = __shfl_sync(full, hd, b >> 1);
          double segsum = (b & 1) ? tail : head;
          int32_t prev = __shfl_up_sync(full, ew, 1);
          if (lane == 0) prev = last_end;
          if (closing) {
            if (ew == prev) segsum = 0.0;                // an empty segment: its end repeats its predecessor's
            else if (b == firstb) segsum += tot;
            const int64_t seg = s + lane;
            y[a.out_row ? (int64_t)__ldg(a.out_row + seg) : seg] = (T)segsum;
          }
          const int k = __popc(cm);                      // closing lanes are a prefix: ends are sorted; k >= 1
          last_end = __shfl_sync(full, ew, k - 1);
          s += k;
          // shift the window by k: lanes take the end k places up, from this window or from the next one
          const int from = lane + k;
          const int32_t near = __shfl_sync(full, ew, from & 31), far = __shfl_sync(full, ew2, from & 31);
          ew = from < 32 ? near : far;
          const int32_t fresh = (s + 32 + lane < a.M) ? __ldg(a.seg_end + s + 32 + lane) : 0x7fffffff;
          ew2 = fresh;
          if (k < 32) break;                             // lane k's end lies beyond this step: nothing more closes
          if (!__any_sync(full, ew <= top)) break;
        }
      }
    }
    const double open = warp_sum(run);
    if (lane == 0) {
      a.carry_seg[tile] = s < a.M ? (int32_t)s : -1;
      a.carry_val[tile] = open;
    }
  }

  // The CTA that finishes last puts the two counters back to zero, the state the next call on this handle
  // expects (no CTA waits for another: each one counts itself done and leaves). This spares a memset per call.
  __syncthreads();
  if (threadIdx.x == 0 && atomicAdd(ctas_done, 1u) == gridDim.x - 1) { *next_tile = 0ull; *ctas_done = 0u; }
}

template <class T, int THREADS, int IPT>
static comet_status_t launch_dot(Context *ctx, SegDotArgs a, cudaStream_t stream) {
  const int64_t total = a.M + a.N;
  a.num_tiles = ceil_div(total, (int64_t)THREADS * IPT);
  const size_t val_bytes = align_up((size_t)a.num_tiles * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  // up to a few thousand tiles the last CTA adds the carries itself: one launch instead of two
  const bool fused = a.num_tiles > 1 && a.num_tiles <= 4096;
  a.ctas_done = fused ? reinterpret_cast<unsigned int *>(ctx->d_status + 35) : nullptr;
  seg_dot_kernel<T, THREADS, IPT><<<(unsigned)a.num_tiles, THREADS, 0, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
  if (a.num_tiles > 1 && !fused) {
    carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, 1, 1, a.y, 1,
                       a.out_row, stream);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}

#ifndef COMET_RES_VC
#define COMET_RES_VC 8          // virtual CTAs per persistent CTA (measured best: 8 x 128 threads x 5 items)
#define COMET_RES_THREADS 128
#define COMET_RES_IPT 5
#endif
constexpr int kResVC = COMET_RES_VC, kResThreads = COMET_RES_THREADS, kResIpt = COMET_RES_IPT;
constexpr size_t kMaxDynamicSmem = 232448;               // 227 KB opt-in limit per CTA on sm_100

template <class T>
static comet_status_t launch_resident(Context *ctx, SegDotArgs a, int64_t x_len, cudaStream_t stream) {
  using RL = ResidentLayout<kResThreads, kResIpt>;
  const int64_t total = a.M + a.N;
  a.num_tiles = ceil_div(total, (int64_t)RL::TILE);
  const size_t val_bytes = align_up((size_t)a.num_tiles * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  const size_t split_bytes = align_up((size_t)(a.num_tiles + 1) * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes + split_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  int32_t *splits = (int32_t *)(scratch + val_bytes + seg_bytes);
  tile_split_kernel<<<(unsigned)ceil_div((a.num_tiles + 1) * 32, 256), 256, 0, stream>>>(a.seg_end, a.M, a.N, RL::TILE,
                                                                                       a.num_tiles, splits);
  COMET_LAUNCH_CHECK(ctx);
  const int32_t x_bytes = (int32_t)align_up((size_t)x_len * sizeof(T), 16);
  const size_t smem = (size_t)x_bytes + (size_t)kResVC * RL::kStageBytes;
  auto kernel = seg_dot_resident_kernel<T, kResVC, kResThreads, kResIpt>;
  COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int64_t ctas = ceil_div(a.num_tiles, kResVC) < kSmCount ? ceil_div(a.num_tiles, kResVC) : kSmCount;
  kernel<<<(unsigned)ctas, kResVC * kResThreads, smem, stream>>>(a, splits, x_len, x_bytes);
  COMET_LAUNCH_CHECK(ctx);
  carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, 1, 1, a.y, 1,
                     a.out_row, stream);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

template <class T>
static comet_status_t launch_stream(Context *ctx, SegDotArgs a, int64_t x_len, bool pairs, cudaStream_t stream) {
  const size_t x_bytes = align_up((size_t)x_len * sizeof(T), 16);
  const bool xsmem = x_bytes <= kMaxDynamicSmem - 1024;
  // the two-entries-per-lane kernel loads pairs with one instruction: the arrays must be aligned for that
  pairs = pairs && (reinterpret_cast<uintptr_t>(a.crd) % 8 == 0) && (reinterpret_cast<uintptr_t>(a.val) % (2 * sizeof(T)) == 0);
  // spans: whole rounds of the kernel (128 entries, or 64 per step of the pair kernel), several per warp of the
  // 148 persistent CTAs so that the tail is short
  const int64_t round = pairs ? 64 * COMET_STREAM2_STEPS : 128;
  const int64_t warps = (int64_t)kSmCount * 32;
  int64_t span = ceil_div(ceil_div(a.N, warps * 10), round) * round;
  if (span < 4 * round) span = 4 * round;
  if (span > 2048 / round * round) span = 2048 / round * round;
  if (const char *e = getenv("COMET_STREAM_SPAN")) { const int v = atoi(e); if (v >= 128 && v % 128 == 0) span = v; }
  a.num_tiles = ceil_div(a.N, span);
  const size_t val_bytes = align_up((size_t)a.num_tiles * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes + 256, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  const int64_t ctas = ceil_div(a.num_tiles, 32) < kSmCount ? ceil_div(a.num_tiles, 32) : kSmCount;
  if (pairs) {
    // span counter and finished-CTA counter live in the handle and are zero between calls (the kernel's last
    // CTA resets them): no memset
    unsigned long long *next_tile = reinterpret_cast<unsigned long long *>(ctx->d_status + 32);
    unsigned int *ctas_done = reinterpret_cast<unsigned int *>(ctx->d_status + 34);
    if (xsmem) {
      auto kernel = seg_dot_stream2_kernel<T, true>;
      COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x_bytes));
      kernel<<<(unsigned)ctas, 1024, x_bytes, stream>>>(a, x_len, (int32_t)span, next_tile, ctas_done);
    } else {
      seg_dot_stream2_kernel<T, false><<<(unsigned)ctas, 1024, 0, stream>>>(a, x_len, (int32_t)span, next_tile, ctas_done);
    }
    COMET_LAUNCH_CHECK(ctx);
    carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, 1, 1, a.y, 1,
                       a.out_row, stream);
    COMET_LAUNCH_CHECK(ctx);
    return COMET_OK;
  }
  unsigned long long *next_tile = (unsigned long long *)(scratch + val_bytes + seg_bytes);
  COMET_CUDA_TRY(ctx, cudaMemsetAsync(next_tile, 0, sizeof(unsigned long long), stream));
  if (xsmem) {
    auto kernel = seg_dot_stream_kernel<T, true>;
    COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x_bytes));
    kernel<<<(unsigned)ctas, 1024, x_bytes, stream>>>(a, x_len, (int32_t)span, next_tile);
  } else {
    seg_dot_stream_kernel<T, false><<<(unsigned)ctas, 1024, 0, stream>>>(a, x_len, (int32_t)span, next_tile);
  }
  COMET_LAUNCH_CHECK(ctx);
  carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, 1, 1, a.y, 1,
                     a.out_row, stream);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

template <class T>
static comet_status_t seg_dot_typed(Context *ctx, int dtype, const int32_t *seg_end, const int32_t *crd, const void *val,
                                    int64_t M, int64_t N, const void *x, int64_t x_len, void *y, const int32_t *out_row,
                                    int64_t out_rows, cudaStream_t stream) {
  if (out_row) {
    comet_status_t st = zero_rows(ctx, y, dtype, out_rows, 1, 1, stream);
    if (st != COMET_OK) return st;
  }
  if (M == 0) return COMET_OK;
  SegDotArgs a{};
  a.seg_end = seg_end; a.crd = crd; a.val = val; a.M = M; a.N = N; a.x = x; a.y = y; a.out_row = out_row;
  // Large problems: the warp-stream kernel (x in shared memory when it fits).
  {
    const char *force = getenv("COMET_SEG_DOT_KERNEL");   // tests: "stream", "resident" or "tile" on any input
    // tests force a kernel on any input: "stream" (32 entries per step), "stream2" (64), "resident" or "tile"
    const bool want_stream = force ? !strncmp(force, "stream", 6) : (N >= (int64_t)kSmCount * 32 * 512 && N > 0);
    // many more segments than entries (hypersparse CSR): segment ends dominate, and the 32-entry kernel closes them cheaper
    const bool pairs = force ? !strcmp(force, "stream2") : M <= N;
    if (want_stream && N > 0) return launch_stream<T>(ctx, a, x_len, pairs, stream);
  }
  // Mid-size problems whose vector fits in shared memory beside the staging: persistent CTAs, x resident.
  {
    using RL = ResidentLayout<kResThreads, kResIpt>;
    const size_t need = align_up((size_t)x_len * sizeof(T), 16) + (size_t)kResVC * RL::kStageBytes;
    const char *force = getenv("COMET_SEG_DOT_KERNEL");
    const bool forced = force && !strcmp(force, "resident");
    if (need <= kMaxDynamicSmem && (forced || M + N >= (int64_t)kSmCount * kResVC * RL::TILE * 8))
      return launch_resident<T>(ctx, a, x_len, stream);
  }
  // Items per thread are odd so that the per-thread walks (stride IPT doubles across lanes) hit all
  // shared-memory banks; an even stride of 8 serialises them 16 ways. Small problems get short tiles so
  // that the grid still covers the 148 SMs.
  if (M + N < (int64_t)kSmCount * 2048 * 2) return launch_dot<T, 128, 5>(ctx, a, stream);
  return launch_dot<T, 256, 9>(ctx, a, stream);
}

comet_status_t seg_dot(Context *ctx, int dtype, const int32_t *seg_end, const int32_t *crd, const void *val, int64_t M,
                       int64_t N, const void *x, int64_t x_len, void *y, const int32_t *out_row, int64_t out_rows,
                       cudaStream_t stream) {
  if (dtype == COMET_F32)
    return seg_dot_typed<float>(ctx, dtype, seg_end, crd, val, M, N, x, x_len, y, out_row, out_rows, stream);
  return seg_dot_typed<double>(ctx, dtype, seg_end, crd, val, M, N, x, x_len, y, out_row, out_rows, stream);
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
  if (M < 0 || N < 0) return COMET_ERR_INVALID_ARG;
  if (M + N > kStaticMaxItems) return COMET_ERR_WORKSPACE;      // beyond the fixed scratch: use comet_spmv
  if (!A->pos[1] || A->pos_len[1] != M + 1 || (N > 0 && (!A->crd[1] || !A->val))) return COMET_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 7) || (reinterpret_cast<uintptr_t>(y) & 7)) return COMET_ERR_MISALIGNED;
  if (M == 0) return COMET_OK;

  void *scratch = nullptr;
  const comet_status_t st = static_scratch_address(&scratch);
  if (st != COMET_OK) return st;

  SegDotArgs a{};
  a.seg_end = A->pos[1] + 1; a.crd = A->crd[1]; a.val = A->val;
  a.M = M; a.N = N; a.x = x; a.y = y; a.out_row = nullptr;
  a.num_tiles = ceil_div(M + N, (int64_t)kStaticThreads * kStaticIpt);
  a.carry_val = (double *)scratch;                               // every tile writes its slot before the
  a.carry_seg = (int32_t *)((char *)scratch + kStaticValBytes);  // fix-up reads it: nothing to clear
  cudaStream_t s = (cudaStream_t)stream;
  seg_dot_kernel<double, kStaticThreads, kStaticIpt><<<(unsigned)a.num_tiles, kStaticThreads, 0, s>>>(a);
  if (a.num_tiles > 1)
    carry_fixup_launch(COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, 1, 1, y, 1, nullptr, s);
  if (cudaGetLastError() != cudaSuccess) return COMET_ERR_CUDA;
  return COMET_OK;
}
