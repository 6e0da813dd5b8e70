// SpMM, long rows by column phases (the SpMM definition of the paper's Sparse Tensor Operations subsection;
// the paper's evaluation names locality of the dense operand and load imbalance as what decides SpMM).
//
// When B is much larger than the L2 cache, every gathered row of B comes from DRAM and the product moves
// nnz * R * 8 bytes instead of reading B once. The entries of a LONG row are the place where that can be
// avoided: a CSR row's column indices ascend, so the part of a row that falls into a block of consecutive
// columns is a contiguous piece of the row, found by a binary search. The long rows are cut into such pieces,
// the pieces into tiles of at most tile_max entries, and the tiles are processed block by block: while block b
// is being worked on, the rows b * block_cols .. of B (a few tens of MB) stay in L2 and are read from DRAM
// about once. A tile lies inside ONE row, so its worker has no segment bookkeeping at all: it keeps a deep
// window of row gathers in flight, adds up, and writes its partial sum to a slot. The slots of a row are
// consecutive and are added in slot order by the fix-up kernel, which WRITES the row of C (deterministic, no
// atomics, no memset). The short rows go through the general kernel, which skips the long ones.
//
// Everything is computed on the device on every call, without a synchronisation; the host sizes the scratch
// by upper bounds (a row of len entries is cut into at most len / piece_target blocks and ceil(len / tile_max)
// + blocks tiles).
#include <stdlib.h>

#include "common.cuh"
#include "kernels.cuh"
#include "spmm_heavy.cuh"

namespace comet {

constexpr int kScanRows = 8;                         // rows per thread of the row-scan kernels
constexpr int kScanCta = kBlockThreads * kScanRows;  // rows per CTA


__device__ __forceinline__ int32_t blocks_of(int32_t len, const HeavyArgs &a) {
  int32_t nb = len / a.piece_target;
  if (nb < 1) nb = 1;
  if (nb > a.P) nb = a.P;
  return 1 << (31 - __clz(nb));                      // power of two, so that it divides P
}
__device__ __forceinline__ int32_t slots_of(int32_t len, const HeavyArgs &a) {
  return (len + a.tile_max - 1) / a.tile_max + blocks_of(len, a);
}

// Exclusive scan of one int per thread over the CTA (256 threads); returns the CTA total in `total`.
__device__ __forceinline__ int32_t block_scan(int32_t v, int32_t &total, int32_t *warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int32_t t = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += t;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int32_t before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kBlockThreads / 32; ++w) {
    const int32_t s = warp_sums[w];
    if (w < warp) before += s;
    all += s;
  }
  __syncthreads();
  total = all;
  return before + inc - v;
}

// The CTA that takes the last ticket turns the per-CTA counts into exclusive offsets (in place).
__device__ void scan_cta_counts(const HeavyArgs &a, int32_t *warp_sums) {
  int32_t run_rows = 0, run_slots = 0;
  for (int32_t base = 0; base < a.num_scan_ctas; base += kBlockThreads) {
    const int32_t i = base + threadIdx.x;
    const int32_t r = i < a.num_scan_ctas ? __ldcg(a.cta_rows + i) : 0;
    const int32_t s = i < a.num_scan_ctas ? __ldcg(a.cta_slots + i) : 0;
    int32_t tr, ts;
    const int32_t er = block_scan(r, tr, warp_sums);
    const int32_t es = block_scan(s, ts, warp_sums);
    if (i < a.num_scan_ctas) { a.cta_rows[i] = run_rows + er; a.cta_slots[i] = run_slots + es; }
    run_rows += tr;
    run_slots += ts;
  }
  if (threadIdx.x == 0) { a.counters[0] = run_rows; a.counters[1] = run_slots; a.counters[3] = 0; a.counters[5] = 0; }
  if (threadIdx.x < 3 * a.P) a.bin[threadIdx.x] = 0;
}

// Pass 1 over the rows: long rows and reserved slots per CTA.
__global__ void __launch_bounds__(kBlockThreads) heavy_count_kernel(const HeavyArgs a) {
  __shared__ int32_t warp_sums[kBlockThreads / 32];
  __shared__ int32_t is_last;
  const int64_t r0 = (int64_t)blockIdx.x * kScanCta + (int64_t)threadIdx.x * kScanRows;
  int32_t cnt = 0, slots = 0;
  if (r0 < a.M) {
    int32_t prev = __ldg(a.pos + r0);
#pragma unroll
    for (int k = 0; k < kScanRows; ++k) {
      if (r0 + k < a.M) {
        const int32_t nxt = __ldg(a.pos + r0 + k + 1);
        const int32_t len = nxt - prev;
        if (len >= a.threshold) { ++cnt; slots += slots_of(len, a); }
        prev = nxt;
      }
    }
  }
  int32_t tc, ts;
  block_scan(cnt, tc, warp_sums);
  block_scan(slots, ts, warp_sums);
  if (threadIdx.x == 0) {
    a.cta_rows[blockIdx.x] = tc;
    a.cta_slots[blockIdx.x] = ts;
    __threadfence();
    is_last = atomicAdd(a.counters + 3, 1) == a.num_scan_ctas - 1;
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    scan_cta_counts(a, warp_sums);
  }
}

// Pass 2: numbers the long rows in ascending order, cuts each into its pieces (one binary search per block
// boundary, a warp per row) and counts the tiles of every phase.
__global__ void __launch_bounds__(kBlockThreads) heavy_pieces_kernel(const HeavyArgs a) {
  if ((int)blockIdx.x >= a.num_scan_ctas) {                    // second role: a thread per boundary of the general tiles
    const int64_t t = (int64_t)(blockIdx.x - a.num_scan_ctas) * kBlockThreads + threadIdx.x;
    if (t > a.part_tiles) return;
    const int64_t total = a.part_M + a.part_N;
    const int64_t d = t * a.part_tile_items < total ? t * a.part_tile_items : total;
    a.part[t] = (int32_t)merge_path_segments(a.part_seg_end, a.part_M, a.part_N, d);
    return;
  }
  __shared__ int32_t warp_sums[kBlockThreads / 32];
  __shared__ int32_t local_h[kScanCta];
  __shared__ int32_t local_n, is_last;
  const int64_t r0 = (int64_t)blockIdx.x * kScanCta + (int64_t)threadIdx.x * kScanRows;
  int32_t len[kScanRows];
  int32_t cnt = 0, slots = 0;
#pragma unroll
  for (int k = 0; k < kScanRows; ++k) len[k] = 0;
  if (r0 < a.M) {
    int32_t prev = __ldg(a.pos + r0);
#pragma unroll
    for (int k = 0; k < kScanRows; ++k) {
      if (r0 + k < a.M) {
        const int32_t nxt = __ldg(a.pos + r0 + k + 1);
        len[k] = nxt - prev;
        if (len[k] >= a.threshold) { ++cnt; slots += slots_of(len[k], a); }
        prev = nxt;
      }
    }
  }
  int32_t tc, ts;
  int32_t my_h = block_scan(cnt, tc, warp_sums);
  int32_t my_slot = block_scan(slots, ts, warp_sums) + __ldcg(a.cta_slots + blockIdx.x);
  const int32_t h_base = __ldcg(a.cta_rows + blockIdx.x);
#pragma unroll
  for (int k = 0; k < kScanRows; ++k) {
    if (len[k] >= a.threshold) {
      const int32_t h = h_base + my_h;
      a.hrow[h] = (int32_t)(r0 + k);
      a.row_slot0[h] = my_slot;
      local_h[my_h] = h;
      ++my_h;
      my_slot += slots_of(len[k], a);
    }
  }
  if (threadIdx.x == 0) local_n = tc;
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int32_t i = warp; i < local_n; i += kBlockThreads / 32) {
    const int32_t h = local_h[i];
    const int32_t row = a.hrow[h];
    const int32_t s = __ldg(a.pos + row), e = __ldg(a.pos + row + 1);
    const int32_t nb = blocks_of(e - s, a);
    const int32_t fine = a.P / nb;                            // blocks of B per piece of this row
    int32_t start = e;
    if (lane < nb) {                                          // first entry with column >= the piece's first column
      const int64_t want = (int64_t)lane * fine * a.block_cols;
      // eight-way search: seven probes per round, all in flight together (the row is cold, so a round costs one
      // memory latency whatever it loads; 5 rounds instead of 14 for a row of 10,000 entries)
      int32_t lo = s, hi = e;
      while (hi - lo > 8) {
        const int32_t step = (hi - lo) >> 3;
        int32_t probe[7];
#pragma unroll
        for (int u = 0; u < 7; ++u) probe[u] = __ldg(a.crd + lo + (u + 1) * step);
        int32_t below = 0;                                   // probes whose column is below the target (they ascend)
#pragma unroll
        for (int u = 0; u < 7; ++u) below += (int64_t)probe[u] < want ? 1 : 0;
        const int32_t nlo = below ? lo + below * step + 1 : lo;
        hi = below < 7 ? lo + (below + 1) * step : hi;
        lo = nlo;
      }
      while (lo < hi && (int64_t)__ldg(a.crd + lo) < want) ++lo;
      start = lo;
    }
    int32_t nxt = __shfl_down_sync(0xffffffffu, start, 1);
    if (lane == 31 || lane + 1 >= nb) nxt = e;
    const int32_t nt = lane < nb ? (nxt - start + a.tile_max - 1) / a.tile_max : 0;
    int32_t inc = nt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t t = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += t;
    }
    if (lane <= nb) a.piece_start[(int64_t)h * (a.P + 1) + lane] = start;   // lane nb holds e
    if (lane == 31) a.row_nt[h] = inc;
    if (nt > 0) atomicAdd(a.bin + lane * fine, nt);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    is_last = atomicAdd(a.counters + 4, 1) == a.num_scan_ctas - 1;
  }
  __syncthreads();
  if (is_last && threadIdx.x == 0) {
    __threadfence();
    int32_t run = 0;
    for (int32_t b = 0; b < a.P; ++b) {
      a.bin[a.P + b] = run;
      run += __ldcg(a.bin + b);
    }
    a.counters[2] = run;
    a.counters[4] = 0;
  }
}

// Pass 3 (a warp per long row, grid-stride): writes the tile records of the row into its phases.
__global__ void __launch_bounds__(kBlockThreads) heavy_tiles_kernel(const HeavyArgs a) {
  const int lane = threadIdx.x & 31;
  const int32_t H = __ldcg(a.counters + 0);
  const int32_t warps = gridDim.x * (kBlockThreads / 32);
  for (int32_t h = blockIdx.x * (kBlockThreads / 32) + (threadIdx.x >> 5); h < H; h += warps) {
    const int32_t row = a.hrow[h];
    const int32_t s = __ldg(a.pos + row), e = __ldg(a.pos + row + 1);
    const int32_t nb = blocks_of(e - s, a);
    const int32_t fine = a.P / nb;
    const int32_t start = lane <= nb ? a.piece_start[(int64_t)h * (a.P + 1) + lane] : e;
    int32_t nxt = __shfl_down_sync(0xffffffffu, start, 1);
    if (lane == 31 || lane + 1 > nb) nxt = e;
    const int32_t nt = lane < nb ? (nxt - start + a.tile_max - 1) / a.tile_max : 0;
    int32_t inc = nt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t t = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += t;
    }
    if (nt > 0) {
      const int32_t phase = lane * fine;
      const int32_t at = __ldcg(a.bin + a.P + phase) + atomicAdd(a.bin + 2 * a.P + phase, nt);
      const int32_t slot = a.row_slot0[h] + inc - nt;
      for (int32_t t = 0; t < nt; ++t) {
        const int32_t j0 = start + t * a.tile_max;
        const int32_t j1 = j0 + a.tile_max < nxt ? j0 + a.tile_max : nxt;
        a.rec[at + t] = make_int4(j0, j1, slot + t, row);
      }
    }
  }
}

static int env_int(const char *name, int dflt) {
  const char *e = getenv(name);
  return e ? atoi(e) : dflt;
}

size_t spmm_heavy_plan(int dtype, int64_t M, int64_t N, int64_t cols, const void *B, int64_t ldb, int64_t R, const void *C,
                       int64_t ldc, int32_t min_threshold, HeavyArgs *out) {
  const size_t elt = dtype == COMET_F32 ? 4 : 8;
  const size_t row_bytes = (size_t)R * elt;
  // Tuning variables (read on every call, so that a test can force the path on a small matrix).
  const int enabled = env_int("COMET_SPMM_LONG_ROWS", 1);
  const int block_mb = env_int("COMET_SPMM_BLOCK_MB", 32);            // target size of a block of B
  const int env_threshold = env_int("COMET_SPMM_LONG_ROW", 512);      // entries that make a row long
  const int env_tile = env_int("COMET_SPMM_LONG_TILE", 128);          // entries per tile of a long row
  const int env_piece = env_int("COMET_SPMM_PIECE", 64);              // a row of len entries is cut into <= len / this blocks
  const int env_ctas = env_int("COMET_SPMM_LONG_CTAS", 3 * kSmCount / 2);
  const int64_t min_nnz = env_int("COMET_SPMM_LONG_MIN_NNZ", 1 << 20);
  const size_t min_b_mb = (size_t)env_int("COMET_SPMM_LONG_MIN_B_MB", 96);   // below: B (nearly) fits in L2, nothing to gain
  if (!enabled || cols <= 0 || M <= 0 || N < min_nnz) return 0;
  if (row_bytes != 256 && row_bytes != 512 && row_bytes != 1024) return 0;   // the vector shapes that carry the role
  const size_t b_bytes = (size_t)cols * row_bytes;
  if (b_bytes < (min_b_mb << 20)) return 0;
  if ((reinterpret_cast<uintptr_t>(B) & 15) || (reinterpret_cast<uintptr_t>(C) & 15) || (ldb * elt) % 16 || (ldc * elt) % 16)
    return 0;

  HeavyArgs a{};
  a.M = M; a.N = N; a.cols = cols;
  a.threshold = env_threshold > min_threshold ? env_threshold : min_threshold;
  int P = 2;
  while (P < 32 && b_bytes / P > ((size_t)(block_mb < 1 ? 1 : block_mb) << 20) * 3 / 2) P *= 2;
  if (const int force = env_int("COMET_SPMM_BLOCKS", 0)) { P = 2; while (P < force && P < 32) P *= 2; }
  a.P = P;
  a.block_cols = (int32_t)ceil_div(cols, P);
  a.tile_max = env_tile < 32 ? 32 : env_tile;
  a.piece_target = env_piece < 8 ? 8 : env_piece;
  a.num_scan_ctas = (int32_t)ceil_div(M, kScanCta);
  a.heavy_ctas = env_ctas < 1 ? 1 : env_ctas;
  a.B = B; a.ldb = ldb; a.C = const_cast<void *>(C); a.ldc = ldc; a.R = (int32_t)R;
  a.carry_ld = (int32_t)align_up((size_t)R, 2);
  a.h_max = N / a.threshold + 1;
  a.t_max = N / a.tile_max + N / a.piece_target + a.h_max;
  size_t off = 0;
  auto take = [&](size_t bytes) { off += align_up(bytes, 256); };
  take(16 * 4); take((size_t)a.num_scan_ctas * 4); take((size_t)a.num_scan_ctas * 4);
  take(a.h_max * 4); take(a.h_max * 4); take(a.h_max * 4);
  take((size_t)a.h_max * (P + 1) * 4); take(3 * 32 * 4); take((size_t)a.t_max * 16);
  take((size_t)a.t_max * a.carry_ld * 8);
  if (off > ((size_t)2 << 30)) return 0;                      // not worth that much scratch: general path only
  *out = a;
  return off;
}

comet_status_t spmm_heavy_prepare(Context *ctx, HeavyArgs *args, const int32_t *pos, const int32_t *crd, const void *val,
                                  char *s, cudaStream_t stream) {
  HeavyArgs &a = *args;
  a.pos = pos; a.crd = crd; a.val = val;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += align_up(bytes, 256); return s + at; };
  a.counters = (int32_t *)take(16 * 4);
  a.cta_rows = (int32_t *)take((size_t)a.num_scan_ctas * 4);
  a.cta_slots = (int32_t *)take((size_t)a.num_scan_ctas * 4);
  a.hrow = (int32_t *)take(a.h_max * 4);
  a.row_slot0 = (int32_t *)take(a.h_max * 4);
  a.row_nt = (int32_t *)take(a.h_max * 4);
  a.piece_start = (int32_t *)take((size_t)a.h_max * (a.P + 1) * 4);
  a.bin = (int32_t *)take(3 * 32 * 4);
  a.rec = (int4 *)take((size_t)a.t_max * 16);
  a.carry_val = (double *)take((size_t)a.t_max * a.carry_ld * 8);
  // the tickets and the tile cursor must start at zero; the scratch is shared with other calls, so clear them here
  COMET_CUDA_TRY(ctx, cudaMemsetAsync(a.counters, 0, 16 * 4, stream));
  heavy_count_kernel<<<a.num_scan_ctas, kBlockThreads, 0, stream>>>(a);
  const int64_t part_ctas = a.part ? ceil_div(a.part_tiles + 1, (int64_t)kBlockThreads) : 0;
  heavy_pieces_kernel<<<(unsigned)(a.num_scan_ctas + part_ctas), kBlockThreads, 0, stream>>>(a);
  heavy_tiles_kernel<<<kSmCount * 2, kBlockThreads, 0, stream>>>(a);
  COMET_LAUNCHED(ctx, 3);
  return COMET_OK;
}

}  // namespace comet
