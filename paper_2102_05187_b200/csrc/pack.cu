// comet_pack: COO -> per-level pos/crd arrays on the GPU (the conversion the paper's input-reading
// runtime function performs; Tensor Storage Format section for what each attribute stores), and
// comet_validate for caller-built descriptors.
//
//   1. keys      one 64-bit key per entry: the coordinates in storage-level order, level 0 in the most
//                significant bits (so key order = lexicographic order); coordinates are range-checked.
//   2. sort      stable LSD radix sort of (key, 32-bit payload), 8 bits per pass, only over the bits in use; the
//                first pass forms the keys from the caller's arrays, so steps 1 and 2 share their launches. The
//                payload is the value itself when it has 32 bits, else the entry's index.
//                Per pass: per-tile digit histogram -> exclusive scan of the (digit, tile) table ->
//                stable scatter (warp-level match ranks, per-warp digit counters in shared memory).
//   3. levels    head flags from key prefixes: entry p opens a new node at level l when the key prefix
//                down to level l differs from its predecessor's. Counting pass -> scan -> ONE host
//                synchronisation to learn the node counts -> exact allocation -> emit pass that writes
//                crd (compaction), pos (rank of the first child at every parent head), and the values in leaf
//                order (64-bit ones gathered through the sorted indices). Equal adjacent keys are duplicates
//                and are reported.
//
// No inter-CTA waiting anywhere: every scan is reduce / scan-of-sums / apply in separate launches.
#include "common.cuh"
#include "kernels.cuh"

#include <stdlib.h>
#include <string.h>

namespace comet {

constexpr int kSortThreads = 256;
constexpr int kSortItems = 8;
constexpr int kSortTile = kSortThreads * kSortItems;   // keys per CTA per pass
constexpr int kSortWarps = kSortThreads / 32;

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

enum { kStatusRange = 0, kStatusDuplicate = 1, kStatusInvalid = 2 };   // words of Context::d_status

struct KeyLayout {
  int order;
  int shift[COMET_MAX_ORDER];      // bit position of level l's coordinate inside the key
  int bits[COMET_MAX_ORDER];
  int total_bits;
  int64_t dim[COMET_MAX_ORDER];    // extent of the mode stored at level l
};

struct CoordPtrs { const int32_t *p[COMET_MAX_ORDER]; };   // level order

// ------------------------------------------------------------------------------------------------ keys
// ORDER is a template parameter so that the per-level loops unroll and the by-value descriptor structs
// are read with constant indices (a runtime index would push them into local memory).
template <int ORDER>
__device__ __forceinline__ uint64_t entry_key(const CoordPtrs &c, const KeyLayout &k, int64_t p, bool &bad) {
  int32_t v[ORDER];
#pragma unroll
  for (int l = 0; l < ORDER; ++l) v[l] = __ldcs(c.p[l] + p);
  uint64_t key = 0;
#pragma unroll
  for (int l = 0; l < ORDER; ++l) {
    bad |= (v[l] < 0) | ((int64_t)v[l] >= k.dim[l]);
    key |= ((uint64_t)(uint32_t)v[l] & ((1ull << k.bits[l]) - 1)) << k.shift[l];
  }
  return key;
}

// Where a sort pass reads its (key, payload) pairs. The payload is one 32-bit word that travels with the key
// through every pass: a 32-bit value itself (as raw bits; nothing is gathered afterwards), else the entry's index
// (64-bit values are gathered through it once, at the end: carrying them would cost more per pass than the gather
// saves from five passes on).
struct SortedPairs {                 // the output of the pass before
  const uint64_t *keys;
  const uint32_t *pay;
  __device__ __forceinline__ uint64_t key(int64_t i, bool &) const { return __ldcs(keys + i); }
  __device__ __forceinline__ uint32_t payload(int64_t i) const { return __ldcs(pay + i); }
};

template <int ORDER>
struct CooEntries {                  // the first pass: the caller's COO arrays; the keys are formed on the fly
  CoordPtrs c;
  KeyLayout k;
  const uint32_t *val32;             // 32-bit values, or null: the payload is the entry's index
  __device__ __forceinline__ uint64_t key(int64_t i, bool &bad) const { return entry_key<ORDER>(c, k, i, bad); }
  __device__ __forceinline__ uint32_t payload(int64_t i) const {
    uint32_t p = (uint32_t)i;
    if (val32) p = __ldcs(val32 + i);
    return p;
  }
};

// Keys and payloads written out as they stand: only for keys of zero bits (every extent 1), where no pass runs.
template <int ORDER>
__global__ void make_keys_kernel(CooEntries<ORDER> src, int64_t n, uint64_t *__restrict__ keys,
                                 uint32_t *__restrict__ pay, int32_t *__restrict__ status) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n) return;
  bool bad = false;
  keys[p] = src.key(p, bad);
  pay[p] = src.payload(p);
  if (bad) atomicOr(status + kStatusRange, 1);
}

// ------------------------------------------------------------------------------------------------ scan
// Exclusive scan of uint32 in three launches: tile sums, scan of the sums by one CTA, apply.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t *s_warp, uint32_t *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = lane < warps ? s_warp[lane] : 0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, w, off);
      if (lane >= off) w += t;
    }
    if (lane < warps) s_warp[lane] = w;        // inclusive over warps
  }
  __syncthreads();
  const uint32_t before = warp > 0 ? s_warp[warp - 1] : 0;
  if (total) *total = s_warp[warps - 1];
  __syncthreads();
  return before + inc - v;
}

__global__ void scan_tile_sums_kernel(const uint32_t *__restrict__ in, int64_t n, uint32_t *__restrict__ sums) {
  __shared__ uint32_t s_warp[32];
  const int64_t base = (int64_t)blockIdx.x * kScanTile;
  uint32_t v = 0;
#pragma unroll
  for (int t = 0; t < kScanItems; ++t) {
    const int64_t i = base + (int64_t)t * kScanThreads + threadIdx.x;
    if (i < n) v += in[i];
  }
  uint32_t total;
  block_exclusive_scan(v, s_warp, &total);
  if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// One CTA: exclusive scan of `sums` in place (any length, chunk by chunk with a running carry);
// the grand total goes to *total_out when given.
__global__ void scan_sums_kernel(uint32_t *__restrict__ sums, int64_t m, uint32_t *__restrict__ total_out) {
  __shared__ uint32_t s_warp[32];
  uint32_t carry = 0;
  for (int64_t base = 0; base < m; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    const uint32_t v = i < m ? sums[i] : 0;
    uint32_t total;
    const uint32_t ex = block_exclusive_scan(v, s_warp, &total);
    if (i < m) sums[i] = carry + ex;
    carry += total;
  }
  if (total_out && threadIdx.x == 0) *total_out = carry;
}

__global__ void scan_apply_kernel(const uint32_t *__restrict__ in, int64_t n, const uint32_t *__restrict__ sums,
                                  uint32_t *__restrict__ out) {
  __shared__ uint32_t s_warp[32];
  const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
  uint32_t v[kScanItems];
  uint32_t mine = 0;
#pragma unroll
  for (int t = 0; t < kScanItems; ++t) {
    v[t] = (base + t < n) ? in[base + t] : 0;
    mine += v[t];
  }
  uint32_t run = sums[blockIdx.x] + block_exclusive_scan(mine, s_warp, nullptr);
#pragma unroll
  for (int t = 0; t < kScanItems; ++t) {
    if (base + t < n) out[base + t] = run;
    run += v[t];
  }
}

// out = exclusive scan of in (may alias); tmp holds scan_tmp_words(n) words; total (device) optional.
int64_t scan_tmp_words(int64_t n) { return ceil_div(n > 0 ? n : 1, kScanTile) + 1; }

comet_status_t exclusive_scan(Context *ctx, const uint32_t *in, uint32_t *out, int64_t n, uint32_t *tmp,
                              uint32_t *total, cudaStream_t s) {
  if (n <= 0) {
    if (total) COMET_CUDA_TRY(ctx, cudaMemsetAsync(total, 0, sizeof(uint32_t), s));
    return COMET_OK;
  }
  const int64_t tiles = ceil_div(n, kScanTile);
  scan_tile_sums_kernel<<<(unsigned)tiles, kScanThreads, 0, s>>>(in, n, tmp);
  scan_sums_kernel<<<1, 1024, 0, s>>>(tmp, tiles, total);
  scan_apply_kernel<<<(unsigned)tiles, kScanThreads, 0, s>>>(in, n, tmp, out);
  COMET_LAUNCHED(ctx, 3);
  return COMET_OK;
}

// ------------------------------------------------------------------------------------------------ radix sort
template <class Src>
__global__ void __launch_bounds__(kSortThreads) radix_histogram_kernel(Src src, int64_t n, int shift, int64_t tiles,
                                                                       uint32_t *__restrict__ table,
                                                                       int32_t *__restrict__ status) {
  __shared__ uint32_t s_cnt[256];
  s_cnt[threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kSortTile;
  bool bad = false;
  uint64_t k[kSortItems];
  const bool full = base + kSortTile <= n;
#pragma unroll
  for (int t = 0; t < kSortItems; ++t) {          // unconditional loads: the eight of a thread are in flight together
    const int64_t i = base + (int64_t)t * kSortThreads + threadIdx.x;
    k[t] = src.key(full || i < n ? i : n - 1, bad);
  }
#pragma unroll
  for (int t = 0; t < kSortItems; ++t) {
    const int64_t i = base + (int64_t)t * kSortThreads + threadIdx.x;
    if (full || i < n) atomicAdd(&s_cnt[(k[t] >> shift) & 255], 1u);
  }
  if (bad) atomicOr(status + kStatusRange, 1);    // only the pass that forms the keys can see a bad coordinate
  __syncthreads();
  table[(int64_t)threadIdx.x * tiles + blockIdx.x] = s_cnt[threadIdx.x];     // digit-major
}

template <class Src>
__global__ void __launch_bounds__(kSortThreads, 4) radix_scatter_kernel(Src src, uint64_t *__restrict__ kout,
                                                                        uint32_t *__restrict__ pout,
                                                                        const uint32_t *__restrict__ table, int64_t n,
                                                                        int shift, int64_t tiles) {
  __shared__ uint32_t s_cnt[kSortWarps][256];     // per-warp digit counts, then where each warp's keys of a digit go
  __shared__ uint32_t s_delta[256];               // global position of digit d's run minus its start inside the tile
  __shared__ uint64_t s_key[kSortTile];           // the tile in sorted order
  __shared__ uint32_t s_pay[kSortTile];
  __shared__ uint32_t s_warp[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int w = 0; w < kSortWarps; ++w) s_cnt[w][tid] = 0;
  // where digit `tid`'s run of this tile starts in the output: asked for now, needed after the ranking
  const uint32_t digit_base = __ldg(table + (int64_t)tid * tiles + blockIdx.x);

  // Item r of lane l of warp w sits at tile_base + w*(32*ITEMS) + r*32 + l: memory order is (w, r, l).
  const int64_t tile_base = (int64_t)blockIdx.x * kSortTile;
  const int64_t warp_base = tile_base + (int64_t)warp * (32 * kSortItems);
  uint64_t key[kSortItems];
  uint32_t pay[kSortItems];
  bool ignored = false;
  if (tile_base + kSortTile <= n) {               // all loads first, none behind a branch
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
      const int64_t i = warp_base + r * 32 + lane;
      key[r] = src.key(i, ignored);
      pay[r] = src.payload(i);
    }
  } else {
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
      const int64_t i = warp_base + r * 32 + lane;
      key[r] = src.key(i < n ? i : n - 1, ignored);
      pay[r] = src.payload(i < n ? i : n - 1);
      if (i >= n) key[r] = ~0ull;                  // slots past the end rank after every real key of the tile
    }
  }
  __syncthreads();
  uint32_t rank[kSortItems];
  const unsigned lt = (1u << lane) - 1u;
#pragma unroll
  for (int r = 0; r < kSortItems; ++r) {
    const uint32_t d = (uint32_t)(key[r] >> shift) & 255u;
    const unsigned peers = __match_any_sync(0xffffffffu, d);
    const int leader = __ffs(peers) - 1;
    uint32_t old = 0;
    if (lane == leader) old = atomicAdd(&s_cnt[warp][d], (uint32_t)__popc(peers));   // one shared-memory operation
    old = __shfl_sync(0xffffffffu, old, leader);
    rank[r] = old + __popc(peers & lt);
    __syncwarp();
  }
  __syncthreads();
  {
    // digit `tid`: tile total -> start of the digit's run inside the tile -> where each warp's keys of the
    // digit start (run start + the counts of the warps before it), so that placing a key costs one lookup
    uint32_t run = 0;
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) run += s_cnt[w][tid];
    const uint32_t start = block_exclusive_scan(run, s_warp, nullptr);
    uint32_t off = start;
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
      const uint32_t c = s_cnt[w][tid];
      s_cnt[w][tid] = off;
      off += c;
    }
    s_delta[tid] = digit_base - start;
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < kSortItems; ++r) {          // local sort: every item to its place in the tile's order
    const uint32_t d = (uint32_t)(key[r] >> shift) & 255u;
    const uint32_t at = s_cnt[warp][d] + rank[r];
    s_key[at] = key[r];
    s_pay[at] = pay[r];
  }
  __syncthreads();
  const int64_t left = n - tile_base;
  const int valid = left < kSortTile ? (int)left : kSortTile;
#pragma unroll
  for (int r = 0; r < kSortItems; ++r) {          // coalesced: consecutive threads write a digit's run contiguously
    const int at = r * kSortThreads + tid;
    if (at < valid) {
      const uint64_t k2 = s_key[at];
      const uint32_t dst = s_delta[(uint32_t)(k2 >> shift) & 255u] + (uint32_t)at;
      kout[dst] = k2;
      pout[dst] = s_pay[at];
    }
  }
}

int64_t radix_sort_table_words(int64_t n) { return 256 * ceil_div(n > 0 ? n : 1, kSortTile); }

// One stable pass over the 8 key bits at `shift`: per-tile digit counts, their scan, the scatter.
template <class Src>
static comet_status_t radix_pass(Context *ctx, const Src &src, uint64_t *kout, uint32_t *pout, int64_t n, int shift,
                                 uint32_t *table, uint32_t *scan_tmp, cudaStream_t s) {
  const int64_t tiles = ceil_div(n, kSortTile);
  radix_histogram_kernel<Src><<<(unsigned)tiles, kSortThreads, 0, s>>>(src, n, shift, tiles, table, ctx->d_status);
  COMET_LAUNCH_CHECK(ctx);
  comet_status_t st = exclusive_scan(ctx, table, table, 256 * tiles, scan_tmp, nullptr, s);
  if (st != COMET_OK) return st;
  radix_scatter_kernel<Src><<<(unsigned)tiles, kSortThreads, 0, s>>>(src, kout, pout, table, n, shift, tiles);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

// Stable LSD radix sort of (key, payload) pairs over the key bits [first_bit, bits), 8 bits per pass. `ka`/`pa`
// hold the input and, on return, the sorted pairs (the pointers are swapped with `kb`/`pb` after every pass); all
// four buffers hold n + 1 elements. `table` holds radix_sort_table_words(n) words, `scan_tmp` scan_tmp_words of
// that.
static comet_status_t radix_sort_from(Context *ctx, uint64_t *&ka, uint64_t *&kb, uint32_t *&pa, uint32_t *&pb,
                                      int64_t n, int first_bit, int bits, uint32_t *table, uint32_t *scan_tmp,
                                      cudaStream_t s) {
  for (int shift = first_bit; shift < bits; shift += 8) {
    const SortedPairs src{ka, pa};
    comet_status_t st = radix_pass(ctx, src, kb, pb, n, shift, table, scan_tmp, s);
    if (st != COMET_OK) return st;
    uint64_t *tk = ka; ka = kb; kb = tk;
    uint32_t *tp = pa; pa = pb; pb = tp;
  }
  return COMET_OK;
}

comet_status_t radix_sort_pairs(Context *ctx, uint64_t *&ka, uint64_t *&kb, uint32_t *&pa, uint32_t *&pb, int64_t n,
                                int bits, uint32_t *table, uint32_t *scan_tmp, cudaStream_t s) {
  if (n <= 0) return COMET_OK;
  return radix_sort_from(ctx, ka, kb, pa, pb, n, 0, bits, table, scan_tmp, s);
}

// The packing's sort: the COO entries by their keys. The first pass reads the caller's arrays and forms the keys
// on the fly (the coordinates are range-checked there); on return `ka`/`pa` hold the sorted keys and payloads.
template <int ORDER>
static comet_status_t sort_entries(Context *ctx, const CoordPtrs &coords, const KeyLayout &key, const uint32_t *val32,
                                   uint64_t *&ka, uint64_t *&kb, uint32_t *&pa, uint32_t *&pb, int64_t n,
                                   uint32_t *table, uint32_t *scan_tmp, cudaStream_t s) {
  const CooEntries<ORDER> src{coords, key, val32};
  if (key.total_bits == 0) {
    make_keys_kernel<ORDER><<<(unsigned)ceil_div(n, 256), 256, 0, s>>>(src, n, ka, pa, ctx->d_status);
    COMET_LAUNCH_CHECK(ctx);
    return COMET_OK;
  }
  comet_status_t st = radix_pass(ctx, src, kb, pb, n, 0, table, scan_tmp, s);
  if (st != COMET_OK) return st;
  uint64_t *tk = ka; ka = kb; kb = tk;
  uint32_t *tp = pa; pa = pb; pb = tp;
  return radix_sort_from(ctx, ka, kb, pa, pb, n, 8, key.total_bits, table, scan_tmp, s);
}

// ------------------------------------------------------------------------------------------------ duplicates
// COMET_PACK_SUM_DUPLICATES: after the sort, entries with equal keys are adjacent and, the sort being stable,
// in the order they were given. The first entry of each run keeps the key; its value becomes the sum of the
// run, added one by one in double in that order (one thread per run: runs are short unless the input is
// degenerate). The level pass then sees distinct keys and the merged values.
__global__ void dup_heads_kernel(const uint64_t *__restrict__ keys, int64_t n, uint32_t *__restrict__ head) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p < n) head[p] = (p == 0 || keys[p] != keys[p - 1]) ? 1u : 0u;
}

// GATHER: the values are the caller's, read through the sorted payload (entry indices); else they are in sorted
// order already.
template <class V, bool GATHER>
__global__ void dup_merge_kernel(const uint64_t *__restrict__ keys, const uint32_t *__restrict__ perm,
                                 const V *__restrict__ val_in, int64_t n, const uint32_t *__restrict__ rank,
                                 uint64_t *__restrict__ keys_out, V *__restrict__ val_out) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n) return;
  const uint64_t k = keys[p];
  if (p > 0 && keys[p - 1] == k) return;
  double sum = (double)val_in[GATHER ? (int64_t)perm[p] : p];
  for (int64_t q = p + 1; q < n && keys[q] == k; ++q) sum = sum + (double)val_in[GATHER ? (int64_t)perm[q] : q];
  const uint32_t r = rank[p];
  keys_out[r] = k;
  val_out[r] = (V)sum;
}

// ------------------------------------------------------------------------------------------------ levels
struct LevelPlan {
  int order;
  int attr[COMET_MAX_ORDER];
  int shift[COMET_MAX_ORDER];
  int bits[COMET_MAX_ORDER];
  int counted[COMET_MAX_ORDER];     // index of the level's node counter (-1: positions are entry ranks or dense)
  int ncounted;
};

__device__ __forceinline__ bool is_head(uint64_t k, uint64_t kprev, bool first, int shift) {
  return first || (k >> shift) != (kprev >> shift);
}

constexpr int kLevelThreads = 256;
constexpr int kLevelItems = 8;
constexpr int kLevelTile = kLevelThreads * kLevelItems;

// Per tile: how many nodes each counted level opens; duplicates (equal adjacent keys) are flagged.
// Counters are indexed by level (slots of uncounted levels stay unused); ORDER is a template parameter
// so that every per-level loop unrolls and the plan is read with constant indices.
template <int ORDER>
__global__ void __launch_bounds__(kLevelThreads) level_count_kernel(const uint64_t *__restrict__ keys, int64_t n,
                                                                    LevelPlan plan, int64_t tiles,
                                                                    uint32_t *__restrict__ counts,
                                                                    int32_t *__restrict__ status) {
  __shared__ uint32_t s_cnt[COMET_MAX_ORDER];
  if (threadIdx.x < COMET_MAX_ORDER) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kLevelTile;
  uint32_t mine[ORDER];
#pragma unroll
  for (int l = 0; l < ORDER; ++l) mine[l] = 0;
  bool dup = false;
  uint64_t key[kLevelItems], prev[kLevelItems];
#pragma unroll
  for (int t = 0; t < kLevelItems; ++t) {         // unconditional loads: all of a thread's in flight together
    const int64_t p = base + (int64_t)t * kLevelThreads + threadIdx.x;
    const int64_t q = p < n ? p : n - 1;
    key[t] = keys[q];
    prev[t] = keys[q > 0 ? q - 1 : 0];
  }
#pragma unroll
  for (int t = 0; t < kLevelItems; ++t) {
    const int64_t p = base + (int64_t)t * kLevelThreads + threadIdx.x;
    if (p < n) {
      const uint64_t k = key[t], kp = prev[t];
      dup |= (p > 0) & (k == kp);
#pragma unroll
      for (int l = 0; l < ORDER; ++l)
        if (plan.counted[l] >= 0 && is_head(k, kp, p == 0, plan.shift[l])) mine[l] += 1;
    }
  }
#pragma unroll
  for (int l = 0; l < ORDER; ++l) {
    if (plan.counted[l] < 0) continue;
    uint32_t v = mine[l];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
    if ((threadIdx.x & 31) == 0 && v) atomicAdd(&s_cnt[l], v);
  }
  if (dup) atomicOr(status + kStatusDuplicate, 1);
  __syncthreads();
  if (threadIdx.x < ORDER && plan.counted[threadIdx.x] >= 0)
    counts[(int64_t)threadIdx.x * tiles + blockIdx.x] = s_cnt[threadIdx.x];
}

struct LevelOut {
  int32_t *pos[COMET_MAX_ORDER];
  int32_t *crd[COMET_MAX_ORDER];
  void *val;                   // fp64 or fp32, as the COO values
  int64_t dim0;                // extent of level 0 (for a dense root)
  uint32_t nodes[COMET_MAX_ORDER];   // node count of every counted level (indexed by level)
};

// Per tile: ranks of the heads (tile-local scan + the tile's scanned offset), then crd / pos / val. GATHER: the
// values are the caller's, read through the sorted payload (entry indices); else they are in sorted order already.
template <int ORDER, class V, bool GATHER>
__global__ void __launch_bounds__(kLevelThreads) level_emit_kernel(const uint64_t *__restrict__ keys,
                                                                   const uint32_t *__restrict__ perm,
                                                                   const V *__restrict__ val_in, int64_t n,
                                                                   LevelPlan plan, int64_t tiles,
                                                                   const uint32_t *__restrict__ offsets,
                                                                   LevelOut out) {
  __shared__ uint32_t s_warp[32];
  const int64_t base = (int64_t)blockIdx.x * kLevelTile + (int64_t)threadIdx.x * kLevelItems;   // blocked: 8 consecutive
  uint64_t k[kLevelItems + 1];
  V vals[kLevelItems];
  k[0] = (base > 0 && base - 1 < n) ? keys[base - 1] : 0;
  if constexpr (GATHER) {
    uint32_t src[kLevelItems];
#pragma unroll
    for (int t = 0; t < kLevelItems; ++t) {
      k[t + 1] = (base + t < n) ? keys[base + t] : 0;
      src[t] = (base + t < n) ? perm[base + t] : 0;
    }
#pragma unroll
    for (int t = 0; t < kLevelItems; ++t) vals[t] = (base + t < n) ? __ldg(val_in + src[t]) : (V)0;   // the random gather, all in flight
  } else {
#pragma unroll
    for (int t = 0; t < kLevelItems; ++t) {
      k[t + 1] = (base + t < n) ? keys[base + t] : 0;
      vals[t] = (base + t < n) ? __ldcs(val_in + base + t) : (V)0;
    }
  }

  // rank[l] = nodes of level l opened before this thread's first entry
  uint32_t rank[ORDER];
#pragma unroll
  for (int l = 0; l < ORDER; ++l) {
    rank[l] = 0;
    if (plan.counted[l] < 0) continue;
    uint32_t mine = 0;
#pragma unroll
    for (int t = 0; t < kLevelItems; ++t)
      if (base + t < n && is_head(k[t + 1], k[t], base + t == 0, plan.shift[l])) mine += 1;
    rank[l] = offsets[(int64_t)l * tiles + blockIdx.x] + block_exclusive_scan(mine, s_warp, nullptr);
  }

#pragma unroll
  for (int t = 0; t < kLevelItems; ++t) {
    const int64_t p = base + t;
    if (p < n) {
      const uint64_t key = k[t + 1], kp = k[t];
      const bool first = p == 0;
      uint32_t parent_pos = 0;       // position of this entry's node at the level above
      bool parent_head = first;      // does this entry open a new node at the level above?
#pragma unroll
      for (int l = 0; l < ORDER; ++l) {
        const int32_t coord = (int32_t)((key >> plan.shift[l]) & ((1ull << plan.bits[l]) - 1));
        const int a = plan.attr[l];
        if (a == COMET_D) {
          parent_pos = (uint32_t)coord;
          parent_head = is_head(key, kp, first, plan.shift[l]);
        } else if (a == COMET_CU) {
          const bool head = is_head(key, kp, first, plan.shift[l]);
          const bool leaf = plan.counted[l] < 0;               // leaf level: one node per entry
          const uint32_t node = leaf ? (uint32_t)p : (head ? rank[l] : rank[l] - 1);
          if (head) {
            out.crd[l][node] = coord;
            if (l == 0) {
              // root: pos = [0, nodes], written by the finisher
            } else if (plan.attr[l > 0 ? l - 1 : 0] == COMET_D) {
              // dense parent: every parent coordinate after the previous node's and up to this one starts here
              if (parent_head) {
                const int sh = plan.shift[l > 0 ? l - 1 : 0], bt = plan.bits[l > 0 ? l - 1 : 0];
                const int64_t prev = first ? -1 : (int64_t)((kp >> sh) & ((1ull << bt) - 1));
                for (int64_t r = prev + 1; r <= (int64_t)parent_pos; ++r) out.pos[l][r] = (int32_t)node;
              }
            } else if (parent_head) {
              out.pos[l][parent_pos] = (int32_t)node;           // first child of parent node parent_pos
            }
          }
          parent_pos = node;
          parent_head = head;
          if (!leaf && head) rank[l] += 1;
        } else {                                                // CN, S: one position per entry
          out.crd[l][p] = coord;
          parent_pos = (uint32_t)p;
          parent_head = true;
        }
      }
      static_cast<V *>(out.val)[p] = vals[t];
    }
  }
}

// Closes the pos arrays: the terminal entry of every compressed level (and the empty tail of a CSR pos).
template <int ORDER>
__global__ void level_finish_kernel(const uint64_t *__restrict__ keys, int64_t n, LevelPlan plan, LevelOut out) {
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t parents = 1;
#pragma unroll
  for (int l = 0; l < ORDER; ++l) {
    const int a = plan.attr[l];
    const uint32_t nodes = plan.counted[l] >= 0 ? out.nodes[l] : (uint32_t)n;
    if (a == COMET_D) {
      if (tid == 0) out.pos[l][0] = (int32_t)out.dim0;
      parents = (uint32_t)out.dim0;
    } else if (a == COMET_CU) {
      if (l == 0) {
        if (tid == 0) { out.pos[0][0] = 0; out.pos[0][1] = (int32_t)nodes; }
      } else if (plan.attr[l > 0 ? l - 1 : 0] == COMET_D) {
        // rows after the last stored one (all rows when the tensor is empty) start at `nodes`
        const int sh = plan.shift[l > 0 ? l - 1 : 0], bt = plan.bits[l > 0 ? l - 1 : 0];
        const int64_t last = n > 0 ? (int64_t)((keys[n - 1] >> sh) & ((1ull << bt) - 1)) : -1;
        for (int64_t r = last + 1 + tid; r <= (int64_t)out.dim0; r += (int64_t)gridDim.x * blockDim.x)
          out.pos[l][r] = (int32_t)nodes;
      } else if (tid == 0) {
        out.pos[l][parents] = (int32_t)nodes;
      }
      parents = nodes;
    } else if (a == COMET_CN) {
      if (tid == 0) { out.pos[l][0] = 0; out.pos[l][1] = (int32_t)n; }
      parents = (uint32_t)n;
    }
  }
}

// ------------------------------------------------------------------------------------------------ validate
__global__ void validate_level_kernel(const int32_t *__restrict__ pos, int64_t parents, const int32_t *__restrict__ crd,
                                      int64_t crd_len, int64_t dim, int attr, int32_t *__restrict__ status) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  bool bad = false;
  if (attr == COMET_CU) {
    if (i == 0) bad |= pos[0] != 0 || (int64_t)pos[parents] != crd_len;
    if (i < parents) {
      const int64_t lo = pos[i], hi = pos[i + 1];
      bad |= lo > hi || lo < 0 || hi > crd_len;
      if (!bad)
        for (int64_t q = lo; q < hi; ++q) {
          const int32_t c = crd[q];
          bad |= c < 0 || c >= dim || (q > lo && crd[q - 1] >= c);
        }
    }
  } else if (i < crd_len) {
    const int32_t c = crd[i];
    bad |= c < 0 || c >= dim;
    if (attr == COMET_CN && i > 0) bad |= crd[i - 1] > c;
  }
  if (bad) atomicOr(status + kStatusInvalid, 1);
}

}  // namespace comet

using namespace comet;

namespace {

int bits_for(int64_t dim) {          // bits needed for coordinates 0 .. dim-1
  int b = 0;
  while (b < 62 && (1ll << b) < dim) ++b;
  return b;
}

bool supported_attrs(int order, const int32_t *attr) {
  bool coo = attr[0] == COMET_CN, csf = attr[0] == COMET_CU, dcs = attr[0] == COMET_D;
  for (int l = 1; l < order; ++l) {
    coo = coo && attr[l] == COMET_S;
    csf = csf && attr[l] == COMET_CU;
    dcs = dcs && attr[l] == COMET_CU;
  }
  return order >= 2 && (coo || csf || dcs);
}

struct TempBlocks {
  Context *ctx;
  cudaStream_t s;
  void *p[12];
  int n = 0;
  TempBlocks(Context *c, cudaStream_t st) : ctx(c), s(st) {}
  void *get(size_t bytes) {
    void *q = ctx_alloc(ctx, bytes, s);
    if (q) p[n++] = q;
    return q;
  }
  ~TempBlocks() { for (int i = 0; i < n; ++i) ctx_free(ctx, p[i], s); }
};

}  // namespace

extern "C" comet_status_t comet_pack(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                                     const int32_t *const *h_coo_crd, const void *coo_val, comet_dtype_t dtype,
                                     const int32_t *h_mode_order, const int32_t *h_attr, void *stream,
                                     comet_sptensor_t *out) {
  return comet_pack_ex(handle, order, h_dims, nnz, h_coo_crd, coo_val, dtype, h_mode_order, h_attr, 0u, stream, out);
}

extern "C" comet_status_t comet_pack_ex(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                                        const int32_t *const *h_coo_crd, const void *coo_val, comet_dtype_t dtype,
                                        const int32_t *h_mode_order, const int32_t *h_attr, uint32_t flags,
                                        void *stream, comet_sptensor_t *out) {
  if (flags & ~(uint32_t)(COMET_PACK_SUM_DUPLICATES | COMET_PACK_CSR_HISTOGRAM)) return COMET_ERR_INVALID_ARG;
  if (!handle || !out || !h_dims || !h_coo_crd || !h_mode_order || !h_attr) return COMET_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  if (order < 1 || order > COMET_MAX_ORDER || nnz < 0) return COMET_ERR_INVALID_ARG;
  if (dtype != COMET_F64 && dtype != COMET_F32) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (nnz > 2147483647ll - 1024) return COMET_ERR_INDEX_OVERFLOW;
  bool seen[COMET_MAX_ORDER] = {false, false, false, false};
  for (int l = 0; l < order; ++l) {
    const int m = h_mode_order[l];
    if (m < 0 || m >= order || seen[m]) return COMET_ERR_INVALID_ARG;
    seen[m] = true;
    if (h_attr[l] < COMET_D || h_attr[l] > COMET_S) return COMET_ERR_INVALID_ARG;
    if (h_dims[l] < 0) return COMET_ERR_INVALID_ARG;
    if (h_dims[l] > 2147483646ll) return COMET_ERR_INDEX_OVERFLOW;
    if (nnz > 0 && !h_coo_crd[l]) return COMET_ERR_INVALID_ARG;
  }
  if (nnz > 0 && !coo_val) return COMET_ERR_INVALID_ARG;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;

  // A singleton level under a dense one asks for ELLPACK: packed as CSR first, then the rows are spread over
  // K slots each (ellpack.cu). The result has three levels, [D, D, S].
  if (order == 2 && h_attr[0] == COMET_D && h_attr[1] == COMET_S) {
    const int32_t csr_attr[2] = {COMET_D, COMET_CU};
    comet_sptensor_t csr;
    comet_status_t st = comet_pack_ex(handle, 2, h_dims, nnz, h_coo_crd, coo_val, dtype, h_mode_order, csr_attr,
                                      flags & ~(uint32_t)COMET_PACK_CSR_HISTOGRAM, stream, &csr);
    if (st != COMET_OK) return st;
    void *owner = owner_new();
    st = owner ? ell_from_csr(ctx, &csr, owner, out, s) : COMET_ERR_ALLOC;
    comet_sptensor_free(handle, &csr, stream);
    if (st != COMET_OK) {
      if (owner) owner_release(ctx, owner, s);
      memset(out, 0, sizeof(*out));
      return st;
    }
    out->owner = owner;
    return COMET_OK;
  }
  if (!supported_attrs(order, h_attr)) return COMET_ERR_UNSUPPORTED_FORMAT;

  // CSR of a matrix with a dense row level: the row structure is a histogram, so the full sort is not needed
  // (pack_csr.cu). On request only (COMET_PACK_CSR_HISTOGRAM): it wins on matrices whose rows are of similar
  // length and loses on skewed ones, where the atomic counters of the heavy rows serialise. The environment
  // variable COMET_PACK_CSR=1 / 0 overrides the flag (tests).
  {
    const char *force = getenv("COMET_PACK_CSR");
    const int64_t rows = h_dims[h_mode_order[0]], cols = h_dims[h_mode_order[1 % order]];
    const bool shape = order == 2 && h_attr[0] == COMET_D && h_attr[1] == COMET_CU &&
                       !(flags & COMET_PACK_SUM_DUPLICATES) && rows <= (1ll << 27) &&
                       rows <= 4 * nnz + 1024;            // a warp visits every row: not for hypersparse matrices
    const bool want = force ? force[0] == '1' : (flags & COMET_PACK_CSR_HISTOGRAM) != 0;
    if (shape && want) {
      void *owner = owner_new();
      if (!owner) return COMET_ERR_ALLOC;
      const size_t val_size = dtype == COMET_F32 ? 4 : 8;
      out->order = 2; out->dtype = dtype; out->nnz = nnz;
      for (int l = 0; l < 2; ++l) { out->dims[l] = h_dims[l]; out->mode_order[l] = h_mode_order[l]; out->attr[l] = h_attr[l]; }
      out->pos_len[0] = 1; out->crd_len[0] = 0; out->pos_len[1] = rows + 1; out->crd_len[1] = nnz;
      out->pos[0] = (int32_t *)owner_alloc(ctx, owner, 4, s);
      out->pos[1] = (int32_t *)owner_alloc(ctx, owner, (size_t)(rows + 1) * 4, s);
      if (nnz > 0) {
        out->crd[1] = (int32_t *)owner_alloc(ctx, owner, (size_t)nnz * 4, s);
        out->val = owner_alloc(ctx, owner, (size_t)nnz * val_size, s);
      }
      comet_status_t st = COMET_OK;
      if (!out->pos[0] || !out->pos[1] || (nnz > 0 && (!out->crd[1] || !out->val))) st = COMET_ERR_ALLOC;
      int fallback = 0;
      if (st == COMET_OK) {
        const int32_t dim0 = (int32_t)rows;
        cudaError_t e = cudaMemcpyAsync(out->pos[0], &dim0, 4, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) st = cuda_fail(ctx, e);
      }
      if (st == COMET_OK)
        st = pack_csr_fast(ctx, dtype, h_coo_crd[h_mode_order[0]], h_coo_crd[h_mode_order[1]], coo_val, nnz, rows, cols,
                           out->pos[1], out->crd[1], out->val, &fallback, s);
      if (st == COMET_OK && !fallback) { out->owner = owner; return COMET_OK; }
      owner_release(ctx, owner, s);
      memset(out, 0, sizeof(*out));
      if (st != COMET_OK) return st;
    }
  }

  KeyLayout key{};
  LevelPlan plan{};
  CoordPtrs coords{};
  key.order = plan.order = order;
  int total_bits = 0;
  for (int l = order - 1; l >= 0; --l) {
    const int m = h_mode_order[l];
    key.dim[l] = h_dims[m];
    key.bits[l] = plan.bits[l] = bits_for(h_dims[m]);
    key.shift[l] = plan.shift[l] = total_bits;
    total_bits += key.bits[l];
    plan.attr[l] = h_attr[l];
    coords.p[l] = h_coo_crd[m];
  }
  if (total_bits > 63) return COMET_ERR_UNSUPPORTED_FORMAT;   // the coordinate bits must fit one 64-bit key
  key.total_bits = total_bits;
  plan.ncounted = 0;
  for (int l = 0; l < order; ++l) {
    // a compressed-unique level above the leaf has fewer nodes than entries and needs a node counter
    plan.counted[l] = (plan.attr[l] == COMET_CU && l < order - 1) ? plan.ncounted++ : -1;
  }
  if (h_attr[0] == COMET_D && h_dims[h_mode_order[0]] == 0 && nnz > 0) return COMET_ERR_COORD_OUT_OF_RANGE;

  int64_t n = nnz;                     // entries the level pass sees (fewer after duplicates are merged)
  const int64_t sort_tiles = ceil_div(n > 0 ? n : 1, kSortTile);
  int64_t level_tiles = ceil_div(n > 0 ? n : 1, kLevelTile);
  const int64_t table_len = radix_sort_table_words(n);
  const int64_t counts_len = (int64_t)COMET_MAX_ORDER * level_tiles;

  TempBlocks tmp(ctx, s);
  uint64_t *keys_a = (uint64_t *)tmp.get((size_t)(n + 1) * 8);
  uint64_t *keys_b = (uint64_t *)tmp.get((size_t)(n + 1) * 8);
  uint32_t *pay_a = (uint32_t *)tmp.get((size_t)(n + 1) * 4);   // fp32 values as raw bits, else entry indices
  uint32_t *pay_b = (uint32_t *)tmp.get((size_t)(n + 1) * 4);
  const int64_t table_words = table_len > counts_len ? table_len : counts_len;
  uint32_t *table = (uint32_t *)tmp.get((size_t)table_words * 4);
  uint32_t *scan_tmp = (uint32_t *)tmp.get((size_t)(ceil_div(table_words, kScanTile) + 1) * 4);
  if (!keys_a || !keys_b || !pay_a || !pay_b || !table || !scan_tmp) return COMET_ERR_ALLOC;

  COMET_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, 16 * sizeof(int32_t), s));
  uint32_t *d_nodes = reinterpret_cast<uint32_t *>(ctx->d_status) + 8;   // node counts live beside the status words

  const void *sorted_val = nullptr;    // the values in sorted order, once some array holds them so
  if (n > 0) {
    {
      const uint32_t *val32 = dtype == COMET_F32 ? static_cast<const uint32_t *>(coo_val) : nullptr;
      comet_status_t st;
      if (order == 2) st = sort_entries<2>(ctx, coords, key, val32, keys_a, keys_b, pay_a, pay_b, n, table, scan_tmp, s);
      else if (order == 3) st = sort_entries<3>(ctx, coords, key, val32, keys_a, keys_b, pay_a, pay_b, n, table, scan_tmp, s);
      else st = sort_entries<4>(ctx, coords, key, val32, keys_a, keys_b, pay_a, pay_b, n, table, scan_tmp, s);
      if (st != COMET_OK) return st;
      if (dtype == COMET_F32) sorted_val = pay_a;
    }
    if (flags & COMET_PACK_SUM_DUPLICATES) {
      // merge runs of equal keys; costs one more synchronisation (the number of distinct cells sizes the rest)
      uint32_t *rank = (uint32_t *)tmp.get((size_t)n * 4);
      void *merged = tmp.get((size_t)n * (dtype == COMET_F32 ? 4 : 8));
      if (!rank || !merged) return COMET_ERR_ALLOC;
      uint32_t *d_distinct = reinterpret_cast<uint32_t *>(ctx->d_status) + 12;
      dup_heads_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, s>>>(keys_a, n, rank);
      COMET_LAUNCH_CHECK(ctx);
      uint32_t *rank_tmp = (uint32_t *)keys_b;                 // free until the merge writes it
      comet_status_t st = exclusive_scan(ctx, rank, rank, n, rank_tmp, d_distinct, s);
      if (st != COMET_OK) return st;
      COMET_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, ctx->d_status, 16 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
      COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));
      if (ctx->h_pinned[kStatusRange]) return COMET_ERR_COORD_OUT_OF_RANGE;
      const int64_t distinct = reinterpret_cast<uint32_t *>(ctx->h_pinned)[12];
      // keys_b is both the scan's scratch and the merge's output: the scan has finished (synchronised above)
      if (dtype == COMET_F32)
        dup_merge_kernel<float, false><<<(unsigned)ceil_div(n, 256), 256, 0, s>>>(keys_a, nullptr, (const float *)sorted_val, n, rank,
                                                                                 keys_b, (float *)merged);
      else
        dup_merge_kernel<double, true><<<(unsigned)ceil_div(n, 256), 256, 0, s>>>(keys_a, pay_a, (const double *)coo_val, n, rank,
                                                                                 keys_b, (double *)merged);
      COMET_LAUNCH_CHECK(ctx);
      keys_a = keys_b;
      sorted_val = merged;
      n = distinct;
      level_tiles = ceil_div(n > 0 ? n : 1, kLevelTile);
    }
    // node counts of the counted levels: per-tile counts -> scanned offsets (kept in `table`) + totals
    if (order == 2) level_count_kernel<2><<<(unsigned)level_tiles, kLevelThreads, 0, s>>>(keys_a, n, plan, level_tiles, table, ctx->d_status);
    else if (order == 3) level_count_kernel<3><<<(unsigned)level_tiles, kLevelThreads, 0, s>>>(keys_a, n, plan, level_tiles, table, ctx->d_status);
    else level_count_kernel<4><<<(unsigned)level_tiles, kLevelThreads, 0, s>>>(keys_a, n, plan, level_tiles, table, ctx->d_status);
    COMET_LAUNCH_CHECK(ctx);
    for (int l = 0; l < order; ++l) {
      if (plan.counted[l] < 0) continue;
      comet_status_t st = exclusive_scan(ctx, table + (int64_t)l * level_tiles, table + (int64_t)l * level_tiles,
                                         level_tiles, scan_tmp, d_nodes + l, s);
      if (st != COMET_OK) return st;
    }
  }
  // the one synchronisation: status words and node counts
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, ctx->d_status, 16 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  if (ctx->h_pinned[kStatusRange]) return COMET_ERR_COORD_OUT_OF_RANGE;
  if (ctx->h_pinned[kStatusDuplicate]) return COMET_ERR_DUPLICATE_COORD;

  // exact allocation
  void *owner = owner_new();
  if (!owner) return COMET_ERR_ALLOC;
  LevelOut lo{};
  bool alloc_ok = true;
  out->order = order;
  out->dtype = dtype;
  out->nnz = n;
  int64_t parents = 1;
  for (int l = 0; l < order; ++l) {
    out->dims[l] = h_dims[l];
    out->mode_order[l] = h_mode_order[l];
    out->attr[l] = h_attr[l];
    const int64_t nodes = plan.counted[l] >= 0 ? (int64_t)reinterpret_cast<uint32_t *>(ctx->h_pinned)[8 + l] : n;
    if (plan.counted[l] >= 0) lo.nodes[l] = (uint32_t)nodes;
    int64_t pos_len = 0, crd_len = 0;
    if (h_attr[l] == COMET_D) { pos_len = 1; parents = key.dim[l]; }
    else if (h_attr[l] == COMET_CU) { pos_len = parents + 1; crd_len = nodes; parents = nodes; }
    else if (h_attr[l] == COMET_CN) { pos_len = 2; crd_len = n; parents = n; }
    else { crd_len = n; }
    out->pos_len[l] = pos_len;
    out->crd_len[l] = crd_len;
    if (pos_len) { out->pos[l] = (int32_t *)owner_alloc(ctx, owner, (size_t)pos_len * 4, s); alloc_ok &= out->pos[l] != nullptr; }
    if (crd_len) { out->crd[l] = (int32_t *)owner_alloc(ctx, owner, (size_t)crd_len * 4, s); alloc_ok &= out->crd[l] != nullptr; }
    lo.pos[l] = out->pos[l];
    lo.crd[l] = out->crd[l];
  }
  const size_t val_size = dtype == COMET_F32 ? 4 : 8;
  if (n > 0) { out->val = owner_alloc(ctx, owner, (size_t)n * val_size, s); alloc_ok &= out->val != nullptr; }
  lo.val = out->val;
  lo.dim0 = key.dim[0];
  if (!alloc_ok) { owner_release(ctx, owner, s); memset(out, 0, sizeof(*out)); return COMET_ERR_ALLOC; }

  if (n > 0) {
    const unsigned g = (unsigned)level_tiles;
    if (dtype == COMET_F32) {
      const float *vin = (const float *)sorted_val;
      if (order == 2) level_emit_kernel<2, float, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
      else if (order == 3) level_emit_kernel<3, float, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
      else level_emit_kernel<4, float, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
    } else if (sorted_val) {
      const double *vin = (const double *)sorted_val;
      if (order == 2) level_emit_kernel<2, double, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
      else if (order == 3) level_emit_kernel<3, double, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
      else level_emit_kernel<4, double, false><<<g, kLevelThreads, 0, s>>>(keys_a, nullptr, vin, n, plan, level_tiles, table, lo);
    } else {
      const double *vin = (const double *)coo_val;
      if (order == 2) level_emit_kernel<2, double, true><<<g, kLevelThreads, 0, s>>>(keys_a, pay_a, vin, n, plan, level_tiles, table, lo);
      else if (order == 3) level_emit_kernel<3, double, true><<<g, kLevelThreads, 0, s>>>(keys_a, pay_a, vin, n, plan, level_tiles, table, lo);
      else level_emit_kernel<4, double, true><<<g, kLevelThreads, 0, s>>>(keys_a, pay_a, vin, n, plan, level_tiles, table, lo);
    }
  }
  if (order == 2) level_finish_kernel<2><<<kSmCount, 256, 0, s>>>(keys_a, n, plan, lo);
  else if (order == 3) level_finish_kernel<3><<<kSmCount, 256, 0, s>>>(keys_a, n, plan, lo);
  else level_finish_kernel<4><<<kSmCount, 256, 0, s>>>(keys_a, n, plan, lo);
  ctx->launches += n > 0 ? 2 : 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { owner_release(ctx, owner, s); memset(out, 0, sizeof(*out)); return cuda_fail(ctx, e); }
  out->owner = owner;
  return COMET_OK;
}

extern "C" comet_status_t comet_validate(comet_handle_t handle, const comet_sptensor_t *t, void *stream) {
  if (!handle || !t) return COMET_ERR_INVALID_ARG;
  if (t->order < 1 || t->order > COMET_MAX_ORDER || t->nnz < 0) return COMET_ERR_INVALID_ARG;
  Context *ctx = reinterpret_cast<Context *>(handle);
  cudaStream_t s = (cudaStream_t)stream;
  // host-visible shape checks first
  int64_t parents = 1;
  for (int l = 0; l < t->order; ++l) {
    const int a = t->attr[l];
    const int64_t dim = t->dims[t->mode_order[l]];
    if (a == COMET_D) {
      if (t->pos_len[l] != 1 || !t->pos[l]) return COMET_ERR_INVALID_TENSOR;
      for (int u = 0; u < l; ++u) if (t->attr[u] != COMET_D) return COMET_ERR_UNSUPPORTED_FORMAT;
      parents *= dim;
    } else if (a == COMET_CU) {
      if (t->pos_len[l] != parents + 1 || !t->pos[l] || (t->crd_len[l] > 0 && !t->crd[l])) return COMET_ERR_INVALID_TENSOR;
      parents = t->crd_len[l];
    } else if (a == COMET_CN) {
      if (l != 0) return COMET_ERR_UNSUPPORTED_FORMAT;
      if (t->pos_len[l] != 2 || !t->pos[l] || t->crd_len[l] != t->nnz) return COMET_ERR_INVALID_TENSOR;
      parents = t->nnz;
    } else if (a == COMET_S) {
      if (l == 0 || (t->attr[l - 1] != COMET_CN && t->attr[l - 1] != COMET_S)) return COMET_ERR_UNSUPPORTED_FORMAT;
      if (t->crd_len[l] != parents) return COMET_ERR_INVALID_TENSOR;
    } else {
      return COMET_ERR_INVALID_ARG;
    }
  }
  if (t->attr[t->order - 1] != COMET_D && parents != t->nnz) return COMET_ERR_INVALID_TENSOR;

  COMET_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, 16 * sizeof(int32_t), s));
  parents = 1;
  for (int l = 0; l < t->order; ++l) {
    const int a = t->attr[l];
    const int64_t dim = t->dims[t->mode_order[l]];
    if (a == COMET_D) { parents *= dim; continue; }
    const int64_t work = a == COMET_CU ? (parents > 0 ? parents : 1) : t->crd_len[l];
    if (work > 0) {
      validate_level_kernel<<<(unsigned)ceil_div(work, 256), 256, 0, s>>>(t->pos[l], parents, t->crd[l], t->crd_len[l],
                                                                          dim, a, ctx->d_status);
      COMET_LAUNCH_CHECK(ctx);
    }
    parents = a == COMET_S ? parents : t->crd_len[l];
  }
  COMET_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->h_pinned, ctx->d_status, 16 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  COMET_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  return ctx->h_pinned[kStatusInvalid] ? COMET_ERR_INVALID_TENSOR : COMET_OK;
}
