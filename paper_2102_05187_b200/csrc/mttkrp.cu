// Root-mode MTTKRP, out[i, :] = sum over entries (i, j, k) of x * P[j, :] * Q[k, :] (the paper names
// the operation without defining it; this is the textbook matricised-tensor-times-Khatri-Rao product),
// for the two storage formats the paper's attributes compose for 3-order tensors:
//   COO [CN,S,S]  sorted entries, an output row is a run of equal root coordinates;
//   CSF [CU,CU,CU] per fiber t = sum x * Q[k, :], then out[i, :] += t * P[j, :] (one P row per fiber).
//
// Same worker scheme as the SpMM/TTM kernel (walk.cuh): a worker is LPN lanes of a warp walking a tile of
// consecutive leaf entries with a rolling window of row gathers in flight. A worker stores the output rows that END in its tile (and zero-fills the
// rows between consecutive stored rows, so no memset is needed), and writes the partial sum of the
// row it stops in to a carry slot that the fix-up kernel adds in tile order (deterministic).
#include <stdlib.h>

#include "common.cuh"
#include "kernels.cuh"
#include "walk.cuh"

#ifndef COMET_PF_COO
#define COMET_PF_COO 2        // entries in flight per worker, two row gathers each
#endif
#ifndef COMET_PF_CSF
#define COMET_PF_CSF 2       // entries in flight per worker (a Q row each, a P row where a fiber closes)
#endif
#ifndef COMET_MINB_COO
#define COMET_MINB_COO 4
#endif
#ifndef COMET_CSF_ROLLED_TAIL
#define COMET_CSF_ROLLED_TAIL true
#endif
#ifndef COMET_MINB_CSF
#define COMET_MINB_CSF 4
#endif


namespace comet {

struct MttkrpArgs {
  // COO: crd0/crd1/crd2/val over N entries. CSF: pos1 (S+1), crd0 (S), crd1 (F), seg_end2 (= pos2+1, F), crd2, val.
  const int32_t *pos1, *crd0, *crd1, *seg_end2, *crd2;
  const void *val;   // values, factors and output are T (double or float)
  int64_t S, F, N, rows;
  const void *P;     // factor gathered by the level-1 coordinate
  int64_t ldp;
  const void *Q;     // factor gathered by the level-2 (leaf) coordinate
  int64_t ldq;
  void *out;
  int64_t ldo;
  int32_t R;
  int32_t tile_items;
  int64_t num_tiles;
  double *carry_val;
  int32_t *carry_seg;
  int32_t carry_ld;
  const int32_t *part_fiber, *part_slice;   // CSF: per tile boundary, from the partition kernel (num_tiles + 1 each)
  bool level1;                              // CSF: the output mode is the one stored at level 1 (atomic accumulation)
};

// ------------------------------------------------------------------------------------------- COO
template <class T, int LPN, int CPL, int VEC>
struct CooPolicy {
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = COMET_PF_COO;   // two rows per entry
  static constexpr bool kAux = true;         // the root coordinate rides in the side ring
  static constexpr bool kFullUnroll = true;
  static constexpr bool kRolledTail = true;  // one copy of the unrolled body (instruction cache)
  struct Slot { T r[2][CPL][VEC]; };

  const MttkrpArgs &a;
  const L &ln;
  const char *pcol, *qcol;               // this lane's piece 0 of row 0 of P and of Q
  int32_t ldp_bytes, ldq_bytes;
  T *ocol;                               // this lane's piece 0 of row 0 of the output
  const T *val;
  double acc[CPL][VEC];
  int32_t cur;                           // output row being accumulated

  __device__ __forceinline__ CooPolicy(const MttkrpArgs &args, const L &lanes, int32_t first_row)
      : a(args), ln(lanes), cur(first_row) {
    ln.zero(acc);
    pcol = reinterpret_cast<const char *>(static_cast<const T *>(a.P) + ln.col0);
    qcol = reinterpret_cast<const char *>(static_cast<const T *>(a.Q) + ln.col0);
    ldp_bytes = (int32_t)(a.ldp * sizeof(T));
    ldq_bytes = (int32_t)(a.ldq * sizeof(T));
    ocol = static_cast<T *>(a.out) + ln.col0;
    val = static_cast<const T *>(a.val);
  }
  __device__ __forceinline__ void fetch(int32_t j, Entry16 &e, int32_t &aux) const {
    e.v = (double)ld_stream(val + j);
    e.a = ld_stream(a.crd1 + j);
    e.b = ld_stream(a.crd2 + j);
    aux = ld_stream(a.crd0 + j);
  }
  __device__ __forceinline__ void prefetch(int32_t cj, int32_t ck, Slot &s) const {
    ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)cj * ldp_bytes), s.r[0]);
    ln.gather(reinterpret_cast<const T *>(qcol + (int64_t)ck * ldq_bytes), s.r[1]);
  }
  __device__ __forceinline__ void begin_chunk(int32_t) {}
  // The run of `cur` ends here: store it. (Rows without entries are zero because the whole output is cleared
  // before the kernel: keeping the zero-fill loops out of here keeps the unrolled chunk body, which holds a copy
  // of this per entry, small enough for the instruction cache; that was worth more than the extra 40 us of
  // writes on the benchmark tensor.)
  __device__ __forceinline__ void next_row(int32_t row) {
    ln.store_row(ocol + (int64_t)cur * a.ldo, acc);
    ln.zero(acc);
    cur = row;
  }
  __device__ __forceinline__ void consume(int, double v, int32_t row, Slot &s) {
    if (row != cur) next_row(row);
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ln.ok[t])
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc[t][k] = fma(v * (double)s.r[0][t][k], (double)s.r[1][t][k], acc[t][k]);
  }
};

template <class T, int LPN, int CPL, int VEC>
__global__ void __launch_bounds__(kBlockThreads, (CPL * VEC * sizeof(T) <= 16 ? COMET_MINB_COO : 1)) mttkrp_coo_kernel(const MttkrpArgs a) {
  using L = Lanes<T, LPN, CPL, VEC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int worker = threadIdx.x / LPN;
  const int64_t tile = (int64_t)blockIdx.x * L::kWorkers + worker;
  if (tile >= a.num_tiles) return;
  using P = CooPolicy<T, LPN, CPL, VEC>;
  const uint32_t smem = smem_u32(smem_raw) + worker * RingLayout<L, true>::kWorkerBytes;
  const L ln(a.R);

  const int64_t j0 = tile * a.tile_items;
  const int64_t j1 = (j0 + a.tile_items < a.N) ? j0 + a.tile_items : a.N;
  const int32_t first = __ldg(a.crd0 + j0);
  P p(a, ln, first);
  walk_tile(ln, p, (int32_t)j0, (int32_t)j1, smem);

  const int64_t nxt = j1 < a.N ? (int64_t)__ldg(a.crd0 + j1) : -1;
  if (nxt == p.cur) {                                    // the row continues in the next tile
    if (ln.g == 0) a.carry_seg[tile] = p.cur;
    ln.store_carry(a.carry_val + tile * a.carry_ld + ln.col0, p.acc);
  } else {
    if (ln.g == 0) a.carry_seg[tile] = -1;
    ln.store_row(p.ocol + (int64_t)p.cur * a.ldo, p.acc);
  }
}

// ------------------------------------------------------------------------------------------- CSF
// Fibers are short (a few entries, most of them one), so what is done per FIBER decides the speed. The fibers
// and slices of a tile are therefore looked at once, before the walk and by all lanes at once: a worker scans the
// fiber ends that fall into its tile (coalesced reads of the level-2 positions and of the level-1 coordinates)
// and leaves, in a shared-memory array with one word per leaf entry of the tile, the P row index at the LAST
// entry of every fiber (-1 elsewhere); a second scan over the slices of the tile sets the top bit at the last
// entry of every slice. The walk then finds everything it needs in the staged entry: an entry that closes a
// fiber has that fiber's P row gathered together with its own Q row (same window, same distance ahead), closing
// a fiber is "slice sum += fiber sum * P row", closing a slice is one row store. No positions are followed and
// nothing is looked up entry by entry.
constexpr int32_t kNoEnd = -1;                      // flag word: no fiber ends at this entry
constexpr uint32_t kSliceEnd = 0x80000000u;         // flag word: P row index, top bit set if the slice ends too
                                                    // (a coordinate is below 2^31 - 1, so the two never collide)
constexpr int kCsfTileCap = 512;                    // leaf entries per tile: 16 mask words
constexpr int kCsfMaskWords = kCsfTileCap / 32;
constexpr int kCsfWorkerBytes = 3 * kCsfMaskWords * 4;   // fiber-end bits, slice-end bits, fiber ends in front of each word

__device__ __forceinline__ void atom_or_shared(uint32_t addr, uint32_t bits) {
  asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(addr), "r"(bits) : "memory");
}

// EXPAND: when the fibers are so short that most entries close one (mean length below 4), following the fibers
// costs more than it saves. The staging then hands EVERY entry the P row index of its fiber (the number of fiber
// ends in front of an entry is its fiber's number), both rows are gathered per entry, and the walk is the one of
// the sorted-COO kernel: slice sum += (x * P row) * Q row, a row store where a slice ends. The P rows of a
// fiber's later entries are L1 hits.
// FORM 2 (kCsfLevel1): the OUTPUT mode is the one stored at level 1. The walk is the same; a fiber's sum, times the
// row of the root mode's factor (P here, one row per slice), is added to output row crd1[fiber] with atomic adds
// (the rows of one output index are spread over the whole tensor, so no tile owns one); nothing is carried from
// tile to tile. Sums are double; the output must be zero when the kernel starts.
constexpr int kCsfFold = 0, kCsfExpand = 1, kCsfLevel1 = 2;

template <class T, int LPN, int CPL, int VEC, int FORM>
struct CsfPolicy {
  static constexpr bool EXPAND = FORM == kCsfExpand;
  static constexpr bool LEVEL1 = FORM == kCsfLevel1;
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = COMET_PF_CSF;
  static constexpr bool kAux = false;
  static constexpr bool kFullUnroll = true;
  static constexpr bool kRolledTail = COMET_CSF_ROLLED_TAIL;
  static constexpr bool kSlotCarries = true;               // value and flag word travel in the window slot
  struct Slot { T r[CPL][VEC]; T p[CPL][VEC]; double v; int32_t flag; };   // Q row of the entry; P row of its fiber if it closes one

  const MttkrpArgs &a;
  const L &ln;
  const char *pcol, *qcol;
  int32_t ldp_bytes, ldq_bytes;
  T *ocol;
  const T *val;
  double tac[CPL][VEC], aac[CPL][VEC];   // open fiber sum, open slice sum
  T arow[CPL][VEC];                      // LEVEL1: the root factor's row of the open slice
  uint32_t ends, slices, before;         // shared addresses of the tile's three word arrays
  int32_t j0, f0;
  int32_t s;                             // open slice
  int32_t f_open;                        // the fiber that is still open behind the tile's last fiber end
  bool a_dirty;

  // The look at the tile's fibers and slices (see above). f0 = first fiber that ends behind j0, s0 = its slice.
  __device__ __forceinline__ CsfPolicy(const MttkrpArgs &args, const L &lanes, int64_t f0_, int64_t f_open_, int64_t s0,
                                       int64_t s_open, int32_t j0_, uint32_t smem_words)
      : a(args), ln(lanes), ends(smem_words), slices(smem_words + kCsfMaskWords * 4), before(smem_words + 2 * kCsfMaskWords * 4),
        j0(j0_), f0((int32_t)f0_), s((int32_t)s0), a_dirty(false) {
    ln.zero(tac);
    ln.zero(aac);
    pcol = reinterpret_cast<const char *>(static_cast<const T *>(a.P) + ln.col0);
    qcol = reinterpret_cast<const char *>(static_cast<const T *>(a.Q) + ln.col0);
    ldp_bytes = (int32_t)(a.ldp * sizeof(T));
    ldq_bytes = (int32_t)(a.ldq * sizeof(T));
    ocol = static_cast<T *>(a.out) + ln.col0;
    val = static_cast<const T *>(a.val);
    if (LEVEL1 && s < a.S) ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)__ldg(a.crd0 + s) * ldp_bytes), arow);
    for (int w = ln.g; w < 2 * kCsfMaskWords; w += LPN) sts_s32(ends + w * 4, 0);
    ln.sync();
    // the fibers f0 .. f_open-1 end inside the tile, the slices s0 .. s_open-1 with them (both bounds come from the
    // partition, so the two scans have known lengths and their loads do not wait for one another)
    f_open = (int32_t)f_open_;
    for (int64_t k = f0_ + ln.g; k < f_open_; k += LPN) {
      const int32_t q = __ldg(a.seg_end2 + k) - 1 - j0;
      atom_or_shared(ends + (q >> 5) * 4, 1u << (q & 31));
    }
    for (int64_t k = s0 + ln.g; k < s_open; k += LPN) {    // slice k ends with fiber pos1[k + 1] - 1
      const int32_t q = __ldg(a.seg_end2 + __ldg(a.pos1 + k + 1) - 1) - 1 - j0;
      atom_or_shared(slices + (q >> 5) * 4, 1u << (q & 31));
    }
    ln.sync();
    for (int w = ln.g; w < kCsfMaskWords; w += LPN) {      // fiber ends in front of each word
      int32_t cnt = 0;
      for (int x = 0; x < w; ++x) cnt += __popc((uint32_t)lds_s32(ends + x * 4));
      sts_s32(before + w * 4, cnt);
    }
    ln.sync();
  }
  __device__ __forceinline__ void begin_chunk(int32_t) {}
  // the flag word of leaf entry j: the P row index of its fiber if it is the fiber's last entry
  __device__ __forceinline__ int32_t flag_of(int32_t j) const {
    const int32_t q = j - j0;
    const uint32_t w = (uint32_t)lds_s32(ends + (q >> 5) * 4);
    const uint32_t bit = 1u << (q & 31);
    if (!EXPAND && !(w & bit)) return kNoEnd;
    const int32_t f = f0 + lds_s32(before + (q >> 5) * 4) + __popc(w & (bit - 1u));
    const uint32_t row = (uint32_t)__ldg(a.crd1 + f);
    return (int32_t)(((uint32_t)lds_s32(slices + (q >> 5) * 4) & bit) ? (row | kSliceEnd) : row);
  }
  __device__ __forceinline__ void fetch(int32_t j, Entry16 &e, int32_t &) const {
    e.v = (double)ld_stream(val + j);
    e.a = ld_stream(a.crd2 + j);
    e.b = flag_of(j);
  }
  __device__ __forceinline__ void prefetch_entry(const Entry16 &e, Slot &sl) const {
    const int32_t ck = e.a, flag = e.b;
    sl.v = e.v;
    sl.flag = flag;
    ln.gather(reinterpret_cast<const T *>(qcol + (int64_t)ck * ldq_bytes), sl.r);
    if (!LEVEL1 && (EXPAND || flag != kNoEnd))
      ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)(int32_t)((uint32_t)flag & ~kSliceEnd) * ldp_bytes), sl.p);
  }
  __device__ __forceinline__ void fold(const T (&prow)[CPL][VEC]) {      // aac += tac * P[crd1[f], :]
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ln.ok[t])
#pragma unroll
        for (int k = 0; k < VEC; ++k) { aac[t][k] = fma(tac[t][k], (double)prow[t][k], aac[t][k]); tac[t][k] = 0.0; }
    a_dirty = true;
  }
  // The slice is complete: this worker owns its row. (The rows that no slice owns are zero-filled by a kernel of
  // their own, so that this stays short.)
  __device__ __forceinline__ void close_slice() {
    ln.store_row(ocol + (int64_t)__ldg(a.crd0 + s) * a.ldo, aac);
    ln.zero(aac);
    a_dirty = false;
    ++s;
  }
  // LEVEL1: out[row, :] += tac * arow (atomic), tac = 0
  __device__ __forceinline__ void scatter_fiber(int32_t row) {
    if constexpr (CPL == 1 && VEC == 2) {
      // A lane holds two ADJACENT columns. Added as they lie, each of the two requests would touch every other
      // pair of the row: twice the 32-byte sectors for L2, which processes atomic adds sector by sector. The
      // lanes exchange their products so that one request covers the first LPN columns and the other the rest.
      const double p0 = tac[0][0] * (double)arow[0][0], p1 = tac[0][1] * (double)arow[0][1];
      tac[0][0] = 0.0; tac[0][1] = 0.0;
      const int lo_src = ln.g >> 1, hi_src = (LPN >> 1) + (ln.g >> 1);
      const double l0 = __shfl_sync(ln.mask, p0, lo_src, LPN), l1 = __shfl_sync(ln.mask, p1, lo_src, LPN);
      const double h0 = __shfl_sync(ln.mask, p0, hi_src, LPN), h1 = __shfl_sync(ln.mask, p1, hi_src, LPN);
      double *base = reinterpret_cast<double *>(a.out) + (int64_t)row * a.ldo + (ln.col0 - ln.g * VEC);
      atomicAdd(base + ln.g, (ln.g & 1) ? l1 : l0);
      atomicAdd(base + LPN + ln.g, (ln.g & 1) ? h1 : h0);
      return;
    }
    double *dst = reinterpret_cast<double *>(a.out) + (int64_t)row * a.ldo + ln.col0;
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ln.ok[t])
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          atomicAdd(dst + t * L::kStride + k, tac[t][k] * (double)arow[t][k]);
          tac[t][k] = 0.0;
        }
  }
  __device__ __forceinline__ void consume_slot(int, Slot &sl) {
    struct { double v; int32_t b; } e{sl.v, sl.flag};
    if (LEVEL1) {
      ln.fma_rows(e.v, sl.r, tac);
      if (e.b != kNoEnd) {
        scatter_fiber((int32_t)((uint32_t)e.b & ~kSliceEnd));
        if (e.b < 0 && ++s < a.S) ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)__ldg(a.crd0 + s) * ldp_bytes), arow);
      }
      return;
    }
    if (EXPAND) {
#pragma unroll
      for (int t = 0; t < CPL; ++t)
        if (ln.ok[t])
#pragma unroll
          for (int k = 0; k < VEC; ++k) aac[t][k] = fma(e.v * (double)sl.p[t][k], (double)sl.r[t][k], aac[t][k]);
      if (e.b < 0) close_slice();
      return;
    }
    ln.fma_rows(e.v, sl.r, tac);
    if (e.b != kNoEnd) {
      fold(sl.p);
      if (e.b < 0) close_slice();
    }
  }
  // After the walk of [j0, j1): the entries behind the last fiber end belong to a fiber that goes on in the next
  // tile; they contribute through distributivity.
  __device__ __forceinline__ void finish(int32_t j1) {
    const int32_t q = j1 - 1 - j0;
    if (EXPAND) {                                          // the slice sum is open unless the last entry closed a slice
      a_dirty = !(((uint32_t)lds_s32(slices + (q >> 5) * 4) >> (q & 31)) & 1u);
      return;
    }
    if (((uint32_t)lds_s32(ends + (q >> 5) * 4) >> (q & 31)) & 1u) return;     // the tile stops at a fiber end
    if (LEVEL1) { scatter_fiber(__ldg(a.crd1 + f_open)); return; }
    T prow[CPL][VEC];
    ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)__ldg(a.crd1 + f_open) * ldp_bytes), prow);
    fold(prow);
  }
};

// Tile boundaries of the CSF kernel, a thread per boundary: the merge-path split of (fiber-end markers, leaf
// positions) at item t * tile_items, then the slice of the first fiber whose entries reach into the tile. The
// slice is stored complemented when that fiber is the one after the split's (its end marker is the next item).
__global__ void __launch_bounds__(kBlockThreads) csf_partition_kernel(const int32_t *__restrict__ seg_end2,
                                                                      const int32_t *__restrict__ pos1, int64_t S, int64_t F,
                                                                      int64_t N, int32_t tile_items, int64_t num_tiles,
                                                                      int32_t *__restrict__ part_fiber,
                                                                      int32_t *__restrict__ part_slice) {
  const int64_t t = (int64_t)blockIdx.x * kBlockThreads + threadIdx.x;
  if (t > num_tiles) return;
  const int64_t total = F + N;
  const int64_t d = t * tile_items < total ? t * tile_items : total;
  int64_t f = merge_path_segments(seg_end2, F, N, d);
  part_fiber[t] = (int32_t)f;
  const bool skip = f < F && (int64_t)__ldg(seg_end2 + f) == d - f;
  if (skip) ++f;
  int64_t lo = 0, hi = S;                                  // slices that end at or before fiber f (every slice is non-empty)
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(pos1 + mid + 1) <= f) lo = mid + 1; else hi = mid;
  }
  part_slice[t] = skip ? ~(int32_t)lo : (int32_t)lo;
}

// Zero-fills the output rows that no slice owns: the rows between the coordinates of consecutive slices, before
// the first and behind the last. A warp looks at 32 slices at a time and clears the gaps it finds together.
template <class T>
__global__ void __launch_bounds__(kBlockThreads) zero_unowned_rows_kernel(const int32_t *__restrict__ crd0, int64_t S, int64_t rows,
                                                                          T *__restrict__ out, int64_t ldo, int32_t R) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * kBlockThreads + threadIdx.x) >> 5;
  const int64_t s = warp * 32 + lane;                      // gap s lies in front of slice s; gap S behind the last slice
  int64_t lo = 0, hi = 0;
  if (s <= S) {
    lo = s > 0 ? (int64_t)__ldg(crd0 + s - 1) + 1 : 0;
    hi = s < S ? (int64_t)__ldg(crd0 + s) : rows;
  }
  unsigned todo = __ballot_sync(0xffffffffu, hi > lo);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const int64_t a = __shfl_sync(0xffffffffu, lo, src), b = __shfl_sync(0xffffffffu, hi, src);
    for (int64_t i = (a * R) + lane; i < b * R; i += 32) {
      const int64_t r = i / R;
      out[r * ldo + (i - r * R)] = (T)0;
    }
  }
}

template <class T, int LPN, int CPL, int VEC, int FORM>
__global__ void __launch_bounds__(kBlockThreads, (CPL * VEC * sizeof(T) <= 16 ? COMET_MINB_CSF : 2)) mttkrp_csf_kernel(const MttkrpArgs a) {
  using L = Lanes<T, LPN, CPL, VEC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int worker = threadIdx.x / LPN;
  const int64_t tile = (int64_t)blockIdx.x * L::kWorkers + worker;
  if (tile >= a.num_tiles) return;
  using P = CsfPolicy<T, LPN, CPL, VEC, FORM>;
  const uint32_t smem = smem_u32(smem_raw) + worker * RingLayout<L, false>::kWorkerBytes;
  const uint32_t flags = smem_u32(smem_raw) + (uint32_t)RingLayout<L, false>::kBlockBytes + worker * kCsfWorkerBytes;
  const L ln(a.R);

  // A tile is a span of the merge list of fiber-end markers and leaf positions (equal work per tile: an entry
  // costs a gather, a fiber another one). It owns the leaf entries of the span and the fibers whose LAST entry
  // is among them.
  // Where the tile starts (fiber, slice) was found by the partition kernel: a worker is sequential, so dependent
  // searches at the head of every tile would cost it a third of its time.
  const int64_t total = a.F + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  const int64_t f0 = __ldg(a.part_fiber + tile), f1 = __ldg(a.part_fiber + tile + 1);
  const int32_t j0 = (int32_t)(d0 - f0), j1 = (int32_t)(d1 - f1);
  if (j0 >= j1) {                                          // nothing but an end marker: its fiber was closed by the tile before
    if (FORM != kCsfLevel1 && ln.g == 0) a.carry_seg[tile] = -1;
    return;
  }
  // The partition stores the slice complemented when the split's fiber has all its entries in front of the split
  // (its end marker is the next item): that fiber belongs to the tile before. So this tile owns the fibers from
  // its own corrected start to the next tile's corrected start, and the slices likewise.
  const int32_t s0 = __ldg(a.part_slice + tile), s1 = __ldg(a.part_slice + tile + 1);
  P p(a, ln, f0 + (s0 < 0 ? 1 : 0), f1 + (s1 < 0 ? 1 : 0), s0 < 0 ? ~s0 : s0, s1 < 0 ? ~s1 : s1, j0, flags);
  walk_tile(ln, p, j0, j1, smem);
  p.finish(j1);
  if (FORM == kCsfLevel1) return;                          // everything went out through atomic adds
  const bool carry = p.a_dirty && p.s < a.S;
  if (ln.g == 0) a.carry_seg[tile] = carry ? (int32_t)p.s : -1;
  if (carry) ln.store_carry(a.carry_val + tile * a.carry_ld + ln.col0, p.aac);
}

// ------------------------------------------------------------------------------------------- host
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <bool CSF, class T, int LPN, int CPL, int VEC>
static comet_status_t launch_mttkrp(Context *ctx, MttkrpArgs a, cudaStream_t stream) {
  constexpr int WORKERS = kBlockThreads / LPN;
  const int64_t total = CSF ? a.F + a.N : a.N;
  using L = Lanes<T, LPN, CPL, VEC>;
  a.tile_items = choose_tile_items(total, WORKERS);
  if (CSF && a.tile_items > kCsfTileCap) a.tile_items = kCsfTileCap;          // one mask bit per leaf entry of a tile
  a.num_tiles = ceil_div(total, a.tile_items);
  a.carry_ld = (int32_t)align_up((size_t)a.R, 2);
  const size_t val_bytes = align_up((size_t)a.num_tiles * a.carry_ld * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  const size_t part_bytes = CSF ? align_up((size_t)(a.num_tiles + 1) * sizeof(int32_t), 256) : 0;
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes + 2 * part_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  if (CSF) {
    int32_t *pf = (int32_t *)(scratch + val_bytes + seg_bytes), *ps = (int32_t *)(scratch + val_bytes + seg_bytes + part_bytes);
    csf_partition_kernel<<<(unsigned)ceil_div(a.num_tiles + 1, kBlockThreads), kBlockThreads, 0, stream>>>(
        a.seg_end2, a.pos1, a.S, a.F, a.N, a.tile_items, a.num_tiles, pf, ps);
    COMET_LAUNCH_CHECK(ctx);
    a.part_fiber = pf;
    a.part_slice = ps;
  }
  const unsigned blocks = (unsigned)ceil_div(a.num_tiles, WORKERS);
  constexpr size_t smem = CSF ? RingLayout<L, false>::kBlockBytes + (size_t)WORKERS * kCsfWorkerBytes
                              : RingLayout<L, true>::kBlockBytes;
  // CSF with short fibers (mean length below 4): the per-entry form; COMET_CSF_FORM=fold / expand forces one
  bool expand = CSF && a.N < 4 * a.F;
  if (const char *e = getenv("COMET_CSF_FORM")) expand = CSF && (e[0] == 'e' ? true : (e[0] == 'f' ? false : expand));
  auto kernel = !CSF ? mttkrp_coo_kernel<T, LPN, CPL, VEC>
                     : (expand ? mttkrp_csf_kernel<T, LPN, CPL, VEC, kCsfExpand> : mttkrp_csf_kernel<T, LPN, CPL, VEC, kCsfFold>);
  if constexpr (CSF && sizeof(T) == 8 && VEC == 2 && CPL == 1) {
    if (a.level1) kernel = mttkrp_csf_kernel<T, LPN, CPL, VEC, kCsfLevel1>;
  }
  if (smem > 48 * 1024)
    COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kernel<<<blocks, kBlockThreads, smem, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
  if (CSF && a.level1) return COMET_OK;
  carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, a.R, a.carry_ld, a.out,
                     a.ldo, CSF ? a.crd0 : nullptr, stream);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

template <bool CSF, class T>
static comet_status_t mttkrp_chunks(Context *ctx, MttkrpArgs base, int64_t R, cudaStream_t stream) {
  constexpr int PER = 16 / sizeof(T);
  const bool vec_ok = aligned16(base.P) && aligned16(base.Q) && aligned16(base.out) && base.ldp % PER == 0 &&
                      base.ldq % PER == 0 && base.ldo % PER == 0;
  int64_t done = 0;
  while (done < R) {
    const int64_t rem = R - done;
    const int64_t chunk = rem < 128 ? rem : 128;
    MttkrpArgs a = base;
    a.P = static_cast<const T *>(base.P) + done;
    a.Q = static_cast<const T *>(base.Q) + done;
    a.out = static_cast<T *>(base.out) + done;
    a.R = (int32_t)chunk;
    const bool v = vec_ok && done % PER == 0 && chunk % PER == 0;
    const int64_t pieces = chunk / PER;
    comet_status_t st;
    if (v && pieces == 64) st = launch_mttkrp<CSF, T, 32, 2, PER>(ctx, a, stream);
    else if (v && pieces == 32) st = launch_mttkrp<CSF, T, 32, 1, PER>(ctx, a, stream);
    else if (v && pieces == 16) st = launch_mttkrp<CSF, T, 16, 1, PER>(ctx, a, stream);
    else if (v && pieces == 8) st = launch_mttkrp<CSF, T, 8, 1, PER>(ctx, a, stream);
    else if (v && pieces == 4) st = launch_mttkrp<CSF, T, 4, 1, PER>(ctx, a, stream);
    else if (v && pieces == 2) st = launch_mttkrp<CSF, T, 2, 1, PER>(ctx, a, stream);
    else if (v && pieces == 1) st = launch_mttkrp<CSF, T, 1, 1, PER>(ctx, a, stream);
    else if (chunk > 64) st = launch_mttkrp<CSF, T, 32, 4, 1>(ctx, a, stream);
    else if (chunk > 32) st = launch_mttkrp<CSF, T, 32, 2, 1>(ctx, a, stream);
    else st = launch_mttkrp<CSF, T, 32, 1, 1>(ctx, a, stream);
    if (st != COMET_OK) return st;
    done += chunk;
  }
  return COMET_OK;
}

comet_status_t mttkrp_coo(Context *ctx, int dtype, const int32_t *crd0, const int32_t *crd1, const int32_t *crd2,
                          const void *val, int64_t N, int64_t rows, const void *P, int64_t ldp, const void *Q,
                          int64_t ldq, int64_t R, void *out, int64_t ldo, cudaStream_t stream) {
  if (ldp >= (1ll << 28) || ldq >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;
  {                                                        // rows without entries stay zero; the others are stored over
    const size_t elt = dtype == COMET_F32 ? 4 : 8;
    if (ldo == R) COMET_CUDA_TRY(ctx, cudaMemsetAsync(out, 0, (size_t)rows * R * elt, stream));
    else {
      const comet_status_t zs = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
      if (zs != COMET_OK) return zs;
    }
  }
  if (N == 0) return COMET_OK;
  MttkrpArgs a{};
  a.crd0 = crd0; a.crd1 = crd1; a.crd2 = crd2; a.val = val; a.N = N; a.rows = rows;
  a.P = P; a.ldp = ldp; a.Q = Q; a.ldq = ldq; a.out = out; a.ldo = ldo;
  return dtype == COMET_F32 ? mttkrp_chunks<false, float>(ctx, a, R, stream) : mttkrp_chunks<false, double>(ctx, a, R, stream);
}

comet_status_t mttkrp_csf(Context *ctx, int dtype, const int32_t *pos1, const int32_t *crd0, const int32_t *crd1,
                          const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S, int64_t F,
                          int64_t N, int64_t rows, const void *P, int64_t ldp, const void *Q, int64_t ldq,
                          int64_t R, void *out, int64_t ldo, cudaStream_t stream) {
  if (ldp >= (1ll << 28) || ldq >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;
  if (N == 0 || S == 0) return zero_rows(ctx, out, dtype, rows, R, ldo, stream);
  MttkrpArgs a{};
  a.pos1 = pos1; a.crd0 = crd0; a.crd1 = crd1; a.seg_end2 = pos2 + 1; a.crd2 = crd2; a.val = val;
  a.S = S; a.F = F; a.N = N; a.rows = rows;
  a.P = P; a.ldp = ldp; a.Q = Q; a.ldq = ldq; a.out = out; a.ldo = ldo;
  {                                                        // rows that no slice owns (all R columns at once)
    const unsigned blocks = (unsigned)ceil_div(S + 1, kBlockThreads);
    if (dtype == COMET_F32) zero_unowned_rows_kernel<float><<<blocks, kBlockThreads, 0, stream>>>(crd0, S, rows, (float *)out, ldo, (int32_t)R);
    else zero_unowned_rows_kernel<double><<<blocks, kBlockThreads, 0, stream>>>(crd0, S, rows, (double *)out, ldo, (int32_t)R);
    COMET_LAUNCH_CHECK(ctx);
  }
  return dtype == COMET_F32 ? mttkrp_chunks<true, float>(ctx, a, R, stream) : mttkrp_chunks<true, double>(ctx, a, R, stream);
}

// CSF, output mode stored at level 1: out[crd1[f], :] += (sum over fiber f of val * Q[crd2, :]) * P[crd0[slice of f], :].
// fp64 with 16-byte aligned operands and R a multiple of 2 up to 64; returns COMET_ERR_UNSUPPORTED_FORMAT otherwise
// (the caller then takes the general scatter kernel). `out` is zero-filled here.
comet_status_t mttkrp_csf_level1(Context *ctx, int dtype, const int32_t *pos1, const int32_t *crd0, const int32_t *crd1,
                                 const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S, int64_t F, int64_t N,
                                 int64_t rows, const void *P, int64_t ldp, const void *Q, int64_t ldq, int64_t R, void *out,
                                 int64_t ldo, cudaStream_t stream) {
  if (dtype != COMET_F64 || !(R == 2 || R == 4 || R == 8 || R == 16 || R == 32 || R == 64) || N == 0 || S == 0)
    return COMET_ERR_UNSUPPORTED_FORMAT;
  if (!aligned16(P) || !aligned16(Q) || !aligned16(out) || ldp % 2 || ldq % 2 || ldo % 2) return COMET_ERR_UNSUPPORTED_FORMAT;
  if (ldp >= (1ll << 28) || ldq >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;
  if (ldo == R) {
    COMET_CUDA_TRY(ctx, cudaMemsetAsync(out, 0, (size_t)rows * R * sizeof(double), stream));
  } else {
    const comet_status_t zs = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
    if (zs != COMET_OK) return zs;
  }
  MttkrpArgs a{};
  a.pos1 = pos1; a.crd0 = crd0; a.crd1 = crd1; a.seg_end2 = pos2 + 1; a.crd2 = crd2; a.val = val;
  a.S = S; a.F = F; a.N = N; a.rows = rows;
  a.P = P; a.ldp = ldp; a.Q = Q; a.ldq = ldq; a.out = out; a.ldo = ldo;
  a.level1 = true;
  return mttkrp_chunks<true, double>(ctx, a, R, stream);
}

}  // namespace comet
