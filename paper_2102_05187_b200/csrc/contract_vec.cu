// Segment-gather contractions with a dense matrix operand: SpMM, TTM (the SpMM/SpTTM definitions of
// the paper's Sparse Tensor Operations subsection). Both are "for every leaf entry p of segment s:
// out[s, :] += val[p] * B[crd[p], :]" where a segment is a CSR row (SpMM) or a CSF fiber (TTM).
//
// Work split (B200): the merge list of segment-end markers and leaf positions is cut into tiles of a
// fixed number of items, one tile per WORKER (a group of LPN lanes of a warp, see walk.cuh). A worker
// walks its tile sequentially with a rolling window of row gathers in flight, stores every segment
// that ENDS inside its tile with plain vector stores (so every output row is written exactly once,
// without a memset), and hands the partial sum of the segment it stops in to a carry slot. A second
// small kernel adds the carries of earlier tiles onto the stored rows in tile order, which makes the
// result deterministic (no atomics anywhere).
#include "common.cuh"
#include "kernels.cuh"
#include "walk.cuh"
#include "spmm_heavy.cuh"

#ifndef COMET_PF_GATHER
#define COMET_PF_GATHER 4      // row gathers in flight per worker (SpMM, TTM); measured best with 4 CTAs/SM
#endif
#ifndef COMET_MINB_GATHER
#define COMET_MINB_GATHER 4    // CTAs per SM the register budget is held to (64 registers)
#endif

namespace comet {

struct SegGatherArgs {
  const int32_t *seg_end;   // M entries: leaf position where segment s ends (= pos + 1)
  const int32_t *crd;       // N leaf coordinates (row index into B)
  const void *val;          // N values (T)
  int64_t M, N;
  const void *B;            // dense operand (T), already offset to this launch's first column
  int64_t ldb;
  void *C;                  // output rows (T), already offset to this launch's first column
  int64_t ldc;
  const int32_t *out_row;   // NULL: segment s -> row s. Else segment s -> row out_row[s] (ascending) and the
  int64_t out_rows;         //   rows in between (and up to out_rows) are zero-filled by the flushing worker
  int32_t R;                // columns handled by this launch
  int32_t tile_items;
  int64_t num_tiles;
  double *carry_val;        // num_tiles x carry_ld
  int32_t *carry_seg;       // num_tiles: segment the carry belongs to, -1 if none
  int32_t carry_ld;
  const int32_t *part;      // num_tiles + 1 merge-path splits (segments in front of each tile boundary), or NULL
  int32_t own_len;          // segments of at most this many entries are processed whole by the tile of their end marker
  int32_t skip_len;         // > 0: segments of at least this many entries are somebody else's (the long-row
                            //      path of SpMM): neither walked nor stored here. Never below tile_items.
};

// What the walker does with one leaf entry: close the segments that end in front of it, accumulate.
template <class T, int LPN, int CPL, int VEC, bool MAPPED, bool PASS_THROUGH = false>
struct SegGatherPolicy {
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = COMET_PF_GATHER;
  static constexpr bool kAux = false;
  static constexpr bool kFullUnroll = true;
  // one copy of the unrolled body where the chunk is long (instruction cache; measured: SpMM config 2 -4 %); the
  // narrow shapes have short tiles of short chunks, where the slower rolled tail costs more than it saves (TTM +5 %)
  static constexpr bool kRolledTail = LPN >= 16;
  struct Slot { T r[CPL][VEC]; };

  const SegGatherArgs &a;
  const L &ln;
  const char *bcol;         // this lane's piece 0 of row 0 of B
  double acc[CPL][VEC];
  // The segment state is three words (the rest is recomputed where a segment closes): registers are what the
  // window of gathers in flight is made of.
  int32_t seg;              // the open segment
  int32_t base, rel_end;    // chunk base; where the open segment ends, relative to it (negative: no segment left)
  uint64_t pass;            // PASS_THROUGH: L2 evict-first policy of the gathers (the other role's block of B stays)

  __device__ __forceinline__ SegGatherPolicy(const SegGatherArgs &args, const L &lanes, int64_t i0, int32_t j0)
      : a(args), ln(lanes), seg((int32_t)i0), base(j0) {
    ln.zero(acc);
    if (PASS_THROUGH) pass = l2_policy_evict_first();
    bcol = reinterpret_cast<const char *>(static_cast<const T *>(a.B) + ln.col0);
    rel_end = end_of_open();
  }
  __device__ __forceinline__ int32_t end_of_open() const {
    return seg < a.M ? __ldg(a.seg_end + seg) - base : (int32_t)0x80000000 / 2;
  }
  __device__ __forceinline__ int64_t segment() const { return seg; }
  __device__ __forceinline__ void fetch(int32_t j, Entry16 &e, int32_t &) const {
    e.v = (double)ld_stream(static_cast<const T *>(a.val) + j);
    e.a = ld_stream(a.crd + j);
  }
  __device__ __forceinline__ void prefetch(int32_t c, int32_t, Slot &s) const {
    const T *row = reinterpret_cast<const T *>(bcol + (int64_t)c * (int32_t)(a.ldb * sizeof(T)));
    if (PASS_THROUGH) ln.gather_hint(row, s.r, pass);
    else ln.gather(row, s.r);
  }
  __device__ __forceinline__ void begin_chunk(int32_t b) { rel_end -= b - base; base = b; }

  // Stores the open segment (and, for a compressed root level, zero-fills the rows in front of it).
  __device__ __forceinline__ void flush() {
    T *cmat = static_cast<T *>(a.C) + ln.col0;
    if (MAPPED) {
      const int64_t i = seg;
      const int64_t r = __ldg(a.out_row + i);
      const int64_t lo = (i > 0) ? (int64_t)__ldg(a.out_row + i - 1) + 1 : 0;
      ln.zero_rows(cmat, a.ldc, lo, r);
      if (i == a.M - 1) ln.zero_rows(cmat, a.ldc, r + 1, a.out_rows);
      ln.store_row(cmat + r * a.ldc, acc);
    } else {
      ln.store_row(cmat + (int64_t)seg * a.ldc, acc);
    }
    ln.zero(acc);
    ++seg;
    rel_end = end_of_open();
  }
  __device__ __forceinline__ void consume(int q, double v, int32_t, Slot &s) {
    while (rel_end == q) flush();              // segments (possibly empty ones) that end in front of this leaf
    ln.fma_rows(v, s.r, acc);
  }
};

// HEAVY: the first h.heavy_ctas CTAs of the grid work on the long rows of an SpMM (spmm_heavy.cuh) while the
// others walk the general tiles and skip those rows. The two roles are bound by different things (the long rows
// by the L2 -> L1 fill rate, the rest by DRAM latency), so sharing the SMs between them is faster than running
// one after the other.
template <class T, int LPN, int CPL, int VEC, bool MAPPED, bool HEAVY>
__global__ void __launch_bounds__(kBlockThreads, (CPL * VEC * sizeof(T) <= 16 ? COMET_MINB_GATHER : 2))
seg_gather_kernel(const SegGatherArgs a, const HeavyArgs h) {
  using L = Lanes<T, LPN, CPL, VEC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (HEAVY && (int)blockIdx.x < h.heavy_ctas) {
    heavy_role<T, LPN, CPL, VEC>(h, smem_raw);
    return;
  }
  const int worker = threadIdx.x / LPN;
  const int64_t tile = (int64_t)(blockIdx.x - (HEAVY ? h.heavy_ctas : 0)) * L::kWorkers + worker;
  if (tile >= a.num_tiles) return;                       // whole groups leave together
  const uint32_t smem = smem_u32(smem_raw) + worker * RingLayout<L, false>::kWorkerBytes;
  const L ln(a.R);

  const int64_t total = a.M + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  // the splits come from the partition kernel when there is one: a worker is sequential, and two dependent
  // searches at the head of every tile are a sizeable part of a short tile
  int64_t i0 = a.part ? (int64_t)__ldg(a.part + tile) : merge_path_segments_coop<LPN>(a.seg_end, a.M, a.N, d0, ln.g, ln.mask);
  const int64_t i1 = a.part ? (int64_t)__ldg(a.part + tile + 1) : merge_path_segments_coop<LPN>(a.seg_end, a.M, a.N, d1, ln.g, ln.mask);
  int32_t j0 = (int32_t)(d0 - i0), j1 = (int32_t)(d1 - i1);
  if (a.skip_len > 0) {
    // A long segment holds more entries than a tile, so it can only be the one open at the tile's start or the
    // one open at its end. Its entries are left out; its end marker (if it is in this tile) stores nothing.
    if (i0 < a.M) {
      const int32_t end0 = __ldg(a.seg_end + i0);
      const int32_t start0 = i0 > 0 ? __ldg(a.seg_end + i0 - 1) : 0;
      if (end0 - start0 >= a.skip_len) {
        if (i0 >= i1) {                                      // the whole tile lies inside the long segment
          if (ln.g == 0) a.carry_seg[tile] = -1;
          return;
        }
        i0 += 1;
        j0 = end0;
      }
    }
    if (i1 < a.M) {
      const int32_t start1 = i1 > 0 ? __ldg(a.seg_end + i1 - 1) : 0;
      if (__ldg(a.seg_end + i1) - start1 >= a.skip_len && start1 < j1) j1 = start1 > j0 ? start1 : j0;
    }
  }

  // A segment of at most `own_len` entries belongs wholly to the tile that holds its end marker: the tile
  // in front leaves the segment's first entries out and this one takes them, so such a segment needs no carry
  // (and no fix-up work). Both tiles look at the same segment and decide alike; longer segments are split as
  // before. The limit is a quarter of a tile, so that tiles stay within 25 % of their nominal size.
  // Measured: config 4 TTM 416 -> 399 us with any limit from an eighth of a tile to a whole one. Not done beside
  // the long-row role (SpMM config 2: 1017 us without, 1020 / 1026 / 1041 / 1079 us with an eighth / a quarter / half
  // a tile / a whole tile: its rows of a few hundred entries make the tiles uneven, which costs more than their
  // carries did).
  if (!HEAVY) {
    if (i0 < a.M) {
      const int32_t start0 = i0 > 0 ? __ldg(a.seg_end + i0 - 1) : 0;
      if (__ldg(a.seg_end + i0) - start0 <= a.own_len && start0 < j0) j0 = start0;
    }
    if (i1 < a.M) {
      const int32_t start1 = i1 > 0 ? __ldg(a.seg_end + i1 - 1) : 0;
      if (__ldg(a.seg_end + i1) - start1 <= a.own_len && start1 < j1) j1 = start1 > j0 ? start1 : j0;
    }
  }

  SegGatherPolicy<T, LPN, CPL, VEC, MAPPED, HEAVY> p(a, ln, i0, j0);
  walk_tile(ln, p, j0, j1, smem);
  while (p.segment() < i1) p.flush();                    // end markers that close the tile

  // leaf entries of a segment that ends in a later tile: the open segment starts in front of the tile's end
  const int64_t seg = p.segment();
  const int32_t open_from = seg > 0 ? __ldg(a.seg_end + seg - 1) : 0;
  const bool carry = seg < a.M && (open_from > j0 ? open_from : j0) < j1;
  if (ln.g == 0) a.carry_seg[tile] = carry ? (int32_t)seg : -1;
  if (carry) ln.store_carry(a.carry_val + tile * a.carry_ld + ln.col0, p.acc);
}

// Merge-path split at every tile boundary, a thread per boundary (a warp per boundary with a 32-way search was
// measured: slower, the boundaries are many and the searches hide each other's latency).
__global__ void __launch_bounds__(kBlockThreads) seg_partition_kernel(const int32_t *__restrict__ seg_end, int64_t M, int64_t N,
                                                                      int32_t tile_items, int64_t num_tiles,
                                                                      int32_t *__restrict__ part) {
  const int64_t t = (int64_t)blockIdx.x * kBlockThreads + threadIdx.x;
  if (t > num_tiles) return;
  const int64_t total = M + N;
  const int64_t d = t * tile_items < total ? t * tile_items : total;
  part[t] = (int32_t)merge_path_segments(seg_end, M, N, d);
}

// Adds the carries onto the stored rows. Tiles that stopped inside the same segment are consecutive;
// the first of such a run sums the run in tile order and updates the row (the only writer of it now).
// A heavy segment spans hundreds of tiles, so the run is read eight tiles at a time with all loads in
// flight together (the additions keep the tile order).
template <class T>
__device__ __forceinline__ void carry_fixup_role(int64_t block, const double *__restrict__ carry_val,
                                                 const int32_t *__restrict__ carry_seg, int64_t num_tiles, int32_t R,
                                                 int32_t carry_ld, T *__restrict__ C, int64_t ldc,
                                                 const int32_t *__restrict__ out_row) {
  const int64_t idx = block * blockDim.x + threadIdx.x;
  const int64_t tile = idx / R;
  const int32_t c = (int32_t)(idx - tile * R);
  if (tile >= num_tiles) return;
  const int32_t seg = carry_seg[tile];
  if (seg < 0) return;
  if (tile > 0 && carry_seg[tile - 1] == seg) return;
  double sum = carry_val[tile * carry_ld + c];
  bool more = true;
  for (int64_t t = tile + 1; more; t += 8) {
    int32_t s[8];
    double v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const bool in = t + u < num_tiles;
      s[u] = in ? __ldg(carry_seg + t + u) : -2;
      v[u] = in ? __ldcs(carry_val + (t + u) * carry_ld + c) : 0.0;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      more = more && s[u] == seg;
      if (more) sum += v[u];
    }
  }
  const int64_t row = out_row ? (int64_t)out_row[seg] : (int64_t)seg;
  C[row * ldc + c] = (T)((double)C[row * ldc + c] + sum);
}

template <class T>
__global__ void __launch_bounds__(kBlockThreads) carry_fixup_kernel(const double *__restrict__ carry_val,
                                                                    const int32_t *__restrict__ carry_seg, int64_t num_tiles,
                                                                    int32_t R, int32_t carry_ld, T *__restrict__ C, int64_t ldc,
                                                                    const int32_t *__restrict__ out_row) {
  carry_fixup_role<T>(blockIdx.x, carry_val, carry_seg, num_tiles, R, carry_ld, C, ldc, out_row);
}

// SpMM with the long-row path: both fix-ups in one launch. They read different scratch and write different rows
// of C (the general tiles leave the long rows out, so no carry names one), so the first `heavy_blocks` CTAs add
// the long rows' slots while the others add the carries.
template <class T>
__global__ void __launch_bounds__(kBlockThreads) spmm_fixups_kernel(const HeavyArgs h, int heavy_blocks,
                                                                    const double *__restrict__ carry_val,
                                                                    const int32_t *__restrict__ carry_seg, int64_t num_tiles,
                                                                    int32_t R, int32_t carry_ld, T *__restrict__ C, int64_t ldc) {
  if ((int)blockIdx.x < heavy_blocks) heavy_fixup_role<T>(h, (int)blockIdx.x, heavy_blocks);
  else carry_fixup_role<T>((int64_t)blockIdx.x - heavy_blocks, carry_val, carry_seg, num_tiles, R, carry_ld, C, ldc, nullptr);
}

void carry_fixup_launch(int dtype, const double *carry_val, const int32_t *carry_seg, int64_t num_tiles, int32_t R,
                        int32_t carry_ld, void *C, int64_t ldc, const int32_t *out_row, cudaStream_t stream) {
  const unsigned blocks = (unsigned)ceil_div(num_tiles * R, 256);
  if (dtype == COMET_F32)
    carry_fixup_kernel<float><<<blocks, 256, 0, stream>>>(carry_val, carry_seg, num_tiles, R, carry_ld, (float *)C, ldc, out_row);
  else
    carry_fixup_kernel<double><<<blocks, 256, 0, stream>>>(carry_val, carry_seg, num_tiles, R, carry_ld, (double *)C, ldc, out_row);
}

template <class T>
__global__ void zero_rows_kernel(T *__restrict__ C, int64_t rows, int32_t R, int64_t ldc) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t r = idx / R;
  if (r < rows) C[r * ldc + (idx - r * R)] = (T)0;
}

comet_status_t zero_rows(Context *ctx, void *C, int dtype, int64_t rows, int64_t R, int64_t ldc, cudaStream_t stream) {
  if (rows <= 0 || R <= 0) return COMET_OK;
  const int64_t n = rows * R;
  if (dtype == COMET_F32) zero_rows_kernel<float><<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>((float *)C, rows, (int32_t)R, ldc);
  else zero_rows_kernel<double><<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>((double *)C, rows, (int32_t)R, ldc);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

int32_t choose_tile_items(int64_t total_items, int workers_per_block) {
  if (const char *e = getenv("COMET_TILE_ITEMS")) {
    int v = atoi(e);
    if (v >= 8 && v <= (1 << 20)) return v;
  }
  // Aim for several tiles per resident worker (148 SMs x 8 blocks), capped so that carries stay a
  // small fraction of the traffic and floored so that the two path searches amortise.
  const int64_t slots = (int64_t)kSmCount * 8 * workers_per_block;
  int64_t t = total_items / (slots * 4);
  if (t < 32) t = 32;
  if (t > 512) t = 512;
  return (int32_t)t;
}

template <class T, int LPN, int CPL, int VEC, bool MAPPED, bool HEAVY>
static comet_status_t launch_mapped(Context *ctx, const SegGatherArgs &a, const HeavyArgs &h, int64_t blocks,
                                    cudaStream_t stream) {
  using L = Lanes<T, LPN, CPL, VEC>;
  constexpr size_t smem = RingLayout<L, false>::kBlockBytes;
  auto kernel = seg_gather_kernel<T, LPN, CPL, VEC, MAPPED, HEAVY>;
  if (smem > 48 * 1024)
    COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kernel<<<(unsigned)(blocks + (HEAVY ? h.heavy_ctas : 0)), kBlockThreads, smem, stream>>>(a, h);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

// The shapes whose rows are 256, 512 or 1024 bytes carry the long-row role of SpMM.
template <class T, int LPN, int CPL, int VEC> constexpr bool kHeavyShape =
    VEC * sizeof(T) == 16 && (LPN * CPL * VEC * sizeof(T) == 256 || LPN * CPL * VEC * sizeof(T) == 512 ||
                              LPN * CPL * VEC * sizeof(T) == 1024) && LPN >= 16;

static size_t carry_bytes(int64_t num_tiles, int32_t carry_ld) {
  return align_up((size_t)num_tiles * carry_ld * sizeof(double), 256) + align_up((size_t)num_tiles * sizeof(int32_t), 256);
}

// `heavy` (optional): the long-row plan of an SpMM; its scratch precedes the carries of this launch.
template <class T, int LPN, int CPL, int VEC>
static comet_status_t launch_one(Context *ctx, SegGatherArgs a, HeavyArgs *heavy, cudaStream_t stream) {
  constexpr int WORKERS = kBlockThreads / LPN;
  const int64_t total = a.M + a.N;
  a.tile_items = choose_tile_items(total, WORKERS);
  a.num_tiles = ceil_div(total, a.tile_items);
  a.own_len = a.tile_items / 4;
  a.carry_ld = (int32_t)align_up((size_t)a.R, 2);
  const size_t val_bytes = align_up((size_t)a.num_tiles * a.carry_ld * sizeof(double), 256);
  size_t heavy_bytes = 0;
  HeavyArgs h{};
  if (kHeavyShape<T, LPN, CPL, VEC> && heavy && !a.out_row)
    heavy_bytes = spmm_heavy_plan(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.M, a.N, heavy->cols, a.B, a.ldb, a.R, a.C, a.ldc,
                                  a.tile_items, &h);
  static const bool use_part = !(getenv("COMET_SEG_PARTITION") && atoi(getenv("COMET_SEG_PARTITION")) == 0);
  const size_t part_bytes = use_part && a.num_tiles >= 1024 ? align_up((size_t)(a.num_tiles + 1) * sizeof(int32_t), 256) : 0;
  char *scratch = (char *)scratch_get(ctx, heavy_bytes + carry_bytes(a.num_tiles, a.carry_ld) + part_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)(scratch + heavy_bytes);
  a.carry_seg = (int32_t *)(scratch + heavy_bytes + val_bytes);
  if (part_bytes) {
    int32_t *part = (int32_t *)(scratch + heavy_bytes + carry_bytes(a.num_tiles, a.carry_ld));
    if (heavy_bytes) {                                     // a role of the long-row path's pieces launch
      h.part_seg_end = a.seg_end; h.part_M = a.M; h.part_N = a.N; h.part_tiles = a.num_tiles;
      h.part_tile_items = a.tile_items; h.part = part;
    } else {
      seg_partition_kernel<<<(unsigned)ceil_div(a.num_tiles + 1, kBlockThreads), kBlockThreads, 0, stream>>>(a.seg_end, a.M, a.N,
                                                                                                           a.tile_items, a.num_tiles, part);
      COMET_LAUNCH_CHECK(ctx);
    }
    a.part = part;
  }
  const int64_t blocks = ceil_div(a.num_tiles, WORKERS);
  comet_status_t st;
  if constexpr (kHeavyShape<T, LPN, CPL, VEC>) {
    if (heavy_bytes) {
      st = spmm_heavy_prepare(ctx, &h, a.seg_end - 1, a.crd, a.val, scratch, stream);
      if (st != COMET_OK) return st;
      a.skip_len = h.threshold;
      st = launch_mapped<T, LPN, CPL, VEC, false, true>(ctx, a, h, blocks, stream);
      if (st != COMET_OK) return st;
      const int heavy_blocks = kSmCount * 8;
      const unsigned fix_blocks = (unsigned)(heavy_blocks + ceil_div(a.num_tiles * a.R, kBlockThreads));
      spmm_fixups_kernel<T><<<fix_blocks, kBlockThreads, 0, stream>>>(h, heavy_blocks, a.carry_val, a.carry_seg, a.num_tiles,
                                                                     (int32_t)a.R, a.carry_ld, static_cast<T *>(a.C), a.ldc);
      COMET_LAUNCH_CHECK(ctx);
      return COMET_OK;
    }
  }
  st = a.out_row ? launch_mapped<T, LPN, CPL, VEC, true, false>(ctx, a, h, blocks, stream)
                 : launch_mapped<T, LPN, CPL, VEC, false, false>(ctx, a, h, blocks, stream);
  if (st != COMET_OK) return st;
  carry_fixup_launch(sizeof(T) == 4 ? COMET_F32 : COMET_F64, a.carry_val, a.carry_seg, a.num_tiles, a.R, a.carry_ld, a.C,
                     a.ldc, a.out_row, stream);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// One launch per chunk of up to 128 columns. A power-of-two chunk on 16-byte-aligned rows takes the
// 128-bit path (LPN lanes x 16 bytes); anything else takes the scalar path (32 lanes, ragged).
template <class T>
static comet_status_t seg_gather_typed(Context *ctx, const int32_t *seg_end, const int32_t *crd, const T *val,
                                       int64_t M, int64_t N, const T *B, int64_t ldb, int64_t R, T *C, int64_t ldc,
                                       const int32_t *out_row, int64_t out_rows, int64_t b_rows, cudaStream_t stream) {
  HeavyArgs hint{};                                        // SpMM on [D,CU] with a known B: long rows by column phases
  hint.cols = b_rows;
  HeavyArgs *heavy = (!out_row && b_rows > 0 && R <= 128) ? &hint : nullptr;
  constexpr int PER = 16 / sizeof(T);                      // elements per 128-bit piece
  const bool vec_ok = aligned16(B) && aligned16(C) && (ldb % PER == 0) && (ldc % PER == 0);
  int64_t done = 0;
  while (done < R) {
    const int64_t rem = R - done;
    SegGatherArgs a{};
    a.seg_end = seg_end; a.crd = crd; a.val = val; a.M = M; a.N = N;
    a.B = B + done; a.ldb = ldb; a.C = C + done; a.ldc = ldc;
    a.out_row = out_row; a.out_rows = out_rows;
    comet_status_t st;
    const int64_t chunk = rem < 128 ? rem : 128;
    a.R = (int32_t)chunk;
    const bool v = vec_ok && done % PER == 0;
    const int64_t pieces = chunk / PER;                    // 128-bit pieces per row when chunk is a multiple
    if (v && chunk % PER == 0 && pieces == 64) st = launch_one<T, 32, 2, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 32) st = launch_one<T, 32, 1, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 16) st = launch_one<T, 16, 1, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 8) st = launch_one<T, 8, 1, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 4) st = launch_one<T, 4, 1, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 2) st = launch_one<T, 2, 1, PER>(ctx, a, heavy, stream);
    else if (v && chunk % PER == 0 && pieces == 1) st = launch_one<T, 1, 1, PER>(ctx, a, heavy, stream);
    else if (chunk > 64) st = launch_one<T, 32, 4, 1>(ctx, a, heavy, stream);
    else if (chunk > 32) st = launch_one<T, 32, 2, 1>(ctx, a, heavy, stream);
    else st = launch_one<T, 32, 1, 1>(ctx, a, heavy, stream);
    if (st != COMET_OK) return st;
    done += a.R;
  }
  return COMET_OK;
}

comet_status_t seg_gather(Context *ctx, int dtype, const int32_t *seg_end, const int32_t *crd, const void *val,
                          int64_t M, int64_t N, const void *B, int64_t ldb, int64_t R, void *C, int64_t ldc,
                          const int32_t *out_row, int64_t out_rows, int64_t b_rows, cudaStream_t stream) {
  if (ldb >= (1ll << 28)) return COMET_ERR_INDEX_OVERFLOW;      // row offsets are formed as int32 bytes * int32 index
  if (M == 0) return out_row ? zero_rows(ctx, C, dtype, out_rows, R, ldc, stream) : COMET_OK;
  if (dtype == COMET_F32)
    return seg_gather_typed<float>(ctx, seg_end, crd, (const float *)val, M, N, (const float *)B, ldb, R, (float *)C, ldc,
                                   out_row, out_rows, b_rows, stream);
  return seg_gather_typed<double>(ctx, seg_end, crd, (const double *)val, M, N, (const double *)B, ldb, R, (double *)C,
                                  ldc, out_row, out_rows, b_rows, stream);
}

}  // namespace comet
