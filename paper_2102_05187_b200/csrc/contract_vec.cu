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

namespace comet {

struct SegGatherArgs {
  const int32_t *seg_end;   // M entries: leaf position where segment s ends (= pos + 1)
  const int32_t *crd;       // N leaf coordinates (row index into B)
  const double *val;        // N values
  int64_t M, N;
  const double *B;
  int64_t ldb;
  double *C;                // output rows
  int64_t ldc;
  const int32_t *out_row;   // NULL: segment s -> row s. Else segment s -> row out_row[s] (ascending) and the
  int64_t out_rows;         //   rows in between (and up to out_rows) are zero-filled by the flushing worker
  int32_t R;                // columns handled by this launch
  int32_t tile_items;
  int64_t num_tiles;
  double *carry_val;        // num_tiles x carry_ld
  int32_t *carry_seg;       // num_tiles: segment the carry belongs to, -1 if none
  int32_t carry_ld;
};

// What the walker does with one leaf entry: close the segments that end in front of it, accumulate.
template <int LPN, int CPL, int VEC, bool MAPPED>
struct SegGatherPolicy {
  using Entry = Entry16;
  using L = Lanes<LPN, CPL, VEC>;
  static constexpr int kRows = 1;
  struct Window { double r[1][CPL][VEC]; };

  const SegGatherArgs &a;
  const L &ln;
  double acc[CPL][VEC];
  int64_t i;          // open segment
  int32_t next_end;   // leaf position where it ends (-1: no segment left)
  int32_t last_flush; // leaf position of the latest flush (entries at or after it are still in acc)

  __device__ __forceinline__ SegGatherPolicy(const SegGatherArgs &args, const L &lanes, int64_t i0, int32_t j0)
      : a(args), ln(lanes), i(i0), last_flush(j0) {
    ln.zero(acc);
    next_end = (i < a.M) ? __ldg(a.seg_end + i) : -1;
  }
  __device__ __forceinline__ Entry fetch(int32_t j) const { return Entry{ld_stream(a.val + j), ld_stream(a.crd + j), 0}; }
  static __device__ __forceinline__ Entry idle() { return Entry{0.0, 0, 0}; }
  __device__ __forceinline__ const double *row(const Entry &e, int) const { return a.B + (int64_t)e.a * a.ldb; }

  // Stores the open segment (and, for a compressed root level, zero-fills the rows in front of it).
  __device__ __forceinline__ void flush(int32_t j) {
    int64_t r = i;
    if (MAPPED) {
      r = __ldg(a.out_row + i);
      const int64_t lo = (i > 0) ? (int64_t)__ldg(a.out_row + i - 1) + 1 : 0;
      ln.zero_rows(a.C, a.ldc, lo, r);
      if (i == a.M - 1) ln.zero_rows(a.C, a.ldc, r + 1, a.out_rows);
    }
    ln.store_row(a.C + r * a.ldc, acc);
    ln.zero(acc);
    ++i;
    next_end = (i < a.M) ? __ldg(a.seg_end + i) : -1;
    last_flush = j;
  }
  __device__ __forceinline__ void consume(int32_t j, const Entry &e, const double (&rows)[1][CPL][VEC]) {
    while (j == next_end) flush(j);          // segments (possibly empty ones) that end in front of leaf j
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ln.ok[t])
#pragma unroll
        for (int k = 0; k < VEC; ++k) acc[t][k] = fma(e.v, rows[0][t][k], acc[t][k]);
  }
};

template <int LPN, int CPL, int VEC, bool MAPPED>
__global__ void __launch_bounds__(kBlockThreads) seg_gather_kernel(const SegGatherArgs a) {
  using L = Lanes<LPN, CPL, VEC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int worker = threadIdx.x / LPN;
  const int64_t tile = (int64_t)blockIdx.x * L::kWorkers + worker;
  if (tile >= a.num_tiles) return;                       // whole groups leave together
  Entry16 *ring = reinterpret_cast<Entry16 *>(smem_raw) + worker * 2 * L::kChunk;
  const L ln(a.R);

  const int64_t total = a.M + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  const int64_t i0 = merge_path_segments(a.seg_end, a.M, a.N, d0);
  const int64_t i1 = merge_path_segments(a.seg_end, a.M, a.N, d1);
  const int32_t j0 = (int32_t)(d0 - i0), j1 = (int32_t)(d1 - i1);

  SegGatherPolicy<LPN, CPL, VEC, MAPPED> p(a, ln, i0, j0);
  walk_tile(ln, p, j0, j1, ring);
  while (p.i < i1) p.flush(j1);                          // end markers that close the tile

  const bool carry = p.i < a.M && j1 > p.last_flush;     // leaf entries of a segment that ends in a later tile
  if (ln.g == 0) a.carry_seg[tile] = carry ? (int32_t)p.i : -1;
  if (carry) ln.store_carry(a.carry_val + tile * a.carry_ld, p.acc);
}

// Adds the carries onto the stored rows. Tiles that stopped inside the same segment are consecutive;
// the first of such a run sums the run in tile order and updates the row (the only writer of it now).
__global__ void carry_fixup_kernel(const double *__restrict__ carry_val, const int32_t *__restrict__ carry_seg,
                                   int64_t num_tiles, int32_t R, int32_t carry_ld, double *__restrict__ C,
                                   int64_t ldc, const int32_t *__restrict__ out_row) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t tile = idx / R;
  const int32_t c = (int32_t)(idx - tile * R);
  if (tile >= num_tiles) return;
  const int32_t seg = carry_seg[tile];
  if (seg < 0) return;
  if (tile > 0 && carry_seg[tile - 1] == seg) return;
  double sum = 0.0;
  for (int64_t t = tile; t < num_tiles && carry_seg[t] == seg; ++t) sum += carry_val[t * carry_ld + c];
  const int64_t row = out_row ? (int64_t)out_row[seg] : (int64_t)seg;
  C[row * ldc + c] += sum;
}

__global__ void zero_rows_kernel(double *__restrict__ C, int64_t rows, int32_t R, int64_t ldc) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t r = idx / R;
  if (r < rows) C[r * ldc + (idx - r * R)] = 0.0;
}

comet_status_t zero_rows(Context *ctx, double *C, int64_t rows, int64_t R, int64_t ldc, cudaStream_t stream) {
  if (rows <= 0 || R <= 0) return COMET_OK;
  const int64_t n = rows * R;
  zero_rows_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(C, rows, (int32_t)R, ldc);
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

template <int LPN, int CPL, int VEC, bool MAPPED>
static comet_status_t launch_mapped(Context *ctx, const SegGatherArgs &a, int64_t blocks, cudaStream_t stream) {
  using L = Lanes<LPN, CPL, VEC>;
  constexpr size_t smem = (size_t)L::kWorkers * 2 * L::kChunk * sizeof(Entry16);
  auto kernel = seg_gather_kernel<LPN, CPL, VEC, MAPPED>;
  if (smem > 48 * 1024)
    COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kernel<<<(unsigned)blocks, kBlockThreads, smem, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

template <int LPN, int CPL, int VEC>
static comet_status_t launch_one(Context *ctx, SegGatherArgs a, cudaStream_t stream) {
  constexpr int WORKERS = kBlockThreads / LPN;
  const int64_t total = a.M + a.N;
  a.tile_items = choose_tile_items(total, WORKERS);
  a.num_tiles = ceil_div(total, a.tile_items);
  a.carry_ld = (int32_t)align_up((size_t)a.R, 2);
  const size_t val_bytes = align_up((size_t)a.num_tiles * a.carry_ld * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  const int64_t blocks = ceil_div(a.num_tiles, WORKERS);
  comet_status_t st = a.out_row ? launch_mapped<LPN, CPL, VEC, true>(ctx, a, blocks, stream)
                                : launch_mapped<LPN, CPL, VEC, false>(ctx, a, blocks, stream);
  if (st != COMET_OK) return st;
  const int64_t fix_threads = a.num_tiles * a.R;
  carry_fixup_kernel<<<(unsigned)ceil_div(fix_threads, 256), 256, 0, stream>>>(
      a.carry_val, a.carry_seg, a.num_tiles, a.R, a.carry_ld, a.C, a.ldc, a.out_row);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

comet_status_t seg_gather(Context *ctx, const int32_t *seg_end, const int32_t *crd, const double *val, int64_t M,
                          int64_t N, const double *B, int64_t ldb, int64_t R, double *C, int64_t ldc,
                          const int32_t *out_row, int64_t out_rows, cudaStream_t stream) {
  if (M == 0) return out_row ? zero_rows(ctx, C, out_rows, R, ldc, stream) : COMET_OK;
  const bool vec_ok = aligned16(B) && aligned16(C) && (ldb % 2 == 0) && (ldc % 2 == 0);
  int64_t done = 0;
  while (done < R) {
    int64_t rem = R - done;
    SegGatherArgs a{};
    a.seg_end = seg_end; a.crd = crd; a.val = val; a.M = M; a.N = N;
    a.B = B + done; a.ldb = ldb; a.C = C + done; a.ldc = ldc;
    a.out_row = out_row; a.out_rows = out_rows;
    comet_status_t st;
    // One launch per chunk of up to 128 columns. A power-of-two chunk on 16-byte-aligned rows takes the
    // 128-bit path (LPN lanes x 2 columns); anything else takes the scalar path (32 lanes, ragged).
    const int64_t chunk = rem < 128 ? rem : 128;
    a.R = (int32_t)chunk;
    const bool v = vec_ok && done % 2 == 0;
    if (v && chunk == 128) st = launch_one<32, 2, 2>(ctx, a, stream);
    else if (v && chunk == 64) st = launch_one<32, 1, 2>(ctx, a, stream);
    else if (v && chunk == 32) st = launch_one<16, 1, 2>(ctx, a, stream);
    else if (v && chunk == 16) st = launch_one<8, 1, 2>(ctx, a, stream);
    else if (v && chunk == 8) st = launch_one<4, 1, 2>(ctx, a, stream);
    else if (v && chunk == 4) st = launch_one<2, 1, 2>(ctx, a, stream);
    else if (v && chunk == 2) st = launch_one<1, 1, 2>(ctx, a, stream);
    else if (chunk > 64) st = launch_one<32, 4, 1>(ctx, a, stream);
    else if (chunk > 32) st = launch_one<32, 2, 1>(ctx, a, stream);
    else st = launch_one<32, 1, 1>(ctx, a, stream);
    if (st != COMET_OK) return st;
    done += a.R;
  }
  return COMET_OK;
}

}  // namespace comet
