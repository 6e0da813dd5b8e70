// Segment-gather contractions with a dense matrix operand: SpMM, TTM (the SpMM/SpTTM definitions of
// the paper's Sparse Tensor Operations subsection). Both are "for every leaf entry p of segment s:
// out[s, :] += val[p] * B[crd[p], :]" where a segment is a CSR row (SpMM) or a CSF fiber (TTM).
//
// Work split (B200): the merge list of segment-end markers and leaf positions is cut into tiles of a
// fixed number of items, one tile per WORKER. A worker is a group of LPN lanes of a warp; lane g of
// the group owns columns {(t*LPN + g)*VEC .. +VEC} for t < CPL, so one gather of a dense row is one
// fully coalesced LPN*VEC*8-byte request and nothing is ever reduced across lanes. A worker walks
// its tile sequentially, keeps up to UNROLL independent row gathers in flight, stores every segment
// that ENDS inside its tile with plain vector stores (so every output row is written exactly once,
// without a memset), and hands the partial sum of the segment it stops in to a carry slot. A second
// small kernel adds the carries of earlier tiles onto the stored rows in tile order, which makes the
// result deterministic (no atomics anywhere).
#include "common.cuh"
#include "kernels.cuh"

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

template <int VEC> struct Piece;
template <> struct Piece<2> {
  static __device__ __forceinline__ void load(const double *p, double *d) {
    double2 v = __ldg(reinterpret_cast<const double2 *>(p));
    d[0] = v.x; d[1] = v.y;
  }
  static __device__ __forceinline__ void store(double *p, const double *d) {
    __stcs(reinterpret_cast<double2 *>(p), make_double2(d[0], d[1]));
  }
  static __device__ __forceinline__ void store_plain(double *p, const double *d) {
    *reinterpret_cast<double2 *>(p) = make_double2(d[0], d[1]);
  }
};
template <> struct Piece<1> {
  static __device__ __forceinline__ void load(const double *p, double *d) { d[0] = __ldg(p); }
  static __device__ __forceinline__ void store(double *p, const double *d) { __stcs(p, d[0]); }
  static __device__ __forceinline__ void store_plain(double *p, const double *d) { *p = d[0]; }
};

template <int LPN> __device__ __forceinline__ unsigned group_mask() {
  if (LPN == 32) return 0xffffffffu;
  const unsigned lane = threadIdx.x & 31;
  return ((1u << LPN) - 1u) << (lane & ~(LPN - 1));
}

template <int LPN, int CPL, int VEC>
__global__ void __launch_bounds__(kBlockThreads) seg_gather_kernel(const SegGatherArgs a) {
  constexpr int UNROLL = LPN < 8 ? LPN : 8;
  constexpr int WORKERS = kBlockThreads / LPN;
  const int g = threadIdx.x & (LPN - 1);
  const int64_t tile = (int64_t)blockIdx.x * WORKERS + threadIdx.x / LPN;
  if (tile >= a.num_tiles) return;                       // whole groups leave together
  const unsigned mask = group_mask<LPN>();

  const int64_t total = a.M + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  int64_t i = merge_path_segments(a.seg_end, a.M, a.N, d0);
  const int64_t j0 = d0 - i;
  const int64_t i1 = merge_path_segments(a.seg_end, a.M, a.N, d1);
  const int64_t j1 = d1 - i1;

  bool col_ok[CPL];
  int64_t col[CPL];
#pragma unroll
  for (int t = 0; t < CPL; ++t) {
    col[t] = (int64_t)(t * LPN + g) * VEC;
    col_ok[t] = col[t] < a.R;                            // only the scalar (VEC == 1) path can be ragged
  }

  double acc[CPL][VEC];
#pragma unroll
  for (int t = 0; t < CPL; ++t)
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;
  bool dirty = false;
  int64_t next_end = (i < a.M) ? (int64_t)__ldg(a.seg_end + i) : -1;

  auto flush = [&]() {
    int64_t row = i;
    if (a.out_row) {
      row = __ldg(a.out_row + i);
      int64_t lo = (i > 0) ? (int64_t)__ldg(a.out_row + i - 1) + 1 : 0;
      const double zero[VEC] = {};
      for (int64_t z = lo; z < row; ++z)
#pragma unroll
        for (int t = 0; t < CPL; ++t)
          if (col_ok[t]) Piece<VEC>::store(a.C + z * a.ldc + col[t], zero);
      if (i == a.M - 1)
        for (int64_t z = row + 1; z < a.out_rows; ++z)
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (col_ok[t]) Piece<VEC>::store(a.C + z * a.ldc + col[t], zero);
    }
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      if (col_ok[t]) Piece<VEC>::store(a.C + row * a.ldc + col[t], acc[t]);
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;
    }
    dirty = false;
    ++i;
    next_end = (i < a.M) ? (int64_t)__ldg(a.seg_end + i) : -1;
  };

  for (int64_t base = j0; base < j1; base += LPN) {
    const int64_t mine = base + g;
    int32_t my_c = 0;
    double my_v = 0.0;
    if (mine < j1) {
      my_c = ld_stream(a.crd + mine);
      my_v = ld_stream(a.val + mine);
    }
    const int n = (j1 - base < LPN) ? (int)(j1 - base) : LPN;
    for (int u0 = 0; u0 < n; u0 += UNROLL) {
      double rows[UNROLL][CPL][VEC];
      double vv[UNROLL];
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        const int src = (u0 + q) & (LPN - 1);
        const int32_t c = __shfl_sync(mask, my_c, src, LPN);
        vv[q] = __shfl_sync(mask, my_v, src, LPN);
        if (u0 + q < n) {
          const double *brow = a.B + (int64_t)c * a.ldb;
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (col_ok[t]) Piece<VEC>::load(brow + col[t], rows[q][t]);
        }
      }
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        if (u0 + q < n) {
          const int64_t jj = base + u0 + q;
          while (jj == next_end) flush();                // segments (possibly empty ones) that end before leaf jj
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (col_ok[t])
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc[t][e] = fma(vv[q], rows[q][t][e], acc[t][e]);
          dirty = true;
        }
      }
    }
  }
  while (i < i1) flush();                                // end markers that close the tile

  if (g == 0) a.carry_seg[tile] = (dirty && i < a.M) ? (int32_t)i : -1;
  if (dirty && i < a.M) {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (col_ok[t]) Piece<VEC>::store_plain(a.carry_val + tile * a.carry_ld + col[t], acc[t]);
  }
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
  seg_gather_kernel<LPN, CPL, VEC><<<(unsigned)blocks, kBlockThreads, 0, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
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
