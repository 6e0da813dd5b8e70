// Root-mode MTTKRP, out[i, :] = sum over entries (i, j, k) of x * P[j, :] * Q[k, :] (the paper names
// the operation without defining it; this is the textbook matricised-tensor-times-Khatri-Rao product),
// for the two storage formats the paper's attributes compose for 3-order tensors:
//   COO [CN,S,S]  sorted entries, an output row is a run of equal root coordinates;
//   CSF [CU,CU,CU] per fiber t = sum x * Q[k, :], then out[i, :] += t * P[j, :] (one P row per fiber).
//
// Same worker scheme as the SpMM/TTM kernel: a worker is LPN lanes of a warp, each owning VEC columns
// of every 16*LPN-byte row piece, walking a tile of consecutive leaf entries with UNROLL independent
// row gathers in flight. A worker stores the output rows that END in its tile (and zero-fills the
// rows between consecutive stored rows, so no memset is needed), and writes the partial sum of the
// row it stops in to a carry slot that the fix-up kernel adds in tile order (deterministic).
#include "common.cuh"
#include "kernels.cuh"

namespace comet {

template <int LPN> __device__ __forceinline__ unsigned lane_group_mask() {
  if (LPN == 32) return 0xffffffffu;
  const unsigned lane = threadIdx.x & 31;
  return ((1u << LPN) - 1u) << (lane & ~(LPN - 1));
}

__device__ __forceinline__ void load_piece(const double *p, double (&d)[2]) {
  const double2 v = __ldg(reinterpret_cast<const double2 *>(p));
  d[0] = v.x; d[1] = v.y;
}
__device__ __forceinline__ void load_piece(const double *p, double (&d)[1]) { d[0] = __ldg(p); }
__device__ __forceinline__ void store_piece(double *p, const double (&d)[2]) {
  __stcs(reinterpret_cast<double2 *>(p), make_double2(d[0], d[1]));
}
__device__ __forceinline__ void store_piece(double *p, const double (&d)[1]) { __stcs(p, d[0]); }
__device__ __forceinline__ void store_piece_plain(double *p, const double (&d)[2]) {
  *reinterpret_cast<double2 *>(p) = make_double2(d[0], d[1]);
}
__device__ __forceinline__ void store_piece_plain(double *p, const double (&d)[1]) { *p = d[0]; }

struct MttkrpArgs {
  // COO: crd0/crd1/crd2/val over N entries. CSF: pos1 (S+1), crd0 (S), crd1 (F), seg_end2 (= pos2+1, F), crd2, val.
  const int32_t *pos1, *crd0, *crd1, *seg_end2, *crd2;
  const double *val;
  int64_t S, F, N, rows;
  const double *P;   // factor gathered by the level-1 coordinate
  int64_t ldp;
  const double *Q;   // factor gathered by the level-2 (leaf) coordinate
  int64_t ldq;
  double *out;
  int64_t ldo;
  int32_t R;
  int32_t tile_items;
  int64_t num_tiles;
  double *carry_val;
  int32_t *carry_seg;
  int32_t carry_ld;
};

template <int LPN, int CPL, int VEC> struct RowOut {
  int64_t col[CPL];
  bool ok[CPL];
  const MttkrpArgs &a;
  __device__ RowOut(const MttkrpArgs &args, int g) : a(args) {
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      col[t] = (int64_t)(t * LPN + g) * VEC;
      ok[t] = col[t] < args.R;
    }
  }
  __device__ __forceinline__ void zero_rows(int64_t lo, int64_t hi) const {   // rows lo .. hi-1
    const double zero[VEC] = {};
    for (int64_t z = lo; z < hi; ++z)
#pragma unroll
      for (int t = 0; t < CPL; ++t)
        if (ok[t]) store_piece(a.out + z * a.ldo + col[t], zero);
  }
  __device__ __forceinline__ void store_row(int64_t row, double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      if (ok[t]) store_piece(a.out + row * a.ldo + col[t], acc[t]);
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;
    }
  }
  __device__ __forceinline__ void store_carry(int64_t tile, const double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) store_piece_plain(a.carry_val + tile * a.carry_ld + col[t], acc[t]);
  }
};

// ------------------------------------------------------------------------------------------- COO
template <int LPN, int CPL, int VEC>
__global__ void __launch_bounds__(kBlockThreads) mttkrp_coo_kernel(const MttkrpArgs a) {
  constexpr int UNROLL = LPN < 8 ? LPN : 8;
  constexpr int WORKERS = kBlockThreads / LPN;
  const int g = threadIdx.x & (LPN - 1);
  const int64_t tile = (int64_t)blockIdx.x * WORKERS + threadIdx.x / LPN;
  if (tile >= a.num_tiles) return;
  const unsigned mask = lane_group_mask<LPN>();
  const RowOut<LPN, CPL, VEC> o(a, g);

  const int64_t j0 = tile * a.tile_items;
  const int64_t j1 = (j0 + a.tile_items < a.N) ? j0 + a.tile_items : a.N;
  int64_t cur = __ldg(a.crd0 + j0);
  {
    const int64_t prev = j0 > 0 ? (int64_t)__ldg(a.crd0 + j0 - 1) : -1;
    if (prev != cur) o.zero_rows(prev + 1, cur);         // the gap in front of a row is filled where the row starts
  }
  double acc[CPL][VEC];
#pragma unroll
  for (int t = 0; t < CPL; ++t)
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;

  for (int64_t base = j0; base < j1; base += LPN) {
    const int64_t mine = base + g;
    int32_t my_i = 0, my_j = 0, my_k = 0;
    double my_v = 0.0;
    if (mine < j1) {
      my_i = ld_stream(a.crd0 + mine);
      my_j = ld_stream(a.crd1 + mine);
      my_k = ld_stream(a.crd2 + mine);
      my_v = ld_stream(a.val + mine);
    }
    const int n = (j1 - base < LPN) ? (int)(j1 - base) : LPN;
    for (int u0 = 0; u0 < n; u0 += UNROLL) {
      double prow[UNROLL][CPL][VEC], qrow[UNROLL][CPL][VEC];
      double vv[UNROLL];
      int32_t ri[UNROLL];
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        const int src = (u0 + q) & (LPN - 1);
        ri[q] = __shfl_sync(mask, my_i, src, LPN);
        const int32_t cj = __shfl_sync(mask, my_j, src, LPN);
        const int32_t ck = __shfl_sync(mask, my_k, src, LPN);
        vv[q] = __shfl_sync(mask, my_v, src, LPN);
        if (u0 + q < n) {
          const double *pr = a.P + (int64_t)cj * a.ldp;
          const double *qr = a.Q + (int64_t)ck * a.ldq;
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (o.ok[t]) {
              load_piece(pr + o.col[t], prow[q][t]);
              load_piece(qr + o.col[t], qrow[q][t]);
            }
        }
      }
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        if (u0 + q < n) {
          if (ri[q] != cur) {
            o.store_row(cur, acc);
            o.zero_rows(cur + 1, ri[q]);
            cur = ri[q];
          }
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (o.ok[t])
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc[t][e] = fma(vv[q] * prow[q][t][e], qrow[q][t][e], acc[t][e]);
        }
      }
    }
  }
  const int64_t nxt = j1 < a.N ? (int64_t)__ldg(a.crd0 + j1) : -1;
  if (nxt == cur) {
    if (g == 0) a.carry_seg[tile] = (int32_t)cur;
    o.store_carry(tile, acc);
  } else {
    if (g == 0) a.carry_seg[tile] = -1;
    o.store_row(cur, acc);
    if (j1 == a.N) o.zero_rows(cur + 1, a.rows);
  }
}

// ------------------------------------------------------------------------------------------- CSF
template <int LPN, int CPL, int VEC>
__global__ void __launch_bounds__(kBlockThreads) mttkrp_csf_kernel(const MttkrpArgs a) {
  constexpr int UNROLL = LPN < 8 ? LPN : 8;
  constexpr int WORKERS = kBlockThreads / LPN;
  const int g = threadIdx.x & (LPN - 1);
  const int64_t tile = (int64_t)blockIdx.x * WORKERS + threadIdx.x / LPN;
  if (tile >= a.num_tiles) return;
  const unsigned mask = lane_group_mask<LPN>();
  const RowOut<LPN, CPL, VEC> o(a, g);

  // tile = a span of the merge list of fiber-end markers and leaf positions
  const int64_t total = a.F + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  int64_t f = merge_path_segments(a.seg_end2, a.F, a.N, d0);
  const int64_t j0 = d0 - f;
  const int64_t f1 = merge_path_segments(a.seg_end2, a.F, a.N, d1);
  const int64_t j1 = d1 - f1;

  // slice that holds fiber f: the largest s with pos1[s] <= f (every slice is non-empty)
  int64_t s;
  {
    int64_t lo = 0, hi = a.S;                            // answer in [0, S]; S only when f == F
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      if ((int64_t)__ldg(a.pos1 + mid + 1) <= f) lo = mid + 1; else hi = mid;
    }
    s = lo;
  }
  int64_t slice_end = s < a.S ? (int64_t)__ldg(a.pos1 + s + 1) : -1;
  int64_t next_end = f < a.F ? (int64_t)__ldg(a.seg_end2 + f) : -1;

  double tac[CPL][VEC], aac[CPL][VEC];                   // open fiber sum, open slice sum
#pragma unroll
  for (int t = 0; t < CPL; ++t)
#pragma unroll
    for (int e = 0; e < VEC; ++e) { tac[t][e] = 0.0; aac[t][e] = 0.0; }
  bool t_dirty = false, a_dirty = false;

  auto fold_fiber = [&]() {                              // aac += tac * P[crd1[f]]
    const double *pr = a.P + (int64_t)__ldg(a.crd1 + f) * a.ldp;
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (o.ok[t]) {
        double p[VEC];
        load_piece(pr + o.col[t], p);
#pragma unroll
        for (int e = 0; e < VEC; ++e) { aac[t][e] = fma(tac[t][e], p[e], aac[t][e]); tac[t][e] = 0.0; }
      }
    t_dirty = false;
    a_dirty = true;
  };
  auto end_fiber = [&]() {
    fold_fiber();
    ++f;
    next_end = f < a.F ? (int64_t)__ldg(a.seg_end2 + f) : -1;
    if (f == slice_end) {                                // the slice is complete: this worker owns its row
      const int64_t row = __ldg(a.crd0 + s);
      const int64_t lo = s > 0 ? (int64_t)__ldg(a.crd0 + s - 1) + 1 : 0;
      o.zero_rows(lo, row);
      o.store_row(row, aac);
      if (s == a.S - 1) o.zero_rows(row + 1, a.rows);
      a_dirty = false;
      ++s;
      slice_end = s < a.S ? (int64_t)__ldg(a.pos1 + s + 1) : -1;
    }
  };

  for (int64_t base = j0; base < j1; base += LPN) {
    const int64_t mine = base + g;
    int32_t my_k = 0;
    double my_v = 0.0;
    if (mine < j1) {
      my_k = ld_stream(a.crd2 + mine);
      my_v = ld_stream(a.val + mine);
    }
    const int n = (j1 - base < LPN) ? (int)(j1 - base) : LPN;
    for (int u0 = 0; u0 < n; u0 += UNROLL) {
      double qrow[UNROLL][CPL][VEC];
      double vv[UNROLL];
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        const int src = (u0 + q) & (LPN - 1);
        const int32_t ck = __shfl_sync(mask, my_k, src, LPN);
        vv[q] = __shfl_sync(mask, my_v, src, LPN);
        if (u0 + q < n) {
          const double *qr = a.Q + (int64_t)ck * a.ldq;
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (o.ok[t]) load_piece(qr + o.col[t], qrow[q][t]);
        }
      }
#pragma unroll
      for (int q = 0; q < UNROLL; ++q) {
        if (u0 + q < n) {
          const int64_t jj = base + u0 + q;
          while (jj == next_end) end_fiber();
#pragma unroll
          for (int t = 0; t < CPL; ++t)
            if (o.ok[t])
#pragma unroll
              for (int e = 0; e < VEC; ++e) tac[t][e] = fma(vv[q], qrow[q][t][e], tac[t][e]);
          t_dirty = true;
        }
      }
    }
  }
  while (f < f1) end_fiber();
  if (t_dirty) fold_fiber();                             // an unfinished fiber contributes through distributivity
  const bool carry = a_dirty && s < a.S;
  if (g == 0) a.carry_seg[tile] = carry ? (int32_t)s : -1;
  if (carry) o.store_carry(tile, aac);
}

// ------------------------------------------------------------------------------------------- host
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <bool CSF, int LPN, int CPL, int VEC>
static comet_status_t launch_mttkrp(Context *ctx, MttkrpArgs a, cudaStream_t stream) {
  constexpr int WORKERS = kBlockThreads / LPN;
  const int64_t total = CSF ? a.F + a.N : a.N;
  a.tile_items = choose_tile_items(total, WORKERS);
  a.num_tiles = ceil_div(total, a.tile_items);
  a.carry_ld = (int32_t)align_up((size_t)a.R, 2);
  const size_t val_bytes = align_up((size_t)a.num_tiles * a.carry_ld * sizeof(double), 256);
  const size_t seg_bytes = align_up((size_t)a.num_tiles * sizeof(int32_t), 256);
  char *scratch = (char *)scratch_get(ctx, val_bytes + seg_bytes, stream);
  if (!scratch) return COMET_ERR_ALLOC;
  a.carry_val = (double *)scratch;
  a.carry_seg = (int32_t *)(scratch + val_bytes);
  const unsigned blocks = (unsigned)ceil_div(a.num_tiles, WORKERS);
  if (CSF) mttkrp_csf_kernel<LPN, CPL, VEC><<<blocks, kBlockThreads, 0, stream>>>(a);
  else mttkrp_coo_kernel<LPN, CPL, VEC><<<blocks, kBlockThreads, 0, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
  carry_fixup_kernel<<<(unsigned)ceil_div(a.num_tiles * a.R, 256), 256, 0, stream>>>(
      a.carry_val, a.carry_seg, a.num_tiles, a.R, a.carry_ld, a.out, a.ldo, CSF ? a.crd0 : nullptr);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

template <bool CSF>
static comet_status_t mttkrp_chunks(Context *ctx, MttkrpArgs base, int64_t R, cudaStream_t stream) {
  const bool vec_ok = aligned16(base.P) && aligned16(base.Q) && aligned16(base.out) && base.ldp % 2 == 0 &&
                      base.ldq % 2 == 0 && base.ldo % 2 == 0;
  int64_t done = 0;
  while (done < R) {
    const int64_t rem = R - done;
    const int64_t chunk = rem < 128 ? rem : 128;
    MttkrpArgs a = base;
    a.P += done; a.Q += done; a.out += done;
    a.R = (int32_t)chunk;
    const bool v = vec_ok && done % 2 == 0;
    comet_status_t st;
    if (v && chunk == 128) st = launch_mttkrp<CSF, 32, 2, 2>(ctx, a, stream);
    else if (v && chunk == 64) st = launch_mttkrp<CSF, 32, 1, 2>(ctx, a, stream);
    else if (v && chunk == 32) st = launch_mttkrp<CSF, 16, 1, 2>(ctx, a, stream);
    else if (v && chunk == 16) st = launch_mttkrp<CSF, 8, 1, 2>(ctx, a, stream);
    else if (v && chunk == 8) st = launch_mttkrp<CSF, 4, 1, 2>(ctx, a, stream);
    else if (v && chunk == 4) st = launch_mttkrp<CSF, 2, 1, 2>(ctx, a, stream);
    else if (v && chunk == 2) st = launch_mttkrp<CSF, 1, 1, 2>(ctx, a, stream);
    else if (chunk > 64) st = launch_mttkrp<CSF, 32, 4, 1>(ctx, a, stream);
    else if (chunk > 32) st = launch_mttkrp<CSF, 32, 2, 1>(ctx, a, stream);
    else st = launch_mttkrp<CSF, 32, 1, 1>(ctx, a, stream);
    if (st != COMET_OK) return st;
    done += chunk;
  }
  return COMET_OK;
}

comet_status_t mttkrp_coo(Context *ctx, const int32_t *crd0, const int32_t *crd1, const int32_t *crd2,
                          const double *val, int64_t N, int64_t rows, const double *P, int64_t ldp, const double *Q,
                          int64_t ldq, int64_t R, double *out, int64_t ldo, cudaStream_t stream) {
  if (N == 0) return zero_rows(ctx, out, rows, R, ldo, stream);
  MttkrpArgs a{};
  a.crd0 = crd0; a.crd1 = crd1; a.crd2 = crd2; a.val = val; a.N = N; a.rows = rows;
  a.P = P; a.ldp = ldp; a.Q = Q; a.ldq = ldq; a.out = out; a.ldo = ldo;
  return mttkrp_chunks<false>(ctx, a, R, stream);
}

comet_status_t mttkrp_csf(Context *ctx, const int32_t *pos1, const int32_t *crd0, const int32_t *crd1,
                          const int32_t *pos2, const int32_t *crd2, const double *val, int64_t S, int64_t F,
                          int64_t N, int64_t rows, const double *P, int64_t ldp, const double *Q, int64_t ldq,
                          int64_t R, double *out, int64_t ldo, cudaStream_t stream) {
  if (N == 0 || S == 0) return zero_rows(ctx, out, rows, R, ldo, stream);
  MttkrpArgs a{};
  a.pos1 = pos1; a.crd0 = crd0; a.crd1 = crd1; a.seg_end2 = pos2 + 1; a.crd2 = crd2; a.val = val;
  a.S = S; a.F = F; a.N = N; a.rows = rows;
  a.P = P; a.ldp = ldp; a.Q = Q; a.ldq = ldq; a.out = out; a.ldo = ldo;
  return mttkrp_chunks<true>(ctx, a, R, stream);
}

}  // namespace comet
