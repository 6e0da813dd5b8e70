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
#include "common.cuh"
#include "kernels.cuh"
#include "walk.cuh"

#ifndef COMET_PF_COO
#define COMET_PF_COO 2        // entries in flight per worker, two row gathers each
#endif
#ifndef COMET_PF_CSF
#define COMET_PF_CSF 4
#endif
#ifndef COMET_MINB_COO
#define COMET_MINB_COO 4
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
};

// ------------------------------------------------------------------------------------------- COO
template <class T, int LPN, int CPL, int VEC>
struct CooPolicy {
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = COMET_PF_COO;   // two rows per entry
  static constexpr bool kAux = true;         // the root coordinate rides in the side ring
  static constexpr bool kFullUnroll = true;
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
  // The run of `cur` ends here: store it, zero-fill the rows up to the next stored row.
  __device__ __forceinline__ void next_row(int32_t row) {
    ln.store_row(ocol + (int64_t)cur * a.ldo, acc);
    ln.zero_rows(ocol, a.ldo, (int64_t)cur + 1, row);
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
  {
    const int64_t prev = j0 > 0 ? (int64_t)__ldg(a.crd0 + j0 - 1) : -1;
    if (prev != first) ln.zero_rows(p.ocol, a.ldo, prev + 1, first);   // the gap in front of a row is filled where it starts
  }
  walk_tile(ln, p, (int32_t)j0, (int32_t)j1, smem);

  const int64_t nxt = j1 < a.N ? (int64_t)__ldg(a.crd0 + j1) : -1;
  if (nxt == p.cur) {                                    // the row continues in the next tile
    if (ln.g == 0) a.carry_seg[tile] = p.cur;
    ln.store_carry(a.carry_val + tile * a.carry_ld + ln.col0, p.acc);
  } else {
    if (ln.g == 0) a.carry_seg[tile] = -1;
    ln.store_row(p.ocol + (int64_t)p.cur * a.ldo, p.acc);
    if (j1 == a.N) ln.zero_rows(p.ocol, a.ldo, (int64_t)p.cur + 1, a.rows);
  }
}

// ------------------------------------------------------------------------------------------- CSF
template <class T, int LPN, int CPL, int VEC>
struct CsfPolicy {
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = COMET_PF_CSF;
  static constexpr bool kAux = false;
  static constexpr bool kFullUnroll = false;   // the fiber/slice epilogue is long: keep the body small
  struct Slot { T r[CPL][VEC]; };

  const MttkrpArgs &a;
  const L &ln;
  const char *pcol, *qcol;
  int32_t ldp_bytes, ldq_bytes;
  T *ocol;
  const T *val;
  double tac[CPL][VEC], aac[CPL][VEC];   // open fiber sum, open slice sum
  T prow[CPL][VEC];                      // P row of the open fiber
  T pnext[CPL][VEC];                     // P row of the fiber after it: fetched one fiber ahead, so that a fold
                                         // never waits for its gather (fibers are a few entries long)
  int32_t end1;                          // leaf position where the fiber after the open one ends
  // cursors instead of indices: the per-fiber path is executed once per fiber and per worker (divergently),
  // so it is kept to pointer bumps and 32-bit compares
  const int32_t *endp;                   // seg_end2 + open fiber
  const int32_t *c1p;                    // crd1 + open fiber
  int32_t fibers_left;                   // fibers from the open one to the last
  int32_t to_slice_end;                  // fibers from the open one to the end of the open slice
  int32_t s;                             // open slice
  int32_t next_end;                      // leaf position where the open fiber ends
  int32_t base, rel_end;
  int32_t last_fold;                     // leaf position of the latest fold (entries at or after it are in tac)
  bool a_dirty;

  __device__ __forceinline__ CsfPolicy(const MttkrpArgs &args, const L &lanes, int64_t f0, int64_t s0, int32_t j0)
      : a(args), ln(lanes), s((int32_t)s0), base(j0), last_fold(j0), a_dirty(false) {
    ln.zero(tac);
    ln.zero(aac);
#pragma unroll
    for (int t = 0; t < CPL; ++t)
#pragma unroll
      for (int k = 0; k < VEC; ++k) { prow[t][k] = (T)0; pnext[t][k] = (T)0; }
    pcol = reinterpret_cast<const char *>(static_cast<const T *>(a.P) + ln.col0);
    qcol = reinterpret_cast<const char *>(static_cast<const T *>(a.Q) + ln.col0);
    ldp_bytes = (int32_t)(a.ldp * sizeof(T));
    ldq_bytes = (int32_t)(a.ldq * sizeof(T));
    ocol = static_cast<T *>(a.out) + ln.col0;
    val = static_cast<const T *>(a.val);
    endp = a.seg_end2 + f0;
    c1p = a.crd1 + f0;
    fibers_left = (int32_t)(a.F - f0);
    next_end = fibers_left > 0 ? __ldg(endp) : -1;
    end1 = fibers_left > 1 ? __ldg(endp + 1) : -1;
    rel_end = next_end - base;
    to_slice_end = s < a.S ? (int32_t)(__ldg(a.pos1 + s + 1) - f0) : -1;
    if (fibers_left > 0) ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)__ldg(c1p) * ldp_bytes), prow);
    fetch_ahead();
  }
  __device__ __forceinline__ int64_t fiber() const { return a.F - fibers_left; }
  __device__ __forceinline__ void fetch_ahead() {        // start fetching the P row of the fiber after the open one
    if (fibers_left > 1) ln.gather(reinterpret_cast<const T *>(pcol + (int64_t)__ldg(c1p + 1) * ldp_bytes), pnext);
  }
  __device__ __forceinline__ void fetch(int32_t j, Entry16 &e, int32_t &) const {
    e.v = (double)ld_stream(val + j);
    e.a = ld_stream(a.crd2 + j);
  }
  __device__ __forceinline__ void prefetch(int32_t ck, int32_t, Slot &sl) const {
    ln.gather(reinterpret_cast<const T *>(qcol + (int64_t)ck * ldq_bytes), sl.r);
  }
  __device__ __forceinline__ void begin_chunk(int32_t b) { base = b; rel_end = next_end - b; }

  __device__ __forceinline__ void fold(int32_t j) {      // aac += tac * P[crd1[f], :]
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ln.ok[t])
#pragma unroll
        for (int k = 0; k < VEC; ++k) { aac[t][k] = fma(tac[t][k], (double)prow[t][k], aac[t][k]); tac[t][k] = 0.0; }
    a_dirty = true;
    last_fold = j;
  }
  __device__ __forceinline__ void close_slice() {        // the slice is complete: this worker owns its row
    const int64_t row = __ldg(a.crd0 + s);
    const int64_t lo = s > 0 ? (int64_t)__ldg(a.crd0 + s - 1) + 1 : 0;
    ln.zero_rows(ocol, a.ldo, lo, row);
    ln.store_row(ocol + row * a.ldo, aac);
    if (s == a.S - 1) ln.zero_rows(ocol, a.ldo, row + 1, a.rows);
    ln.zero(aac);
    a_dirty = false;
    ++s;
    to_slice_end = s < a.S ? __ldg(a.pos1 + s + 1) - __ldg(a.pos1 + s) : -1;
  }
  __device__ __forceinline__ void end_fiber(int32_t j) {
    fold(j);
    ++endp;
    ++c1p;
    --fibers_left;
    next_end = end1;                                     // loaded one fiber ago
    end1 = fibers_left > 1 ? __ldg(endp + 1) : -1;
    rel_end = next_end - base;
#pragma unroll
    for (int t = 0; t < CPL; ++t)
#pragma unroll
      for (int k = 0; k < VEC; ++k) prow[t][k] = pnext[t][k];
    fetch_ahead();
    if (--to_slice_end == 0) close_slice();
  }
  __device__ __forceinline__ void consume(int q, double v, int32_t, Slot &sl) {
    while (rel_end == q) end_fiber(base + q);
    ln.fma_rows(v, sl.r, tac);
  }
};

template <class T, int LPN, int CPL, int VEC>
__global__ void __launch_bounds__(kBlockThreads, (CPL * VEC * sizeof(T) <= 16 ? COMET_MINB_CSF : 2)) mttkrp_csf_kernel(const MttkrpArgs a) {
  using L = Lanes<T, LPN, CPL, VEC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int worker = threadIdx.x / LPN;
  const int64_t tile = (int64_t)blockIdx.x * L::kWorkers + worker;
  if (tile >= a.num_tiles) return;
  using P = CsfPolicy<T, LPN, CPL, VEC>;
  const uint32_t smem = smem_u32(smem_raw) + worker * RingLayout<L, false>::kWorkerBytes;
  const L ln(a.R);

  // tile = a span of the merge list of fiber-end markers and leaf positions
  const int64_t total = a.F + a.N;
  const int64_t d0 = tile * a.tile_items;
  const int64_t d1 = (d0 + a.tile_items < total) ? d0 + a.tile_items : total;
  const int64_t f0 = merge_path_segments_coop<LPN>(a.seg_end2, a.F, a.N, d0, ln.g, ln.mask);
  const int64_t f1 = merge_path_segments_coop<LPN>(a.seg_end2, a.F, a.N, d1, ln.g, ln.mask);
  const int32_t j0 = (int32_t)(d0 - f0), j1 = (int32_t)(d1 - f1);

  // slice that holds fiber f0: the number of slices that end at or before it (every slice is non-empty)
  int64_t lo = 0, hi = a.S;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(a.pos1 + mid + 1) <= f0) lo = mid + 1; else hi = mid;
  }

  P p(a, ln, f0, lo, j0);
  walk_tile(ln, p, j0, j1, smem);
  while (p.fiber() < f1) p.end_fiber(j1);
  if (j1 > p.last_fold) p.fold(j1);                      // an unfinished fiber contributes through distributivity
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
  using L = Lanes<T, LPN, CPL, VEC>;
  constexpr size_t smem = CSF ? RingLayout<L, false>::kBlockBytes : RingLayout<L, true>::kBlockBytes;
  auto kernel = CSF ? mttkrp_csf_kernel<T, LPN, CPL, VEC> : mttkrp_coo_kernel<T, LPN, CPL, VEC>;
  if (smem > 48 * 1024)
    COMET_CUDA_TRY(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kernel<<<blocks, kBlockThreads, smem, stream>>>(a);
  COMET_LAUNCH_CHECK(ctx);
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
  if (N == 0) return zero_rows(ctx, out, dtype, rows, R, ldo, stream);
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
  return dtype == COMET_F32 ? mttkrp_chunks<true, float>(ctx, a, R, stream) : mttkrp_chunks<true, double>(ctx, a, R, stream);
}

}  // namespace comet
