// The long-row path of SpMM: what the general gather kernel needs to run its tiles (spmm_heavy.cu has the rest).
#pragma once

#include "common.cuh"
#include "walk.cuh"

#ifndef COMET_PF_HEAVY
#define COMET_PF_HEAVY 8       // row gathers in flight per worker
#endif

namespace comet {

struct HeavyArgs {
  const int32_t *pos;        // M + 1
  const int32_t *crd;
  const void *val;
  int64_t M, N, cols;
  int32_t threshold;         // a row with at least this many entries is long
  int32_t P;                 // column blocks (power of two, at most 32)
  int32_t block_cols;        // columns per block
  int32_t tile_max;
  int32_t piece_target;
  int32_t num_scan_ctas;
  int32_t heavy_ctas;        // CTAs of the gather kernel that take the long-row role
  int64_t h_max, t_max;      // capacity of the per-row and per-tile arrays
  int32_t *counters;         // 0: long rows, 1: slots reserved, 2: tiles, 3 / 4: finished-CTA tickets, 5: next tile
  int32_t *cta_rows, *cta_slots;            // per scan CTA: counts, then exclusive offsets
  int32_t *hrow, *row_slot0, *row_nt;       // per long row: row id, first slot, slots in use
  int32_t *piece_start;                     // per long row: P + 1 leaf positions
  int32_t *bin;                             // P tile counts per phase, P starts, P cursors
  int4 *rec;                                // tiles in processing order: first entry, end, slot, row
  double *carry_val;
  int32_t carry_ld;
  const void *B;
  int64_t ldb;
  void *C;
  int64_t ldc;
  int32_t R;
  // the tile boundaries of the GENERAL tiles (merge-path splits), computed by extra CTAs of the pieces launch
  const int32_t *part_seg_end;
  int64_t part_M, part_N, part_tiles;
  int32_t part_tile_items;
  int32_t *part;
};

// A tile of one row: no segment ends, only the window of gathers and the sum.
template <class T, int LPN, int CPL, int VEC>
struct HeavyPolicy {
  using L = Lanes<T, LPN, CPL, VEC>;
  static constexpr int kPF = CPL > 1 ? COMET_PF_HEAVY / 2 : COMET_PF_HEAVY;   // register budget: 64
  static constexpr bool kAux = false;
  static constexpr bool kFullUnroll = true;
  static constexpr bool kRolledTail = true;
  struct Slot { T r[CPL][VEC]; };
  const L &ln;
  const T *val;
  const int32_t *crd;
  const char *bcol;
  int32_t ldb_bytes;
  uint64_t keep;            // L2 policy: the block of B in work stays while the other role streams its rows through
  double acc[CPL][VEC];
  __device__ __forceinline__ HeavyPolicy(const HeavyArgs &a, const L &lanes) : ln(lanes) {
    keep = l2_policy_evict_last();
    val = static_cast<const T *>(a.val);
    crd = a.crd;
    bcol = reinterpret_cast<const char *>(static_cast<const T *>(a.B) + ln.col0);
    ldb_bytes = (int32_t)(a.ldb * sizeof(T));
  }
  __device__ __forceinline__ void fetch(int32_t j, Entry16 &e, int32_t &) const {
    e.v = (double)ld_stream(val + j);
    e.a = ld_stream(crd + j);
  }
  __device__ __forceinline__ void prefetch(int32_t c, int32_t, Slot &s) const {
    ln.gather_hint(reinterpret_cast<const T *>(bcol + (int64_t)c * ldb_bytes), s.r, keep);
  }
  __device__ __forceinline__ void begin_chunk(int32_t) {}
  __device__ __forceinline__ void consume(int, double v, int32_t, Slot &s) { ln.fma_rows(v, s.r, acc); }
};

// The CTAs that take this role draw tiles until none is left.
template <class T, int LPN, int CPL, int VEC>
__device__ __forceinline__ void heavy_role(const HeavyArgs &a, unsigned char *smem_raw) {
  using L = Lanes<T, LPN, CPL, VEC>;
  const int worker = threadIdx.x / LPN;
  const uint32_t smem = smem_u32(smem_raw) + worker * RingLayout<L, false>::kWorkerBytes;
  const L ln(a.R);
  HeavyPolicy<T, LPN, CPL, VEC> p(a, ln);
  const int32_t tiles = __ldcg(a.counters + 2);
  for (;;) {
    int32_t t = 0;
    if (ln.g == 0) t = atomicAdd(a.counters + 5, 1);
    t = __shfl_sync(ln.mask, t, 0, LPN);
    if (t >= tiles) break;
    const int4 rec = __ldcg(a.rec + t);
    ln.zero(p.acc);
    walk_tile(ln, p, rec.x, rec.y, smem);
    ln.store_carry(a.carry_val + (int64_t)rec.z * a.carry_ld + ln.col0, p.acc);
    ln.sync();                                               // the ring is re-used by the next tile
  }
}

// Host side (spmm_heavy.cu). plan: decides whether the path applies (returns 0 if not) and how much scratch it
// needs; prepare: lays the arrays out in `scratch` and runs the three analysis kernels. The fix-up that writes the
// long rows of C after the gather kernel is heavy_fixup_role below.
size_t spmm_heavy_plan(int dtype, int64_t M, int64_t N, int64_t cols, const void *B, int64_t ldb, int64_t R, const void *C,
                       int64_t ldc, int32_t min_threshold, HeavyArgs *out);
comet_status_t spmm_heavy_prepare(Context *ctx, HeavyArgs *args, const int32_t *pos, const int32_t *crd, const void *val,
                                  char *scratch, cudaStream_t stream);


// The long rows' fix-up, a role of the fix-up launch (contract_vec.cu; `block` of `blocks` CTAs play it):
// C[row, :] = the sum of the row's slots, a long row per CTA and step. The 256 threads are G groups of R columns
// (G = 256 / R, at least 1); group g adds the slots g, g + G, g + 2G, ... in that order (up to sixteen loads in
// flight), and the groups' sums are then added in group order: a fixed order, so results stay bit-identical from
// run to run.
template <class T>
__device__ __forceinline__ void heavy_fixup_role(const HeavyArgs &a, int block, int blocks) {
  __shared__ double s_part[kBlockThreads];
  const int32_t H = __ldcg(a.counters + 0);
  T *C = static_cast<T *>(a.C);
  const int R = a.R;
  const int G = R < kBlockThreads ? kBlockThreads / R : 1;      // R is a power of two here (the shapes of the long-row path)
  const int g = threadIdx.x / R;
  for (int32_t h = block; h < H; h += blocks) {
    const int32_t n = a.row_nt[h];
    for (int c = threadIdx.x % R; c < R; c += kBlockThreads) {  // one sweep unless R > 256
      const double *src = a.carry_val + (int64_t)a.row_slot0[h] * a.carry_ld + c;
      double sum = 0.0;
      int32_t t = g;
      for (; t + 15 * G < n; t += 16 * G) {
        double v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = __ldcs(src + (int64_t)(t + u * G) * a.carry_ld);
#pragma unroll
        for (int u = 0; u < 16; ++u) sum += v[u];
      }
      for (; t < n; t += G) sum += __ldcs(src + (int64_t)t * a.carry_ld);
      if (G > 1) {
        __syncthreads();                                        // the sums of the row before have been read
        s_part[threadIdx.x] = sum;
        __syncthreads();
        if (g == 0) {
          for (int x = 1; x < G; ++x) sum += s_part[x * R + c];
          C[(int64_t)a.hrow[h] * a.ldc + c] = (T)sum;
        }
      } else {
        C[(int64_t)a.hrow[h] * a.ldc + c] = (T)sum;
      }
    }
  }
}


}  // namespace comet
