// The tile walker shared by the matrix-operand contractions (SpMM, TTM, MTTKRP).
//
// A WORKER is a group of LPN lanes of one warp. Lane g of the group owns VEC consecutive columns of
// each of CPL row pieces: columns (t*LPN + g)*VEC .. +VEC for t < CPL, so one gather of a dense-operand
// row by the group is one contiguous LPN*VEC*8-byte request and no value ever crosses lanes.
//
// A worker walks a tile of consecutive leaf entries [j0, j1):
//   * the leaf arrays (coordinates, value) are read with coalesced group loads, kChunk entries at a
//     time, one refill ahead of use, and parked in a per-worker shared-memory ring (2 x kChunk
//     entries) from which every lane re-reads them with one broadcast LDS per entry;
//   * the dense-operand rows of the next kPF entries are always in flight (a rolling register
//     window), so the gather latency is hidden inside one worker, not only across warps;
//   * what is done with an entry and its gathered rows (segment ends, accumulation, stores) is the
//     policy's business: consume().
//
// Policy interface (all members called by every lane of the group, group-uniform control flow):
//   typename Entry                       16- or 32-byte POD staged per leaf entry
//   static constexpr int kRows           dense rows gathered per entry (1 or 2)
//   Entry fetch(int j) const             read leaf entry j from global memory
//   static Entry idle()                  a harmless entry (row 0, value 0) for slots past the tile
//   const double *row(const Entry &, int which) const   base pointer of the row to gather
//   struct Window { double r[kRows][CPL][VEC]; }   the gathered rows of one entry
//   void consume(int j, const Entry &, const double (&rows)[kRows][CPL][VEC])
#pragma once

#include "common.cuh"

namespace comet {

struct Entry16 { double v; int32_t a; int32_t b; };
struct Entry32 { double v; int32_t a; int32_t b; int32_t c; int32_t pad0; int64_t pad1; };
static_assert(sizeof(Entry16) == 16 && sizeof(Entry32) == 32, "staged entries are whole 16-byte words");

template <int VEC> struct Piece;
template <> struct Piece<2> {
  static __device__ __forceinline__ void load(const double *p, double (&d)[2]) {
    const double2 v = __ldg(reinterpret_cast<const double2 *>(p));
    d[0] = v.x; d[1] = v.y;
  }
  static __device__ __forceinline__ void store_stream(double *p, const double (&d)[2]) {
    __stcs(reinterpret_cast<double2 *>(p), make_double2(d[0], d[1]));
  }
  static __device__ __forceinline__ void store(double *p, const double (&d)[2]) {
    *reinterpret_cast<double2 *>(p) = make_double2(d[0], d[1]);
  }
};
template <> struct Piece<1> {
  static __device__ __forceinline__ void load(const double *p, double (&d)[1]) { d[0] = __ldg(p); }
  static __device__ __forceinline__ void store_stream(double *p, const double (&d)[1]) { __stcs(p, d[0]); }
  static __device__ __forceinline__ void store(double *p, const double (&d)[1]) { *p = d[0]; }
};

template <int LPN, int CPL, int VEC> struct Lanes {
  static constexpr int kChunk = LPN >= 4 ? 32 : 8 * LPN;   // leaf entries per refill of the ring
  static constexpr int kPer = kChunk / LPN;                // entries each lane loads per refill
  static constexpr int kPF = 8;                            // gathers in flight per worker
  static constexpr int kWorkers = kBlockThreads / LPN;     // workers per CTA
  static_assert(kChunk % kPF == 0, "the rolling window must divide the chunk");

  int g;            // lane within the group
  unsigned mask;    // the group's lanes
  int32_t col[CPL]; // first column of each owned piece
  bool ok[CPL];     // piece inside the R columns of this launch (only the scalar path is ever ragged)

  __device__ __forceinline__ Lanes(int R) {
    g = threadIdx.x & (LPN - 1);
    const unsigned lane = threadIdx.x & 31;
    mask = LPN == 32 ? 0xffffffffu : (((1u << LPN) - 1u) << (lane & ~(LPN - 1)));
#pragma unroll
    for (int t = 0; t < CPL; ++t) {
      col[t] = (t * LPN + g) * VEC;
      ok[t] = VEC == 2 ? true : col[t] < R;
    }
  }
  __device__ __forceinline__ void sync() const { __syncwarp(mask); }

  __device__ __forceinline__ void zero(double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;
  }
  __device__ __forceinline__ void gather(const double *row, double (&dst)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) Piece<VEC>::load(row + col[t], dst[t]);
  }
  // out_row[0..R) = acc, streaming stores (written once, never re-read by this kernel)
  __device__ __forceinline__ void store_row(double *row, const double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) Piece<VEC>::store_stream(row + col[t], acc[t]);
  }
  __device__ __forceinline__ void store_carry(double *row, const double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) Piece<VEC>::store(row + col[t], acc[t]);
  }
  __device__ __forceinline__ void zero_rows(double *base, int64_t ld, int64_t lo, int64_t hi) const {
    double z[CPL][VEC];
    zero(z);
    for (int64_t r = lo; r < hi; ++r) store_row(base + r * ld, z);
  }
};

// Walks leaf entries [j0, j1) of one tile. `ring` is this worker's 2*kChunk-entry shared-memory ring.
template <class L, class Policy>
__device__ __forceinline__ void walk_tile(const L &ln, Policy &p, int32_t j0, int32_t j1,
                                          typename Policy::Entry *ring) {
  using Entry = typename Policy::Entry;
  constexpr int kChunk = L::kChunk, kPer = L::kPer, kPF = L::kPF, kRows = Policy::kRows;
  constexpr int LPN = kChunk / kPer;
  if (j0 >= j1) return;

  Entry regs[kPer];
  auto load_regs = [&](int32_t base) {
#pragma unroll
    for (int t = 0; t < kPer; ++t) {
      const int32_t j = base + t * LPN + ln.g;
      regs[t] = (j < j1) ? p.fetch(j) : Policy::idle();   // base may run past the tile: idle entries
    }
  };
  auto store_regs = [&](int half) {
#pragma unroll
    for (int t = 0; t < kPer; ++t) ring[half * kChunk + t * LPN + ln.g] = regs[t];
  };

  load_regs(j0);
  store_regs(0);
  load_regs(j0 + kChunk);
  ln.sync();

  Entry e[kPF];
  typename Policy::Window win[kPF];
#pragma unroll
  for (int u = 0; u < kPF; ++u) {
    e[u] = ring[u];
#pragma unroll
    for (int w = 0; w < kRows; ++w) ln.gather(p.row(e[u], w), win[u].r[w]);
  }

  int half = 0;
  for (int32_t base = j0; base < j1; base += kChunk, half ^= 1) {
    ln.sync();                       // every lane is done reading the half that is refilled next
    store_regs(half ^ 1);            // entries of the next chunk (idle entries past the tile)
    ln.sync();
    load_regs(base + 2 * kChunk);    // and the chunk after it goes into registers
    const int n = (j1 - base < kChunk) ? (j1 - base) : kChunk;
    if (n == kChunk) {
      for (int q0 = 0; q0 < kChunk; q0 += kPF) {
#pragma unroll
        for (int u = 0; u < kPF; ++u) {
          p.consume(base + q0 + u, e[u], win[u].r);
          e[u] = ring[(half * kChunk + q0 + u + kPF) & (2 * kChunk - 1)];
#pragma unroll
          for (int w = 0; w < kRows; ++w) ln.gather(p.row(e[u], w), win[u].r[w]);
        }
      }
    } else {
      for (int q0 = 0; q0 < n; q0 += kPF) {
#pragma unroll
        for (int u = 0; u < kPF; ++u) {
          if (q0 + u < n) p.consume(base + q0 + u, e[u], win[u].r);
          e[u] = ring[(half * kChunk + q0 + u + kPF) & (2 * kChunk - 1)];
#pragma unroll
          for (int w = 0; w < kRows; ++w) ln.gather(p.row(e[u], w), win[u].r[w]);
        }
      }
    }
  }
}

}  // namespace comet
