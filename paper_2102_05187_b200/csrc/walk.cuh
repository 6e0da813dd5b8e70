// The tile walker shared by the matrix-operand contractions (SpMM, TTM, MTTKRP).
//
// A WORKER is a group of LPN lanes of one warp. Lane g of the group owns VEC consecutive columns of
// each of CPL row pieces: columns (t*LPN + g)*VEC .. +VEC for t < CPL, so one gather of a dense-operand
// row by the group is one contiguous LPN*VEC*8-byte request and no value ever crosses lanes.
//
// A worker walks a tile of consecutive leaf entries [j0, j1):
//   * the leaf arrays (value, coordinates) are read with coalesced group loads, kChunk entries at a
//     time and one refill ahead of use, and parked in a per-worker shared-memory ring (2 x kChunk
//     16-byte entries, plus an optional int32 side ring) from which every lane re-reads an entry with
//     one broadcast 128-bit LDS;
//   * the dense-operand rows of the next kPF entries are always in flight in a rolling REGISTER window
//     (slot q % kPF). Gathered rows never touch shared memory: staging them there was measured and
//     saturates the L1/shared-memory pipe (90 % on TTM) long before L2 does;
//   * the chunk body is fully unrolled, so window slots, ring offsets and the position inside the
//     chunk are compile-time constants;
//   * what is done with an entry and its gathered rows (segment ends, accumulation, stores) is the
//     policy's business.
//
// Policy interface (called by every lane of the group; control flow is group-uniform):
//   static constexpr int kPF            entries whose rows are in flight
//   static constexpr bool kAux          whether a second int32 per entry is staged
//   static constexpr bool kFullUnroll   unroll the whole chunk (cheap consume) or only kPF-wide steps
//   struct Slot                         the gathered rows of one in-flight entry (nothing else: the value
//                                       and the aux word are re-read from the ring when the entry is consumed)
//   void fetch(int32_t j, Entry16 &e, int32_t &aux) const   read leaf entry j from global memory
//   void prefetch(int32_t a, int32_t b, Slot &s) const      issue the row gathers of an entry (its two coordinates)
//   void begin_chunk(int32_t base)      positions inside the chunk are relative to `base`
//   void consume(int q, double v, int32_t aux, Slot &s)     entry at position base + q
#pragma once

#include "common.cuh"

namespace comet {

struct Entry16 { double v; int32_t a; int32_t b; };

// 32-bit shared-memory addressing through PTX: one LDS/STS each, no generic-pointer conversions.
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ Entry16 lds_entry(uint32_t addr) {
  int x, y, z, w;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(addr));
  Entry16 e;
  e.v = __hiloint2double(y, x);
  e.a = z;
  e.b = w;
  return e;
}
__device__ __forceinline__ double lds_f64(uint32_t addr) {
  double v;
  asm volatile("ld.shared.f64 %0, [%1];" : "=d"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void lds_coords(uint32_t entry_addr, int32_t &a, int32_t &b) {   // words 2, 3 of an entry
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+8];" : "=r"(a), "=r"(b) : "r"(entry_addr));
}
__device__ __forceinline__ void sts_entry(uint32_t addr, const Entry16 &e) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(__double2loint(e.v)),
               "r"(__double2hiint(e.v)), "r"(e.a), "r"(e.b)
               : "memory");
}
__device__ __forceinline__ int32_t lds_s32(uint32_t addr) {
  int32_t v;
  asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_s32(uint32_t addr, int32_t v) {
  asm volatile("st.shared.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// A lane's piece of a dense row: VEC elements of T. Vector pieces are 16 bytes (2 doubles or 4 floats);
// VEC == 1 is the scalar path for ragged widths or unaligned operands. Loads are volatile so that the
// gathers keep their program order relative to the ring reads: exactly the rolling window is in flight
// (the scheduler otherwise hoists loads of far-ahead entries and spills).
template <class T, int VEC> struct Piece;
// L2 eviction policies for the gathers of a kernel whose CTAs play two roles at once: rows that are re-used out
// of L2 are kept (evict_last) while rows that are read once pass through (evict_first).
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
template <> struct Piece<double, 2> {
  static __device__ __forceinline__ void load(const double *p, double (&d)[2]) {
    asm volatile("ld.global.nc.v2.f64 {%0, %1}, [%2];" : "=d"(d[0]), "=d"(d[1]) : "l"(p));
  }
  static __device__ __forceinline__ void load_hint(const double *p, double (&d)[2], uint64_t pol) {
    asm volatile("ld.global.nc.L2::cache_hint.v2.f64 {%0, %1}, [%2], %3;" : "=d"(d[0]), "=d"(d[1]) : "l"(p), "l"(pol));
  }
  static __device__ __forceinline__ void store_stream(double *p, const double (&d)[2]) {
    __stcs(reinterpret_cast<double2 *>(p), make_double2(d[0], d[1]));
  }
};
template <> struct Piece<double, 1> {
  static __device__ __forceinline__ void load(const double *p, double (&d)[1]) {
    asm volatile("ld.global.nc.f64 %0, [%1];" : "=d"(d[0]) : "l"(p));
  }
  static __device__ __forceinline__ void store_stream(double *p, const double (&d)[1]) { __stcs(p, d[0]); }
};
template <> struct Piece<float, 4> {
  static __device__ __forceinline__ void load(const float *p, float (&d)[4]) {
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "l"(p));
  }
  static __device__ __forceinline__ void load_hint(const float *p, float (&d)[4], uint64_t pol) {
    asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "l"(p), "l"(pol));
  }
  static __device__ __forceinline__ void store_stream(float *p, const double (&d)[4]) {
    __stcs(reinterpret_cast<float4 *>(p), make_float4((float)d[0], (float)d[1], (float)d[2], (float)d[3]));
  }
};
template <> struct Piece<float, 1> {
  static __device__ __forceinline__ void load(const float *p, float (&d)[1]) {
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(d[0]) : "l"(p));
  }
  static __device__ __forceinline__ void store_stream(float *p, const double (&d)[1]) { __stcs(p, (float)d[0]); }
};

// T is the storage type of values and dense operands (double or float); sums are always kept in double.
template <class T_, int LPN_, int CPL_, int VEC_> struct Lanes {
  using T = T_;
  static constexpr int LPN = LPN_, CPL = CPL_, VEC = VEC_;
  // leaf entries per refill of the ring (8 for the narrow shapes: 16 was measured 3 % slower on TTM config 4,
  // the staging registers of a second entry per lane are better spent elsewhere)
  static constexpr int kChunk = LPN >= 16 ? 32 : 8;
  static constexpr int kPer = kChunk / LPN;                // entries each lane loads per refill
  static constexpr int kWorkers = kBlockThreads / LPN;     // workers per CTA
  static constexpr int kStride = LPN * VEC;                // columns between a lane's consecutive pieces
  static constexpr bool kVector = VEC * sizeof(T) == 16;   // 128-bit pieces: the launch width is never ragged

  int g;            // lane within the group
  unsigned mask;    // the group's lanes
  int32_t col0;     // first column of piece 0; piece t starts at col0 + t * kStride
  bool ok[CPL];     // piece inside the R columns of this launch (only the scalar path is ever ragged)

  __device__ __forceinline__ Lanes(int R) {
    g = threadIdx.x & (LPN - 1);
    const unsigned lane = threadIdx.x & 31;
    mask = LPN == 32 ? 0xffffffffu : (((1u << LPN) - 1u) << (lane & ~(LPN - 1)));
    col0 = g * VEC;
#pragma unroll
    for (int t = 0; t < CPL; ++t) ok[t] = kVector ? true : (col0 + t * kStride) < R;
  }
  __device__ __forceinline__ void sync() const { __syncwarp(mask); }

  __device__ __forceinline__ void zero(double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[t][e] = 0.0;
  }
  // `row` already points at this lane's piece 0 (row base + col0)
  __device__ __forceinline__ void gather(const T *row, T (&dst)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) Piece<T, VEC>::load(row + t * kStride, dst[t]);
  }
  // the same with an L2 eviction policy (128-bit pieces only; the other shapes never carry two roles)
  __device__ __forceinline__ void gather_hint(const T *row, T (&dst)[CPL][VEC], uint64_t pol) const {
    if constexpr (VEC * sizeof(T) == 16) {
#pragma unroll
      for (int t = 0; t < CPL; ++t) Piece<T, VEC>::load_hint(row + t * kStride, dst[t], pol);
    } else {
      gather(row, dst);
    }
  }
  __device__ __forceinline__ void store_row(T *row, const double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t]) Piece<T, VEC>::store_stream(row + t * kStride, acc[t]);
  }
  __device__ __forceinline__ void store_carry(double *row, const double (&acc)[CPL][VEC]) const {   // carries stay double
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t])
#pragma unroll
        for (int e = 0; e < VEC; ++e) row[t * kStride + e] = acc[t][e];
  }
  // rows lo .. hi-1 of a matrix whose lane-piece-0 pointer of row 0 is `base`
  __device__ __forceinline__ void zero_rows(T *base, int64_t ld, int64_t lo, int64_t hi) const {
    double z[CPL][VEC];
    zero(z);
    for (int64_t r = lo; r < hi; ++r) store_row(base + r * ld, z);
  }
  __device__ __forceinline__ void fma_rows(double v, const T (&row)[CPL][VEC], double (&acc)[CPL][VEC]) const {
#pragma unroll
    for (int t = 0; t < CPL; ++t)
      if (ok[t])
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[t][e] = fma(v, (double)row[t][e], acc[t][e]);
  }
};

// Shared memory of one worker: the entry ring, then (when the policy stages an aux word) the side ring.
template <class L, bool AUX> struct RingLayout {
  static constexpr int kEntryBytes = 2 * L::kChunk * 16;
  // +16: the workers of one warp read the same ring position in the same instruction; without the skew
  // their rings are a multiple of 128 bytes apart and every broadcast read is a 2- to 8-way bank conflict
  static constexpr int kWorkerBytes = kEntryBytes + (AUX ? 2 * L::kChunk * 4 : 0) + 16;
  static constexpr size_t kBlockBytes = (size_t)L::kWorkers * kWorkerBytes;
};

// A policy that declares `static constexpr bool kPositional = true` is told WHERE the entry it prefetches sits
// (position `at` of the current or of the next chunk) through prefetch_at(at, in_current_chunk, a, b, slot):
// for policies that keep per-chunk information about the entries (the CSF fiber-end masks).
template <class P, class = void> struct policy_is_positional { static constexpr bool value = false; };
template <class P> struct policy_is_positional<P, decltype((void)P::kPositional)> { static constexpr bool value = P::kPositional; };

// A policy that declares `static constexpr bool kTwoSpeed = true` has two ways to consume an entry: the full
// consume(), and consume_plain() for the chunks for which plain_chunk() says that the rare, long part of
// consume() cannot happen (end_plain_chunk() then settles the bookkeeping for the whole chunk). Only the plain
// form is unrolled; the full form runs as a loop, so the code stays small enough for the instruction cache.
template <class P, class = void> struct policy_is_two_speed { static constexpr bool value = false; };
template <class P> struct policy_is_two_speed<P, decltype((void)P::kTwoSpeed)> { static constexpr bool value = P::kTwoSpeed; };

// kEntryConsume: the policy wants the whole staged entry (value and both coordinate words, one 128-bit read)
// when it consumes it, through consume_entry(q, entry, slot): for flags that travel in the coordinate words.
template <class P, class = void> struct policy_consumes_entry { static constexpr bool value = false; };
template <class P> struct policy_consumes_entry<P, decltype((void)P::kEntryConsume)> { static constexpr bool value = P::kEntryConsume; };

// kSlotCarries: the policy keeps what it needs of an entry (value, flags) in the window slot, filled when the
// entry's rows are requested: prefetch_entry(entry, slot) gets the whole staged entry (one 128-bit read) and
// consume_slot(q, slot) reads nothing from shared memory. One shared-memory read per entry instead of two.
template <class P, class = void> struct policy_slot_carries { static constexpr bool value = false; };
template <class P> struct policy_slot_carries<P, decltype((void)P::kSlotCarries)> { static constexpr bool value = P::kSlotCarries; };

template <class P, class = void> struct policy_rolls_tail { static constexpr bool value = false; };
template <class P> struct policy_rolls_tail<P, decltype((void)P::kRolledTail)> { static constexpr bool value = P::kRolledTail; };

// One chunk, unrolled: positions 0..n-1 of the ring half at shared address `cur`; `nxt` is the other half. Ring
// offsets and positions are immediates.
template <class L, class Policy, bool TAIL, bool PLAIN>
__device__ __forceinline__ void walk_chunk_unrolled(Policy &p, typename Policy::Slot (&win)[Policy::kPF], uint32_t cur,
                                                    uint32_t nxt, uint32_t cur_aux, uint32_t nxt_aux, int n) {
  constexpr int kChunk = L::kChunk, kPF = Policy::kPF;
#pragma unroll
  for (int q = 0; q < kChunk; ++q) {
    if (TAIL && q >= n) break;
    if constexpr (policy_slot_carries<Policy>::value) p.consume_slot(q, win[q % kPF]);
    else if constexpr (PLAIN) p.consume_plain(q, lds_f64(cur + q * 16), win[q % kPF]);
    else if constexpr (policy_consumes_entry<Policy>::value) p.consume_entry(q, lds_entry(cur + q * 16), win[q % kPF]);
    else p.consume(q, lds_f64(cur + q * 16), Policy::kAux ? lds_s32(cur_aux + q * 4) : 0, win[q % kPF]);
    // refill the slot with the entry kPF ahead (it may sit in the next chunk's half of the ring);
    // the last, partial chunk only looks ahead inside itself
    if (TAIL && q + kPF >= n) continue;
    const bool in_cur = q + kPF < kChunk;
    const int at = in_cur ? q + kPF : q + kPF - kChunk;
    if constexpr (policy_slot_carries<Policy>::value) {
      p.prefetch_entry(lds_entry((in_cur ? cur : nxt) + at * 16), win[q % kPF]);
    } else {
      int32_t ca, cb;
      lds_coords((in_cur ? cur : nxt) + at * 16, ca, cb);
      if constexpr (policy_is_positional<Policy>::value) p.prefetch_at(at, in_cur, ca, cb, win[q % kPF]);
      else p.prefetch(ca, cb, win[q % kPF]);
    }
  }
}

// One chunk as a loop of kPF-wide unrolled steps (for heavy per-segment work, where code size matters more).
template <class L, class Policy, bool TAIL>
__device__ __forceinline__ void walk_chunk_rolled(Policy &p, typename Policy::Slot (&win)[Policy::kPF], uint32_t cur,
                                                  uint32_t nxt, uint32_t cur_aux, uint32_t nxt_aux, int n) {
  constexpr int kChunk = L::kChunk, kPF = Policy::kPF;
  // the two halves are adjacent in shared memory: position q + kPF of `cur` wraps into `nxt`
  const uint32_t lo = cur < nxt ? cur : nxt, lo_aux = cur_aux < nxt_aux ? cur_aux : nxt_aux;
  const int off = cur < nxt ? 0 : kChunk;
#pragma unroll 1
  for (int q0 = 0; q0 < (TAIL ? n : kChunk); q0 += kPF) {
#pragma unroll
    for (int u = 0; u < kPF; ++u) {
      const int q = q0 + u;
      if (TAIL && q >= n) break;
      const int r = off + q;
      if constexpr (policy_slot_carries<Policy>::value) p.consume_slot(q, win[u]);
      else if constexpr (policy_consumes_entry<Policy>::value) p.consume_entry(q, lds_entry(lo + r * 16), win[u]);
      else p.consume(q, lds_f64(lo + r * 16), Policy::kAux ? lds_s32(lo_aux + r * 4) : 0, win[u]);
      if (TAIL && q + kPF >= n) continue;
      if constexpr (policy_slot_carries<Policy>::value) {
        p.prefetch_entry(lds_entry(lo + ((r + kPF) & (2 * kChunk - 1)) * 16), win[u]);
      } else {
        int32_t ca, cb;
        lds_coords(lo + ((r + kPF) & (2 * kChunk - 1)) * 16, ca, cb);
        if constexpr (policy_is_positional<Policy>::value) p.prefetch_at((q + kPF) & (kChunk - 1), q + kPF < kChunk, ca, cb, win[u]);
        else p.prefetch(ca, cb, win[u]);
      }
    }
  }
}

template <class L, class Policy, bool TAIL>
__device__ __forceinline__ void walk_chunk(Policy &p, typename Policy::Slot (&win)[Policy::kPF], uint32_t cur,
                                           uint32_t nxt, uint32_t cur_aux, uint32_t nxt_aux, int n) {
  if constexpr (policy_is_two_speed<Policy>::value) {
    if (!TAIL && p.plain_chunk()) {
      walk_chunk_unrolled<L, Policy, false, true>(p, win, cur, nxt, cur_aux, nxt_aux, n);
      p.end_plain_chunk();
    } else {
      walk_chunk_rolled<L, Policy, TAIL>(p, win, cur, nxt, cur_aux, nxt_aux, n);
    }
  } else if constexpr (Policy::kFullUnroll) {
    // kRolledTail: the one partial chunk of a tile runs as a loop, so that only one copy of the unrolled body exists
    if constexpr (TAIL && policy_rolls_tail<Policy>::value) walk_chunk_rolled<L, Policy, true>(p, win, cur, nxt, cur_aux, nxt_aux, n);
    else walk_chunk_unrolled<L, Policy, TAIL, false>(p, win, cur, nxt, cur_aux, nxt_aux, n);
  } else {
    walk_chunk_rolled<L, Policy, TAIL>(p, win, cur, nxt, cur_aux, nxt_aux, n);
  }
}

// Walks leaf entries [j0, j1) of one tile. `smem` is the shared address of this worker's ring memory.
template <class L, class Policy>
__device__ __forceinline__ void walk_tile(const L &ln, Policy &p, int32_t j0, int32_t j1, uint32_t smem) {
  constexpr int kChunk = L::kChunk, kPer = L::kPer, kPF = Policy::kPF, LPN = L::LPN;
  static_assert(kChunk % kPF == 0 && kPF <= kChunk, "the rolling window must divide the chunk");
  if (j0 >= j1) return;
  const uint32_t s_aux = smem + RingLayout<L, Policy::kAux>::kEntryBytes;

  Entry16 regs[kPer];
  int32_t regs_aux[kPer];
  auto load_regs = [&](int32_t base) {                   // base may run past the tile: idle entries
#pragma unroll
    for (int t = 0; t < kPer; ++t) {
      const int32_t j = base + t * LPN + ln.g;
      regs[t] = Entry16{0.0, 0, 0};
      regs_aux[t] = 0;
      if (j < j1) p.fetch(j, regs[t], regs_aux[t]);
    }
  };
  auto store_regs = [&](int half) {
#pragma unroll
    for (int t = 0; t < kPer; ++t) {
      const int at = half * kChunk + t * LPN + ln.g;
      sts_entry(smem + at * 16, regs[t]);
      if (Policy::kAux) sts_s32(s_aux + at * 4, regs_aux[t]);
    }
  };

  load_regs(j0);
  store_regs(0);
  load_regs(j0 + kChunk);
  ln.sync();

  typename Policy::Slot win[kPF];
#pragma unroll
  for (int u = 0; u < kPF; ++u) {
    if constexpr (policy_slot_carries<Policy>::value) {
      p.prefetch_entry(lds_entry(smem + u * 16), win[u]);
    } else {
      int32_t ca, cb;
      lds_coords(smem + u * 16, ca, cb);
      if constexpr (policy_is_positional<Policy>::value) p.prefetch_at(u, true, ca, cb, win[u]);
      else p.prefetch(ca, cb, win[u]);
    }
  }

  int half = 0;
  for (int32_t base = j0; base < j1; base += kChunk, half ^= 1) {
    ln.sync();                       // every lane is done reading the half that is refilled next
    store_regs(half ^ 1);            // entries of the next chunk (idle entries past the tile)
    ln.sync();
    load_regs(base + 2 * kChunk);    // and the chunk after it goes into registers
    const uint32_t cur = smem + half * (kChunk * 16), nxt = smem + (half ^ 1) * (kChunk * 16);
    const uint32_t cur_aux = s_aux + half * (kChunk * 4), nxt_aux = s_aux + (half ^ 1) * (kChunk * 4);
    p.begin_chunk(base);
    const int n = j1 - base;
    if (n >= kChunk) walk_chunk<L, Policy, false>(p, win, cur, nxt, cur_aux, nxt_aux, kChunk);
    else walk_chunk<L, Policy, true>(p, win, cur, nxt, cur_aux, nxt_aux, n);
  }
}

}  // namespace comet
