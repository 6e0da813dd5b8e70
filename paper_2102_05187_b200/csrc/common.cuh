// Shared device/host helpers of libcomet (sm_100a). Internal: not part of the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/comet.h"

namespace comet {

constexpr int kSmCount = 148;            // B200: 2 dies x 74 SMs; grids are sized against this
constexpr int kBlockThreads = 256;

struct Context {
  comet_allocator_t allocator;            // user allocator or the cudaMalloc fallback
  bool user_allocator;
  int device;
  int last_cuda_error;
  void *scratch;                          // cached scratch, grown on demand
  size_t scratch_bytes;
  int32_t *h_pinned;                      // small pinned buffer for device->host size reads
  int32_t *d_status;                      // device words written by checking kernels
  int64_t launches;                       // kernels launched through this handle (for accounting)
  cudaStream_t last_stream;               // stream of the latest call that used the scratch or the counters
  bool has_last_stream;
  bool counters_dirty;                    // a CUDA call failed: the device counters may not be back at zero
  bool has_copy_streams;                  // comet_spmm_from_host: its two copy streams and events, made on first use
  cudaStream_t copy_in, copy_out;
  cudaEvent_t copy_event[2 * 8 + 2];
};
constexpr int kCopyChunks = 8;            // most column chunks of comet_spmm_from_host
constexpr int kCopyEvents = 2 * kCopyChunks + 2;
void host_streams_destroy(Context *ctx);

// Grows the cached scratch buffer to at least `bytes` and returns it (NULL on allocation failure).
void *scratch_get(Context *ctx, size_t bytes, cudaStream_t stream);
void *ctx_alloc(Context *ctx, size_t bytes, cudaStream_t stream);
void ctx_free(Context *ctx, void *p, cudaStream_t stream);
comet_status_t cuda_fail(Context *ctx, cudaError_t e);

#define COMET_CUDA_TRY(ctx, expr)                         \
  do {                                                    \
    cudaError_t e__ = (expr);                             \
    if (e__ != cudaSuccess) return cuda_fail((ctx), e__); \
  } while (0)

// After a kernel launch (or `n` back-to-back launches): count them and surface a launch error.
#define COMET_LAUNCHED(ctx, n)                       \
  do {                                               \
    (ctx)->launches += (n);                          \
    COMET_CUDA_TRY((ctx), cudaGetLastError());       \
  } while (0)
#define COMET_LAUNCH_CHECK(ctx) COMET_LAUNCHED(ctx, 1)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------------------------------------
// device helpers

// Streaming (read-once) loads: evict-first so that index/value streams do not displace the dense
// operand rows that are re-used out of L2.
__device__ __forceinline__ int32_t ld_stream(const int32_t *p) { return __ldcs(p); }
__device__ __forceinline__ double ld_stream(const double *p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream(const float *p) { return __ldcs(p); }

// Merge-path split: the merge list interleaves segment-end markers (segment s ends at leaf position
// seg_end[s]) with the leaf positions 0..N-1; at state (i, j) the next item is leaf j if
// j < seg_end[i], else the end marker of segment i. Marker s is therefore item number seg_end[s] + s.
// Returns how many markers lie among the first `diag` items; the leaf count is diag minus that.
__device__ __forceinline__ int64_t merge_path_segments(const int32_t *__restrict__ seg_end, int64_t M, int64_t N,
                                                       int64_t diag) {
  int64_t lo = diag > N ? diag - N : 0;
  int64_t hi = diag < M ? diag : M;
  while (lo < hi) {
    int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(seg_end + mid) + mid < diag) lo = mid + 1; else hi = mid;
  }
  return lo;
}


// The same split found cooperatively by W consecutive lanes (W a power of two, `mask` = those lanes,
// `k` = this lane's index among them): a W-ary search, log_W(M) rounds of one coalesced-ish probe per
// lane instead of log_2(M) dependent loads by one thread. Every lane returns the result.
template <int W>
__device__ __forceinline__ int64_t merge_path_segments_coop(const int32_t *__restrict__ seg_end, int64_t M, int64_t N,
                                                            int64_t diag, int k, unsigned mask) {
  int64_t lo = diag > N ? diag - N : 0;
  int64_t hi = diag < M ? diag : M;                 // markers below lo are inside, markers from hi on are not
  const int shift = (threadIdx.x & 31) & ~(W - 1);
  while (lo < hi) {
    const int64_t stride = (hi - lo + W - 1) / W;
    const int64_t s = lo + (int64_t)k * stride + stride - 1;     // last marker of this lane's sub-range
    const bool inside = s < hi && (int64_t)__ldg(seg_end + s) + s < diag;
    const unsigned votes = (__ballot_sync(mask, inside) >> shift) & (W == 32 ? 0xffffffffu : ((1u << W) - 1u));
    const int full = __popc(votes);                // sub-ranges that lie wholly inside (the predicate is monotone)
    lo += (int64_t)full * stride;
    const int64_t cap = lo + stride - 1;           // the last marker of the first mixed sub-range is outside
    if (cap < hi) hi = cap;
  }
  return lo;
}

}  // namespace comet
