// MTTKRP for an output mode that is NOT stored first (levels 1 and 2 of a 3-level tensor), on the
// tensor as it is: nothing is re-packed or permuted.
//
// With the output mode below the root the terms of one output row are spread over the whole tensor
// (the entries are sorted by the root mode first), so no tile owns a row. The terms are therefore
// added into the output with floating-point atomic adds. Two consequences, both stated in the header:
// the summation order is not fixed (results agree from run to run only up to rounding, unlike every
// other kernel of the library), and the output is zero-filled first. Sums are kept in double: for
// fp32 tensors the atomics go to a double scratch matrix that is rounded into the output at the end.
//
// CSF [CU,CU,CU], coordinates (i, j, k) at levels 0..2, A / B = the factors of the two other modes:
//   level 1:  out[j, :] += (sum over the fiber's entries of val * B[k, :]) * A[i, :]     one add per fiber
//   level 2:  out[k, :] += val * (A[i, :] * B[j, :])                                     one add per entry
// COO [CN,S,S]:  out[c_out, :] += val * A[c_a, :] * B[c_b, :]                            one add per entry
//
// A worker is G lanes (G = the power of two covering min(R, 32) columns); it owns a few consecutive
// fibers (CSF) or entries (COO), finds its slice once by binary search in the level-1 pos array and
// then advances it. Lanes of a worker touch consecutive columns, so row reads and atomic adds are
// one contiguous request per worker.
#include "common.cuh"
#include "kernels.cuh"

namespace comet {

struct ScatterArgs {
  const int32_t *pos1, *crd0, *crd1, *pos2, *crd2;   // CSF levels (COO: crd0/crd1/crd2 = out / a / b coordinates)
  const void *val;
  int64_t S, F, N;
  const void *A, *B;
  int64_t lda, ldb;
  double *acc;                                         // rows x R sums, leading dimension ldacc
  int64_t ldacc;
  int32_t R;
  int32_t per_worker;                                  // fibers (CSF) or entries (COO) per worker
};

constexpr int kScatterThreads = 256;

template <class T, int LEVEL, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_csf_scatter_kernel(const ScatterArgs a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t f0 = worker * a.per_worker;
  if (f0 >= a.F) return;
  const int64_t f1 = f0 + a.per_worker < a.F ? f0 + a.per_worker : a.F;
  // the slice of fiber f0: the largest s with pos1[s] <= f0 (pos1[0] = 0 and pos1[S] = F > f0 bracket it)
  int64_t lo = 0, hi = a.S;
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(a.pos1 + mid) <= f0) lo = mid; else hi = mid;
  }
  int64_t s = lo;
  int64_t s_end = __ldg(a.pos1 + s + 1);
  for (int64_t f = f0; f < f1; ++f) {
    while (f >= s_end && s + 1 < a.S) { ++s; s_end = __ldg(a.pos1 + s + 1); }
    const int64_t i = __ldg(a.crd0 + s), j = __ldg(a.crd1 + f);
    const int64_t p0 = __ldg(a.pos2 + f), p1 = __ldg(a.pos2 + f + 1);
    for (int c = g; c < a.R; c += G) {
      if (LEVEL == 1) {
        double t = 0.0;
        for (int64_t p = p0; p < p1; ++p)
          t += (double)ld_stream(val + p) * (double)__ldg(B + (int64_t)__ldg(a.crd2 + p) * a.ldb + c);
        atomicAdd(a.acc + j * a.ldacc + c, t * (double)__ldg(A + i * a.lda + c));
      } else {
        const double w = (double)__ldg(A + i * a.lda + c) * (double)__ldg(B + j * a.ldb + c);
        for (int64_t p = p0; p < p1; ++p)
          atomicAdd(a.acc + (int64_t)__ldg(a.crd2 + p) * a.ldacc + c, (double)ld_stream(val + p) * w);
      }
    }
  }
}

template <class T, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_coo_scatter_kernel(const ScatterArgs a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t p0 = worker * a.per_worker;
  const int64_t p1 = p0 + a.per_worker < a.N ? p0 + a.per_worker : a.N;
  for (int64_t p = p0; p < p1; ++p) {
    const int64_t ro = __ldg(a.crd0 + p), ia = __ldg(a.crd1 + p), ib = __ldg(a.crd2 + p);
    const double v = (double)ld_stream(val + p);
    for (int c = g; c < a.R; c += G)
      atomicAdd(a.acc + ro * a.ldacc + c, v * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c));
  }
}

__global__ void zero_acc_kernel(double *__restrict__ acc, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) acc[i] = 0.0;
}

// out[r, c] = (float)acc[r, c]: the one rounding of an fp32 result
__global__ void round_acc_kernel(const double *__restrict__ acc, int64_t rows, int32_t R, float *__restrict__ out,
                                 int64_t ldo) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t r = i / R;
  if (r < rows) out[r * ldo + (i - r * R)] = (float)acc[i];
}

template <class T, int G>
static void launch_scatter(int kind, const ScatterArgs &a, int64_t units, cudaStream_t stream) {
  const int64_t workers = ceil_div(units, a.per_worker);
  const unsigned blocks = (unsigned)ceil_div(workers * G, kScatterThreads);
  if (kind == 0) mttkrp_coo_scatter_kernel<T, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 1) mttkrp_csf_scatter_kernel<T, 1, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else mttkrp_csf_scatter_kernel<T, 2, G><<<blocks, kScatterThreads, 0, stream>>>(a);
}

template <class T>
static void launch_scatter_width(int kind, const ScatterArgs &a, int64_t units, cudaStream_t stream) {
  if (a.R > 16) launch_scatter<T, 32>(kind, a, units, stream);
  else if (a.R > 8) launch_scatter<T, 16>(kind, a, units, stream);
  else if (a.R > 4) launch_scatter<T, 8>(kind, a, units, stream);
  else if (a.R > 2) launch_scatter<T, 4>(kind, a, units, stream);
  else if (a.R > 1) launch_scatter<T, 2>(kind, a, units, stream);
  else launch_scatter<T, 1>(kind, a, units, stream);
}

// kind 0: COO (crd0 = output-mode coordinates, crd1 / crd2 = coordinates of A's / B's modes);
// kind 1 / 2: CSF with the output mode at level 1 / 2.
comet_status_t mttkrp_scatter(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *crd0,
                              const int32_t *crd1, const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S,
                              int64_t F, int64_t N, int64_t rows, const void *A, int64_t lda, const void *B, int64_t ldb,
                              int64_t R, void *out, int64_t ldo, cudaStream_t stream) {
  if (R > 2147483647ll) return COMET_ERR_INDEX_OVERFLOW;
  ScatterArgs a{};
  a.pos1 = pos1; a.crd0 = crd0; a.crd1 = crd1; a.pos2 = pos2; a.crd2 = crd2; a.val = val;
  a.S = S; a.F = F; a.N = N; a.A = A; a.lda = lda; a.B = B; a.ldb = ldb; a.R = (int32_t)R;
  if (dtype == COMET_F32) {
    if (rows == 0) return COMET_OK;
    const int64_t n = rows * R;
    a.acc = (double *)scratch_get(ctx, (size_t)n * sizeof(double), stream);
    if (!a.acc) return COMET_ERR_ALLOC;
    a.ldacc = R;
    zero_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, n);
    COMET_LAUNCH_CHECK(ctx);
  } else {
    comet_status_t st = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
    if (st != COMET_OK) return st;
    a.acc = (double *)out;
    a.ldacc = ldo;
  }
  if (N > 0) {
    a.per_worker = kind == 0 ? 16 : 8;
    const int64_t units = kind == 0 ? N : F;
    if (dtype == COMET_F32) launch_scatter_width<float>(kind, a, units, stream);
    else launch_scatter_width<double>(kind, a, units, stream);
    COMET_LAUNCH_CHECK(ctx);
  }
  if (dtype == COMET_F32) {
    const int64_t n = rows * R;
    round_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, rows, (int32_t)R, (float *)out, ldo);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}


// ------------------------------------------------------------------------------------------- 4-order tensors
// The same accumulation for tensors of four modes, every output mode (the mode stored first included: there
// is no tiled kernel for 4-order tensors). CSF [CU,CU,CU,CU], coordinates (c0, c1, c2, c3) at levels 0..3; a
// worker owns a few consecutive level-2 fibers and tracks the level-1 fiber and the slice that hold them.
//   output at level 3:   out[c3, :] += val * (A[c0, :] * B[c1, :] * C[c2, :])                 one add per entry
//   output at level < 3: out[c_L, :] += (sum over the fiber of val * C[c3, :]) * A[.] * B[.]   one add per fiber
// (A, B, C = the factors of the three other levels in storage order.) COO [CN,S,S,S]: one add per entry.
struct Scatter4Args {
  const int32_t *pos1, *pos2, *pos3, *crd[4];   // COO: crd[0] = output coordinates, crd[1..3] = those of A, B, C
  const void *val;
  int64_t S, F1, F2, N;
  const void *A, *B, *C;
  int64_t lda, ldb, ldc;
  double *acc;
  int64_t ldacc;
  int32_t R;
  int32_t per_worker;
};

__device__ __forceinline__ int64_t last_at_or_below(const int32_t *pos, int64_t n, int64_t x) {
  int64_t lo = 0, hi = n;                       // pos[0] = 0 <= x < pos[n]: the largest index with pos[index] <= x
  while (hi - lo > 1) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(pos + mid) <= x) lo = mid; else hi = mid;
  }
  return lo;
}

template <class T, int LEVEL, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_csf4_scatter_kernel(const Scatter4Args a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B), *const Cf = static_cast<const T *>(a.C);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t f0 = worker * a.per_worker;
  if (f0 >= a.F2) return;
  const int64_t f1 = f0 + a.per_worker < a.F2 ? f0 + a.per_worker : a.F2;
  int64_t u = last_at_or_below(a.pos2, a.F1, f0);          // level-1 fiber that holds level-2 fiber f0
  int64_t s = last_at_or_below(a.pos1, a.S, u);            // slice that holds it
  int64_t u_end = __ldg(a.pos2 + u + 1), s_end = __ldg(a.pos1 + s + 1);
  for (int64_t f = f0; f < f1; ++f) {
    while (f >= u_end && u + 1 < a.F1) { ++u; u_end = __ldg(a.pos2 + u + 1); }
    while (u >= s_end && s + 1 < a.S) { ++s; s_end = __ldg(a.pos1 + s + 1); }
    const int64_t c0 = __ldg(a.crd[0] + s), c1 = __ldg(a.crd[1] + u), c2 = __ldg(a.crd[2] + f);
    const int64_t p0 = __ldg(a.pos3 + f), p1 = __ldg(a.pos3 + f + 1);
    // the upper coordinates that index A and B (and C when the output is the leaf), and the output's
    const int64_t ia = LEVEL == 0 ? c1 : c0;
    const int64_t ib = LEVEL <= 1 ? c2 : c1;
    const int64_t io = LEVEL == 0 ? c0 : (LEVEL == 1 ? c1 : c2);
    for (int c = g; c < a.R; c += G) {
      if (LEVEL == 3) {
        const double w = (double)__ldg(A + c0 * a.lda + c) * (double)__ldg(B + c1 * a.ldb + c) *
                         (double)__ldg(Cf + c2 * a.ldc + c);
        for (int64_t p = p0; p < p1; ++p)
          atomicAdd(a.acc + (int64_t)__ldg(a.crd[3] + p) * a.ldacc + c, (double)ld_stream(val + p) * w);
      } else {
        double t = 0.0;
        for (int64_t p = p0; p < p1; ++p)
          t += (double)ld_stream(val + p) * (double)__ldg(Cf + (int64_t)__ldg(a.crd[3] + p) * a.ldc + c);
        atomicAdd(a.acc + io * a.ldacc + c, t * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c));
      }
    }
  }
}

template <class T, int G>
__global__ void __launch_bounds__(kScatterThreads) mttkrp_coo4_scatter_kernel(const Scatter4Args a) {
  const T *const val = static_cast<const T *>(a.val);
  const T *const A = static_cast<const T *>(a.A), *const B = static_cast<const T *>(a.B), *const Cf = static_cast<const T *>(a.C);
  const int g = threadIdx.x % G;
  const int64_t worker = ((int64_t)blockIdx.x * kScatterThreads + threadIdx.x) / G;
  const int64_t p0 = worker * a.per_worker;
  const int64_t p1 = p0 + a.per_worker < a.N ? p0 + a.per_worker : a.N;
  for (int64_t p = p0; p < p1; ++p) {
    const int64_t ro = __ldg(a.crd[0] + p), ia = __ldg(a.crd[1] + p), ib = __ldg(a.crd[2] + p), ic = __ldg(a.crd[3] + p);
    const double v = (double)ld_stream(val + p);
    for (int c = g; c < a.R; c += G)
      atomicAdd(a.acc + ro * a.ldacc + c, v * (double)__ldg(A + ia * a.lda + c) * (double)__ldg(B + ib * a.ldb + c) *
                                              (double)__ldg(Cf + ic * a.ldc + c));
  }
}

template <class T, int G>
static void launch_scatter4(int kind, const Scatter4Args &a, int64_t units, cudaStream_t stream) {
  const int64_t workers = ceil_div(units, a.per_worker);
  const unsigned blocks = (unsigned)ceil_div(workers * G, kScatterThreads);
  if (kind < 0) mttkrp_coo4_scatter_kernel<T, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 0) mttkrp_csf4_scatter_kernel<T, 0, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 1) mttkrp_csf4_scatter_kernel<T, 1, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else if (kind == 2) mttkrp_csf4_scatter_kernel<T, 2, G><<<blocks, kScatterThreads, 0, stream>>>(a);
  else mttkrp_csf4_scatter_kernel<T, 3, G><<<blocks, kScatterThreads, 0, stream>>>(a);
}

template <class T>
static void launch_scatter4_width(int kind, const Scatter4Args &a, int64_t units, cudaStream_t stream) {
  if (a.R > 16) launch_scatter4<T, 32>(kind, a, units, stream);
  else if (a.R > 8) launch_scatter4<T, 16>(kind, a, units, stream);
  else if (a.R > 4) launch_scatter4<T, 8>(kind, a, units, stream);
  else if (a.R > 2) launch_scatter4<T, 4>(kind, a, units, stream);
  else if (a.R > 1) launch_scatter4<T, 2>(kind, a, units, stream);
  else launch_scatter4<T, 1>(kind, a, units, stream);
}

// kind -1: COO (crd[0] = output-mode coordinates, crd[1..3] = coordinates of A's, B's, C's modes);
// kind 0..3: CSF with the output mode at that level (crd = the four levels' coordinate arrays).
comet_status_t mttkrp_scatter4(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *pos2,
                               const int32_t *pos3, const int32_t *const *crd, const void *val, int64_t S, int64_t F1,
                               int64_t F2, int64_t N, int64_t rows, const void *A, int64_t lda, const void *B,
                               int64_t ldb, const void *C, int64_t ldc, int64_t R, void *out, int64_t ldo,
                               cudaStream_t stream) {
  if (R > 2147483647ll) return COMET_ERR_INDEX_OVERFLOW;
  Scatter4Args a{};
  a.pos1 = pos1; a.pos2 = pos2; a.pos3 = pos3; a.val = val;
  for (int l = 0; l < 4; ++l) a.crd[l] = crd[l];
  a.S = S; a.F1 = F1; a.F2 = F2; a.N = N;
  a.A = A; a.lda = lda; a.B = B; a.ldb = ldb; a.C = C; a.ldc = ldc; a.R = (int32_t)R;
  if (dtype == COMET_F32) {
    if (rows == 0) return COMET_OK;
    const int64_t n = rows * R;
    a.acc = (double *)scratch_get(ctx, (size_t)n * sizeof(double), stream);
    if (!a.acc) return COMET_ERR_ALLOC;
    a.ldacc = R;
    zero_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, n);
    COMET_LAUNCH_CHECK(ctx);
  } else {
    comet_status_t st = zero_rows(ctx, out, dtype, rows, R, ldo, stream);
    if (st != COMET_OK) return st;
    a.acc = (double *)out;
    a.ldacc = ldo;
  }
  if (N > 0) {
    a.per_worker = kind < 0 ? 16 : 8;
    const int64_t units = kind < 0 ? N : F2;
    if (dtype == COMET_F32) launch_scatter4_width<float>(kind, a, units, stream);
    else launch_scatter4_width<double>(kind, a, units, stream);
    COMET_LAUNCH_CHECK(ctx);
  }
  if (dtype == COMET_F32) {
    const int64_t n = rows * R;
    round_acc_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(a.acc, rows, (int32_t)R, (float *)out, ldo);
    COMET_LAUNCH_CHECK(ctx);
  }
  return COMET_OK;
}

}  // namespace comet
