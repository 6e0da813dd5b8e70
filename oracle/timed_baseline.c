/* Timed CPU baseline of the benchmark: the SpMM definition of the paper's Sparse Tensor Operations subsection,
 * C[i, r] += x * B[j, r] over the raw COO entries, exactly the loop of the parity oracle (comet_oracle.c) but
 * with `double` accumulators and compiled -O3 -march=native, on one thread or on several (each thread owns a
 * contiguous range of output rows and walks all entries, keeping those of its rows: no sort, no atomics).
 *
 * TEST INFRASTRUCTURE ONLY, like the rest of oracle/: a reported baseline, never a fallback of the library. */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int64_t nnz, R, row_lo, row_hi;
  const int32_t *ci, *cj;
  const double *val, *B;
  double *C;
} job_t;

static void *run(void *arg) {
  const job_t *j = (const job_t *)arg;
  const int64_t R = j->R;
  for (int64_t e = 0; e < j->nnz; ++e) {
    const int64_t i = j->ci[e];
    if (i < j->row_lo || i >= j->row_hi) continue;
    const double x = j->val[e];
    const double *b = j->B + (int64_t)j->cj[e] * R;
    double *c = j->C + i * R;
    for (int64_t r = 0; r < R; ++r) c[r] += x * b[r];
  }
  return NULL;
}

/* C (rows x R, row-major) = A * B for A given as nnz COO entries; threads >= 1. Returns 0, or -1 on a failed thread start. */
int timed_spmm(int64_t rows, int64_t nnz, const int32_t *ci, const int32_t *cj, const double *val, const double *B, int64_t R,
               double *C, int threads) {
  memset(C, 0, (size_t)rows * (size_t)R * sizeof(double));
  if (threads < 1) threads = 1;
  if (threads > 256) threads = 256;
  job_t jobs[256];
  pthread_t tid[256];
  for (int t = 0; t < threads; ++t) {
    jobs[t] = (job_t){nnz, R, rows * t / threads, rows * (t + 1) / threads, ci, cj, val, B, C};
  }
  if (threads == 1) { run(&jobs[0]); return 0; }
  int started = 0, rc = 0;
  for (; started < threads; ++started)
    if (pthread_create(&tid[started], NULL, run, &jobs[started]) != 0) { rc = -1; break; }
  for (int t = 0; t < started; ++t) pthread_join(tid[t], NULL);
  return rc;
}
