/*
 * CPU oracle for the sparse x dense contractions and the format packing.
 *
 * TEST INFRASTRUCTURE ONLY: plain, slow, single-threaded, obviously-correct C. Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it; the CUDA library shares no code
 * with it and never calls it.
 *
 * Contractions iterate the RAW (unsorted) COO entries exactly as the index-notation definitions of
 * the paper's "Sparse Tensor Operations" subsection read, accumulate each output element in
 * long double (64-bit mantissa on x86-64) and round once to double. Beside each output element the
 * normaliser S = sum |x| * |b| (* |c|) is accumulated in double; a result r passes a comparison when
 * |r - oracle| <= tol * S.
 *
 * Packing follows the attribute definitions of the paper's "Tensor Storage Format" section (D, CU,
 * CN, S) with Table 1's loop forms deciding what `pos` is indexed by (the parent position).
 *
 * All functions return 0 on success and a negative code on a malformed request.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_ORDER 4

enum { ATTR_D = 0, ATTR_CU = 1, ATTR_CN = 2, ATTR_S = 3 };

enum {
  ORACLE_OK = 0,
  ORACLE_ERR_ARG = -1,
  ORACLE_ERR_FORMAT = -2,
  ORACLE_ERR_RANGE = -3,
  ORACLE_ERR_DUPLICATE = -4,
  ORACLE_ERR_ALLOC = -6
};

static double abs_d(double v) { return v < 0 ? -v : v; }

/* ------------------------------------------------------------------------------------------ SpMV
 * y_i = sum_j x_ij v_j  (SpMV definition). row_slot (may be NULL) maps a row to its output slot or
 * to -1 when the row is not wanted (sampled evaluation); n_out is the number of output slots. */
int oracle_spmv(int64_t nnz, const int32_t *ci, const int32_t *cj, const double *val, int64_t I, int64_t J,
                const double *v, const int64_t *row_slot, int64_t n_out, double *y, double *ynorm) {
  if (nnz < 0 || I < 0 || J < 0 || n_out < 0) return ORACLE_ERR_ARG;
  long double *acc = (long double *)calloc((size_t)(n_out > 0 ? n_out : 1), sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (int64_t o = 0; o < n_out; ++o) ynorm[o] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    int64_t i = ci[e], j = cj[e];
    if (i < 0 || i >= I || j < 0 || j >= J) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t o = row_slot ? row_slot[i] : i;
    if (o < 0) continue;
    acc[o] += (long double)val[e] * (long double)v[j];
    ynorm[o] += abs_d(val[e]) * abs_d(v[j]);
  }
  for (int64_t o = 0; o < n_out; ++o) y[o] = (double)acc[o];
  free(acc);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ SpMM
 * y_ir = sum_j x_ij u_jr  (SpMM definition); U is J x R row-major with leading dimension ldu, the
 * output is n_out x R row-major, dense (the index-variable rule vIdx = vIdx * SIZE + coord). */
int oracle_spmm(int64_t nnz, const int32_t *ci, const int32_t *cj, const double *val, int64_t I, int64_t J,
                const double *U, int64_t R, int64_t ldu, const int64_t *row_slot, int64_t n_out, double *Y,
                double *Ynorm) {
  if (nnz < 0 || R < 0 || ldu < R || n_out < 0) return ORACLE_ERR_ARG;
  size_t cells = (size_t)n_out * (size_t)R;
  long double *acc = (long double *)calloc(cells ? cells : 1, sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (size_t c = 0; c < cells; ++c) Ynorm[c] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    int64_t i = ci[e], j = cj[e];
    if (i < 0 || i >= I || j < 0 || j >= J) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t o = row_slot ? row_slot[i] : i;
    if (o < 0) continue;
    for (int64_t r = 0; r < R; ++r) {
      double u = U[j * ldu + r];
      acc[o * R + r] += (long double)val[e] * (long double)u;
      Ynorm[o * R + r] += abs_d(val[e]) * abs_d(u);
    }
  }
  for (size_t c = 0; c < cells; ++c) Y[c] = (double)acc[c];
  free(acc);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------- fiber bookkeeping
 * TTV and TTM in mode n produce one output fiber per distinct pair of the two kept coordinates
 * (a, b) = the kept modes in increasing mode order. The oracle keeps the output as a map keyed by
 * a * dim_b + b: the sorted list of distinct keys, looked up by binary search. */
static int cmp_i64(const void *p, const void *q) {
  int64_t a = *(const int64_t *)p, b = *(const int64_t *)q;
  return (a > b) - (a < b);
}

static int64_t find_key(const int64_t *keys, int64_t n, int64_t k) {
  int64_t lo = 0, hi = n;
  while (lo < hi) {
    int64_t mid = lo + (hi - lo) / 2;
    if (keys[mid] < k) lo = mid + 1; else hi = mid;
  }
  return (lo < n && keys[lo] == k) ? lo : -1;
}

static void kept_modes(int mode, int *a, int *b) {
  *a = (mode == 0) ? 1 : 0;
  *b = (mode == 2) ? 1 : 2;
}

/* Distinct output-fiber keys of X x_n (.), ascending. keys must hold nnz entries; returns the count. */
int64_t oracle_fiber_keys(int64_t nnz, const int32_t *c0, const int32_t *c1, const int32_t *c2,
                          const int64_t *dims, int mode, int64_t *keys) {
  const int32_t *c[3] = {c0, c1, c2};
  int a, b;
  if (mode < 0 || mode > 2) return ORACLE_ERR_ARG;
  kept_modes(mode, &a, &b);
  for (int64_t e = 0; e < nnz; ++e) keys[e] = (int64_t)c[a][e] * dims[b] + (int64_t)c[b][e];
  qsort(keys, (size_t)nnz, sizeof(int64_t), cmp_i64);
  int64_t n = 0;
  for (int64_t e = 0; e < nnz; ++e)
    if (e == 0 || keys[e] != keys[e - 1]) keys[n++] = keys[e];
  return n;
}

/* ------------------------------------------------------------------------------------------ TTV
 * Y = X x_n v: y_ab = sum_{i_n} x_{i1 i2 i3} v_{i_n}; the output has one order less (SpTTV
 * definition; the paper prints n = 1, `mode` selects n, 0-based). Output fiber f corresponds to
 * keys[f]; entries whose key is not in `keys` are skipped (sampled evaluation). */
int oracle_ttv(int64_t nnz, const int32_t *c0, const int32_t *c1, const int32_t *c2, const double *val,
               const int64_t *dims, int mode, const double *v, const int64_t *keys, int64_t nkeys, double *y,
               double *ynorm) {
  const int32_t *c[3] = {c0, c1, c2};
  int a, b;
  if (mode < 0 || mode > 2 || nnz < 0 || nkeys < 0) return ORACLE_ERR_ARG;
  kept_modes(mode, &a, &b);
  long double *acc = (long double *)calloc((size_t)(nkeys ? nkeys : 1), sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (int64_t f = 0; f < nkeys; ++f) ynorm[f] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    for (int m = 0; m < 3; ++m)
      if (c[m][e] < 0 || c[m][e] >= dims[m]) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t f = find_key(keys, nkeys, (int64_t)c[a][e] * dims[b] + (int64_t)c[b][e]);
    if (f < 0) continue;
    double w = v[c[mode][e]];
    acc[f] += (long double)val[e] * (long double)w;
    ynorm[f] += abs_d(val[e]) * abs_d(w);
  }
  for (int64_t f = 0; f < nkeys; ++f) y[f] = (double)acc[f];
  free(acc);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ TTM
 * Y = X x_n U with U in R^{I_n x R} (rows indexed by the contracted mode): mode n is replaced by r
 * in place, y_{a b r} = sum_{i_n} x_{i1 i2 i3} u_{i_n r} (SpTTM definition). Output: nkeys dense
 * fibers of length R, row-major. */
int oracle_ttm(int64_t nnz, const int32_t *c0, const int32_t *c1, const int32_t *c2, const double *val,
               const int64_t *dims, int mode, const double *U, int64_t R, int64_t ldu, const int64_t *keys,
               int64_t nkeys, double *Y, double *Ynorm) {
  const int32_t *c[3] = {c0, c1, c2};
  int a, b;
  if (mode < 0 || mode > 2 || nnz < 0 || nkeys < 0 || R < 0 || ldu < R) return ORACLE_ERR_ARG;
  kept_modes(mode, &a, &b);
  size_t cells = (size_t)nkeys * (size_t)R;
  long double *acc = (long double *)calloc(cells ? cells : 1, sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (size_t q = 0; q < cells; ++q) Ynorm[q] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    for (int m = 0; m < 3; ++m)
      if (c[m][e] < 0 || c[m][e] >= dims[m]) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t f = find_key(keys, nkeys, (int64_t)c[a][e] * dims[b] + (int64_t)c[b][e]);
    if (f < 0) continue;
    int64_t k = c[mode][e];
    for (int64_t r = 0; r < R; ++r) {
      double u = U[k * ldu + r];
      acc[f * R + r] += (long double)val[e] * (long double)u;
      Ynorm[f * R + r] += abs_d(val[e]) * abs_d(u);
    }
  }
  for (size_t q = 0; q < cells; ++q) Y[q] = (double)acc[q];
  free(acc);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------- TTV / TTM, any order
 * The same two definitions for a tensor of `order` modes (2 <= order <= 4): the mode-n product
 * contracts mode n and keeps the others. An output fiber is identified by the kept coordinates,
 * linearised in increasing mode order (the last kept mode varies fastest): key = sum c_m * stride_m.
 * `coords` holds one pointer per mode. Plain loops over the raw COO entries, long-double sums. */
static int64_t kept_key(int order, const int32_t *const *c, const int64_t *dims, int mode, int64_t e) {
  int64_t key = 0;
  for (int m = 0; m < order; ++m)
    if (m != mode) key = key * dims[m] + (int64_t)c[m][e];
  return key;
}

int64_t oracle_fiber_keys_n(int order, int64_t nnz, const int32_t *const *coords, const int64_t *dims, int mode,
                            int64_t *keys) {
  if (order < 2 || order > 4 || mode < 0 || mode >= order) return ORACLE_ERR_ARG;
  for (int64_t e = 0; e < nnz; ++e) keys[e] = kept_key(order, coords, dims, mode, e);
  qsort(keys, (size_t)nnz, sizeof(int64_t), cmp_i64);
  int64_t n = 0;
  for (int64_t e = 0; e < nnz; ++e)
    if (e == 0 || keys[e] != keys[e - 1]) keys[n++] = keys[e];
  return n;
}

/* U is I_mode x R (ldu >= R); R = 1 with ldu = 1 is the tensor-times-vector product. */
int oracle_ttm_n(int order, int64_t nnz, const int32_t *const *coords, const double *val, const int64_t *dims,
                 int mode, const double *U, int64_t R, int64_t ldu, const int64_t *keys, int64_t nkeys, double *Y,
                 double *Ynorm) {
  if (order < 2 || order > 4 || mode < 0 || mode >= order || nnz < 0 || nkeys < 0 || R < 0 || ldu < R)
    return ORACLE_ERR_ARG;
  size_t cells = (size_t)nkeys * (size_t)R;
  long double *acc = (long double *)calloc(cells ? cells : 1, sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (size_t q = 0; q < cells; ++q) Ynorm[q] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    for (int m = 0; m < order; ++m)
      if (coords[m][e] < 0 || coords[m][e] >= dims[m]) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t f = find_key(keys, nkeys, kept_key(order, coords, dims, mode, e));
    if (f < 0) continue;
    int64_t k = coords[mode][e];
    for (int64_t r = 0; r < R; ++r) {
      double u = U[k * ldu + r];
      acc[f * R + r] += (long double)val[e] * (long double)u;
      Ynorm[f * R + r] += abs_d(val[e]) * abs_d(u);
    }
  }
  for (size_t q = 0; q < cells; ++q) Y[q] = (double)acc[q];
  free(acc);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------- MTTKRP
 * Mode-n matricised-tensor-times-Khatri-Rao product (the paper only names it; this is the textbook
 * definition): out_{i_n r} = sum over the other two modes of x * P_{p r} * Q_{q r}, where P and Q are
 * the factors of the two other modes in increasing mode order. The product is formed as (x * P) * Q. */
int oracle_mttkrp(int64_t nnz, const int32_t *c0, const int32_t *c1, const int32_t *c2, const double *val,
                  const int64_t *dims, int mode, const double *F0, const double *F1, const double *F2,
                  const int64_t *ld, int64_t R, const int64_t *row_slot, int64_t n_out, double *A,
                  double *Anorm) {
  const int32_t *c[3] = {c0, c1, c2};
  const double *F[3] = {F0, F1, F2};
  int a, b;
  if (mode < 0 || mode > 2 || nnz < 0 || n_out < 0 || R < 0) return ORACLE_ERR_ARG;
  kept_modes(mode, &a, &b);
  size_t cells = (size_t)n_out * (size_t)R;
  long double *acc = (long double *)calloc(cells ? cells : 1, sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (size_t q = 0; q < cells; ++q) Anorm[q] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    for (int m = 0; m < 3; ++m)
      if (c[m][e] < 0 || c[m][e] >= dims[m]) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t i = c[mode][e];
    int64_t o = row_slot ? row_slot[i] : i;
    if (o < 0) continue;
    int64_t p = c[a][e], q = c[b][e];
    for (int64_t r = 0; r < R; ++r) {
      double fp = F[a][p * ld[a] + r], fq = F[b][q * ld[b] + r];
      acc[o * R + r] += ((long double)val[e] * (long double)fp) * (long double)fq;
      Anorm[o * R + r] += abs_d(val[e]) * abs_d(fp) * abs_d(fq);
    }
  }
  for (size_t q = 0; q < cells; ++q) A[q] = (double)acc[q];
  free(acc);
  return ORACLE_OK;
}

/* MTTKRP for tensors of order 3 or 4: out_{i_n r} = sum over the entries of x * prod_{m != n} F_m[i_m, r]
 * (the textbook definition for any order). The product is formed left to right in increasing mode
 * order, ((x * F_a) * F_b) * F_c, so that the 3-order case is the function above, operation for
 * operation. `factors` / `ld` hold one entry per mode (the one at `mode` is ignored). */
int oracle_mttkrp_n(int order, int64_t nnz, const int32_t *const *coords, const double *val, const int64_t *dims,
                    int mode, const double *const *factors, const int64_t *ld, int64_t R, const int64_t *row_slot,
                    int64_t n_out, double *A, double *Anorm) {
  if (order < 3 || order > 4 || mode < 0 || mode >= order || nnz < 0 || n_out < 0 || R < 0) return ORACLE_ERR_ARG;
  size_t cells = (size_t)n_out * (size_t)R;
  long double *acc = (long double *)calloc(cells ? cells : 1, sizeof(long double));
  if (!acc) return ORACLE_ERR_ALLOC;
  for (size_t q = 0; q < cells; ++q) Anorm[q] = 0.0;
  for (int64_t e = 0; e < nnz; ++e) {
    for (int m = 0; m < order; ++m)
      if (coords[m][e] < 0 || coords[m][e] >= dims[m]) { free(acc); return ORACLE_ERR_RANGE; }
    int64_t i = coords[mode][e];
    int64_t o = row_slot ? row_slot[i] : i;
    if (o < 0) continue;
    for (int64_t r = 0; r < R; ++r) {
      long double term = (long double)val[e];
      double mag = abs_d(val[e]);
      for (int m = 0; m < order; ++m) {
        if (m == mode) continue;
        double f = factors[m][(int64_t)coords[m][e] * ld[m] + r];
        term *= (long double)f;
        mag *= abs_d(f);
      }
      acc[o * R + r] += term;
      Anorm[o * R + r] += mag;
    }
  }
  for (size_t q = 0; q < cells; ++q) A[q] = (double)acc[q];
  free(acc);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ Pack
 * COO -> per-level pos/crd arrays from the level attributes.
 *
 * Step 1: stable merge sort of the entries by the coordinate tuple in storage-level order
 *         (level l holds tensor mode mode_order[l]).
 * Step 2: one left-to-right walk per level. P_{l-1} is the number of parent positions (P_{-1} = 1):
 *   D : pos = [dim], no crd; an entry's position is parent_position * dim + coordinate
 *       (allowed only while every ancestor is D).
 *   CU: a new node starts whenever the parent position or the coordinate changes; crd holds the
 *       nodes' coordinates, pos has P_{l-1} + 1 entries with pos[p+1] - pos[p] = children of p.
 *   CN: (root only) crd = every entry's coordinate, pos = [0, N]; position = entry rank.
 *   S : crd[p] = the coordinate of the entry at parent position p (parent must be CN or S).
 * Finally every entry must sit at its own leaf position (else two entries share all coordinates).
 */
typedef struct {
  int32_t c[ORACLE_MAX_ORDER];
  int64_t src;
} rec_t;

static int rec_less(const rec_t *x, const rec_t *y, int order) {
  for (int l = 0; l < order; ++l) {
    if (x->c[l] < y->c[l]) return 1;
    if (x->c[l] > y->c[l]) return 0;
  }
  return 0;
}

static void merge_sort(rec_t *a, rec_t *tmp, int64_t lo, int64_t hi, int order) {
  if (hi - lo < 2) return;
  int64_t mid = lo + (hi - lo) / 2;
  merge_sort(a, tmp, lo, mid, order);
  merge_sort(a, tmp, mid, hi, order);
  int64_t i = lo, j = mid, k = lo;
  while (i < mid && j < hi) {
    if (rec_less(&a[j], &a[i], order)) tmp[k++] = a[j++];   /* take right only if strictly smaller: stable */
    else tmp[k++] = a[i++];
  }
  while (i < mid) tmp[k++] = a[i++];
  while (j < hi) tmp[k++] = a[j++];
  memcpy(a + lo, tmp + lo, (size_t)(hi - lo) * sizeof(rec_t));
}

typedef struct {
  int32_t order;
  int64_t nnz;
  int32_t *pos[ORACLE_MAX_ORDER];
  int64_t pos_len[ORACLE_MAX_ORDER];
  int32_t *crd[ORACLE_MAX_ORDER];
  int64_t crd_len[ORACLE_MAX_ORDER];
  double *val;
  int64_t *perm; /* perm[p] = index of the input entry stored at leaf position p */
} oracle_packed_t;

void oracle_packed_free(oracle_packed_t *t) {
  if (!t) return;
  for (int l = 0; l < ORACLE_MAX_ORDER; ++l) {
    free(t->pos[l]);
    free(t->crd[l]);
    t->pos[l] = t->crd[l] = NULL;
  }
  free(t->val);
  free(t->perm);
  t->val = NULL;
  t->perm = NULL;
}

/* Entries that share all coordinates are merged into one whose value is their sum, added one by one in
 * double in the order the entries were given (a stable sort keeps that order inside a run of equal
 * coordinates). Writes the merged entries (in sorted storage order, which the packing does not need
 * but which makes the result unique) and returns how many there are; out_coo[m] / out_val hold nnz
 * slots. `first[k]` receives the input index of the first entry of merged entry k. */
int64_t oracle_sum_duplicates(int32_t order, int64_t nnz, const int32_t *const *coo, const double *val,
                              const int32_t *mode_order, int32_t *const *out_coo, double *out_val, int64_t *first) {
  if (order < 1 || order > ORACLE_MAX_ORDER || nnz < 0) return ORACLE_ERR_ARG;
  size_t n1 = (size_t)(nnz ? nnz : 1);
  rec_t *rec = (rec_t *)malloc(n1 * sizeof(rec_t));
  rec_t *tmp = (rec_t *)malloc(n1 * sizeof(rec_t));
  if (!rec || !tmp) { free(rec); free(tmp); return ORACLE_ERR_ALLOC; }
  for (int64_t e = 0; e < nnz; ++e) {
    for (int l = 0; l < order; ++l) rec[e].c[l] = coo[mode_order[l]][e];
    rec[e].src = e;
  }
  merge_sort(rec, tmp, 0, nnz, order);
  int64_t m = 0;
  for (int64_t e = 0; e < nnz; ++e) {
    if (e > 0 && !rec_less(&rec[e - 1], &rec[e], order)) {
      out_val[m - 1] = out_val[m - 1] + val[rec[e].src];      /* same coordinates: add to the open entry */
    } else {
      for (int l = 0; l < order; ++l) out_coo[mode_order[l]][m] = rec[e].c[l];
      out_val[m] = val[rec[e].src];
      first[m] = rec[e].src;
      m += 1;
    }
  }
  free(rec); free(tmp);
  return m;
}

int oracle_pack(int32_t order, const int64_t *dims, int64_t nnz, const int32_t *const *coo, const double *val,
                const int32_t *mode_order, const int32_t *attr, oracle_packed_t *out) {
  if (order < 1 || order > ORACLE_MAX_ORDER || nnz < 0 || !out) return ORACLE_ERR_ARG;
  memset(out, 0, sizeof(*out));
  int seen[ORACLE_MAX_ORDER] = {0, 0, 0, 0};
  for (int l = 0; l < order; ++l) {
    if (mode_order[l] < 0 || mode_order[l] >= order || seen[mode_order[l]]) return ORACLE_ERR_ARG;
    seen[mode_order[l]] = 1;
    if (attr[l] < ATTR_D || attr[l] > ATTR_S) return ORACLE_ERR_ARG;
    if (attr[l] == ATTR_D) for (int a = 0; a < l; ++a) if (attr[a] != ATTR_D) return ORACLE_ERR_FORMAT;
    if (attr[l] == ATTR_CN && l != 0) return ORACLE_ERR_FORMAT;
    if (attr[l] == ATTR_S && (l == 0 || (attr[l - 1] != ATTR_CN && attr[l - 1] != ATTR_S))) return ORACLE_ERR_FORMAT;
  }
  if (attr[order - 1] == ATTR_D) return ORACLE_ERR_FORMAT; /* a sparse tensor's leaf level stores entries */

  size_t n1 = (size_t)(nnz ? nnz : 1);
  rec_t *rec = (rec_t *)malloc(n1 * sizeof(rec_t));
  rec_t *tmp = (rec_t *)malloc(n1 * sizeof(rec_t));
  int64_t *ppos = (int64_t *)malloc(n1 * sizeof(int64_t)); /* parent position of each sorted entry */
  int64_t *cpos = (int64_t *)malloc(n1 * sizeof(int64_t)); /* its position at the current level */
  if (!rec || !tmp || !ppos || !cpos) { free(rec); free(tmp); free(ppos); free(cpos); return ORACLE_ERR_ALLOC; }
  int rc = ORACLE_OK;

  for (int64_t e = 0; e < nnz; ++e) {
    for (int l = 0; l < order; ++l) {
      int32_t c = coo[mode_order[l]][e];
      if (c < 0 || c >= dims[mode_order[l]]) { rc = ORACLE_ERR_RANGE; goto done; }
      rec[e].c[l] = c;
    }
    rec[e].src = e;
  }
  merge_sort(rec, tmp, 0, nnz, order);
  for (int64_t e = 1; e < nnz; ++e) /* two entries with the same full coordinate are rejected */
    if (!rec_less(&rec[e - 1], &rec[e], order)) { rc = ORACLE_ERR_DUPLICATE; goto done; }

  out->order = order;
  out->nnz = nnz;
  for (int64_t e = 0; e < nnz; ++e) ppos[e] = 0;
  int64_t P_prev = 1;
  for (int l = 0; l < order; ++l) {
    int64_t dim = dims[mode_order[l]];
    int64_t P = 0;
    if (attr[l] == ATTR_D) {
      out->pos[l] = (int32_t *)malloc(sizeof(int32_t));
      out->pos[l][0] = (int32_t)dim;
      out->pos_len[l] = 1;
      out->crd_len[l] = 0;
      for (int64_t e = 0; e < nnz; ++e) cpos[e] = ppos[e] * dim + rec[e].c[l];
      P = P_prev * dim;
    } else if (attr[l] == ATTR_CU) {
      int32_t *pos = (int32_t *)calloc((size_t)P_prev + 1, sizeof(int32_t));
      int32_t *crd = (int32_t *)malloc(n1 * sizeof(int32_t));
      int64_t nodes = 0;
      for (int64_t e = 0; e < nnz; ++e) {
        int fresh = (e == 0) || (ppos[e] != ppos[e - 1]) || (rec[e].c[l] != rec[e - 1].c[l]);
        if (fresh) {
          crd[nodes] = rec[e].c[l];
          pos[ppos[e] + 1] += 1;          /* one more child of this parent position */
          nodes += 1;
        }
        cpos[e] = nodes - 1;
      }
      for (int64_t p = 0; p < P_prev; ++p) pos[p + 1] += pos[p];
      out->pos[l] = pos;
      out->pos_len[l] = P_prev + 1;
      out->crd[l] = (int32_t *)realloc(crd, (size_t)(nodes ? nodes : 1) * sizeof(int32_t));
      out->crd_len[l] = nodes;
      P = nodes;
    } else if (attr[l] == ATTR_CN) {
      int32_t *pos = (int32_t *)malloc(2 * sizeof(int32_t));
      int32_t *crd = (int32_t *)malloc(n1 * sizeof(int32_t));
      pos[0] = 0;
      pos[1] = (int32_t)nnz;
      for (int64_t e = 0; e < nnz; ++e) { crd[e] = rec[e].c[l]; cpos[e] = e; }
      out->pos[l] = pos;
      out->pos_len[l] = 2;
      out->crd[l] = crd;
      out->crd_len[l] = nnz;
      P = nnz;
    } else { /* ATTR_S */
      int32_t *crd = (int32_t *)malloc((size_t)(P_prev ? P_prev : 1) * sizeof(int32_t));
      for (int64_t e = 0; e < nnz; ++e) {
        if (e > 0 && ppos[e] == ppos[e - 1]) { free(crd); rc = ORACLE_ERR_DUPLICATE; goto done; }
        crd[ppos[e]] = rec[e].c[l];
        cpos[e] = ppos[e];
      }
      out->pos_len[l] = 0;
      out->crd[l] = crd;
      out->crd_len[l] = P_prev;
      P = P_prev;
    }
    int64_t *swap = ppos; ppos = cpos; cpos = swap;
    P_prev = P;
  }
  /* every entry must own its leaf position */
  for (int64_t e = 0; e < nnz; ++e)
    if (ppos[e] != e) { rc = ORACLE_ERR_DUPLICATE; goto done; }
  if (P_prev != nnz) { rc = ORACLE_ERR_DUPLICATE; goto done; }

  out->val = (double *)malloc(n1 * sizeof(double));
  out->perm = (int64_t *)malloc(n1 * sizeof(int64_t));
  for (int64_t p = 0; p < nnz; ++p) {
    out->perm[p] = rec[p].src;
    out->val[p] = val[rec[p].src];
  }
done:
  free(rec); free(tmp); free(ppos); free(cpos);
  if (rc != ORACLE_OK) oracle_packed_free(out);
  return rc;
}
