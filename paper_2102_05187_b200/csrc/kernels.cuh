// Internal launchers shared between the translation units of libcomet. Not part of the C ABI.
#pragma once

#include "common.cuh"

namespace comet {

// out[row(s), 0..R) = sum over leaf entries p of segment s of val[p] * B[crd[p], 0..R)   (SpMM, TTM)
// seg_end[s] = leaf position where segment s ends; seg_end - 1 must be readable and hold 0 (seg_end = pos + 1).
// out_row == NULL: row(s) = s; otherwise row(s) = out_row[s] (ascending) and all other rows below out_rows are
// zero-filled. b_rows = number of rows of B (0: unknown; only used to decide on the long-row path of SpMM).
comet_status_t seg_gather(Context *ctx, int dtype, const int32_t *seg_end, const int32_t *crd, const void *val,
                          int64_t M, int64_t N, const void *B, int64_t ldb, int64_t R, void *C, int64_t ldc,
                          const int32_t *out_row, int64_t out_rows, int64_t b_rows, cudaStream_t stream);


// y[row(s)] = sum over leaf entries p of segment s of val[p] * x[crd[p]]                    (SpMV, TTV)
comet_status_t seg_dot(Context *ctx, int dtype, const int32_t *seg_end, const int32_t *crd, const void *val, int64_t M,
                       int64_t N, const void *x, int64_t x_len, void *y, const int32_t *out_row,
                       int64_t out_rows, cudaStream_t stream);

// Sorted COO [CN,S,S]: out[crd0[p], :] += val[p] * P[crd1[p], :] * Q[crd2[p], :]; every row < rows written.
comet_status_t mttkrp_coo(Context *ctx, int dtype, const int32_t *crd0, const int32_t *crd1, const int32_t *crd2,
                          const void *val, int64_t N, int64_t rows, const void *P, int64_t ldp, const void *Q,
                          int64_t ldq, int64_t R, void *out, int64_t ldo, cudaStream_t stream);

// CSF [CU,CU,CU]: per fiber t = sum val * Q[crd2]; out[crd0[slice], :] += t * P[crd1[fiber], :].
comet_status_t mttkrp_csf(Context *ctx, int dtype, const int32_t *pos1, const int32_t *crd0, const int32_t *crd1,
                          const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S, int64_t F,
                          int64_t N, int64_t rows, const void *P, int64_t ldp, const void *Q, int64_t ldq,
                          int64_t R, void *out, int64_t ldo, cudaStream_t stream);

// CSF with the output mode stored at level 1, on the tiled walker (mttkrp.cu): fp64, R a power of two up to 64 and
// aligned operands; COMET_ERR_UNSUPPORTED_FORMAT otherwise (take mttkrp_scatter then). P = the ROOT mode's factor.
comet_status_t mttkrp_csf_level1(Context *ctx, int dtype, const int32_t *pos1, const int32_t *crd0, const int32_t *crd1,
                                 const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S, int64_t F, int64_t N,
                                 int64_t rows, const void *P, int64_t ldp, const void *Q, int64_t ldq, int64_t R, void *out,
                                 int64_t ldo, cudaStream_t stream);

// MTTKRP with the output mode NOT stored first, by atomic accumulation (see mttkrp_scatter.cu). kind 0: COO,
// crd0 = output-mode coordinates and crd1 / crd2 those of A's / B's modes; kind 1 / 2: CSF, output mode at
// level 1 / 2, A = the root mode's factor, B = the factor of the remaining mode. rows / a_rows / b_rows: the
// extents of the output mode and of A's and B's modes.
comet_status_t mttkrp_scatter(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *crd0,
                              const int32_t *crd1, const int32_t *pos2, const int32_t *crd2, const void *val, int64_t S,
                              int64_t F, int64_t N, int64_t rows, int64_t a_rows, int64_t b_rows, const void *A,
                              int64_t lda, const void *B, int64_t ldb, int64_t R, void *out, int64_t ldo,
                              cudaStream_t stream);

// The same for 4-order tensors, every output mode. kind -1: COO (crd[0] = output-mode coordinates, crd[1..3] =
// those of A's, B's, C's modes); kind 0..3: CSF, output mode at that level, A / B / C = the factors of the three
// other levels in storage order.
comet_status_t mttkrp_scatter4(Context *ctx, int dtype, int kind, const int32_t *pos1, const int32_t *pos2,
                               const int32_t *pos3, const int32_t *const *crd, const void *val, int64_t S, int64_t F1,
                               int64_t F2, int64_t N, int64_t rows, const void *A, int64_t lda, const void *B,
                               int64_t ldb, const void *C, int64_t ldc, int64_t R, void *out, int64_t ldo,
                               cudaStream_t stream);

comet_status_t zero_rows(Context *ctx, void *C, int dtype, int64_t rows, int64_t R, int64_t ldc, cudaStream_t stream);
// Exclusive scan of uint32 words in three launches (tile sums, scan of the sums, apply); defined in pack.cu.
// `out` may alias `in`; `tmp` holds scan_tmp_words(n) words; `total` (device, optional) receives the sum.
int64_t scan_tmp_words(int64_t n);
comet_status_t exclusive_scan(Context *ctx, const uint32_t *in, uint32_t *out, int64_t n, uint32_t *tmp,
                              uint32_t *total, cudaStream_t s);

// Stable LSD radix sort of (64-bit key, 32-bit payload) pairs over the low `bits` key bits (pack.cu). The sorted
// pairs end up behind `ka` / `pa` (the pointers are swapped with `kb` / `pb` after every pass); every buffer holds
// n + 1 elements, `table` radix_sort_table_words(n) words and `scan_tmp` scan_tmp_words(that) words.
int64_t radix_sort_table_words(int64_t n);
comet_status_t radix_sort_pairs(Context *ctx, uint64_t *&ka, uint64_t *&kb, uint32_t *&pa, uint32_t *&pb, int64_t n,
                                int bits, uint32_t *table, uint32_t *scan_tmp, cudaStream_t s);

// COO -> CSR without the full sort (pack_csr.cu): fills pos_out (rows + 1), crd_out (n), val_out (n); synchronises
// the stream once. *fallback = 1 with COMET_OK when a row is too long for it: run the generic path instead.
comet_status_t pack_csr_fast(Context *ctx, int dtype, const int32_t *row, const int32_t *col, const void *val, int64_t n,
                             int64_t rows, int64_t cols, int32_t *pos_out, int32_t *crd_out, void *val_out,
                             int *fallback, cudaStream_t s);

// ELLPACK [D,D,S] (ellpack.cu): conversion from a CSR tensor (arrays allocated into `owner`; synchronises), the
// descriptor test and the two products.
comet_status_t ell_from_csr(Context *ctx, const comet_sptensor_t *csr, void *owner, comet_sptensor_t *out, cudaStream_t s);
bool is_ellpack(const comet_sptensor_t *A);
comet_status_t ell_check(const comet_sptensor_t *A);
comet_status_t ell_spmv(Context *ctx, const comet_sptensor_t *A, const void *x, void *y, cudaStream_t s);
comet_status_t ell_spmm(Context *ctx, const comet_sptensor_t *A, const void *B, int64_t ldb, int64_t R, void *C, int64_t ldc,
                        cudaStream_t s);

// out[p] = val[p] * B[coordinates of leaf position p] (elementwise.cu); h_strides: element stride of every MODE in B.
comet_status_t elementwise_mul(Context *ctx, const comet_sptensor_t *A, const void *B, const int64_t *h_strides, void *out,
                               cudaStream_t s);

int32_t choose_tile_items(int64_t total_items, int workers_per_block);

// Block list of a library-owned tensor (what comet_sptensor_free releases).
void *owner_new();
void *owner_alloc(Context *ctx, void *owner, size_t bytes, cudaStream_t stream);
void owner_release(Context *ctx, void *owner, cudaStream_t stream);

// Carry fix-up shared by all contraction kernels (defined in contract_vec.cu): adds the per-tile open sums
// carry_val[tile, 0..R) onto row carry_seg[tile] of C (mapped through out_row when given). One launch of
// num_tiles * R threads on `stream`; the caller checks the launch.
void carry_fixup_launch(int dtype, const double *carry_val, const int32_t *carry_seg, int64_t num_tiles, int32_t R,
                        int32_t carry_ld, void *C, int64_t ldc, const int32_t *out_row, cudaStream_t stream);

}  // namespace comet
