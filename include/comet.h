/*
 * comet.h -- C ABI of libcomet: mixed sparse x dense tensor contractions on one B200 (sm_100a),
 * driven by per-dimension storage-level attributes.
 *
 * A sparse tensor is `order` storage levels. Level l stores tensor mode mode_order[l] with one of
 * four attributes and a (pos, crd) pair of int32 arrays, plus one value array (the paper's
 * "Tensor Storage Format" section and its sparse-tensor struct: per-dimension pos/crd of i32 and
 * values of f64):
 *
 *   D  (dense)                pos = [dim] (1 entry), no crd; position = parent_position*dim + coordinate
 *   CU (compressed, unique)   crd = the distinct coordinates under each parent position, ascending;
 *                             pos has parents+1 entries: children of parent p are crd[pos[p] .. pos[p+1])
 *                             (the loop form of Table 1: pos is indexed by the position that the level above
 *                             produced, 0 at the first level, and brackets that parent's range of crd)
 *   CN (compressed, nonunique) first level only: crd = every entry's coordinate, pos = [0, nnz]
 *   S  (singleton)            crd[p] = coordinate of the entry at parent position p, no pos
 *
 * COO = [CN,S(,S)], CSR = [D,CU], DCSR = [CU,CU], CSF = [CU,CU,CU]. Every packed format is in
 * lexicographic order of (mode_order[0], mode_order[1], ...) coordinates. Indices are 0-based.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the parameter name starts with h_ (host memory).
 *   - Inputs are borrowed and never modified. Dense outputs are caller-allocated and are
 *     OVERWRITTEN (C = A.B, not +=); rows / fibers without a stored entry become +0.0.
 *   - Dense operands are row-major with an explicit leading dimension in elements.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Contractions
 *     are asynchronous on that stream; comet_pack and the *_symbolic calls synchronise the stream
 *     once to learn data-dependent sizes. Exceptions, all on the host side of a contraction call:
 *     the handle's scratch grows on demand, and the call that grows it waits for the stream before the
 *     old buffer is released (so the first call, or the first larger one, may synchronise);
 *     comet_spmv / comet_spmm on a [CN,S] matrix allocate and release a row index on every call;
 *     a call on another stream than the handle's previous call first waits for that previous stream.
 *   - A handle caches scratch memory and device counters: one call at a time. Calls on one handle
 *     from several host threads, or overlapping on the GPU, are not supported (use a handle each).
 *   - Errors are return codes; nothing aborts, throws or traps. Errors detectable on the host are
 *     returned before anything is launched.
 *   - Limits: nnz, every extent and every pos value must be < 2^31 - 1 (int32 indices); leading
 *     dimensions of gathered dense operands must be < 2^28 elements (COMET_ERR_INDEX_OVERFLOW).
 *   - Values are fp64 (COMET_F64) or fp32 (COMET_F32); a tensor's dtype is also the type of every dense
 *     operand and output of a call on it (no mixing: the library cannot see a dense buffer's type, so the
 *     caller must get this right; a sparse OUTPUT of another dtype is COMET_ERR_INVALID_ARG). Products and
 *     sums are formed in double for both types and rounded once when stored; with fp32 a row that spans
 *     several tiles is rounded once more when its carry is added. Dense pointers must be aligned to one
 *     element (COMET_ERR_MISALIGNED).
 */
#ifndef COMET_H
#define COMET_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { COMET_D = 0, COMET_CU = 1, COMET_CN = 2, COMET_S = 3 } comet_attr_t;
typedef enum { COMET_F64 = 0, COMET_F32 = 1 } comet_dtype_t;

typedef enum {
  COMET_OK = 0,
  COMET_ERR_INVALID_ARG = -1,        /* NULL pointer, negative size, bad enum, bad mode_order */
  COMET_ERR_UNSUPPORTED_FORMAT = -2, /* attribute combination / dtype this entry point does not handle */
  COMET_ERR_COORD_OUT_OF_RANGE = -3, /* an input coordinate lies outside [0, dim) */
  COMET_ERR_DUPLICATE_COORD = -4,    /* two input entries share all coordinates */
  COMET_ERR_INDEX_OVERFLOW = -5,     /* nnz or an extent does not fit int32 */
  COMET_ERR_ALLOC = -6,              /* the allocator returned NULL */
  COMET_ERR_CUDA = -7,               /* a CUDA runtime call failed; see comet_last_cuda_error */
  COMET_ERR_WORKSPACE = -8,          /* a fixed-size workspace is too small for this problem */
  COMET_ERR_MISALIGNED = -9,         /* a pointer is not aligned to its element type */
  COMET_ERR_INVALID_TENSOR = -10     /* comet_validate: pos/crd arrays violate the level invariants */
} comet_status_t;

#define COMET_MAX_ORDER 4

/* Tuning variables read from the environment (for experiments and tests; the defaults are the measured best):
 *   COMET_TILE_ITEMS=n          items (leaf entries + segment ends) per tile of the matrix-operand kernels
 *   COMET_SEG_DOT_KERNEL=name   SpMV/TTV kernel: resident | stream | stream2 (default: chosen by size)
 *   COMET_STREAM_SPAN=n         entries per span of the SpMV/TTV stream kernels (multiple of 128)
 *   COMET_PACK_CSR=1|0          forces / forbids the histogram CSR packing of comet_pack_ex (COMET_PACK_CSR_HISTOGRAM)
 *   COMET_SEG_PARTITION=0       matrix-operand kernels search their tile boundaries themselves (no pre-pass)
 *   COMET_CSF_FORM=fold|expand  root-mode CSF MTTKRP: per-fiber or per-entry form (default: by mean fiber length)
 *   COMET_MTTKRP_HOT_ROWS=0|1   per-entry MTTKRP (CSF leaf mode, COO non-root modes): never / always keep the most popular output rows in shared memory
 *                               (default: for R >= 16 and at least 2^20 entries)
 *   COMET_HOST_CHUNK_BYTES=n    comet_spmm_from_host: bytes per row of a column chunk of B and C (default 256; 0 = one chunk)
 *   COMET_SPMM_LONG_ROWS=0      comet_spmm without the long-row path; COMET_SPMM_LONG_ROW, _LONG_TILE, _PIECE,
 *                               _BLOCK_MB, _BLOCKS, _LONG_CTAS, _LONG_MIN_NNZ, _LONG_MIN_B_MB: its threshold
 *                               (entries), tile and piece sizes, block size / count of B, CTAs of the long-row
 *                               role, and the matrix / operand sizes from which it switches itself on */

/* The sparse tensor descriptor (a plain struct the caller may also fill in by hand for arrays it
 * built itself; run comet_validate on such a tensor before contracting it). */
typedef struct {
  int32_t order;
  int32_t dtype;                        /* comet_dtype_t of val */
  int64_t dims[COMET_MAX_ORDER];        /* extent of tensor MODE m (not of level m) */
  int32_t mode_order[COMET_MAX_ORDER];  /* storage level l holds tensor mode mode_order[l] */
  int32_t attr[COMET_MAX_ORDER];        /* comet_attr_t per level */
  int32_t *pos[COMET_MAX_ORDER];        /* device; D: 1 entry; CU: parents+1; CN: 2; S: NULL */
  int64_t pos_len[COMET_MAX_ORDER];
  int32_t *crd[COMET_MAX_ORDER];        /* device; D: NULL; CU: #nodes; CN, S: #positions */
  int64_t crd_len[COMET_MAX_ORDER];
  void *val;                            /* device; nnz values in leaf order */
  int64_t nnz;
  void *owner;                          /* non-NULL: arrays were allocated by the library (see comet_sptensor_free) */
} comet_sptensor_t;

typedef struct comet_context *comet_handle_t;

/* Device-memory allocator used for library-owned outputs (packed tensors, symbolic outputs) and
 * scratch. alloc returns a device pointer aligned to at least 256 bytes, or NULL. Both callbacks
 * may be called from any comet_* call and must not call back into the library. */
typedef struct {
  void *(*alloc)(void *ctx, size_t bytes, void *stream);
  void (*free)(void *ctx, void *ptr, void *stream);
  void *ctx;
} comet_allocator_t;

/* Create / destroy a handle on the current CUDA device. `allocator` may be NULL: cudaMalloc/cudaFree
 * are then used. Returns COMET_ERR_INVALID_ARG for a NULL out-pointer, COMET_ERR_CUDA if no device. */
comet_status_t comet_create(comet_handle_t *handle, const comet_allocator_t *allocator);
comet_status_t comet_destroy(comet_handle_t handle);
const char *comet_status_string(comet_status_t status);
/* The cudaError_t (as int) of the last failing CUDA call seen by this handle, 0 if none. */
int comet_last_cuda_error(comet_handle_t handle);
/* Number of CUDA kernels this handle has launched since comet_create (accounting for benchmarks). */
int64_t comet_kernel_launches(comet_handle_t handle);

/* COO -> packed format (the format conversion the paper's input-reading runtime function performs
 * after reading a COO file; Tensor Storage Format section for what each level holds).
 *   h_dims[order]       extents per tensor mode
 *   h_coo_crd[order]    HOST array of DEVICE pointers, one int32[nnz] coordinate array per mode
 *   coo_val             DEVICE, nnz values, copied bitwise into leaf order
 *   h_mode_order[order] a permutation of 0..order-1; h_attr[order] one comet_attr_t per level
 * Supported attribute tuples: [CN,S,...,S], [CU,...,CU], [D,CU,...,CU] (orders 2..4), and [D,S] for a matrix, which
 * asks for ELLPACK (below), provided the
 * coordinate bit widths (ceil(log2(extent)) per mode) sum to <= 63. Input order is arbitrary; duplicates and out-of-range
 * coordinates are detected on the device and reported (COMET_ERR_DUPLICATE_COORD,
 * COMET_ERR_COORD_OUT_OF_RANGE); `out` is then left zeroed. On success `out` owns its arrays
 * (allocated through the handle's allocator) until comet_sptensor_free. Synchronises `stream` once.  *
 * ELLPACK (named in the Tensor Storage Format section among the formats the four attributes compose; the paper
 * does not spell the composition out, this is the reading used): order 2 with h_attr = {COMET_D, COMET_S} gives a
 * descriptor of THREE levels [D, D, S]: the rows (dense), K slots per row (dense; listed as a third "mode" of
 * extent K = the longest row: dims[2] = K, mode_order = {row mode, 2, column mode}), and one singleton column
 * coordinate per slot. pos[0] = [rows], pos[1] = [K], crd[2] and val hold rows * K entries (nnz = rows * K): a row's
 * entries first, columns ascending, then padding with column -1 and value 0. comet_spmv, comet_spmm and
 * comet_elementwise_mul accept it. Synchronises `stream` twice more than the CSR packing it goes through. */
comet_status_t comet_pack(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                          const int32_t *const *h_coo_crd, const void *coo_val, comet_dtype_t dtype,
                          const int32_t *h_mode_order, const int32_t *h_attr, void *stream,
                          comet_sptensor_t *out);

/* comet_pack with options. flags: a bitwise OR of
 *   COMET_PACK_SUM_DUPLICATES  entries that share all coordinates are merged into one entry whose value is
 *                              their sum, added one by one in double in the order the entries were given
 *                              (fp32 values: summed in double, rounded once), instead of being reported as
 *                              COMET_ERR_DUPLICATE_COORD. out->nnz is then the number of distinct cells. The
 *                              paper does not say what a duplicate means; this is the common reading of a COO
 *                              file and costs one more stream synchronisation and one more pass.
 *   COMET_PACK_CSR_HISTOGRAM   a hint for [D,CU] matrices: build the row structure as a histogram (count the rows,
 *                              scan, drop the entries into their rows, sort inside each row) instead of sorting
 *                              all entries. Same result, bit for bit. Faster when the rows are of similar length
 *                              (20 M uniform entries in 1,048,576^2: 1.36 ms against 1.85 ms), slower when a few
 *                              rows hold much of the matrix (the benchmark's Zipf rows: 2.3 ms against 1.8 ms),
 *                              because the per-row counters of heavy rows serialise. Ignored where it does not
 *                              apply (other formats, rows longer than 12,288 entries, far more rows than entries,
 *                              or together with COMET_PACK_SUM_DUPLICATES); synchronises once like comet_pack.
 * Any other bit: COMET_ERR_INVALID_ARG. flags = 0 is comet_pack. */
#define COMET_PACK_SUM_DUPLICATES 1u
#define COMET_PACK_CSR_HISTOGRAM 2u
comet_status_t comet_pack_ex(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                             const int32_t *const *h_coo_crd, const void *coo_val, comet_dtype_t dtype,
                             const int32_t *h_mode_order, const int32_t *h_attr, uint32_t flags, void *stream,
                             comet_sptensor_t *out);

/* Releases the arrays of a library-owned tensor (no-op for caller-built descriptors) and zeroes it. */
comet_status_t comet_sptensor_free(comet_handle_t handle, comet_sptensor_t *tensor, void *stream);

/* Checks a caller-built descriptor against the level invariants (the paper keeps the caller's layout
 * and only describes it with attributes): pos monotone from 0 to the level's crd length, CU
 * coordinates strictly ascending inside each parent, every coordinate inside its extent.
 * Synchronises `stream`; returns COMET_ERR_INVALID_TENSOR on a violation. */
comet_status_t comet_validate(comet_handle_t handle, const comet_sptensor_t *tensor, void *stream);

/* SpMV  y_i = sum_j A_ij x_j  (SpMV definition in the Sparse Tensor Operations subsection).
 * A: 2 levels, [D,CU] (CSR), [CU,CU] (DCSR) or [CN,S] (COO; its row structure is rebuilt into a
 * temporary obtained from the handle's allocator). x: dims[mode_order[1]] values;
 * y: dims[mode_order[0]] values, every entry written. */
comet_status_t comet_spmv(comet_handle_t handle, const comet_sptensor_t *A, const void *x, void *y, void *stream);

/* SpMM  C_ir = sum_j A_ij B_jr  (SpMM definition). B: dims[mode_order[1]] x R, leading dimension
 * ldb >= R; C: dims[mode_order[0]] x R, leading dimension ldc >= R; every row of C is written.
 * Formats as for comet_spmv. Any R >= 1; columns are processed in chunks of up to 128, and a chunk of
 * 2^k 16-byte pieces (fp64: 2..128 columns, fp32: 4..128) on 16-byte-aligned rows takes the vectorised path. */
comet_status_t comet_spmm(comet_handle_t handle, const comet_sptensor_t *A, const void *B, int64_t R, int64_t ldb,
                          void *C, int64_t ldc, void *stream);

/* The SpMM path from HOST buffers in one call: copies the COO entries and B to the device, packs the matrix
 * to CSR ([D,CU], comet_pack), multiplies (comet_spmm) and copies C back; returns when C has landed in h_C.
 * The transfers overlap: B and C travel in column chunks of 256 bytes per row on two copy streams of the handle,
 * so C's first chunk leaves while the rest of B still arrives (COMET_HOST_CHUNK_BYTES=n changes the chunk width,
 * 0 = one chunk). Every h_ pointer is HOST memory and should be pinned (page-locked): with pageable memory the
 * copies are staged by the driver and nothing overlaps. Device buffers come from the handle's allocator and are
 * released before the call returns.
 *   h_dims[2]      rows, columns;   h_row / h_col / h_val: nnz coordinates (int32) and values, any order, distinct cells
 *   h_B            columns x R, row-major, leading dimension ldb;   h_C: rows x R, leading dimension ldc, every row written
 * Errors as for comet_pack and comet_spmm. */
comet_status_t comet_spmm_from_host(comet_handle_t handle, const int64_t *h_dims, int64_t nnz, const int32_t *h_row,
                                    const int32_t *h_col, const void *h_val, comet_dtype_t dtype, const void *h_B,
                                    int64_t ldb, int64_t R, void *h_C, int64_t ldc, void *stream);

/* TTV  Y = X x_n v  (SpTTV definition; `mode` = n, 0-based, must be the mode of X's LAST level).
 * X: 3 levels, [CU,CU,CU] (CSF) or [CN,S,S] (sorted COO), or 4 levels, [CU,CU,CU,CU] (CSF) or [CN,S,S,S] (sorted
 * COO; its symbolic call derives the compressed levels by packing the entries once more). The result
 * is sparse, one order lower: comet_ttv_symbolic builds its structure over the kept modes in storage
 * order (Y's modes are renumbered 0..order-2) with h_out_attr[order-1] level attributes: {D,CU} (CSR) or
 * {CU,CU} (DCSR) for a 3-order X, {CU,CU,CU} (CSF) for a 4-order X; values are then (re)computed by
 * comet_ttv, which writes only Y->val. The structure depends on X's structure alone, never on values. Y owns its
 * arrays; X need not outlive it.
 * COO input: the fibers (runs of equal leading coordinate pairs) are not stored, so the symbolic call
 * derives them from the sorted coordinates (head flags, two scans, one synchronisation to read the
 * counts) and leaves the fiber boundary array (#fibers + 1 positions into X's entries) in the first
 * level slot BEYOND Y's own levels: Y->pos[2] / pos_len[2] for TTV, Y->pos[3] / pos_len[3] for TTM.
 * The numeric call reads it from there, so it must be given the Y that was built from this X
 * (anything else is COMET_ERR_INVALID_ARG when the sizes disagree). The slot is owned by Y. */
comet_status_t comet_ttv_symbolic(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                                  const int32_t *h_out_attr, void *stream, comet_sptensor_t *Y);
comet_status_t comet_ttv(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, const void *v,
                         comet_sptensor_t *Y, void *stream);

/* TTM  Y = X x_n U, U in R^{I_n x R} with rows indexed by the contracted mode (SpTTM definition);
 * mode n is replaced by r in place. `mode` must be the mode of X's last level. The result is
 * semi-sparse, [CU,CU,D] for a 3-order X and [CU,CU,CU,D] for a 4-order X: its sparse levels equal X's
 * upper levels and every stored fiber is a dense row of R values (val is #fibers x R, row-major). comet_ttm_symbolic builds that structure,
 * comet_ttm writes only Y->val. Formats of X as for comet_ttv (COO: see the note there). */
comet_status_t comet_ttm_symbolic(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, int64_t R,
                                  void *stream, comet_sptensor_t *Y);
/* comet_ttm_symbolic with a choice of result format. h_out_attr (one attribute per level of Y): the default
 * {CU,..,CU,D}, or, for a 3-order X, the mode-generic form {CN,S,D} that the paper names for semi-sparse
 * tensors: pos[0] = [0, #fibers], crd[0] / crd[1] hold one coordinate pair per stored fiber (sorted), and val is
 * the same #fibers x R matrix. NULL selects the default. comet_ttm takes either kind of Y. */
comet_status_t comet_ttm_symbolic_ex(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, int64_t R,
                                     const int32_t *h_out_attr, void *stream, comet_sptensor_t *Y);
comet_status_t comet_ttm(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode, const void *U, int64_t R,
                         int64_t ldu, comet_sptensor_t *Y, void *stream);

/* MTTKRP  out_{i_n r} = sum x_{i1 i2 i3} P_{p r} Q_{q r} over the two other modes p < q (the paper
 * names the operation without defining it; this is the textbook matricised-tensor-times-Khatri-Rao
 * product). X: [CN,S,S] (COO) or [CU,CU,CU] (CSF); `mode` = n may be ANY of the three modes, so that
 * one packed tensor serves the all-modes sequence of CP-ALS:
 *   - n stored at X's FIRST level: tiled kernels, every output row written by exactly one CTA, results
 *     bit-identical from run to run;
 *   - n stored at level 1 or 2: the tensor is used as stored (nothing is re-packed); the terms of an
 *     output row are then spread over the whole tensor and are added with atomic adds in double, so
 *     the summation ORDER is not fixed and results agree from run to run only up to rounding (still
 *     within the stated tolerance). About 2-4x slower than the first-level case; callers that repeat the
 *     same mode many times may prefer a second comet_pack with that mode first. For fp32 tensors this
 *     path takes rows x R doubles of handle scratch. The leaf mode of a large CSF tensor keeps its most
 *     popular output rows in shared memory (adds to one address retire one by one in L2) and allocates
 *     4 bytes per fiber and 8 per output row for the duration of the call.
 * 4-order tensors ([CN,S,S,S] or [CU,CU,CU,CU]; out_{i_n r} = sum x * the three other factors' entries): every
 * mode, all by atomic accumulation (the note on the summation order applies to all four modes).
 *   h_factors[order]  HOST array of DEVICE pointers, factor of mode m is dims[m] x R with leading
 *                 dimension h_ld[m] (h_ld has `order` entries too); the entry at `mode` is ignored
 *   out           dims[mode] x R, leading dimension ldo, every row written. */
comet_status_t comet_mttkrp(comet_handle_t handle, const comet_sptensor_t *X, int32_t mode,
                            const void *const *h_factors, const int64_t *h_ld, int64_t R, void *out, int64_t ldo,
                            void *stream);

/* Reordering pre-pass (Data Reordering section: sort one dimension at a time lexicographically by the
 * coordinates of its entries in the other dimensions, all dimensions in turn, to gather the entries around the
 * diagonal). The paper gives no further detail; this call keeps the first element of each index's sorted entry
 * list: in a step for mode m, key(x) = the smallest tuple (current numbers of the other modes' coordinates, in
 * increasing mode order) over the entries with mode-m index x, +infinity for an index without entries, and the
 * indices are re-numbered in ascending key order, ties in the order of their current numbers. One iteration is
 * a step for every mode in turn.
 *   h_coo_crd[order]    HOST array of DEVICE pointers: int32[nnz] coordinates per mode (COO, any order;
 *                       duplicates allowed); orders 2 to 4
 *   h_new_label[order]  HOST array of DEVICE pointers: int32[dims[m]] OUT, new_label[m][x] = the new number of
 *                       original index x (a permutation of 0..dims[m]-1; the identity for iterations = 0)
 * The caller applies it: coordinates become new_label[m][c], row j of a dense operand indexed by mode m moves to
 * row new_label[m][j], and row i of a result indexed by mode m is found at row new_label[m][i]. The result of
 * a contraction is unchanged up to that relabelling. Synchronises `stream` once (coordinate range check);
 * COMET_ERR_COORD_OUT_OF_RANGE leaves the labels at the identity. */
comet_status_t comet_reorder(comet_handle_t handle, int32_t order, const int64_t *h_dims, int64_t nnz,
                             const int32_t *const *h_coo_crd, int32_t iterations, int32_t *const *h_new_label,
                             void *stream);

/* Element-wise product with a dense operand (Language section: `*` between operands whose indices are not
 * contraction indices is element-wise): C = A .* B, sparse with A's structure. out_val[p] = val[p] * B[coordinates
 * of A's leaf position p]; out_val (device, A->nnz values of A's dtype, caller-allocated, may be A->val itself)
 * is the value array of a tensor that otherwise shares A's level arrays. B is dense over A's modes: element
 * (i_0, i_1, ...) in MODE order (not storage order) sits at B[sum_m i_m * h_strides[m]] (h_strides: host array,
 * one non-negative element stride per mode). Any attribute tuple the descriptor may hold, of order 1..4, and
 * ELLPACK (two strides; padding slots give 0). Asynchronous on `stream`; a caller-built A is trusted as in the
 * contractions. */
comet_status_t comet_elementwise_mul(comet_handle_t handle, const comet_sptensor_t *A, const void *B,
                                     const int64_t *h_strides, void *out_val, void *stream);

/* CSR SpMV without any allocation (the paper has no counterpart; this exists for deployment only).
 *
 * Who needs it: callers that cannot obtain device memory at call time. Examples are a service whose
 * whole GPU has been handed to another component's memory pool, so that a driver allocation would
 * fail or stall, and a latency-critical loop in which a driver allocation (it can take a lock and
 * synchronise the device) is not acceptable. comet_spmv needs a handle, and a handle gets its
 * scratch from an allocator; this entry point needs neither. It calls no cudaMalloc, cudaFree or
 * any other allocating routine, directly or through a library.
 *
 * The same product as comet_spmv for A = [D,CU] with fp64 values, equal to it up to rounding (the two tile the
 * matrix differently); other formats or fp32: COMET_ERR_UNSUPPORTED_FORMAT. The caller
 * still passes the inputs and the output (device pointers, y has dims[mode_order[0]] entries and is
 * fully overwritten). The per-tile carry slots live in a fixed 768 KiB device array that is part of
 * the library image: every GPU that loads the library holds it until the process exits.
 *   - Limit: rows + nnz <= 134,217,728 (65,536 tiles of 2,048 merge items); larger problems return
 *     COMET_ERR_WORKSPACE and must use comet_spmv.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and remembers it; make that first call outside any stream capture.
 *   - All calls share the one array, which keeps whatever the previous call left in it (each call
 *     overwrites every slot it reads, so nothing has to be cleared). Two calls that overlap on the
 *     GPU -- different streams, or different threads -- race on it: serialise them.
 *   - Asynchronous on `stream`; errors are return codes as everywhere else. */
comet_status_t comet_spmv_static(const comet_sptensor_t *A, const void *x, void *y, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* COMET_H */
