// Element-wise product of a sparse tensor with a dense one (the `*` of the paper's Language section between
// operands whose indices are not contraction indices): C = A .* B has A's structure and the values
// val[p] * B[coordinates of leaf entry p]. A thread per stored leaf position climbs the levels from the leaf to
// the root to find its coordinates, by the rule of each level's attribute: a compressed or singleton level reads
// its coordinate array (a compressed-unique level then finds its parent by a search in pos), a dense level splits
// the position into (parent, coordinate). Any attribute tuple a descriptor may hold, ELLPACK's padding included.
#include "common.cuh"
#include "kernels.cuh"

namespace comet {

struct ElementwiseArgs {
  int32_t order;
  int32_t attr[COMET_MAX_ORDER];
  const int32_t *pos[COMET_MAX_ORDER];
  int64_t pos_len[COMET_MAX_ORDER];
  const int32_t *crd[COMET_MAX_ORDER];
  int64_t dim[COMET_MAX_ORDER];        // extent of the mode stored at level l
  int64_t stride[COMET_MAX_ORDER];     // element stride in B of the mode stored at level l (0: the level stores no mode of B)
  int64_t positions;                   // stored leaf positions
};

template <class T>
__global__ void __launch_bounds__(kBlockThreads) elementwise_mul_kernel(const ElementwiseArgs a, const T *__restrict__ val,
                                                                        const T *__restrict__ B, T *__restrict__ out) {
  const int64_t p = (int64_t)blockIdx.x * kBlockThreads + threadIdx.x;
  if (p >= a.positions) return;
  int64_t at = p, offset = 0;
  bool padding = false;
#pragma unroll
  for (int l = COMET_MAX_ORDER - 1; l >= 0; --l) {
    if (l >= a.order) continue;
    int64_t coord;
    if (a.attr[l] == COMET_D) {
      coord = at % a.dim[l];
      at /= a.dim[l];
    } else {
      coord = __ldg(a.crd[l] + at);
      if (a.attr[l] == COMET_CU && l > 0) {                 // parent = the last position whose range starts at or before `at`
        int64_t lo = 0, hi = a.pos_len[l] - 1;
        while (hi - lo > 1) {
          const int64_t mid = (lo + hi) >> 1;
          if ((int64_t)__ldg(a.pos[l] + mid) <= at) lo = mid; else hi = mid;
        }
        at = lo;
      } else if (a.attr[l] != COMET_S) {
        at = 0;                                             // a root level hangs under the single root position
      }
    }
    padding |= coord < 0;
    offset += coord * a.stride[l];
  }
  out[p] = padding ? (T)0 : (T)((double)val[p] * (double)__ldg(B + offset));
}

comet_status_t elementwise_mul(Context *ctx, const comet_sptensor_t *A, const void *B, const int64_t *h_strides, void *out,
                               cudaStream_t s) {
  ElementwiseArgs a{};
  a.order = A->order;
  const bool ell = is_ellpack(A);
  for (int l = 0; l < A->order; ++l) {
    a.attr[l] = A->attr[l];
    a.pos[l] = A->pos[l];
    a.pos_len[l] = A->pos_len[l];
    a.crd[l] = A->crd[l];
    a.dim[l] = A->dims[A->mode_order[l]];
    a.stride[l] = (ell && l == 1) ? 0 : h_strides[A->mode_order[l]];
    if (a.attr[l] == COMET_D && a.dim[l] <= 0) return COMET_OK;          // no position at all
  }
  a.positions = A->nnz;
  if (a.positions == 0) return COMET_OK;
  const unsigned blocks = (unsigned)ceil_div(a.positions, kBlockThreads);
  if (A->dtype == COMET_F32)
    elementwise_mul_kernel<float><<<blocks, kBlockThreads, 0, s>>>(a, (const float *)A->val, (const float *)B, (float *)out);
  else
    elementwise_mul_kernel<double><<<blocks, kBlockThreads, 0, s>>>(a, (const double *)A->val, (const double *)B, (double *)out);
  COMET_LAUNCH_CHECK(ctx);
  return COMET_OK;
}

}  // namespace comet
