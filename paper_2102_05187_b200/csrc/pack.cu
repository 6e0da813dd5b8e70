// Placeholder translation unit: replaced by the GPU packing path.
#include "common.cuh"
extern "C" comet_status_t comet_pack(comet_handle_t, int32_t, const int64_t *, int64_t, const int32_t *const *,
                                     const void *, comet_dtype_t, const int32_t *, const int32_t *, void *,
                                     comet_sptensor_t *) { return COMET_ERR_UNSUPPORTED_FORMAT; }
extern "C" comet_status_t comet_validate(comet_handle_t, const comet_sptensor_t *, void *) {
  return COMET_ERR_UNSUPPORTED_FORMAT;
}
