// Host helpers shared by the .cu translation units: descriptor validation, image offsets,
// CUDA error bookkeeping.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rwkvq.h"
#include "format.h"

namespace rwkvq {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up_sz(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline rwkvq_status check_matrix_desc(const rwkvq_desc* d) {
  if (!d) return RWKVQ_EINVAL;
  if (d->oc <= 0 || d->ic <= 0) return RWKVQ_ESHAPE;
  if (d->method == RWKVQ_SQ) {
    if (d->bits != 3 || d->group != 128) return RWKVQ_EUNSUPPORTED;
    if (d->oc % 16 || d->ic % 128) return RWKVQ_ESHAPE;
    if (d->oc_pad != (int)round_up_sz(d->oc, 128) || d->ic_pad != (int)round_up_sz(d->ic, 256)) return RWKVQ_EINVAL;
  } else if (d->method == RWKVQ_VQ) {
    if ((d->bits != 6 && d->bits != 8) || d->vec_dim != 2 || d->tile != 256) return RWKVQ_EUNSUPPORTED;
    if (d->entries != (1 << d->bits)) return RWKVQ_EINVAL;
    if (d->oc % 256 || d->ic % 256) return RWKVQ_ESHAPE;
    if (d->oc_pad != d->oc || d->ic_pad != d->ic) return RWKVQ_EINVAL;
  } else {
    return RWKVQ_EINVAL;
  }
  return RWKVQ_OK;
}

inline rwkvq_status check_vector_desc(const rwkvq_desc* d, int ic) {
  if (!d) return RWKVQ_EINVAL;
  if (d->method != RWKVQ_VQ || d->oc != 1) return RWKVQ_EINVAL;
  if ((d->bits != 6 && d->bits != 8) || d->vec_dim != 2) return RWKVQ_EUNSUPPORTED;
  if (d->entries != (1 << d->bits)) return RWKVQ_EINVAL;
  if (d->ic != ic || ic % 2) return RWKVQ_ESHAPE;
  return RWKVQ_OK;
}

inline size_t matrix_aux_offset(const rwkvq_desc* d) {
  size_t rb = d->method == RWKVQ_SQ ? RWKVQ_SQ_RECORD_BYTES : rwkvq_vq_record_bytes(d->bits);
  return RWKVQ_HEADER_BYTES + (size_t)(d->oc_pad / 128) * (d->ic_pad / 256) * 8 * rb;
}
inline size_t vector_aux_offset(const rwkvq_desc* d) {
  return RWKVQ_HEADER_BYTES + round_up_sz(((size_t)(d->ic / 2) * d->bits + 7) / 8, 16);
}

void set_last_cuda_error(cudaError_t e);
inline rwkvq_status cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return RWKVQ_OK;
  set_last_cuda_error(e);
  return RWKVQ_ECUDA;
}

}  // namespace rwkvq
