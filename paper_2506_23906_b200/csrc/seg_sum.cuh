// Segmented sum over CSR offsets and CSR SpMV (placeholder until the kernels land).
#pragma once
#include "../../include/mmv.h"
#include "common.cuh"

namespace mmv {
inline bool seg_sum_set_attributes() { return true; }
inline mmv_status seg_sum_csr_launch(const void*, const int32_t*, long long, long long, mmv_dtype, void*, void*,
                                     size_t, void*) {
    return MMV_ERR_UNSUPPORTED;
}
inline mmv_status spmv_csr_launch(const int32_t*, const int32_t*, const void*, const float*, float*, long long,
                                  long long, long long, void*, size_t, void*) {
    return MMV_ERR_UNSUPPORTED;
}
}  // namespace mmv
