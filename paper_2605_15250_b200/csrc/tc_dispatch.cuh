// Host-side dispatch to the tensor-core (tcgen05) kernels.  Each function returns
// GQLA_ERR_UNSUPPORTED when the shape is outside what those kernels cover, in which case
// the caller falls through to the generic SIMT kernels.
#pragma once
#include "../../include/gqla.h"
#include "common.cuh"

namespace gqla {

// path: 0 = absorb, 1 = GQA
inline bool tc_covers(const gqla_dims& d, gqla_dtype dtype, int32_t s_q, int32_t path) {
    (void)d; (void)dtype; (void)s_q; (void)path;
    return false;
}

inline gqla_status tc_absorb_q(const gqla_dims&, gqla_dtype, int32_t, int32_t, const void*, const void*, const void*,
                               void*, cudaStream_t) {
    return GQLA_ERR_UNSUPPORTED;
}
inline gqla_status tc_up_proj(const gqla_dims&, gqla_dtype, int32_t, int32_t, const void*, const void*, void*,
                              cudaStream_t) {
    return GQLA_ERR_UNSUPPORTED;
}
inline gqla_status tc_expand_cache(const gqla_dims&, gqla_dtype, int64_t, const void*, int64_t, const void*,
                                   const void*, void*, void*, void*, cudaStream_t) {
    return GQLA_ERR_UNSUPPORTED;
}
inline gqla_status tc_decode_absorb(const gqla_dims&, int32_t, int32_t, float, int32_t, const void*, const void*,
                                    int64_t, const int64_t*, const int32_t*, float*, float*, int32_t*, cudaStream_t) {
    return GQLA_ERR_UNSUPPORTED;
}
inline gqla_status tc_decode_gqa(const gqla_dims&, int32_t, int32_t, float, int32_t, const void*, const void*,
                                 const void*, const void*, int64_t, const int64_t*, const int32_t*, float*, float*,
                                 int32_t*, cudaStream_t) {
    return GQLA_ERR_UNSUPPORTED;
}

}  // namespace gqla
