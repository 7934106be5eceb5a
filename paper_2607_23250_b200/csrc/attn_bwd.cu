// Backward pool attention (placeholder translation unit until the kernels land).
#include "common.h"

using namespace libra;

extern "C" size_t libra_attn_pool_bwd_workspace_bytes(const libra_plan_t* plan, const libra_dims* dims) {
    if (!plan || !dims || dims->hq <= 0 || dims->head_dim <= 0) return 0;
    const size_t T = (size_t)plan->T;
    size_t dq_acc = T * (size_t)dims->hq * (size_t)dims->head_dim * sizeof(float);
    size_t drow = (size_t)dims->hq * T * sizeof(float);
    dq_acc = (dq_acc + 255) & ~(size_t)255;
    drow = (drow + 255) & ~(size_t)255;
    return dq_acc + drow;
}

extern "C" int libra_attn_pool_bwd(const void*, const void*, const void*, const void*, const float*, const void*,
                                   const int32_t*, const libra_plan_t*, void*, void*, void*, void*,
                                   const libra_dims*, void*) {
    return LIBRA_ERR_UNSUPPORTED;
}
