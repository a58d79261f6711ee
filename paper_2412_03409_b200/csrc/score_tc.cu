// Importance score (Sec. 3.2), tensor-core path for bf16 inputs (tcgen05 / TMEM / TMA).
#include "common.cuh"

namespace pkv {

bool score_tc_usable(const pkv_shape *, const void *, pkv_strides, const void *, pkv_strides)
{
    return false;
}

int launch_score_tc(const pkv_shape *, const void *, pkv_strides, const void *, pkv_strides,
                    const float *, const float *, float *, void *, cudaStream_t)
{
    return PKV_ERR_UNSUPPORTED;
}

}  // namespace pkv
