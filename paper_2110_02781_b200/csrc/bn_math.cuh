// Batch-norm / activation arithmetic shared by the streaming kernels and by the kernels that apply a batch norm
// to their input operand while they load it: one expression, so both routes give the same bits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace ftp {

__device__ __forceinline__ float act_f(float v, int act) {
    if (act == 1) return fmaxf(v, 0.f);
    if (act == 2) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}
__device__ __forceinline__ bool act_pass(float z, int act) {      // derivative is 1 strictly inside the linear range
    if (act == 1) return z > 0.f;
    if (act == 2) return z > 0.f && z < 6.f;
    return true;
}

// Normalised value: the mean is a two-float sum and is subtracted first, so that the result keeps
// float accuracy relative to its own size even when the mean dwarfs the spread.
__device__ __forceinline__ float bn_z(float y, float mh, float ml, float scale, float beta) {
    return fmaf((y - mh) - ml, scale, beta);
}

// the same batch norm + activation in the form used by kernels that normalise what they load: the float part of the mean
// is subtracted, its remainder is folded into offset = beta - mean_lo * scale, then the clamp (lo, hi) of the activation
__device__ __forceinline__ float xf_z(float y, float mean, float scale, float offset, float lo, float hi) {
    return fminf(fmaxf(fmaf(y - mean, scale, offset), lo), hi);
}

// a value as the tensor of element type T would hold it
template <typename T> __device__ __forceinline__ float as_stored(float v);
template <> __device__ __forceinline__ float as_stored<float>(float v) { return v; }
template <> __device__ __forceinline__ float as_stored<__nv_bfloat16>(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

}  // namespace ftp
