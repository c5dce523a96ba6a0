// Small device helpers shared by the convolution kernels.
#ifndef RTOSS_CONV_COMMON_CUH
#define RTOSS_CONV_COMMON_CUH

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "rtoss_internal.h"

namespace rtoss_dev {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// Packed value i of the given storage type, widened to fp32.
__device__ __forceinline__ float load_val(const void* val, size_t i, int dtype) {
    if (dtype == RTOSS_F32) return reinterpret_cast<const float*>(val)[i];
    if (dtype == RTOSS_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(val)[i]);
    return __half2float(reinterpret_cast<const __half*>(val)[i]);
}

// Fused epilogue: bias was already added by the caller; activation in fp32.
__device__ __forceinline__ float activate(float v, int act) {
    if (act == RTOSS_ACT_RELU) return fmaxf(v, 0.f);
    if (act == RTOSS_ACT_SILU) return v / (1.f + __expf(-v));
    return v;
}

}  // namespace rtoss_dev

#endif
