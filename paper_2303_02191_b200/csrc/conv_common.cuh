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

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic stream
// serialization and begins with pdl_enter(): it lets the NEXT kernel of the stream be scheduled already (launch
// latency and block start-up then overlap this kernel's run) and then waits until every kernel before it in the
// stream has completed and its writes are visible.  No kernel touches memory before that wait, so the stream's
// order of reads and writes is unchanged.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The kernels that WRITE a packed handle's arrays (values, ids, order, the tensor path's weights and issue words) begin
// with this instead: they wait like every other kernel but never let the next kernel start early.  The tensor-path
// convolution relies on it: it fetches its weights before its own wait (they are constant while a network runs), which is
// safe because whatever may still be writing them -- one of these kernels -- has completed before the convolution starts.
__device__ __forceinline__ void pdl_enter_handle_writer() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<Args&&>(args)...);
}

// The same with thread-block clusters of `cluster` CTAs along x (1 = no clusters).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<Args&&>(args)...);
}

}  // namespace rtoss_dev

#endif
