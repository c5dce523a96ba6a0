// Glue operations between the convolutions of a detector (not part of the paper's method; they are what a
// whole-network run needs besides the pattern convolutions): k x k max-pooling, nearest-neighbour 2x
// up-sampling, element-wise addition with an optional activation.  All are bandwidth-bound element-wise
// kernels; outputs may be channel slices of a wider tensor so that a concatenation is a write, not a copy.
#include "conv_common.cuh"

namespace {

using namespace rtoss_dev;

struct GlueArgs {
    const void* x;
    const void* x2;
    void* y;
    int N, C, H, W, Ho, Wo;
    int k, stride, pad;
    int layout, act;
    int y_c_off, y_c_stride;
};

__device__ __forceinline__ size_t idx_of(int layout, int n, int c, int h, int w, int C, int H, int W) {
    return layout == RTOSS_NCHW ? (((size_t)n * C + c) * H + h) * W + w : (((size_t)n * H + h) * W + w) * C + c;
}

// One thread per output element, channel fastest for NHWC and column fastest for NCHW (coalesced both ways).
template <typename T>
__global__ void maxpool_kernel(const GlueArgs a) {
    rtoss_dev::pdl_enter();
    const size_t total = (size_t)a.N * a.C * a.Ho * a.Wo;
    const T* __restrict__ x = reinterpret_cast<const T*>(a.x);
    T* __restrict__ y = reinterpret_cast<T*>(a.y);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int n, c, oh, ow;
        size_t r = i;
        if (a.layout == RTOSS_NCHW) {
            ow = (int)(r % a.Wo); r /= a.Wo;
            oh = (int)(r % a.Ho); r /= a.Ho;
            c = (int)(r % a.C);
            n = (int)(r / a.C);
        } else {
            c = (int)(r % a.C); r /= a.C;
            ow = (int)(r % a.Wo); r /= a.Wo;
            oh = (int)(r % a.Ho);
            n = (int)(r / a.Ho);
        }
        float m = -INFINITY;  // padding never wins
        for (int dy = 0; dy < a.k; ++dy) {
            const int ih = oh * a.stride + dy - a.pad;
            if (ih < 0 || ih >= a.H) continue;
            for (int dx = 0; dx < a.k; ++dx) {
                const int iw = ow * a.stride + dx - a.pad;
                if (iw < 0 || iw >= a.W) continue;
                m = fmaxf(m, to_f32<T>(x[idx_of(a.layout, n, c, ih, iw, a.C, a.H, a.W)]));
            }
        }
        y[idx_of(a.layout, n, a.y_c_off + c, oh, ow, a.y_c_stride, a.Ho, a.Wo)] = from_f32<T>(m);
    }
}

template <typename T>
__global__ void upsample2x_kernel(const GlueArgs a) {
    rtoss_dev::pdl_enter();
    const size_t total = (size_t)a.N * a.C * a.Ho * a.Wo;
    const T* __restrict__ x = reinterpret_cast<const T*>(a.x);
    T* __restrict__ y = reinterpret_cast<T*>(a.y);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int n, c, oh, ow;
        size_t r = i;
        if (a.layout == RTOSS_NCHW) {
            ow = (int)(r % a.Wo); r /= a.Wo;
            oh = (int)(r % a.Ho); r /= a.Ho;
            c = (int)(r % a.C);
            n = (int)(r / a.C);
        } else {
            c = (int)(r % a.C); r /= a.C;
            ow = (int)(r % a.Wo); r /= a.Wo;
            oh = (int)(r % a.Ho);
            n = (int)(r / a.Ho);
        }
        y[idx_of(a.layout, n, a.y_c_off + c, oh, ow, a.y_c_stride, a.Ho, a.Wo)] =
            x[idx_of(a.layout, n, c, oh >> 1, ow >> 1, a.C, a.H, a.W)];
    }
}

template <typename T>
__global__ void add_act_kernel(const T* __restrict__ p, const T* __restrict__ q, T* __restrict__ y, size_t n, int act) {
    rtoss_dev::pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        y[i] = from_f32<T>(activate(to_f32<T>(p[i]) + to_f32<T>(q[i]), act));
}

int grid_for(size_t n) {
    size_t g = (n + 255) / 256;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

bool ok_dtype(int d) { return d == RTOSS_F32 || d == RTOSS_BF16 || d == RTOSS_F16; }

}  // namespace

extern "C" {

rtoss_status rtoss_maxpool2d(const void* x_dev, void* y_dev, int N, int C, int H, int W, int k, int stride, int pad,
                             rtoss_layout layout, rtoss_dtype dtype, int y_channel_offset, int y_channel_stride,
                             void* cuda_stream) {
    if (!x_dev || !y_dev || N < 1 || C < 1 || H < 1 || W < 1 || k < 1 || stride < 1 || pad < 0 || !ok_dtype(dtype) || (layout != RTOSS_NCHW && layout != RTOSS_NHWC))
        return RTOSS_ERR_INVALID_ARG;
    if (pad > k / 2) return RTOSS_ERR_INVALID_ARG;  // a window must always contain an input pixel
    const int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
    if (Ho < 1 || Wo < 1) return RTOSS_ERR_INVALID_ARG;
    const int cs = y_channel_stride ? y_channel_stride : C;
    if (y_channel_offset < 0 || cs < y_channel_offset + C) return RTOSS_ERR_INVALID_ARG;
    GlueArgs a{x_dev, nullptr, y_dev, N, C, H, W, Ho, Wo, k, stride, pad, (int)layout, 0, y_channel_offset, cs};
    const int grid = grid_for((size_t)N * C * Ho * Wo);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == RTOSS_F32) rtoss_dev::launch_pdl(maxpool_kernel<float>, grid, 256, 0, s, a);
    else if (dtype == RTOSS_BF16) rtoss_dev::launch_pdl(maxpool_kernel<__nv_bfloat16>, grid, 256, 0, s, a);
    else rtoss_dev::launch_pdl(maxpool_kernel<__half>, grid, 256, 0, s, a);
    return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
}

rtoss_status rtoss_upsample2x(const void* x_dev, void* y_dev, int N, int C, int H, int W, rtoss_layout layout,
                              rtoss_dtype dtype, int y_channel_offset, int y_channel_stride, void* cuda_stream) {
    if (!x_dev || !y_dev || N < 1 || C < 1 || H < 1 || W < 1 || !ok_dtype(dtype) ||
        (layout != RTOSS_NCHW && layout != RTOSS_NHWC))
        return RTOSS_ERR_INVALID_ARG;
    const int cs = y_channel_stride ? y_channel_stride : C;
    if (y_channel_offset < 0 || cs < y_channel_offset + C) return RTOSS_ERR_INVALID_ARG;
    GlueArgs a{x_dev, nullptr, y_dev, N, C, H, W, 2 * H, 2 * W, 0, 0, 0, (int)layout, 0, y_channel_offset, cs};
    const int grid = grid_for((size_t)N * C * 4 * H * W);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == RTOSS_F32) rtoss_dev::launch_pdl(upsample2x_kernel<float>, grid, 256, 0, s, a);
    else if (dtype == RTOSS_BF16) rtoss_dev::launch_pdl(upsample2x_kernel<__nv_bfloat16>, grid, 256, 0, s, a);
    else rtoss_dev::launch_pdl(upsample2x_kernel<__half>, grid, 256, 0, s, a);
    return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
}

rtoss_status rtoss_add_act(const void* a_dev, const void* b_dev, void* y_dev, int64_t n_elements, rtoss_dtype dtype,
                           rtoss_act act, void* cuda_stream) {
    if (!a_dev || !b_dev || !y_dev || n_elements < 1 || !ok_dtype(dtype) ||
        (act != RTOSS_ACT_NONE && act != RTOSS_ACT_RELU && act != RTOSS_ACT_SILU))
        return RTOSS_ERR_INVALID_ARG;
    const int grid = grid_for((size_t)n_elements);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype == RTOSS_F32)
        rtoss_dev::launch_pdl(add_act_kernel<float>, grid, 256, 0, s, (const float*)a_dev, (const float*)b_dev, (float*)y_dev, (size_t)n_elements, (int)act);
    else if (dtype == RTOSS_BF16)
        rtoss_dev::launch_pdl(add_act_kernel<__nv_bfloat16>, grid, 256, 0, s, (const __nv_bfloat16*)a_dev, (const __nv_bfloat16*)b_dev,
                                                            (__nv_bfloat16*)y_dev, (size_t)n_elements, (int)act);
    else
        rtoss_dev::launch_pdl(add_act_kernel<__half>, grid, 256, 0, s, (const __half*)a_dev, (const __half*)b_dev, (__half*)y_dev, (size_t)n_elements, (int)act);
    return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
}

}  // extern "C"
