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

// ---- 16-bit NHWC tensors whose channel counts, slices and pointers allow it: eight channels (16 bytes) per thread.
// The scalar kernels above move two bytes per thread and spend their time on index arithmetic; these are the ones
// a chained network runs.  Results are the same bits (a maximum selects one of its inputs; the sum is formed per
// element exactly as above).
template <typename T> struct Pair;
template <> struct Pair<__nv_bfloat16> { using type = __nv_bfloat162; };
template <> struct Pair<__half> { using type = __half2; };

template <typename T>
__device__ __forceinline__ uint4 max8(uint4 p, uint4 q) {
    using P = typename Pair<T>::type;
    uint4 r;
    P* rp = reinterpret_cast<P*>(&r);
    const P* pp = reinterpret_cast<const P*>(&p);
    const P* qp = reinterpret_cast<const P*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) rp[i] = __hmax2(pp[i], qp[i]);   // like fmaxf: a NaN loses against a number
    return r;
}

template <typename T>
__global__ void maxpool_vec8_kernel(const GlueArgs a) {
    rtoss_dev::pdl_enter();
    const int C8 = a.C >> 3;
    const size_t total = (size_t)a.N * a.Ho * a.Wo * C8;
    const T* __restrict__ x = reinterpret_cast<const T*>(a.x);
    T* __restrict__ y = reinterpret_cast<T*>(a.y);
    const T ninf = from_f32<T>(-INFINITY);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int c8 = (int)(r % C8); r /= C8;
        const int ow = (int)(r % a.Wo); r /= a.Wo;
        const int oh = (int)(r % a.Ho);
        const int n = (int)(r / a.Ho);
        __align__(16) T init[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) init[j] = ninf;   // padding never wins
        uint4 m = *reinterpret_cast<const uint4*>(init);
        for (int dy = 0; dy < a.k; ++dy) {
            const int ih = oh * a.stride + dy - a.pad;
            if (ih < 0 || ih >= a.H) continue;
            for (int dx = 0; dx < a.k; ++dx) {
                const int iw = ow * a.stride + dx - a.pad;
                if (iw < 0 || iw >= a.W) continue;
                m = max8<T>(m, *reinterpret_cast<const uint4*>(x + (((size_t)n * a.H + ih) * a.W + iw) * a.C + c8 * 8));
            }
        }
        *reinterpret_cast<uint4*>(y + (((size_t)n * a.Ho + oh) * a.Wo + ow) * a.y_c_stride + a.y_c_off + c8 * 8) = m;
    }
}

template <typename T>
__global__ void upsample2x_vec8_kernel(const GlueArgs a) {
    rtoss_dev::pdl_enter();
    const int C8 = a.C >> 3;
    const size_t total = (size_t)a.N * a.Ho * a.Wo * C8;
    const T* __restrict__ x = reinterpret_cast<const T*>(a.x);
    T* __restrict__ y = reinterpret_cast<T*>(a.y);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int c8 = (int)(r % C8); r /= C8;
        const int ow = (int)(r % a.Wo); r /= a.Wo;
        const int oh = (int)(r % a.Ho);
        const int n = (int)(r / a.Ho);
        *reinterpret_cast<uint4*>(y + (((size_t)n * a.Ho + oh) * a.Wo + ow) * a.y_c_stride + a.y_c_off + c8 * 8) =
            *reinterpret_cast<const uint4*>(x + (((size_t)n * a.H + (oh >> 1)) * a.W + (ow >> 1)) * a.C + c8 * 8);
    }
}

template <typename T>
__global__ void add_act_vec8_kernel(const T* __restrict__ p, const T* __restrict__ q, T* __restrict__ y, size_t n8, int act) {
    rtoss_dev::pdl_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 pv = reinterpret_cast<const uint4*>(p)[i], qv = reinterpret_cast<const uint4*>(q)[i];
        const T* pe = reinterpret_cast<const T*>(&pv);
        const T* qe = reinterpret_cast<const T*>(&qv);
        __align__(16) T o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j] = from_f32<T>(activate(to_f32<T>(pe[j]) + to_f32<T>(qe[j]), act));
        reinterpret_cast<uint4*>(y)[i] = *reinterpret_cast<const uint4*>(o);
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// 16-bit NHWC, channels and the output slice in multiples of eight, 16-byte aligned pointers
inline bool vec8_ok(const GlueArgs& a, int dtype) {
    return dtype != RTOSS_F32 && a.layout == RTOSS_NHWC && a.C % 8 == 0 && a.y_c_off % 8 == 0 && a.y_c_stride % 8 == 0 &&
           aligned16(a.x) && aligned16(a.y);
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
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (vec8_ok(a, (int)dtype)) {
        const int g8 = grid_for((size_t)N * (C / 8) * Ho * Wo);
        if (dtype == RTOSS_BF16) rtoss_dev::launch_pdl(maxpool_vec8_kernel<__nv_bfloat16>, g8, 256, 0, s, a);
        else rtoss_dev::launch_pdl(maxpool_vec8_kernel<__half>, g8, 256, 0, s, a);
        return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
    }
    const int grid = grid_for((size_t)N * C * Ho * Wo);
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
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (vec8_ok(a, (int)dtype)) {
        const int g8 = grid_for((size_t)N * (C / 8) * 4 * H * W);
        if (dtype == RTOSS_BF16) rtoss_dev::launch_pdl(upsample2x_vec8_kernel<__nv_bfloat16>, g8, 256, 0, s, a);
        else rtoss_dev::launch_pdl(upsample2x_vec8_kernel<__half>, g8, 256, 0, s, a);
        return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
    }
    const int grid = grid_for((size_t)N * C * 4 * H * W);
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
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (dtype != RTOSS_F32 && n_elements % 8 == 0 && aligned16(a_dev) && aligned16(b_dev) && aligned16(y_dev)) {
        const size_t n8 = (size_t)n_elements / 8;
        const int g8 = grid_for(n8);
        if (dtype == RTOSS_BF16)
            rtoss_dev::launch_pdl(add_act_vec8_kernel<__nv_bfloat16>, g8, 256, 0, s, (const __nv_bfloat16*)a_dev,
                                  (const __nv_bfloat16*)b_dev, (__nv_bfloat16*)y_dev, n8, (int)act);
        else
            rtoss_dev::launch_pdl(add_act_vec8_kernel<__half>, g8, 256, 0, s, (const __half*)a_dev, (const __half*)b_dev,
                                  (__half*)y_dev, n8, (int)act);
        return cudaGetLastError() == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
    }
    const int grid = grid_for((size_t)n_elements);
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
