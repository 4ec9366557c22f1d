// kop_bn_relu_avgpool: a = relu(x * scale[c] + shift[c]) written once, pooled[n,c] = mean over the
// (h, w) plane of the unrounded fp32 activations, in the same pass. NCHW planes are contiguous, so
// a CTA (or a warp, for small planes) streams one plane with 16-byte vectors and reduces it.
#include "kop_common.cuh"

namespace kop {
namespace {

// IEEE-compare ReLU: NaN fails (v > 0) and (v <= 0) alike and is passed through.
__device__ __forceinline__ float relu_keep_nan(float v) { return v > 0.0f ? v : (v <= 0.0f ? 0.0f : v); }

// One CTA per plane; every thread issues up to UNROLL independent 16-byte loads per trip.
template <typename T, int UNROLL>
__global__ void __launch_bounds__(1024)
bn_plane_block_kernel(const T* __restrict__ x, const float* __restrict__ scale,
                      const float* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                      int nvec, int64_t plane_elems, int C, float inv_plane)
{
    constexpr int E = Elem<T>::kPerVec;
    __shared__ float red[32];
    const int64_t p = blockIdx.x;
    const int c = (int)(p % C);
    const float sc = __ldg(scale + c), sh = __ldg(shift + c);
    const T* xp = x + p * plane_elems;
    T* yp = y + p * plane_elems;
    float sum = 0.0f;
    for (int base = 0; base < nvec; base += UNROLL * blockDim.x) {
        Vec16 raw[UNROLL];
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const int v = base + k * blockDim.x + threadIdx.x;
            if (v < nvec) raw[k] = ld_stream(xp + (int64_t)v * E);
        }
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const int v = base + k * blockDim.x + threadIdx.x;
            if (v < nvec) {
                float f[E];
                Elem<T>::unpack(raw[k], f);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    f[e] = relu_keep_nan(fmaf(f[e], sc, sh));
                    sum += f[e];
                }
                st_stream(yp + (int64_t)v * E, Elem<T>::pack(f));
            }
        }
    }
    sum = block_sum(sum, red);
    if (threadIdx.x == 0) pooled[p] = sum * inv_plane;
}

// One warp per plane (small planes), scalar or vector by template flag.
template <typename T, bool kVec>
__global__ void __launch_bounds__(256)
bn_plane_warp_kernel(const T* __restrict__ x, const float* __restrict__ scale,
                     const float* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                     int64_t planes, int64_t plane_elems, int C, float inv_plane)
{
    constexpr int E = Elem<T>::kPerVec;
    const int lane = threadIdx.x & 31;
    const int64_t p = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (p < planes) {
        const int c = (int)(p % C);
        const float sc = __ldg(scale + c), sh = __ldg(shift + c);
        const T* xp = x + p * plane_elems;
        T* yp = y + p * plane_elems;
        float sum = 0.0f;
        if (kVec) {
            const int64_t nvec = plane_elems / E;
            for (int64_t v = lane; v < nvec; v += 32) {
                float f[E];
                Elem<T>::unpack(ld_stream(xp + v * E), f);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    f[e] = relu_keep_nan(fmaf(f[e], sc, sh));
                    sum += f[e];
                }
                st_stream(yp + v * E, Elem<T>::pack(f));
            }
        } else {
            for (int64_t j = lane; j < plane_elems; j += 32) {
                const float a = relu_keep_nan(fmaf(Elem<T>::load1(xp + j), sc, sh));
                sum += a;
                Elem<T>::store1(yp + j, a);
            }
        }
        sum = warp_sum(sum);
        if (lane == 0) pooled[p] = sum * inv_plane;
    }
}

// Large planes that cannot be vectorised: one CTA per plane, scalar loads.
template <typename T>
__global__ void __launch_bounds__(256)
bn_plane_scalar_kernel(const T* __restrict__ x, const float* __restrict__ scale,
                       const float* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                       int64_t plane_elems, int C, float inv_plane)
{
    __shared__ float red[32];
    const int64_t p = blockIdx.x;
    const int c = (int)(p % C);
    const float sc = __ldg(scale + c), sh = __ldg(shift + c);
    const T* xp = x + p * plane_elems;
    T* yp = y + p * plane_elems;
    float sum = 0.0f;
    for (int64_t j = threadIdx.x; j < plane_elems; j += blockDim.x) {
        const float a = relu_keep_nan(fmaf(Elem<T>::load1(xp + j), sc, sh));
        sum += a;
        Elem<T>::store1(yp + j, a);
    }
    sum = block_sum(sum, red);
    if (threadIdx.x == 0) pooled[p] = sum * inv_plane;
}

template <typename T>
kop_status_t launch_bn(const void* xv, const float* scale, const float* shift, void* yv, float* pooled,
                       int64_t N, int64_t C, int64_t H, int64_t W, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    T* y = static_cast<T*>(yv);
    constexpr int E = Elem<T>::kPerVec;
    const int64_t plane = H * W, planes = N * C;
    const float inv_plane = (float)(1.0 / (double)plane);
    const bool vec = aligned_to(x, 16) && aligned_to(y, 16) && (plane % E) == 0;
    const int64_t nvec64 = plane / E;
    if (plane <= 1024 || planes > 0x7FFFFFFFLL) {
        const int64_t ctas = (planes + 7) / 8;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        const unsigned grid = (unsigned)ctas;
        if (vec)
            bn_plane_warp_kernel<T, true><<<grid, 256, 0, stream>>>(x, scale, shift, y, pooled, planes, plane, (int)C, inv_plane);
        else
            bn_plane_warp_kernel<T, false><<<grid, 256, 0, stream>>>(x, scale, shift, y, pooled, planes, plane, (int)C, inv_plane);
        return launch_status();
    }
    if (vec && nvec64 <= 0x7FFFFFFF) {
        const int nvec = (int)nvec64;
        // Four vectors per thread per trip; a 56x56 fp32 plane (784 vectors) gets 224 threads
        // and a single trip (196 threads would cover it exactly; 224 is the next warp multiple).
        int threads = ((nvec + 3) / 4 + 31) / 32 * 32;
        if (threads > 512) threads = 512;
        bn_plane_block_kernel<T, 4><<<(unsigned)planes, threads, 0, stream>>>(x, scale, shift, y, pooled, nvec, plane, (int)C, inv_plane);
        return launch_status();
    }
    bn_plane_scalar_kernel<T><<<(unsigned)planes, 256, 0, stream>>>(x, scale, shift, y, pooled, plane, (int)C, inv_plane);
    return launch_status();
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_bn_relu_avgpool(const void* x, const float* scale, const float* shift,
                                            void* y, float* pooled, int64_t N, int64_t C, int64_t H,
                                            int64_t W, const int64_t x_strides[4],
                                            const int64_t y_strides[4], kop_dtype_t dtype,
                                            kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    if (N < 0 || C <= 0 || H <= 0 || W <= 0) return KOP_ERR_BAD_SHAPE;
    if (N == 0) return KOP_OK;
    if (!x || !scale || !shift || !y || !pooled || !x_strides || !y_strides) return KOP_ERR_NULL_POINTER;
    if (C > 0x7FFFFFFF || H > kMaxElems || W > kMaxElems || N > kMaxElems) return KOP_ERR_BAD_SHAPE;
    if (H > kMaxElems / W) return KOP_ERR_BAD_SHAPE;
    const int64_t plane = H * W;
    if (C > kMaxElems / plane) return KOP_ERR_BAD_SHAPE;
    if (N > 0 && C * plane > kMaxElems / N) return KOP_ERR_BAD_SHAPE;
    const int64_t want[4] = {C * plane, plane, W, 1};
    for (int i = 0; i < 4; ++i)
        if (x_strides[i] != want[i] || y_strides[i] != want[i]) return KOP_ERR_BAD_STRIDE;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || !aligned_to(scale, 4) || !aligned_to(shift, 4) ||
        !aligned_to(pooled, 4))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, C * plane, y, C * plane, N, C * plane, esz, true)) return KOP_ERR_BAD_ALIAS;
    kop_status_t st = check_device();
    if (st != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_bn<float>(x, scale, shift, y, pooled, N, C, H, W, s)
                            : launch_bn<__nv_bfloat16>(x, scale, shift, y, pooled, N, C, H, W, s);
}
