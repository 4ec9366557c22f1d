// kop_bn_relu_avgpool: a = relu(x * scale[c] + shift[c]) written once, pooled[n,c] = mean over the
// (h, w) plane of the unrounded fp32 activations, in the same pass. NCHW planes are contiguous, so
// a CTA (or a warp, for small planes) streams one plane with 16-byte vectors and reduces it; the
// channels-last kernels are at the end of the file.
#include "kop_common.cuh"

namespace kop {
namespace {

// IEEE-compare ReLU: NaN fails (v > 0) and (v <= 0) alike and is passed through.
__device__ __forceinline__ float relu_keep_nan(float v) { return v > 0.0f ? v : (v <= 0.0f ? 0.0f : v); }

// One CTA per plane; every thread issues up to UNROLL independent 16-byte loads per trip.
template <typename T, typename PT, int UNROLL>
__global__ void __launch_bounds__(1024)
bn_plane_block_kernel(const T* __restrict__ x, const PT* __restrict__ scale,
                      const PT* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                      int nvec, int64_t plane_elems, int C, float inv_plane)
{
    constexpr int E = Elem<T>::kPerVec;
    __shared__ float red[32];
    const int64_t p = blockIdx.x;
    const int c = (int)(p % C);
    const float sc = param1(scale, c), sh = param1(shift, c);
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
template <typename T, typename PT, bool kVec>
__global__ void __launch_bounds__(256)
bn_plane_warp_kernel(const T* __restrict__ x, const PT* __restrict__ scale,
                     const PT* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                     int64_t planes, int64_t plane_elems, int C, float inv_plane)
{
    constexpr int E = Elem<T>::kPerVec;
    const int lane = threadIdx.x & 31;
    const int64_t p = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (p < planes) {
        const int c = (int)(p % C);
        const float sc = param1(scale, c), sh = param1(shift, c);
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

// Small planes (7x7, 14x14, ...: the usual input of a global average pool) are shorter than a warp's
// worth of vectors and often not a whole number of them, but consecutive planes are contiguous. A CTA
// therefore takes a run of G planes (G a multiple of the vector length, so every run starts on a 16-byte
// boundary) as one flat array: 16-byte loads and stores across plane boundaries, the plane of each
// element found by one small division per vector and carried along it, per-plane scale / shift staged in
// shared memory, the activations parked in shared memory, and the plane sums taken from there by one
// warp per plane in a fixed order.
constexpr int kFlatThreads = 256;
constexpr int kFlatMaxElems = 4096;                       // activations parked per CTA (16 KB)

template <typename T, typename PT>
__global__ void __launch_bounds__(kFlatThreads)
bn_flat_kernel(const T* __restrict__ x, const PT* __restrict__ scale, const PT* __restrict__ shift,
               T* __restrict__ y, float* __restrict__ pooled, int64_t planes, int plane, int G, int C,
               float inv_plane)
{
    constexpr int E = Elem<T>::kPerVec;
    __shared__ __align__(16) float act[kFlatMaxElems];
    __shared__ float sc_s[kFlatMaxElems / 4], sh_s[kFlatMaxElems / 4];      // G <= chunk / plane, plane >= 1 ...
    const int64_t p0 = (int64_t)blockIdx.x * G;
    const int g_here = (int)(planes - p0 < G ? planes - p0 : G);
    const int elems = g_here * plane;
    const T* xc = x + p0 * plane;
    T* yc = y + p0 * plane;
    for (int g = threadIdx.x; g < g_here; g += kFlatThreads) {
        const int c = (int)((p0 + g) % C);
        sc_s[g] = param1(scale, c);
        sh_s[g] = param1(shift, c);
    }
    __syncthreads();
    const float inv = 1.0f / (float)plane;
    const int nvec = elems / E;
    for (int v = threadIdx.x; v < nvec; v += kFlatThreads) {
        float f[E];
        Elem<T>::unpack(ld_stream(xc + (int64_t)v * E), f);
        const int i0 = v * E;
        int pl = (int)((float)i0 * inv);                 // i0 / plane: float estimate, one-step fix-up
        int rem = i0 - pl * plane;
        if (rem >= plane) { rem -= plane; ++pl; }
        if (rem < 0) { rem += plane; --pl; }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            f[e] = relu_keep_nan(fmaf(f[e], sc_s[pl], sh_s[pl]));
            act[i0 + e] = f[e];
            if (++rem == plane) { rem = 0; ++pl; }
        }
        st_stream(yc + (int64_t)v * E, Elem<T>::pack(f));
    }
    // the last run of the tensor may end inside a vector: its tail goes element by element
    for (int i = nvec * E + threadIdx.x; i < elems; i += kFlatThreads) {
        const int pl = i / plane;
        const float a = relu_keep_nan(fmaf(Elem<T>::load1(xc + i), sc_s[pl], sh_s[pl]));
        act[i] = a;
        Elem<T>::store1(yc + i, a);
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int g = warp; g < g_here; g += kFlatThreads / 32) {
        float s = 0.0f;
        for (int j = lane; j < plane; j += 32) s += act[g * plane + j];
        s = warp_sum(s);
        if (lane == 0) pooled[p0 + g] = s * inv_plane;
    }
}

// Large planes that cannot be vectorised: one CTA per plane, scalar loads.
template <typename T, typename PT>
__global__ void __launch_bounds__(256)
bn_plane_scalar_kernel(const T* __restrict__ x, const PT* __restrict__ scale,
                       const PT* __restrict__ shift, T* __restrict__ y, float* __restrict__ pooled,
                       int64_t plane_elems, int C, float inv_plane)
{
    __shared__ float red[32];
    const int64_t p = blockIdx.x;
    const int c = (int)(p % C);
    const float sc = param1(scale, c), sh = param1(shift, c);
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

template <typename T, typename PT>
kop_status_t launch_bn(const void* xv, const void* scalev, const void* shiftv, void* yv, float* pooled,
                       int64_t N, int64_t C, int64_t H, int64_t W, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    const PT* scale = static_cast<const PT*>(scalev);
    const PT* shift = static_cast<const PT*>(shiftv);
    T* y = static_cast<T*>(yv);
    constexpr int E = Elem<T>::kPerVec;
    const int64_t plane = H * W, planes = N * C;
    const float inv_plane = (float)(1.0 / (double)plane);
    const bool vec = aligned_to(x, 16) && aligned_to(y, 16) && (plane % E) == 0;
    const int64_t nvec64 = plane / E;
    // (planes that are whole vectors and at least two warp-loads long do better with a warp each: 14x14
    // fp32 measured 46 us with the warp kernel against 52 us flat; 7x7 52 us against 40 us flat)
    if (plane <= 1024 && aligned_to(x, 16) && aligned_to(y, 16) && (plane % E != 0 || plane < 64)) {
        // G planes per CTA: a multiple of the vector length, about 3K elements, at most 1024 planes
        int64_t G = (3072 / plane) / E * E;
        if (G < E) G = E;
        if (G > 1024) G = 1024;
        if (G * plane <= kFlatMaxElems) {
            const int64_t ctas = (planes + G - 1) / G;
            if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
            bn_flat_kernel<T, PT><<<(unsigned)ctas, kFlatThreads, 0, stream>>>(x, scale, shift, y, pooled, planes,
                                                                          (int)plane, (int)G, (int)C, inv_plane);
            return launch_status();
        }
    }
    if (plane <= 1024 || planes > 0x7FFFFFFFLL) {
        const int64_t ctas = (planes + 7) / 8;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        const unsigned grid = (unsigned)ctas;
        if (vec)
            bn_plane_warp_kernel<T, PT, true><<<grid, 256, 0, stream>>>(x, scale, shift, y, pooled, planes, plane, (int)C, inv_plane);
        else
            bn_plane_warp_kernel<T, PT, false><<<grid, 256, 0, stream>>>(x, scale, shift, y, pooled, planes, plane, (int)C, inv_plane);
        return launch_status();
    }
    if (vec && nvec64 <= 0x7FFFFFFF) {
        const int nvec = (int)nvec64;
        // Four vectors per thread per trip; a 56x56 fp32 plane (784 vectors) gets 224 threads
        // and a single trip (196 threads would cover it exactly; 224 is the next warp multiple).
        int threads = ((nvec + 3) / 4 + 31) / 32 * 32;
        if (threads > 512) threads = 512;
        bn_plane_block_kernel<T, PT, 4><<<(unsigned)planes, threads, 0, stream>>>(x, scale, shift, y, pooled, nvec, plane, (int)C, inv_plane);
        return launch_status();
    }
    bn_plane_scalar_kernel<T, PT><<<(unsigned)planes, 256, 0, stream>>>(x, scale, shift, y, pooled, plane, (int)C, inv_plane);
    return launch_status();
}

// ---- channels-last (NHWC memory): x[n][h*w][c] --------------------------------------------------------
// The channel is the innermost index, so the pooled mean is a column sum. A CTA owns one image, a tile of
// TV 16-byte vectors of channels (up to 256 contiguous bytes per row) and a slab of rows; thread t keeps
// column t % TV and walks rows t / TV, t / TV + R, ... of the slab (R = 256 / TV rows per sweep, U of them
// in flight) with its scale / shift values and running column sums in registers. When an image has too
// few (tile) CTAs to fill the GPU its rows are split over a thread-block cluster of up to 8 CTAs: each
// writes its column sums into the first CTA's shared memory (distributed shared memory) once all CTAs of
// the cluster are known to run, one cluster barrier, and the first CTA adds them in rank order. No atomics, no workspace, and for a given call
// shape a fixed summation order.
constexpr int kBnMaxSlabs = 8;      // portable cluster size

template <typename T, typename PT, int TV, int U, bool kCluster>
__global__ void __launch_bounds__(256)
bn_nhwc_kernel(const T* __restrict__ x, const PT* __restrict__ scale, const PT* __restrict__ shift,
               T* __restrict__ y, float* __restrict__ pooled, int64_t hw, int cvec, int tiles, int slabs,
               float inv_hw)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int NT = 256, R = NT / TV;
    __shared__ float part[R][TV * E];
    __shared__ float from_ranks[kCluster ? kBnMaxSlabs : 1][TV * E];
    // "This CTA has started": distributed shared memory may only be touched once every CTA of the cluster is
    // running, so each arrives here and waits (below) just before the first remote store. The row sweep in
    // between hides the wait.
    if (kCluster) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    const int col = threadIdx.x % TV, phase = threadIdx.x / TV;
    const int slab = kCluster ? (int)cluster_rank() : 0;     // consecutive CTAs form a cluster
    const int64_t unit = blockIdx.x / slabs;                 // (image, channel tile)
    const int64_t n = unit / tiles;
    const int tile = (int)(unit - n * tiles);
    const int cv = tile * TV + col;                          // this thread's channel vector
    const bool live = cv < cvec;
    const int64_t C = (int64_t)cvec * E;
    const int64_t slab_rows = (hw + slabs - 1) / slabs;
    const int64_t r_begin = slab * slab_rows;
    const int64_t r_end = r_begin + slab_rows < hw ? r_begin + slab_rows : hw;
    float sc[E], sh[E], acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        sc[e] = live ? param1(scale, (int64_t)cv * E + e) : 0.0f;
        sh[e] = live ? param1(shift, (int64_t)cv * E + e) : 0.0f;
        acc[e] = 0.0f;
    }
    const T* xn = x + n * hw * C + (int64_t)cv * E;
    T* yn = y + n * hw * C + (int64_t)cv * E;
    if (live) {
        for (int64_t r0 = r_begin + phase; r0 < r_end; r0 += (int64_t)R * U) {
            Vec16 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t r = r0 + (int64_t)u * R;
                if (r < r_end) raw[u] = ld_stream(xn + r * C);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t r = r0 + (int64_t)u * R;
                if (r < r_end) {
                    float f[E];
                    Elem<T>::unpack(raw[u], f);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        f[e] = relu_keep_nan(fmaf(f[e], sc[e], sh[e]));
                        acc[e] += f[e];
                    }
                    st_stream(yn + r * C, Elem<T>::pack(f));
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) part[phase][col * E + e] = acc[e];
    __syncthreads();
    float s = 0.0f;
    if (threadIdx.x < TV * E) {
#pragma unroll 8
        for (int r = 0; r < R; ++r) s += part[r][threadIdx.x];
    }
    if (kCluster) {
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");    // every CTA of the cluster has started
        if (threadIdx.x < TV * E) store_to_cluster_cta(&from_ranks[slab][threadIdx.x], 0u, s);
        cluster_barrier();                                   // the stores have landed in the first CTA
        if (slab != 0) return;
        if (threadIdx.x < TV * E) {
            s = 0.0f;
            for (int k = 0; k < slabs; ++k) s += from_ranks[k][threadIdx.x];
        }
    }
    if (threadIdx.x < TV * E) {
        const int64_t c = (int64_t)tile * TV * E + threadIdx.x;
        if (c < C) pooled[n * C + c] = s * inv_hw;
    }
}

// Any channel count / alignment: lanes along channels with scalar loads, warps along rows.
template <typename T, typename PT>
__global__ void __launch_bounds__(256)
bn_nhwc_scalar_kernel(const T* __restrict__ x, const PT* __restrict__ scale, const PT* __restrict__ shift,
                      T* __restrict__ y, float* __restrict__ pooled, int64_t hw, int64_t C, int tiles,
                      float inv_hw)
{
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t n = blockIdx.x / tiles;
    const int64_t c = (blockIdx.x - n * tiles) * 32 + lane;
    float acc = 0.0f;
    if (c < C) {
        const float sc = param1(scale, c), sh = param1(shift, c);
        const T* xn = x + n * hw * C + c;
        T* yn = y + n * hw * C + c;
        for (int64_t r = warp; r < hw; r += 8) {
            const float a = relu_keep_nan(fmaf(Elem<T>::load1(xn + r * C), sc, sh));
            acc += a;
            Elem<T>::store1(yn + r * C, a);
        }
    }
    part[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < C) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += part[w][lane];
        pooled[n * C + c] = s * inv_hw;
    }
}

template <typename T, typename PT>
kop_status_t launch_bn_nhwc(const void* xv, const void* scalev, const void* shiftv, void* yv, float* pooled,
                            int64_t N, int64_t C, int64_t H, int64_t W, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    const PT* scale = static_cast<const PT*>(scalev);
    const PT* shift = static_cast<const PT*>(shiftv);
    T* y = static_cast<T*>(yv);
    constexpr int E = Elem<T>::kPerVec;
    const int64_t hw = H * W;
    const float inv_hw = (float)(1.0 / (double)hw);
    const bool vec = aligned_to(x, 16) && aligned_to(y, 16) && (C % E) == 0;
    if (vec) {
        const int cvec = (int)(C / E);
        // a tile as wide as the channel count allows, up to 16 vectors (one 256-byte run per row)
        int tv = 16;
        while (tv > 1 && tv / 2 >= cvec) tv >>= 1;
        const int tiles = (cvec + tv - 1) / tv;
        // rows split over a cluster until there are ~6 CTAs per SM, each slab keeping at least four sweeps
        const int64_t want = 6LL * sm_count();
        const int64_t sweep = (256 / tv) * 4;
        int slabs = 1;
        while (slabs < kBnMaxSlabs && N * tiles * slabs < want && hw / (2 * slabs) >= 4 * sweep) slabs <<= 1;
        const int64_t grid = N * tiles * slabs;
        if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid, 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)slabs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = slabs > 1 ? 1 : 0;
        cudaError_t err;
#define KOP_BN_NHWC(TVV)                                                                                         \
    err = slabs > 1 ? cudaLaunchKernelEx(&cfg, bn_nhwc_kernel<T, PT, TVV, 4, true>, x, scale, shift, y, pooled, hw,   \
                                         cvec, tiles, slabs, inv_hw)                                              \
                    : cudaLaunchKernelEx(&cfg, bn_nhwc_kernel<T, PT, TVV, 4, false>, x, scale, shift, y, pooled, hw,  \
                                         cvec, tiles, slabs, inv_hw)
        switch (tv) {
        case 16: KOP_BN_NHWC(16); break;
        case 8: KOP_BN_NHWC(8); break;
        case 4: KOP_BN_NHWC(4); break;
        case 2: KOP_BN_NHWC(2); break;
        default: KOP_BN_NHWC(1); break;
        }
#undef KOP_BN_NHWC
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return KOP_ERR_CUDA;
        }
        return launch_status();
    }
    const int64_t tiles = (C + 31) / 32;
    if (N * tiles > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    bn_nhwc_scalar_kernel<T, PT><<<(unsigned)(N * tiles), 256, 0, stream>>>(x, scale, shift, y, pooled, hw, C, (int)tiles, inv_hw);
    return launch_status();
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

kop_status_t bn_entry(const void* x, const void* scale, const void* shift, void* y, float* pooled, int64_t N, int64_t C,
                      int64_t H, int64_t W, const int64_t x_strides[4], const int64_t y_strides[4], kop_dtype_t dtype,
                      kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    if (N < 0 || C <= 0 || H <= 0 || W <= 0) return KOP_ERR_BAD_SHAPE;
    if (N == 0) return KOP_OK;
    if (!x || !scale || !shift || !y || !pooled || !x_strides || !y_strides) return KOP_ERR_NULL_POINTER;
    if (C > 0x7FFFFFFF || H > kMaxElems || W > kMaxElems || N > kMaxElems) return KOP_ERR_BAD_SHAPE;
    if (H > kMaxElems / W) return KOP_ERR_BAD_SHAPE;
    const int64_t plane = H * W;
    if (C > kMaxElems / plane) return KOP_ERR_BAD_SHAPE;
    if (N > 0 && C * plane > kMaxElems / N) return KOP_ERR_BAD_SHAPE;
    // Two layouts, the same for x and y: contiguous NCHW, or channels-last (NHWC memory addressed with
    // NCHW indices). When both descriptions fit (C == 1 or H * W == 1) the layouts coincide.
    const int64_t nchw[4] = {C * plane, plane, W, 1};
    const int64_t nhwc[4] = {C * plane, 1, W * C, C};
    const int64_t dims[4] = {N, C, H, W};
    bool is_nchw = true, is_nhwc = true;
    for (int i = 0; i < 4; ++i) {
        if (dims[i] == 1) continue;                          // the stride of an extent-1 dimension is never used
        is_nchw = is_nchw && x_strides[i] == nchw[i] && y_strides[i] == nchw[i];
        is_nhwc = is_nhwc && x_strides[i] == nhwc[i] && y_strides[i] == nhwc[i];
    }
    if (!is_nchw && !is_nhwc) return KOP_ERR_BAD_STRIDE;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || !aligned_to(scale, elem_size(pdtype)) ||
        !aligned_to(shift, elem_size(pdtype)) ||
        !aligned_to(pooled, 4))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, C * plane, y, C * plane, N, C * plane, esz, true)) return KOP_ERR_BAD_ALIAS;
    kop_status_t st = check_device();
    if (st != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
#define KOP_BN_NHWC_GO(T, PT) launch_bn_nhwc<T, PT>(x, scale, shift, y, pooled, N, C, H, W, s)
#define KOP_BN_GO(T, PT) launch_bn<T, PT>(x, scale, shift, y, pooled, N, C, H, W, s)
    if (!is_nchw) return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_BN_NHWC_GO);
    return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_BN_GO);
#undef KOP_BN_NHWC_GO
#undef KOP_BN_GO
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_bn_relu_avgpool(const void* x, const float* scale, const float* shift,
                                            void* y, float* pooled, int64_t N, int64_t C, int64_t H,
                                            int64_t W, const int64_t x_strides[4],
                                            const int64_t y_strides[4], kop_dtype_t dtype,
                                            kop_stream_t stream)
{
    return kop::bn_entry(x, scale, shift, y, pooled, N, C, H, W, x_strides, y_strides, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_bn_relu_avgpool_ex(const void* x, const void* scale, const void* shift, void* y,
                                               float* pooled, int64_t N, int64_t C, int64_t H, int64_t W,
                                               const int64_t x_strides[4], const int64_t y_strides[4],
                                               kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream)
{
    return kop::bn_entry(x, scale, shift, y, pooled, N, C, H, W, x_strides, y_strides, dtype, param_dtype, stream);
}
