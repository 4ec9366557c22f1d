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

// Planes of at most 1024 elements: L lanes per plane (2 .. 32, a power of two chosen from the plane's size), 32 / L
// planes per warp, eight warps per CTA. A lane sweeps its share of the plane in batches that keep 64 bytes of loads in
// flight, with the widest load that divides a plane's bytes and both tensors' alignment (VB = 16, 8, 4 bytes or one
// element); every value is activated, stored back at the same width and added to the lane's sum, and a butterfly
// over the plane's lanes finishes the mean. No shared memory, no barrier; a fixed summation order.
template <int VB>
struct BnRaw {
    uint32_t w[VB >= 4 ? VB / 4 : 1];
};

template <typename T, typename PT, int VB, int L>
__global__ void __launch_bounds__(256)
bn_plane_group_kernel(const T* __restrict__ x, const PT* __restrict__ scale, const PT* __restrict__ shift,
                      T* __restrict__ y, float* __restrict__ pooled, int64_t planes, int plane, int C, float inv_plane,
                      int64_t p_first = 0)                   // index of plane 0 in the tensor (its channel is p_first mod C)
{
    constexpr int EV = VB / (int)sizeof(T);
    constexpr int U = VB >= 16 ? 4 : (VB == 8 ? 8 : 16);
    constexpr int kPerWarp = 32 / L;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t p = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * kPerWarp + lane / L;
    const bool live = p < planes;
    float sc = 1.0f, sh = 0.0f;
    if (live) {
        const int c = (int)((p_first + p) % C);
        sc = param1(scale, c);
        sh = param1(shift, c);
    }
    const T* xp = x + (live ? p : 0) * plane;
    T* yp = y + (live ? p : 0) * plane;
    const int n = live ? plane / EV : 0;
    float sum = 0.0f;
    for (int base = 0; base < n; base += U * L) {
        BnRaw<VB> raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * L + sub;
            if (v < n) {
                const T* q = xp + (int64_t)v * EV;
                if constexpr (VB == 16) {
                    const Vec16 t = ld_stream(q);
                    raw[k].w[0] = t.w[0], raw[k].w[1] = t.w[1], raw[k].w[2] = t.w[2], raw[k].w[3] = t.w[3];
                } else if constexpr (VB == 8) {
                    const uint2 t = __ldg(reinterpret_cast<const uint2*>(q));
                    raw[k].w[0] = t.x, raw[k].w[1] = t.y;
                } else if constexpr (VB == 4) {
                    raw[k].w[0] = __ldg(reinterpret_cast<const uint32_t*>(q));
                } else {
                    raw[k].w[0] = __ldg(reinterpret_cast<const unsigned short*>(q));
                }
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * L + sub;
            if (v < n) {
                T* q = yp + (int64_t)v * EV;
                if constexpr (VB == 16) {
                    float f[EV];
                    Elem<T>::unpack(Vec16{{raw[k].w[0], raw[k].w[1], raw[k].w[2], raw[k].w[3]}}, f);
#pragma unroll
                    for (int e = 0; e < EV; ++e) {
                        f[e] = relu_keep_nan(fmaf(f[e], sc, sh));
                        sum += f[e];
                    }
                    st_stream(q, Elem<T>::pack(f));
                } else if constexpr (sizeof(T) == 4) {           // one or two fp32
                    float f[EV];
#pragma unroll
                    for (int e = 0; e < EV; ++e) {
                        f[e] = relu_keep_nan(fmaf(__uint_as_float(raw[k].w[e]), sc, sh));
                        sum += f[e];
                    }
                    if constexpr (EV == 2) *reinterpret_cast<float2*>(q) = make_float2(f[0], f[1]);
                    else *q = f[0];
                } else if constexpr (VB >= 4) {                  // two or four 16-bit values
                    T o[EV];
#pragma unroll
                    for (int i = 0; i < VB / 4; ++i) {
                        float2 a;
                        Elem<T>::unpack_pair(raw[k].w[i], a);
                        a.x = relu_keep_nan(fmaf(a.x, sc, sh));
                        a.y = relu_keep_nan(fmaf(a.y, sc, sh));
                        sum += a.x;
                        sum += a.y;
                        Elem<T>::store1(&o[2 * i], a.x);
                        Elem<T>::store1(&o[2 * i + 1], a.y);
                    }
                    if constexpr (VB == 8) *reinterpret_cast<uint2*>(q) = *reinterpret_cast<const uint2*>(o);
                    else *reinterpret_cast<uint32_t*>(q) = *reinterpret_cast<const uint32_t*>(o);
                } else {                                         // one 16-bit value
                    float2 a;
                    Elem<T>::unpack_pair(raw[k].w[0], a);
                    a.x = relu_keep_nan(fmaf(a.x, sc, sh));
                    sum += a.x;
                    Elem<T>::store1(q, a.x);
                }
            }
        }
    }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        sum = (lane & o) ? other + sum : sum + other;            // the lower lane's term first: both lanes agree
    }
    if (live && sub == 0) pooled[p] = sum * inv_plane;
}

// ---- planes that are not whole vectors, bundled -----------------------------------------------------------------
// A 7 x 7 plane is 196 bytes of fp32 or 98 of bf16: nothing wider than one element divides it, and element accesses
// are bound by the L1 (7 x 7 fp32 4.4 TB/s, bf16 2.1; the head of every ResNet). B consecutive planes (2, 4 or 8)
// together are a whole number of 16-byte vectors, so a team of L lanes takes such a bundle: 16-byte loads and stores
// over the bundle, every vector's elements in at most two planes (scale / shift picked per element between the two),
// the activations parked in shared memory as fp32, and after a warp barrier one lane per plane adds its plane's
// values in index order.
__device__ __forceinline__ int bn_div_small(int i, int d, float inv_d)
{
    int q = (int)((float)i * inv_d);
    const int r = i - q * d;
    q += (r >= d) ? 1 : 0;
    q -= (r < 0) ? 1 : 0;
    return q;
}

template <typename T, typename PT, int L, int NV>
__global__ void __launch_bounds__(256)
bn_bundle_kernel(const T* __restrict__ x, const PT* __restrict__ scale, const PT* __restrict__ shift,
                 T* __restrict__ y, float* __restrict__ pooled, int64_t bundles, int B, int plane, int nvec, int C,
                 float inv_plane, float inv_plane_f, int tile_floats)
{
    constexpr int E = Elem<T>::kPerVec;
    extern __shared__ __align__(16) float bn_tile[];
    const int sub = threadIdx.x & (L - 1), team = threadIdx.x / L;
    const int64_t b = (int64_t)blockIdx.x * (blockDim.x / L) + team;
    const bool live = b < bundles;
    float* tile = bn_tile + team * tile_floats;
    const int64_t p0 = (live ? b : 0) * B;
    const T* xb = x + p0 * plane;
    T* yb = y + p0 * plane;
    const int c_p0 = (int)(p0 % C);
    const int n = live ? nvec : 0;
    Vec16 raw[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int v = k * L + sub;
        if (v < n) raw[k] = ld_stream(xb + (int64_t)v * E);
    }
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int v = k * L + sub;
        if (v < n) {
            const int i0 = v * E;
            const int pl = bn_div_small(i0, plane, inv_plane_f);
            const int left = plane - (i0 - pl * plane);              // elements of this vector in plane pl
            int c = c_p0 + pl;
            while (c >= C) c -= C;
            const float sc0 = param1(scale, c), sh0 = param1(shift, c);
            float sc1 = sc0, sh1 = sh0;
            if (left < E) {
                const int c1 = c + 1 == C ? 0 : c + 1;
                sc1 = param1(scale, c1);
                sh1 = param1(shift, c1);
            }
            float f[E];
            Elem<T>::unpack(raw[k], f);
#pragma unroll
            for (int e = 0; e < E; ++e) f[e] = relu_keep_nan(fmaf(f[e], e < left ? sc0 : sc1, e < left ? sh0 : sh1));
            float4* dst = reinterpret_cast<float4*>(tile + i0);
#pragma unroll
            for (int q = 0; q < E / 4; ++q) dst[q] = make_float4(f[4 * q], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
            st_stream(yb + i0, Elem<T>::pack(f));
        }
    }
    __syncwarp();
    if (live && sub < B) {
        const float* t = tile + sub * plane;
        float s = 0.0f;
        for (int j = 0; j < plane; ++j) s += t[j];
        pooled[p0 + sub] = s * inv_plane;
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
    // planes of at most 1024 elements: lanes per plane. (A warp per plane, and for planes that are not whole vectors
    // runs of planes copied flat through shared memory, were here before: fp32 28 x 28 / 14 x 14 / 7 x 7 planes 5.4 / 5.1 /
    // 3.2 TB/s, bf16 3.8 / 2.6 / 1.8; now 6.1 / 6.3 / 4.0 and 5.8 / 5.5 / 1.9.)
    // planes that nothing wider than four bytes divides, in bundles of 4 or 8 (7 x 7: 49 vectors a bundle for every data
    // type; fp32 / bf16 TB/s 4.4 / 2.1 from the lanes-per-plane kernel, 5.6 / 3.1 here). Planes that 8-byte accesses
    // divide stay there (bf16 14 x 14 and 10 x 10: 6.1 / 5.4 against 2.9 / 3.4 in bundles of two).
    if (plane <= 256 && plane >= E && aligned_to(x, 16) && aligned_to(y, 16) && (plane * sizeof(T)) % 8 != 0) {
        const int pbytes = (int)plane * (int)sizeof(T);
        int B = 2;
        while ((B * pbytes) % 16 != 0) B *= 2;                       // at most 8: a plane is a whole number of elements
        const int nvec = B * pbytes / 16;
        const int64_t bundles = planes / B, rest = planes - bundles * B;
        // fp32: eight lanes a bundle, eight vectors a lane. 16-bit data: sixteen lanes, four vectors a lane, 46 registers
        // instead of 64 (bf16 7 x 7 with eight lanes: warps active 46 %, long-scoreboard stalls first, 3.1 TB/s; 4.2 this
        // way; fp32 the other way round, 5.6 against 5.1). Beyond 64 vectors a bundle: sixteen lanes, eight vectors.
        const bool wide = sizeof(T) == 2 || nvec > 64;
        const int L = wide ? 16 : 8;
        const int tile_floats = (B * (int)plane + 3) / 4 * 4;
        int threads = 256;                                           // the teams' tiles stay within the default 48 KB
        while (threads > 32 && (size_t)(threads / L) * tile_floats * sizeof(float) > 46 * 1024) threads /= 2;
        const int teams = threads / L;
        const int64_t ctas = (bundles + teams - 1) / teams;
        const size_t smem = (size_t)teams * tile_floats * sizeof(float);
        if (nvec <= 128 && bundles > 0 && ctas <= 0x7FFFFFFFLL && smem <= 46 * 1024) {
            const float inv_plane_f = 1.0f / (float)plane;
#define KOP_BN_BUNDLE(LL, NVV) \
    bn_bundle_kernel<T, PT, LL, NVV><<<(unsigned)ctas, threads, smem, stream>>>(x, scale, shift, y, pooled, bundles, B, (int)plane, nvec, (int)C, inv_plane, inv_plane_f, tile_floats)
            if (!wide) KOP_BN_BUNDLE(8, 8);
            else if (nvec <= 64) KOP_BN_BUNDLE(16, 4);
            else KOP_BN_BUNDLE(16, 8);
#undef KOP_BN_BUNDLE
            if (rest > 0) {
                // the planes after the last whole bundle: lanes per plane with element accesses
                const int64_t pf = bundles * B;
                bn_plane_group_kernel<T, PT, (int)sizeof(T), 8><<<(unsigned)((rest + 31) / 32), 256, 0, stream>>>(
                    x + pf * plane, scale, shift, y + pf * plane, pooled + pf, rest, (int)plane, (int)C, inv_plane, pf);
            }
            return launch_status();
        }
    }
    if (plane <= 1024 && planes <= 0x7FFFFFFFLL * 8) {
        const int pbytes = (int)plane * (int)sizeof(T);
        const int vb = (pbytes % 16 == 0 && aligned_to(x, 16) && aligned_to(y, 16)) ? 16
                       : (pbytes % 8 == 0 && aligned_to(x, 8) && aligned_to(y, 8)) ? 8
                       : (pbytes % 4 == 0 && aligned_to(x, 4) && aligned_to(y, 4)) ? 4 : (int)sizeof(T);
        // loads a lane: 64 bytes in flight with 16- and 8-byte units; eight narrower ones, so that more lanes share a plane
        // and a warp's load covers longer runs (7 x 7 fp32 / bf16 planes: 4.4 / 2.1 TB/s with sixteen, 5.0 / 2.6 with eight)
        const int units = pbytes / vb, per_lane = vb >= 16 ? 4 : 8;
        int L = 2;
        while (L < 32 && L * per_lane < units) L *= 2;
        const int per_cta = 8 * (32 / L);
        const int64_t ctas = (planes + per_cta - 1) / per_cta;
        if (ctas <= 0x7FFFFFFFLL) {
#define KOP_BN_GROUP_L(V, LL) \
    bn_plane_group_kernel<T, PT, V, LL><<<(unsigned)ctas, 256, 0, stream>>>(x, scale, shift, y, pooled, planes, (int)plane, (int)C, inv_plane)
#define KOP_BN_GROUP(V)                           \
    do {                                          \
        if (L == 2) KOP_BN_GROUP_L(V, 2);         \
        else if (L == 4) KOP_BN_GROUP_L(V, 4);    \
        else if (L == 8) KOP_BN_GROUP_L(V, 8);    \
        else if (L == 16) KOP_BN_GROUP_L(V, 16);  \
        else KOP_BN_GROUP_L(V, 32);               \
    } while (0)
            if (vb == 16) KOP_BN_GROUP(16);
            else if (vb == 8) KOP_BN_GROUP(8);
            else if (vb == 4) KOP_BN_GROUP(4);
            else KOP_BN_GROUP((int)sizeof(T));
#undef KOP_BN_GROUP
#undef KOP_BN_GROUP_L
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
