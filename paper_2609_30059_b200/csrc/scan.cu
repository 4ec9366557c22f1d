// kop_cumsum_rows: running sums along each row (inclusive or exclusive, forward or reverse, optionally
// masked), one HBM pass.
//
// A CTA owns a row. Vectors are dealt to threads round-robin (vector k * NT + t of a tile goes to thread t),
// so every warp load is one contiguous 512-byte run; the scan order is then (k, thread, element). Each
// thread scans its vector, the warp scans the vector totals with shuffles, lane 31 publishes the warp
// total, and after ONE barrier every warp scans the published totals of its tile for itself (no second
// barrier, no serial thread). Rows longer than a tile (4 vectors x up to 1024 threads) loop over tiles
// with a running carry; the published totals are double-buffered so the loop keeps one barrier per tile.
// A reverse scan is the same code on mirrored indices (vector nvec-1-v, elements of a vector backwards).
// All prefixes are formed by shifting inclusive sums, never by subtracting an element back out, so an
// infinity or NaN affects exactly the outputs at and after its position.
#include "kop_common.cuh"

namespace kop {
namespace {

constexpr int kScanU = 4;

__device__ __forceinline__ float warp_inclusive(float v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Mask bytes of one vector (E of them), widened to a bit per element. Requires E-byte alignment.
template <int E>
__device__ __forceinline__ unsigned mask_bits(const unsigned char* p)
{
    unsigned bits = 0;
    if (E == 4) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(p));
#pragma unroll
        for (int e = 0; e < 4; ++e) bits |= ((w >> (8 * e)) & 0xFFu) ? (1u << e) : 0u;
    } else {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(p));
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            bits |= ((w.x >> (8 * e)) & 0xFFu) ? (1u << e) : 0u;
            bits |= ((w.y >> (8 * e)) & 0xFFu) ? (1u << (e + 4)) : 0u;
        }
    }
    return bits;
}

template <typename T, bool kMask, bool kRev>
__global__ void __launch_bounds__(1024)
cumsum_row_kernel(const T* __restrict__ x, const unsigned char* __restrict__ mask, T* __restrict__ y, int nvec,
                  int64_t x_stride, int64_t m_stride, int64_t y_stride, int exclusive)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int U = kScanU;
    __shared__ float totals[2][U][32];

    const int NT = blockDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = NT >> 5;
    const T* xr = x + (int64_t)blockIdx.x * x_stride;
    T* yr = y + (int64_t)blockIdx.x * y_stride;
    const unsigned char* mr = kMask ? mask + (int64_t)blockIdx.x * m_stride : nullptr;
    const int tile_vecs = U * NT;

    float carry = 0.0f;
    int buf = 0;
    for (int base = 0; base < nvec; base += tile_vecs, buf ^= 1) {
        // loads of the whole tile first: U vectors in flight per thread
        Vec16 raw[U];
        unsigned keep[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int lv = base + k * NT + (int)threadIdx.x;         // position in scan order
            const int pv = kRev ? nvec - 1 - lv : lv;                // position in memory
            if (lv < nvec) {
                raw[k] = ld_stream(xr + (int64_t)pv * E);
                keep[k] = kMask ? mask_bits<E>(mr + (int64_t)pv * E) : 0xFFu;
            } else {
                raw[k] = Vec16{{0u, 0u, 0u, 0u}};
                keep[k] = 0u;
            }
        }
        // scan inside each vector (in scan order), then across the warp
        float f[U][E];       // running sums inside the vector (inclusive or exclusive as asked)
        float tot[U], inc[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float v[E];
            Elem<T>::unpack(raw[k], v);
            float run = 0.0f;
#pragma unroll
            for (int s = 0; s < E; ++s) {
                const int e = kRev ? E - 1 - s : s;                  // element visited at scan step s
                const float val = (keep[k] >> e) & 1u ? v[e] : 0.0f;
                f[k][e] = exclusive ? run : run + val;
                run += val;
            }
            tot[k] = run;
        }
#pragma unroll
        for (int k = 0; k < U; ++k) inc[k] = tot[k];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const float t = __shfl_up_sync(0xFFFFFFFFu, inc[k], o);
                if (lane >= o) inc[k] += t;
            }
        }
        if (lane == 31) {
#pragma unroll
            for (int k = 0; k < U; ++k) totals[buf][k][warp] = inc[k];
        }
        __syncthreads();
        float batch_base = carry;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            // prefix of this thread inside its warp: the left neighbour's inclusive sum
            float before = __shfl_up_sync(0xFFFFFFFFu, inc[k], 1);
            if (lane == 0) before = 0.0f;
            // every warp scans the tile's warp totals for itself
            const float t = lane < nw ? totals[buf][k][lane] : 0.0f;
            const float S = warp_inclusive(t, lane);
            float warps_before = __shfl_sync(0xFFFFFFFFu, S, warp > 0 ? warp - 1 : 0);
            if (warp == 0) warps_before = 0.0f;
            const float batch_total = __shfl_sync(0xFFFFFFFFu, S, 31);
            const float prefix = (batch_base + warps_before) + before;
            const int lv = base + k * NT + (int)threadIdx.x;
            if (lv < nvec) {
                const int pv = kRev ? nvec - 1 - lv : lv;
                float o[E];
#pragma unroll
                for (int e = 0; e < E; ++e) o[e] = prefix + f[k][e];
                st_stream(yr + (int64_t)pv * E, Elem<T>::pack(o));
            }
            batch_base += batch_total;
        }
        carry = batch_base;
    }
}

// Short rows: L lanes of a warp per row (L = 1 .. 32), 32 / L rows per warp, eight warps per CTA; the scan
// across the row's lanes is a shuffle scan of width L, with no shared memory and no barrier; a row longer than
// 4 L vectors takes several batches with a running carry.
template <typename T, bool kMask, bool kRev, int L, bool kOne>
__global__ void __launch_bounds__(256)
cumsum_group_kernel(const T* __restrict__ x, const unsigned char* __restrict__ mask, T* __restrict__ y, int64_t rows,
                    int nvec, int64_t x_stride, int64_t m_stride, int64_t y_stride, int exclusive)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int U = kScanU;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t row = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * (32 / L) + lane / L;
    const bool live = row < rows;
    const int64_t r = live ? row : 0;
    const T* xr = x + r * x_stride;
    T* yr = y + r * y_stride;
    const unsigned char* mr = kMask ? mask + r * m_stride : nullptr;
    const int n = live ? nvec : 0;
    float batch_base = 0.0f;                                         // running carry over the batches of a row
    // every lane of the warp runs the same number of batches (the shuffles need all of them); kOne: the row is
    // one batch (nvec <= 4 L), no loop
    for (int base = 0; base < (kOne ? 1 : nvec); base += U * L) {
        Vec16 raw[U];
        unsigned keep[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int lv = base + k * L + sub;                       // position in scan order
            const int pv = kRev ? n - 1 - lv : lv;                   // position in memory
            if (lv < n) {
                raw[k] = ld_stream(xr + (int64_t)pv * E);
                keep[k] = kMask ? mask_bits<E>(mr + (int64_t)pv * E) : 0xFFu;
            } else {
                raw[k] = Vec16{{0u, 0u, 0u, 0u}};
                keep[k] = 0u;
            }
        }
        float f[U][E], inc[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float v[E];
            Elem<T>::unpack(raw[k], v);
            float run = 0.0f;
#pragma unroll
            for (int s = 0; s < E; ++s) {
                const int e = kRev ? E - 1 - s : s;
                const float val = (keep[k] >> e) & 1u ? v[e] : 0.0f;
                f[k][e] = exclusive ? run : run + val;
                run += val;
            }
            inc[k] = run;
        }
#pragma unroll
        for (int o = 1; o < L; o <<= 1) {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const float t = __shfl_up_sync(0xFFFFFFFFu, inc[k], o, L);
                if (sub >= o) inc[k] += t;
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float before = __shfl_up_sync(0xFFFFFFFFu, inc[k], 1, L);
            if (sub == 0) before = 0.0f;
            const float batch_total = __shfl_sync(0xFFFFFFFFu, inc[k], L - 1, L);
            const float prefix = batch_base + before;
            const int lv = base + k * L + sub;
            if (lv < n) {
                const int pv = kRev ? n - 1 - lv : lv;
                float o[E];
#pragma unroll
                for (int e = 0; e < E; ++e) o[e] = prefix + f[k][e];
                st_stream(yr + (int64_t)pv * E, Elem<T>::pack(o));
            }
            batch_base += batch_total;
        }
    }
}

// Any length / alignment: every thread owns a contiguous segment of the row in scan order; pass 1 sums the
// segments, one block scan orders them, pass 2 walks each segment again and writes the outputs.
template <typename T>
__global__ void __launch_bounds__(256)
cumsum_row_scalar_kernel(const T* __restrict__ x, const unsigned char* __restrict__ mask, T* __restrict__ y,
                         int64_t cols, int64_t x_stride, int64_t m_stride, int64_t y_stride, int exclusive,
                         int reverse)
{
    __shared__ float totals[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const T* xr = x + (int64_t)blockIdx.x * x_stride;
    T* yr = y + (int64_t)blockIdx.x * y_stride;
    const unsigned char* mr = mask != nullptr ? mask + (int64_t)blockIdx.x * m_stride : nullptr;
    const int64_t seg = (cols + blockDim.x - 1) / blockDim.x;
    const int64_t s0 = (int64_t)threadIdx.x * seg;
    const int64_t s1 = s0 + seg < cols ? s0 + seg : cols;
    float sum = 0.0f;
    for (int64_t s = s0; s < s1; ++s) {
        const int64_t j = reverse ? cols - 1 - s : s;
        const float v = Elem<T>::load1(xr + j);
        sum += (mr == nullptr || mr[j] != 0) ? v : 0.0f;
    }
    const float inc = warp_inclusive(sum, lane);
    if (lane == 31) totals[warp] = inc;
    __syncthreads();
    float before = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
    if (lane == 0) before = 0.0f;
    const float t = lane < (int)(blockDim.x >> 5) ? totals[lane] : 0.0f;
    const float S = warp_inclusive(t, lane);
    float warps_before = __shfl_sync(0xFFFFFFFFu, S, warp > 0 ? warp - 1 : 0);
    if (warp == 0) warps_before = 0.0f;
    float run = warps_before + before;
    for (int64_t s = s0; s < s1; ++s) {
        const int64_t j = reverse ? cols - 1 - s : s;
        const float v = Elem<T>::load1(xr + j);
        const float val = (mr == nullptr || mr[j] != 0) ? v : 0.0f;
        Elem<T>::store1(yr + j, exclusive ? run : run + val);
        run += val;
    }
}

template <typename T>
kop_status_t launch_cumsum(const void* x, const unsigned char* mask, void* y, int64_t rows, int64_t cols,
                           int64_t xs, int64_t ms, int64_t ys, int exclusive, int reverse, cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    const T* xt = static_cast<const T*>(x);
    T* yt = static_cast<T*>(y);
    const bool vec = vec_ok(x, cols, xs, sizeof(T)) && vec_ok(y, cols, ys, sizeof(T)) && cols / E <= 0x7FFFFFFF &&
                     (mask == nullptr || (aligned_to(mask, E) && ms % E == 0));
    // Lanes of a warp per row: rows of at most 128 vectors in one batch (2 to 32 lanes); 16-bit rows up to 2048
    // vectors a warp each with a carry (5.0 - 5.1 TB/s at 2048 - 16384 columns against 4.0 - 4.6 for a CTA per
    // row; fp32 rows of that length do better with the CTA: 6.2 - 6.4 TB/s).
    if (vec && cols / E <= (sizeof(T) == 2 ? 2048 : 128)) {
        const int nvec = (int)(cols / E);
        const int lanes = nvec > 64 ? 32 : nvec > 32 ? 16 : nvec > 16 ? 8 : nvec > 8 ? 4 : nvec > 4 ? 2 : 1;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
        const unsigned grid = (unsigned)ctas;
#define KOP_SCAN_GROUP_L(M, R, L, ONE) \
    cumsum_group_kernel<T, M, R, L, ONE><<<grid, 256, 0, stream>>>(xt, mask, yt, rows, nvec, xs, ms, ys, exclusive)
#define KOP_SCAN_GROUP(L, ONE)                                                     \
    do {                                                                           \
        if (mask != nullptr) {                                                     \
            if (reverse) KOP_SCAN_GROUP_L(true, true, L, ONE);                     \
            else KOP_SCAN_GROUP_L(true, false, L, ONE);                            \
        } else {                                                                   \
            if (reverse) KOP_SCAN_GROUP_L(false, true, L, ONE);                    \
            else KOP_SCAN_GROUP_L(false, false, L, ONE);                           \
        }                                                                          \
    } while (0)
        switch (lanes) {
        case 32:
            if (nvec <= 128) KOP_SCAN_GROUP(32, true);
            else KOP_SCAN_GROUP(32, false);
            break;
        case 16: KOP_SCAN_GROUP(16, true); break;
        case 8: KOP_SCAN_GROUP(8, true); break;
        case 4: KOP_SCAN_GROUP(4, true); break;
        case 2: KOP_SCAN_GROUP(2, true); break;
        default: KOP_SCAN_GROUP(1, true); break;
        }
#undef KOP_SCAN_GROUP_L
#undef KOP_SCAN_GROUP
        return launch_status();
    }
    if (vec) {
        const int nvec = (int)(cols / E);
        int threads = ((nvec + kScanU - 1) / kScanU + 31) / 32 * 32;
        if (threads > 1024) threads = 1024;
        const unsigned grid = (unsigned)rows;
#define KOP_SCAN_LAUNCH(M, R) \
    cumsum_row_kernel<T, M, R><<<grid, threads, 0, stream>>>(xt, mask, yt, nvec, xs, ms, ys, exclusive)
        if (mask != nullptr) {
            if (reverse) KOP_SCAN_LAUNCH(true, true);
            else KOP_SCAN_LAUNCH(true, false);
        } else {
            if (reverse) KOP_SCAN_LAUNCH(false, true);
            else KOP_SCAN_LAUNCH(false, false);
        }
#undef KOP_SCAN_LAUNCH
        return launch_status();
    }
    cumsum_row_scalar_kernel<T><<<(unsigned)rows, 256, 0, stream>>>(xt, mask, yt, cols, xs, ms, ys, exclusive, reverse);
    return launch_status();
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_cumsum_rows(const void* x, const unsigned char* mask, void* y, int64_t rows,
                                        int64_t cols, int64_t x_row_stride, int64_t mask_row_stride,
                                        int64_t y_row_stride, int exclusive, int reverse, kop_dtype_t dtype,
                                        kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;                 // one CTA per row
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, cols, rows)) != KOP_OK) return st;
    if (mask != nullptr && (st = check_row_stride(mask_row_stride, cols, rows)) != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz)) return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, cols, esz, true)) return KOP_ERR_BAD_ALIAS;
    if (mask != nullptr) {
        // the mask is read while y is written: it must not overlap y
        uintptr_t m0, m1, y0, y1;
        span_of(mask, rows, cols, mask_row_stride, 1, &m0, &m1);
        span_of(y, rows, cols, y_row_stride, esz, &y0, &y1);
        if (!(m1 <= y0 || y1 <= m0)) return KOP_ERR_BAD_ALIAS;
    }
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    const int ex = exclusive != 0, rv = reverse != 0;
    return dtype == KOP_F32
               ? launch_cumsum<float>(x, mask, y, rows, cols, x_row_stride, mask_row_stride, y_row_stride, ex, rv, s)
               : dtype == KOP_BF16 ? launch_cumsum<__nv_bfloat16>(x, mask, y, rows, cols, x_row_stride, mask_row_stride, y_row_stride, ex, rv, s)
               : launch_cumsum<__half>(x, mask, y, rows, cols, x_row_stride, mask_row_stride, y_row_stride, ex, rv, s);
}
