// kop_row_scale and kop_matvec_bias: the two memory-bound kernels that the paper's case studies
// reduce a GEMM to (diag(a) * B -> row scaling; Linear -> Sum -> ... -> a mat-vec with precomputed
// column sums). Both stream their matrix once.
#include "kop_common.cuh"

namespace kop {
namespace {

// ---- out[i, :] = a[i] * B[i, :] -----------------------------------------------------------------------
// A CTA covers U * blockDim.x consecutive vectors of one row; a[i] is one broadcast load per CTA.
template <typename T, int U, bool kFull>
__global__ void __launch_bounds__(256)
row_scale_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, int nvec,
                 int tiles_per_row, int64_t b_stride, int64_t o_stride)
{
    constexpr int E = Elem<T>::kPerVec;
    const unsigned urow = blockIdx.x / (unsigned)tiles_per_row;
    const int tile = (int)(blockIdx.x - urow * (unsigned)tiles_per_row);
    const int64_t row = urow;
    const float s = Elem<T>::load1(a + row);
    const T* br = b + row * b_stride;
    T* orow = out + row * o_stride;
    const int v0 = tile * (U * blockDim.x) + threadIdx.x;
    Vec16 raw[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int v = v0 + k * blockDim.x;
        if (kFull || v < nvec) raw[k] = ld_stream(br + (int64_t)v * E);
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int v = v0 + k * blockDim.x;
        if (kFull || v < nvec) {
            float f[E];
            Elem<T>::unpack(raw[k], f);
#pragma unroll
            for (int e = 0; e < E; ++e) f[e] *= s;
            st_stream(orow + (int64_t)v * E, Elem<T>::pack(f));
        }
    }
}

// Rows shorter than a tile (or with a mostly empty last tile): the CTA's U * blockDim.x vectors are taken in
// row-major order across rows; a[row] is then one load per vector (L1-resident: neighbours share it).
template <typename T, int U>
__global__ void __launch_bounds__(256)
row_scale_flat_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, int nvec,
                      int64_t nvec_total, int64_t b_stride, int64_t o_stride)
{
    constexpr int E = Elem<T>::kPerVec;
    const int64_t g0 = (int64_t)blockIdx.x * (U * blockDim.x) + threadIdx.x;
    int64_t row[U];
    int v[U];
    bool live[U];
    Vec16 raw[U];
    float s[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int64_t g = g0 + k * blockDim.x;
        live[k] = g < nvec_total;
        flat_position(live[k] ? g : 0, nvec, &row[k], &v[k]);
        if (live[k]) {
            raw[k] = ld_stream(b + row[k] * b_stride + (int64_t)v[k] * E);
            s[k] = Elem<T>::load1(a + row[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
        if (live[k]) {
            float f[E];
            Elem<T>::unpack(raw[k], f);
#pragma unroll
            for (int e = 0; e < E; ++e) f[e] *= s[k];
            st_stream(out + row[k] * o_stride + (int64_t)v[k] * E, Elem<T>::pack(f));
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
row_scale_scalar_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, int64_t rows,
                        int64_t cols, int64_t b_stride, int64_t o_stride)
{
    const int64_t total = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols, j = i - r * cols;
        Elem<T>::store1(out + r * o_stride + j, Elem<T>::load1(a + r) * Elem<T>::load1(b + r * b_stride + j));
    }
}

// ---- out[i] = sum_k X[i,k] * w[k] + b_sum -------------------------------------------------------------
// A CTA takes R consecutive rows. Per trip every thread fetches the fp32 weights of U vector columns
// once and multiplies them into those columns of all R rows, so the weight traffic through L1 is 1/R
// of what one row per CTA would need.
template <typename T, int R, int U, bool kWide>
__global__ void __launch_bounds__(256)
matvec_rows_kernel(const T* __restrict__ x, const float* __restrict__ w, float b_sum, float* __restrict__ out,
                   int64_t rows, int nvec, int64_t x_stride)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;
    __shared__ float red[R][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * R;
    float2 acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = make_float2(0.0f, 0.0f);
    // U vector columns per trip: U * R matrix loads are in flight before the first FMA.
    for (int v0 = threadIdx.x; v0 < nvec; v0 += U * blockDim.x) {
        Vec16 raw[U][R];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * blockDim.x;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (v < nvec && row0 + r < rows) raw[u][r] = ld_stream(x + (row0 + r) * x_stride + (int64_t)v * E);
                else raw[u][r] = Vec16{{0u, 0u, 0u, 0u}};
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * blockDim.x;
            float2 wv[P];
            if (v < nvec) load_params<E, kWide>(w + (int64_t)v * E, wv);
            else {
#pragma unroll
                for (int q = 0; q < P; ++q) wv[q] = make_float2(0.0f, 0.0f);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float2 f[P];
                Elem<T>::unpack2(raw[u][r], f);
#pragma unroll
                for (int q = 0; q < P; ++q) acc[r] = __ffma2_rn(f[q], wv[q], acc[r]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const float s = warp_sum(acc[r].x + acc[r].y);
        if (lane == 0) red[r][warp] = s;
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float s = warp_sum(lane < nw ? red[r][lane] : 0.0f);
            if (lane == 0 && row0 + r < rows) out[row0 + r] = s + b_sum;
        }
    }
}

// Short rows (at most 4 L vectors): L lanes of a warp per row, 32 / L rows per warp, eight warps per CTA; the
// dot product is a butterfly over the row's lanes.
template <typename T, int L>
__global__ void __launch_bounds__(256)
matvec_group_kernel(const T* __restrict__ x, const float* __restrict__ w, float b_sum, float* __restrict__ out,
                    int64_t rows, int nvec, int64_t x_stride)
{
    constexpr int E = Elem<T>::kPerVec, P = E / 2, VPL = 4;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t row = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * (32 / L) + lane / L;
    const bool live = row < rows;
    const T* xr = x + (live ? row : 0) * x_stride;
    Vec16 raw[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        raw[k] = Vec16{{0u, 0u, 0u, 0u}};
        if (live && v < nvec) raw[k] = ld_stream(xr + (int64_t)v * E);
    }
    float2 acc = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        if (v < nvec) {
            float2 wv[P], f[P];
            load_params<E, false>(w + (int64_t)v * E, wv);
            Elem<T>::unpack2(raw[k], f);
#pragma unroll
            for (int q = 0; q < P; ++q) acc = __ffma2_rn(f[q], wv[q], acc);
        }
    }
    float s = acc.x + acc.y;
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (live && sub == 0) out[row] = s + b_sum;
}

template <typename T>
__global__ void __launch_bounds__(256)
matvec_scalar_kernel(const T* __restrict__ x, const float* __restrict__ w, float b_sum, float* __restrict__ out,
                     int64_t K, int64_t x_stride)
{
    __shared__ float red[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    float acc = 0.0f;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) acc = fmaf(Elem<T>::load1(xr + k), __ldg(w + k), acc);
    acc = block_sum(acc, red);
    if (threadIdx.x == 0) out[row] = acc + b_sum;
}

inline unsigned scalar_grid(int64_t total)
{
    const int64_t want = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 32;
    return (unsigned)(want < cap ? (want > 0 ? want : 1) : cap);
}

template <typename T>
kop_status_t launch_row_scale(const void* av, const void* bv, void* ov, int64_t rows, int64_t cols, int64_t bs,
                              int64_t os, cudaStream_t stream)
{
    const T* a = static_cast<const T*>(av);
    const T* b = static_cast<const T*>(bv);
    T* out = static_cast<T*>(ov);
    constexpr int E = Elem<T>::kPerVec;
    const bool vec = vec_ok(b, cols, bs, sizeof(T)) && vec_ok(out, cols, os, sizeof(T));
    const int64_t nvec64 = cols / E;
    if (vec && nvec64 <= 0x7FFFFFFF) {
        const int nvec = (int)nvec64;
        // 256 threads x 2 vectors: 24.1 us on 4096 x 4096 fp32 against 24.5 (128 x 4) and 25.5 (128 x 1); a launch of this
        // size is about 3.5 us of ramp and tail whatever the tiling (8192 x 8192 runs at the copy peak)
        const int threads = 256;
        constexpr int U = 2;
        const int tiles = (nvec + threads * U - 1) / (threads * U);
        if (nvec < threads * U || ((int64_t)tiles * threads * U - nvec) * 4 > nvec) {
            const int64_t total = rows * nvec, fgrid = (total + 256 * U - 1) / (256 * U);
            if (fgrid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
            row_scale_flat_kernel<T, U><<<(unsigned)fgrid, 256, 0, stream>>>(a, b, out, nvec, total, bs, os);
            return launch_status();
        }
        const int64_t grid = rows * tiles;
        if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        if (nvec % (threads * U) == 0)
            row_scale_kernel<T, U, true><<<(unsigned)grid, threads, 0, stream>>>(a, b, out, nvec, tiles, bs, os);
        else
            row_scale_kernel<T, U, false><<<(unsigned)grid, threads, 0, stream>>>(a, b, out, nvec, tiles, bs, os);
        return launch_status();
    }
    row_scale_scalar_kernel<T><<<scalar_grid(rows * cols), 256, 0, stream>>>(a, b, out, rows, cols, bs, os);
    return launch_status();
}

template <typename T>
kop_status_t launch_matvec(const void* xv, const float* w, float b_sum, float* out, int64_t M, int64_t K,
                           int64_t xs, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    constexpr int E = Elem<T>::kPerVec;
    const bool vec = vec_ok(x, K, xs, sizeof(T)) && aligned_to(w, 16);
    const int64_t nvec64 = K / E;
    if (vec && nvec64 <= 0x7FFFFFFF) {
        const int nvec = (int)nvec64;
        if (nvec <= 128) {                                   // short rows: lanes of a warp per row
            const int lanes = nvec > 64 ? 32 : nvec > 32 ? 16 : nvec > 16 ? 8 : nvec > 8 ? 4 : 2;
            const int64_t rows_per_cta = 8 * (32 / lanes);
            const int64_t ctas = (M + rows_per_cta - 1) / rows_per_cta;
            if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
#define KOP_MV_GROUP(L) matvec_group_kernel<T, L><<<(unsigned)ctas, 256, 0, stream>>>(x, w, b_sum, out, M, nvec, xs)
            switch (lanes) {
            case 32: KOP_MV_GROUP(32); break;
            case 16: KOP_MV_GROUP(16); break;
            case 8: KOP_MV_GROUP(8); break;
            case 4: KOP_MV_GROUP(4); break;
            default: KOP_MV_GROUP(2); break;
            }
#undef KOP_MV_GROUP
            return launch_status();
        }
        // Two rows per CTA, 64 threads, four vector columns per trip (eight matrix loads in flight per
        // thread). Measured on [32768, 4096] bf16: 43.5 us; eight rows per CTA 59 us, one row 47.7 us,
        // a warp-per-row variant without barriers 44.3 us.
        constexpr int R = 2;
        const int64_t grid = (M + R - 1) / R;
        if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        // long rows get up to 256 threads (a 64-thread CTA would loop 64 times over a 65536-column fp32 row with too
        // few CTAs to fill the GPU: 1.2 TB/s against 4.0; rows of 16384 columns 4.0 - 4.4 against 4.9 - 5.5)
        const int cap = nvec > 1024 ? 256 : 64;
        int threads = 32;
        while (threads < cap && threads * 4 < nvec) threads *= 2;
        if (E == 8 && aligned_to(w, 32))
            matvec_rows_kernel<T, R, 4, true><<<(unsigned)grid, threads, 0, stream>>>(x, w, b_sum, out, M, nvec, xs);
        else
            matvec_rows_kernel<T, R, 4, false><<<(unsigned)grid, threads, 0, stream>>>(x, w, b_sum, out, M, nvec, xs);
        return launch_status();
    }
    if (M > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    matvec_scalar_kernel<T><<<(unsigned)M, 256, 0, stream>>>(x, w, b_sum, out, K, xs);
    return launch_status();
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_row_scale(const void* a, const void* b, void* out, int64_t rows, int64_t cols,
                                      int64_t b_row_stride, int64_t out_row_stride, kop_dtype_t dtype,
                                      kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!a || !b || !out) return KOP_ERR_NULL_POINTER;
    if ((st = check_row_stride(b_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(out_row_stride, cols, rows)) != KOP_OK) return st;
    const int esz = elem_size(dtype);
    if (!aligned_to(a, esz) || !aligned_to(b, esz) || !aligned_to(out, esz)) return KOP_ERR_MISALIGNED;
    if (!alias_ok(b, b_row_stride, out, out_row_stride, rows, cols, esz, true)) return KOP_ERR_BAD_ALIAS;
    {
        // `a` is read by every CTA of its row while `out` is being written: no overlap allowed.
        uintptr_t a0 = reinterpret_cast<uintptr_t>(a), a1 = a0 + (uintptr_t)rows * esz, o0, o1;
        span_of(out, rows, cols, out_row_stride, esz, &o0, &o1);
        if (!(a1 <= o0 || o1 <= a0)) return KOP_ERR_BAD_ALIAS;
    }
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_row_scale<float>(a, b, out, rows, cols, b_row_stride, out_row_stride, s)
                            : dtype == KOP_BF16 ? launch_row_scale<__nv_bfloat16>(a, b, out, rows, cols, b_row_stride, out_row_stride, s)
                            : launch_row_scale<__half>(a, b, out, rows, cols, b_row_stride, out_row_stride, s);
}

extern "C" kop_status_t kop_matvec_bias(const void* x, const float* w, float b_sum, float* out, int64_t rows,
                                        int64_t k, int64_t x_row_stride, kop_dtype_t dtype,
                                        kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, k);
    if (st != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || !w || !out) return KOP_ERR_NULL_POINTER;
    if ((st = check_row_stride(x_row_stride, k, rows)) != KOP_OK) return st;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(w, 4) || !aligned_to(out, 4)) return KOP_ERR_MISALIGNED;
    {
        uintptr_t x0, x1, o0 = reinterpret_cast<uintptr_t>(out), o1 = o0 + (uintptr_t)rows * 4;
        span_of(x, rows, k, x_row_stride, esz, &x0, &x1);
        if (!(x1 <= o0 || o1 <= x0)) return KOP_ERR_BAD_ALIAS;
    }
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_matvec<float>(x, w, b_sum, out, rows, k, x_row_stride, s)
                            : dtype == KOP_BF16 ? launch_matvec<__nv_bfloat16>(x, w, b_sum, out, rows, k, x_row_stride, s)
                            : launch_matvec<__half>(x, w, b_sum, out, rows, k, x_row_stride, s);
}
