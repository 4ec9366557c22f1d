// kop_lp_normalize_rows: y = x / max(||x||_p, eps) per row (p = 1 or 2), the norms optionally written too, in one
// HBM pass. The same four row shapes as the other norm kernels: 2 .. 32 lanes of a warp per short row, a CTA per
// row with the row in registers, two sweeps with vector loads (the second backwards, out of the L2) beyond one
// CTA's registers, and a scalar kernel for rows that cannot take 16-byte vectors.
#include "kop_common.cuh"

namespace kop {
namespace {

// |v| or v^2 of a packed pair, added to acc
template <int P>
__device__ __forceinline__ float2 accumulate(float2 acc, float2 v)
{
    if (P == 1) return __fadd2_rn(acc, make_float2(fabsf(v.x), fabsf(v.y)));
    return __ffma2_rn(v, v, acc);
}
// 1 / max(norm, eps) from the row's sum; a NaN sum stays NaN (fmaxf would drop it)
template <int P>
__device__ __forceinline__ float inv_norm(float s, float eps, float* norm)
{
    const float n = P == 1 ? s : sqrtf(s);
    *norm = n;
    return n != n ? n : 1.0f / fmaxf(n, eps);
}

// kRagged (all three vector kernels): rows that are not whole aligned vectors; `nvec` then carries the row length in
// elements, a row is split into head elements up to the first 16-byte boundary, whole vectors and tail elements, and the
// edge elements go to the row's lanes (one or two each) or one to a thread. x and y rows sit at the same offset from a
// boundary.
template <typename T, int L, int P, bool kRagged = false>
__global__ void __launch_bounds__(256)
lpnorm_group_kernel(const T* __restrict__ x, T* __restrict__ y, float* __restrict__ norm_out, int64_t rows, int nvec,
                    int64_t x_stride, int64_t y_stride, float eps)
{
    constexpr int E = Elem<T>::kPerVec, Q = E / 2, VPL = 4;
    constexpr int KE = kRagged ? (2 * (E - 1) + L - 1) / L : 1;      // edge elements a lane holds at most
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t row = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * (32 / L) + lane / L;
    const bool live = row < rows;
    const int64_t r = live ? row : 0;
    const T* xr = x + r * x_stride;
    T* yr = y + r * y_stride;
    int edge_col[KE];                                        // this lane's edge columns (-1: none) and their values
    float ev[KE];
#pragma unroll
    for (int q = 0; q < KE; ++q) edge_col[q] = -1, ev[q] = 0.0f;
    const T* xm = xr;                                        // first whole vector of the row
    T* ym = yr;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, nvec);
#pragma unroll
        for (int q = 0; q < KE; ++q)
            if (live && sub + q * L < sp.edges()) {
                edge_col[q] = sp.edge_col(sub + q * L);
                ev[q] = Elem<T>::load1(xr + edge_col[q]);
            }
        nvec = sp.nvec;
        xm += sp.head;
        ym += sp.head;
    }
    Vec16 raw[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        raw[k] = Vec16{{0u, 0u, 0u, 0u}};
        if (live && v < nvec) raw[k] = ld_stream(xm + (int64_t)v * E);
    }
    float2 val[VPL][Q];
    float2 acc = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        Elem<T>::unpack2(raw[k], val[k]);
#pragma unroll
        for (int q = 0; q < Q; ++q) acc = accumulate<P>(acc, val[k][q]);
    }
    float s = acc.x + acc.y;
    if constexpr (kRagged) {
#pragma unroll
        for (int q = 0; q < KE; ++q) s = P == 1 ? s + fabsf(ev[q]) : fmaf(ev[q], ev[q], s);
    }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    float n;
    const float inv = inv_norm<P>(s, eps, &n);
    if (live && sub == 0 && norm_out != nullptr) norm_out[row] = n;
    const float2 inv2 = make_float2(inv, inv);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        if (live && v < nvec) {
            float2 o[Q];
#pragma unroll
            for (int q = 0; q < Q; ++q) o[q] = __fmul2_rn(val[k][q], inv2);
            st_stream(ym + (int64_t)v * E, Elem<T>::pack2(o));
        }
    }
    if constexpr (kRagged) {
#pragma unroll
        for (int q = 0; q < KE; ++q)
            if (edge_col[q] >= 0) Elem<T>::store1(yr + edge_col[q], ev[q] * inv);
    }
}

template <typename T, int VPT, int P, bool kRagged = false>
__global__ void __launch_bounds__(max_threads_for(VPT * Elem<T>::kPerVec))
lpnorm_block_kernel(const T* __restrict__ x, T* __restrict__ y, float* __restrict__ norm_out, int nvec, int64_t x_stride,
                    int64_t y_stride, float eps)
{
    constexpr int E = Elem<T>::kPerVec, Q = E / 2;
    __shared__ float red[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    const T* xm = xr;
    T* ym = yr;
    int edge_col = -1;
    float ev = 0.0f;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, nvec);
        if ((int)threadIdx.x < sp.edges()) {
            edge_col = sp.edge_col(threadIdx.x);
            ev = Elem<T>::load1(xr + edge_col);
        }
        nvec = sp.nvec;
        xm += sp.head;
        ym += sp.head;
    }
    Vec16 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        raw[k] = Vec16{{0u, 0u, 0u, 0u}};
        if (v < nvec) raw[k] = ld_stream(xm + (int64_t)v * E);
    }
    float2 val[VPT][Q];
    float2 acc = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        Elem<T>::unpack2(raw[k], val[k]);
#pragma unroll
        for (int q = 0; q < Q; ++q) acc = accumulate<P>(acc, val[k][q]);
    }
    float part = acc.x + acc.y;
    if constexpr (kRagged) part = P == 1 ? part + fabsf(ev) : fmaf(ev, ev, part);
    float n;
    const float inv = inv_norm<P>(block_sum(part, red), eps, &n);
    if (threadIdx.x == 0 && norm_out != nullptr) norm_out[row] = n;
    const float2 inv2 = make_float2(inv, inv);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        if (v < nvec) {
            float2 o[Q];
#pragma unroll
            for (int q = 0; q < Q; ++q) o[q] = __fmul2_rn(val[k][q], inv2);
            st_stream(ym + (int64_t)v * E, Elem<T>::pack2(o));
        }
    }
    if constexpr (kRagged) {
        if (edge_col >= 0) Elem<T>::store1(yr + edge_col, ev * inv);
    }
}

template <typename T, int P, bool kRagged = false>
__global__ void __launch_bounds__(512)
lpnorm_long_kernel(const T* __restrict__ x, T* __restrict__ y, float* __restrict__ norm_out, int nvec, int64_t x_stride,
                   int64_t y_stride, float eps)
{
    constexpr int E = Elem<T>::kPerVec, Q = E / 2, U = 4;
    __shared__ float red[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    int edge_col = -1;
    float ev = 0.0f;
    T* edge_dst = yr;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, nvec);
        if ((int)threadIdx.x < sp.edges()) {
            edge_col = sp.edge_col(threadIdx.x);
            ev = Elem<T>::load1(xr + edge_col);
            edge_dst = yr + edge_col;
        }
        nvec = sp.nvec;
        xr += sp.head;
        yr += sp.head;
    }
    const int step = U * blockDim.x;
    const int nbatch = (nvec + step - 1) / step;
    const uint64_t keep = l2_policy_keep(), drop = l2_policy_drop();
    float2 acc = make_float2(0.0f, 0.0f);
    for (int b = 0; b < nbatch; ++b) {
        Vec16 raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            raw[k] = Vec16{{0u, 0u, 0u, 0u}};
            if (v < nvec) raw[k] = ld_stream_hint(xr + (int64_t)v * E, keep);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            float2 val[Q];
            Elem<T>::unpack2(raw[k], val);
#pragma unroll
            for (int q = 0; q < Q; ++q) acc = accumulate<P>(acc, val[q]);
        }
    }
    float part = acc.x + acc.y;
    if constexpr (kRagged) part = P == 1 ? part + fabsf(ev) : fmaf(ev, ev, part);
    float n;
    const float inv = inv_norm<P>(block_sum(part, red), eps, &n);
    if (threadIdx.x == 0 && norm_out != nullptr) norm_out[row] = n;
    const float2 inv2 = make_float2(inv, inv);
    if constexpr (kRagged) {
        if (edge_col >= 0) Elem<T>::store1(edge_dst, ev * inv);
    }
    // backwards: the end of the row is what the first sweep left in the L2; y[v] is written by the thread that
    // read x[v], after every thread has finished the first sweep (the barrier in block_sum)
    for (int b = nbatch - 1; b >= 0; --b) {
        Vec16 raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            if (v < nvec) raw[k] = ld_stream_hint(xr + (int64_t)v * E, drop);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            if (v < nvec) {
                float2 val[Q];
                Elem<T>::unpack2(raw[k], val);
#pragma unroll
                for (int q = 0; q < Q; ++q) val[q] = __fmul2_rn(val[q], inv2);
                st_stream_hint(yr + (int64_t)v * E, Elem<T>::pack2(val), drop);
            }
        }
    }
}

template <typename T, int P>
__global__ void __launch_bounds__(256)
lpnorm_scalar_kernel(const T* __restrict__ x, T* __restrict__ y, float* __restrict__ norm_out, int64_t cols,
                     int64_t x_stride, int64_t y_stride, float eps)
{
    __shared__ float red[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    float acc = 0.0f;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float v = Elem<T>::load1(xr + j);
        acc = P == 1 ? acc + fabsf(v) : fmaf(v, v, acc);
    }
    float n;
    const float inv = inv_norm<P>(block_sum(acc, red), eps, &n);
    if (threadIdx.x == 0 && norm_out != nullptr) norm_out[row] = n;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) Elem<T>::store1(yr + j, Elem<T>::load1(xr + j) * inv);
}

template <typename T, int P>
kop_status_t launch_lpnorm(const void* xv, void* yv, float* norm_out, int64_t rows, int64_t cols, int64_t xs, int64_t ys,
                           float eps, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    T* y = static_cast<T*>(yv);
    constexpr int E = Elem<T>::kPerVec;
    const bool vec = vec_ok(x, cols, xs, sizeof(T)) && vec_ok(y, cols, ys, sizeof(T));
    const int64_t nvec64 = cols / E;
    if (vec && nvec64 <= 128) {
        const int nvec = (int)nvec64;
        const int lanes = nvec > 64 ? 32 : nvec > 32 ? 16 : nvec > 16 ? 8 : nvec > 8 ? 4 : 2;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
#define KOP_LP_GROUP(L) lpnorm_group_kernel<T, L, P><<<(unsigned)ctas, 256, 0, stream>>>(x, y, norm_out, rows, nvec, xs, ys, eps)
        switch (lanes) {
        case 32: KOP_LP_GROUP(32); break;
        case 16: KOP_LP_GROUP(16); break;
        case 8: KOP_LP_GROUP(8); break;
        case 4: KOP_LP_GROUP(4); break;
        default: KOP_LP_GROUP(2); break;
        }
#undef KOP_LP_GROUP
        return launch_status();
    }
    if (rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    if (vec && cols <= kMaxRegisterRow) {
        const int nvec = (int)nvec64;
        int vals = 32;
        if (cols <= 1024) vals = 16;
        if ((nvec + vals / E - 1) / (vals / E) > max_threads_for(vals)) vals = 64;
        const int vpt = vals / E;
        const int threads = ((nvec + vpt - 1) / vpt + 31) / 32 * 32;
#define KOP_LP_BLOCK(V) lpnorm_block_kernel<T, V, P><<<(unsigned)rows, threads, 0, stream>>>(x, y, norm_out, nvec, xs, ys, eps)
        switch (vals) {
        case 16: KOP_LP_BLOCK(16 / E); break;
        case 32: KOP_LP_BLOCK(32 / E); break;
        default: KOP_LP_BLOCK(64 / E); break;
        }
#undef KOP_LP_BLOCK
        return launch_status();
    }
    if (vec && nvec64 <= 0x7FFFFFFF) {
        lpnorm_long_kernel<T, P><<<(unsigned)rows, 512, 0, stream>>>(x, y, norm_out, (int)nvec64, xs, ys, eps);
        return launch_status();
    }
    // rows that are not whole aligned vectors, x and y rows at the same offset from a 16-byte boundary: head elements,
    // aligned vectors, tail elements in the same three kernels
    const bool ragged = !vec && (reinterpret_cast<uintptr_t>(x) - reinterpret_cast<uintptr_t>(y)) % 16 == 0 &&
                        ((xs - ys) * (int64_t)sizeof(T)) % 16 == 0 && cols <= 0x7FFFFFFFLL;
    if (ragged && nvec64 <= 128) {
        const int lanes = nvec64 > 64 ? 32 : nvec64 > 32 ? 16 : 8;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
#define KOP_LP_RAG(L) lpnorm_group_kernel<T, L, P, true><<<(unsigned)ctas, 256, 0, stream>>>(x, y, norm_out, rows, (int)cols, xs, ys, eps)
        if (lanes == 32) KOP_LP_RAG(32);
        else if (lanes == 16) KOP_LP_RAG(16);
        else KOP_LP_RAG(8);
#undef KOP_LP_RAG
        return launch_status();
    }
    if (ragged && cols <= kMaxRegisterRow) {
        const int nvec = (int)nvec64;
        int vals = 32;
        if (cols <= 1024) vals = 16;
        if ((nvec + vals / E - 1) / (vals / E) > max_threads_for(vals)) vals = 64;
        const int vpt = vals / E;
        const int threads = ((nvec + vpt - 1) / vpt + 31) / 32 * 32;
#define KOP_LP_BLOCK_RAG(V) lpnorm_block_kernel<T, V, P, true><<<(unsigned)rows, threads, 0, stream>>>(x, y, norm_out, (int)cols, xs, ys, eps)
        switch (vals) {
        case 16: KOP_LP_BLOCK_RAG(16 / E); break;
        case 32: KOP_LP_BLOCK_RAG(32 / E); break;
        default: KOP_LP_BLOCK_RAG(64 / E); break;
        }
#undef KOP_LP_BLOCK_RAG
        return launch_status();
    }
    if (ragged) {
        lpnorm_long_kernel<T, P, true><<<(unsigned)rows, 512, 0, stream>>>(x, y, norm_out, (int)cols, xs, ys, eps);
        return launch_status();
    }
    lpnorm_scalar_kernel<T, P><<<(unsigned)rows, 256, 0, stream>>>(x, y, norm_out, cols, xs, ys, eps);
    return launch_status();
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_lp_normalize_rows(const void* x, void* y, float* norm_out, int64_t rows, int64_t cols,
                                              int64_t x_row_stride, int64_t y_row_stride, int p, float eps,
                                              kop_dtype_t dtype, kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if ((p != 1 && p != 2) || !(eps >= 0.0f)) return KOP_ERR_BAD_SHAPE;
    if (rows == 0) return KOP_OK;
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, cols, rows)) != KOP_OK) return st;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (norm_out && !aligned_to(norm_out, 4))) return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, cols, esz, true)) return KOP_ERR_BAD_ALIAS;
    if (norm_out != nullptr) {
        // the norms overlap neither tensor
        uintptr_t n0 = reinterpret_cast<uintptr_t>(norm_out), n1 = n0 + (uintptr_t)rows * 4, a0, a1, b0, b1;
        span_of(x, rows, cols, x_row_stride, esz, &a0, &a1);
        span_of(y, rows, cols, y_row_stride, esz, &b0, &b1);
        if (!(n1 <= a0 || a1 <= n0) || !(n1 <= b0 || b1 <= n0)) return KOP_ERR_BAD_ALIAS;
    }
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
#define KOP_LP_GO(T) \
    return p == 1 ? launch_lpnorm<T, 1>(x, y, norm_out, rows, cols, x_row_stride, y_row_stride, eps, s) \
                  : launch_lpnorm<T, 2>(x, y, norm_out, rows, cols, x_row_stride, y_row_stride, eps, s)
    if (dtype == KOP_F32) KOP_LP_GO(float);
    if (dtype == KOP_BF16) KOP_LP_GO(__nv_bfloat16);
    KOP_LP_GO(__half);
#undef KOP_LP_GO
}
