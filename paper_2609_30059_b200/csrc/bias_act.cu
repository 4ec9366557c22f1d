// kop_bias_act: y = act(x + bias[j]), the pointwise tail of a Linear / GEMM call written once ("activation +
// bias fusion"). Pure streaming: 16-byte loads and stores, the bias vector through L1, fp32 arithmetic, one
// compile-time activation per kernel. fp32 data uses the accurate math functions where the approximate
// ones would eat into the 1e-5 gate (tanh, erf, expm1); 16-bit data uses the hardware approximations, whose
// error is far below the output rounding.
#include "kop_common.cuh"

namespace kop {
namespace {

enum {
    kActIdentity = 0, kActRelu, kActLeakyRelu, kActGeluTanh, kActGeluErf, kActSilu, kActSigmoid, kActTanh, kActMish,
    kActHardswish, kActElu, kActCount
};

template <int ACT, bool kFast>
__device__ __forceinline__ float act_dev(float u, float alpha)
{
    switch (ACT) {
    case kActRelu: {
        float r;
        asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(u), "f"(0.0f));      // NaN stays NaN
        return r;
    }
    case kActLeakyRelu: return u > 0.0f ? u : alpha * u;
    case kActGeluTanh: {
        const float k0 = 0.7978845608028654f, k1 = 0.7978845608028654f * 0.044715f;
        const float inner = u * fmaf(k1, u * u, k0);
        const float t = kFast ? tanh_approx(inner) : tanhf(inner);
        const float hu = 0.5f * u;
        return fmaf(hu, t, hu);
    }
    case kActGeluErf: return 0.5f * u * (1.0f + erf_fast(u * 0.7071067811865476f));
    case kActSilu: return u * rcp_approx(1.0f + ex2_approx(-u * kLog2e));      // ~3e-7 relative
    case kActSigmoid: return rcp_approx(1.0f + ex2_approx(-u * kLog2e));
    case kActTanh: return kFast ? tanh_approx(u) : tanhf(u);
    case kActMish: {
        // tanh(ln(1 + e^u)) = n / (n + 2) with n = e^u (e^u + 2); beyond u = 20 the quotient is 1 in fp32
        const float e = ex2_approx(fminf(u, 20.0f) * kLog2e);
        const float n = e * (e + 2.0f);
        return u > 20.0f ? u : u * n * rcp_approx(n + 2.0f);
    }
    case kActHardswish: return u * fminf(fmaxf(u + 3.0f, 0.0f), 6.0f) * (1.0f / 6.0f);   // NaN * 0 is NaN
    case kActElu: return u > 0.0f ? u : alpha * (kFast ? ex2_approx(u * kLog2e) - 1.0f : expm1f(u));
    default: return u;
    }
}

// kFlat: rows shorter than a tile; the CTA takes U * blockDim.x vectors in row-major order across rows
// (nvec_total = rows * nvec). Otherwise a CTA is one tile of one row.
// kBias: a bias is present (a compile-time variant: tested at run time, its loads and adds stay in the code of the
// activation-only call as predicated-off instructions)
template <typename T, typename PT, int ACT, bool kFlat, bool kBias>
__global__ void __launch_bounds__(256)
bias_act_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y, int nvec,
                int tiles_per_row, int64_t nvec_total, int64_t x_stride, int64_t y_stride, float alpha)
{
    constexpr int E = Elem<T>::kPerVec, U = 4;
    constexpr bool kFast = sizeof(T) == 2;
    int64_t row[U];
    int v[U];
    bool live[U];
    if (kFlat) {
        const int64_t g0 = (int64_t)blockIdx.x * (U * blockDim.x) + threadIdx.x;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int64_t g = g0 + k * blockDim.x;
            live[k] = g < nvec_total;
            flat_position(live[k] ? g : 0, nvec, &row[k], &v[k]);
        }
    } else {
        const int64_t r = blockIdx.x / tiles_per_row;
        const int tile = (int)(blockIdx.x - r * tiles_per_row);
#pragma unroll
        for (int k = 0; k < U; ++k) {
            row[k] = r;
            v[k] = tile * (U * blockDim.x) + threadIdx.x + k * blockDim.x;
            live[k] = v[k] < nvec;
        }
    }
    Vec16 raw[U];
#pragma unroll
    for (int k = 0; k < U; ++k)
        if (live[k]) raw[k] = ld_stream(x + row[k] * x_stride + (int64_t)v[k] * E);
#pragma unroll
    for (int k = 0; k < U; ++k) {
        if (live[k]) {
            float f[E];
            Elem<T>::unpack(raw[k], f);
            if (kBias) {
#pragma unroll
                for (int q = 0; q < E / 4; ++q) {
                    const float4 b = ldg_p4(bias + (int64_t)v[k] * E + 4 * q);
                    f[4 * q] += b.x;
                    f[4 * q + 1] += b.y;
                    f[4 * q + 2] += b.z;
                    f[4 * q + 3] += b.w;
                }
            }
#pragma unroll
            for (int e = 0; e < E; ++e) f[e] = act_dev<ACT, kFast>(f[e], alpha);
            st_stream(y + row[k] * y_stride + (int64_t)v[k] * E, Elem<T>::pack(f));
        }
    }
}

template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(256)
bias_act_scalar_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y, int64_t rows,
                       int64_t cols, int64_t x_stride, int64_t y_stride, float alpha)
{
    constexpr bool kFast = sizeof(T) == 2;
    const int64_t total = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols, j = i - r * cols;
        const float u = Elem<T>::load1(x + r * x_stride + j) + (bias != nullptr ? param1(bias, j) : 0.0f);
        Elem<T>::store1(y + r * y_stride + j, act_dev<ACT, kFast>(u, alpha));
    }
}

// ---- the general chain: y = act(clamp((x + bias) * scale + residual * residual_scale, lo, hi)) ----------
struct ChainArgs {
    float scale, residual_scale, lo, hi, alpha;
};

__device__ __forceinline__ float chain_value(float x, float b, float r, const ChainArgs& a)
{
    float u = fmaf(r, a.residual_scale, (x + b) * a.scale);
    float c;                                   // clamp with NaN-propagating min / max: a NaN stays a NaN
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(c) : "f"(u), "f"(a.lo));
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(u) : "f"(c), "f"(a.hi));
    return u;
}

// kRes: a residual is present (tested at run time its loads, widenings and multiply-adds stay in the code as
// predicated-off instructions, which 16-bit data without a residual pays for: bf16 bias + clamp + SiLU 4.6 TB/s)
template <typename T, typename PT, int ACT, bool kFlat, bool kRes>
__global__ void __launch_bounds__(256)
chain_kernel(const T* __restrict__ x, const PT* __restrict__ bias, const T* __restrict__ res, T* __restrict__ y,
             int nvec, int tiles_per_row, int64_t nvec_total, int64_t x_stride, int64_t r_stride, int64_t y_stride,
             ChainArgs a)
{
    constexpr int E = Elem<T>::kPerVec, U = 2;
    constexpr bool kFast = sizeof(T) == 2;
    int64_t row[U];
    int v[U];
    bool live[U];
    if (kFlat) {
        const int64_t g0 = (int64_t)blockIdx.x * (U * blockDim.x) + threadIdx.x;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int64_t g = g0 + k * blockDim.x;
            live[k] = g < nvec_total;
            flat_position(live[k] ? g : 0, nvec, &row[k], &v[k]);
        }
    } else {
        const int64_t r = blockIdx.x / tiles_per_row;
        const int tile = (int)(blockIdx.x - r * tiles_per_row);
#pragma unroll
        for (int k = 0; k < U; ++k) {
            row[k] = r;
            v[k] = tile * (U * blockDim.x) + threadIdx.x + k * blockDim.x;
            live[k] = v[k] < nvec;
        }
    }
    Vec16 rx[U], rres[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
        if (live[k]) {
            rx[k] = ld_stream(x + row[k] * x_stride + (int64_t)v[k] * E);
            if (kRes) rres[k] = ld_stream(res + row[k] * r_stride + (int64_t)v[k] * E);
        }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
        if (live[k]) {
            float f[E], g[E], b[E];
            Elem<T>::unpack(rx[k], f);
            if (kRes) Elem<T>::unpack(rres[k], g);
#pragma unroll
            for (int q = 0; q < E / 4; ++q) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (bias != nullptr) t = ldg_p4(bias + (int64_t)v[k] * E + 4 * q);
                b[4 * q] = t.x;
                b[4 * q + 1] = t.y;
                b[4 * q + 2] = t.z;
                b[4 * q + 3] = t.w;
            }
#pragma unroll
            for (int e = 0; e < E; ++e)
                f[e] = act_dev<ACT, kFast>(chain_value(f[e], b[e], kRes ? g[e] : 0.0f, a), a.alpha);
            st_stream(y + row[k] * y_stride + (int64_t)v[k] * E, Elem<T>::pack(f));
        }
    }
}

template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(256)
chain_scalar_kernel(const T* __restrict__ x, const PT* __restrict__ bias, const T* __restrict__ res,
                    T* __restrict__ y, int64_t rows, int64_t cols, int64_t x_stride, int64_t r_stride,
                    int64_t y_stride, ChainArgs a)
{
    constexpr bool kFast = sizeof(T) == 2;
    const int64_t total = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols, j = i - r * cols;
        const float u = chain_value(Elem<T>::load1(x + r * x_stride + j), bias != nullptr ? param1(bias, j) : 0.0f,
                                    res != nullptr ? Elem<T>::load1(res + r * r_stride + j) : 0.0f, a);
        Elem<T>::store1(y + r * y_stride + j, act_dev<ACT, kFast>(u, a.alpha));
    }
}

// ---- contiguous tensors whose rows are not whole aligned vectors ------------------------------------------
// The tensor as one span: head elements up to the first 16-byte boundary, aligned vectors that run across the row
// boundaries, tail elements. A vector's first column comes from its flat index by a multiply-shift remainder
// (magic = ceil(2^64 / cols), exact below 2^64 / cols); the following columns wrap at most once (cols >= the vector
// length); the bias is read per element. x, y and the residual sit at the same offset from a boundary.
template <typename T, typename PT, int ACT, bool kChain>
__global__ void __launch_bounds__(256)
span_kernel(const T* __restrict__ x, const PT* __restrict__ bias, const T* __restrict__ res, T* __restrict__ y,
            int64_t total, int cols, unsigned long long magic, ChainArgs a)
{
    constexpr int E = Elem<T>::kPerVec, U = kChain ? 2 : 4;
    constexpr bool kFast = sizeof(T) == 2;
    int64_t head = (int64_t)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / (unsigned)sizeof(T));
    if (head > total) head = total;
    const int64_t nv = (total - head) / E;
    const int tail = (int)(total - head - nv * E);
    auto value = [&](float xv, float rv, int c) {
        const float b = bias != nullptr ? param1(bias, c) : 0.0f;
        if constexpr (kChain) return act_dev<ACT, kFast>(chain_value(xv, b, rv, a), a.alpha);
        else return act_dev<ACT, kFast>(xv + b, a.alpha);
    };
    if (blockIdx.x == 0 && (int)threadIdx.x < (int)head + tail) {
        const int64_t j = (int64_t)threadIdx.x < head ? (int64_t)threadIdx.x : head + nv * E + ((int64_t)threadIdx.x - head);
        const float rv = kChain && res != nullptr ? Elem<T>::load1(res + j) : 0.0f;
        Elem<T>::store1(y + j, value(Elem<T>::load1(x + j), rv, (int)(j % cols)));
    }
    const T* xm = x + head;
    const T* rm = res != nullptr ? res + head : nullptr;
    T* ym = y + head;
    const int64_t g0 = (int64_t)blockIdx.x * (U * blockDim.x) + threadIdx.x;
    Vec16 rx[U], rres[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int64_t g = g0 + k * blockDim.x;
        if (g < nv) {
            rx[k] = ld_stream(xm + g * E);
            if (kChain && res != nullptr) rres[k] = ld_stream(rm + g * E);
        }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
        const int64_t g = g0 + k * blockDim.x;
        if (g < nv) {
            const unsigned long long i0 = (unsigned long long)(head + g * E);
            int c = (int)(i0 - __umul64hi(i0, magic) * (unsigned)cols);
            float f[E], r[E];
            Elem<T>::unpack(rx[k], f);
            if (kChain && res != nullptr) Elem<T>::unpack(rres[k], r);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                f[e] = value(f[e], kChain && res != nullptr ? r[e] : 0.0f, c);
                c = c + 1 == cols ? 0 : c + 1;
            }
            st_stream(ym + g * E, Elem<T>::pack(f));
        }
    }
}

// Launches span_kernel when the tensors qualify; false when they do not.
template <typename T, typename PT, int ACT, bool kChain>
bool launch_span(const T* x, const PT* bias, const T* res, T* y, int64_t rows, int64_t cols, int64_t xs, int64_t rs,
                 int64_t ys, const ChainArgs& a, cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec, U = kChain ? 2 : 4;
    if (xs != cols || ys != cols || (res != nullptr && rs != cols) || cols < E || cols > 0x7FFFFFFFLL) return false;
    const uintptr_t off = reinterpret_cast<uintptr_t>(x) & 15u;
    if ((reinterpret_cast<uintptr_t>(y) & 15u) != off || (res != nullptr && (reinterpret_cast<uintptr_t>(res) & 15u) != off))
        return false;
    const int64_t total = rows * cols;
    const int64_t grid = (total / E + U * 256 - 1) / (U * 256) + 1;
    if (grid > 0x7FFFFFFFLL) return false;
    const unsigned long long magic = (~0ull) / (unsigned long long)cols + 1ull;
    span_kernel<T, PT, ACT, kChain><<<(unsigned)grid, 256, 0, stream>>>(x, bias, res, y, total, (int)cols, magic, a);
    return true;
}

template <typename T, typename PT, int ACT>
kop_status_t launch_chain_a(const T* x, const PT* bias, const T* res, T* y, int64_t rows, int64_t cols, int64_t xs,
                            int64_t rs, int64_t ys, const ChainArgs& a, cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    const bool vec = vec_ok(x, cols, xs, sizeof(T)) && vec_ok(y, cols, ys, sizeof(T)) && cols / E <= 0x3FFFFFFF &&
                     (res == nullptr || vec_ok(res, cols, rs, sizeof(T))) && (bias == nullptr || aligned_to(bias, 16));
    if (vec) {
        const int nvec = (int)(cols / E);
        // a CTA is one tile of one row, sized to the row (32 to 256 threads); rows too short for that, or whose
        // last tile would be mostly empty, take tiles that cross rows
        int threads = ((nvec + 1) / 2 + 31) / 32 * 32;
        if (threads > 256) threads = 256;
        const int tiles = (nvec + 2 * threads - 1) / (2 * threads);
        if (nvec < 64 || ((int64_t)tiles * 2 * threads - nvec) * 4 > nvec) {
            const int64_t total = rows * nvec, grid = (total + 511) / 512;
            if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
            if (res != nullptr) chain_kernel<T, PT, ACT, true, true><<<(unsigned)grid, 256, 0, stream>>>(x, bias, res, y, nvec, 1, total, xs, rs, ys, a);
            else chain_kernel<T, PT, ACT, true, false><<<(unsigned)grid, 256, 0, stream>>>(x, bias, res, y, nvec, 1, total, xs, rs, ys, a);
            return launch_status();
        }
        const int64_t grid = rows * tiles;
        if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        if (res != nullptr) chain_kernel<T, PT, ACT, false, true><<<(unsigned)grid, threads, 0, stream>>>(x, bias, res, y, nvec, tiles, 0, xs, rs, ys, a);
        else chain_kernel<T, PT, ACT, false, false><<<(unsigned)grid, threads, 0, stream>>>(x, bias, res, y, nvec, tiles, 0, xs, rs, ys, a);
        return launch_status();
    }
    if (launch_span<T, PT, ACT, true>(x, bias, res, y, rows, cols, xs, rs, ys, a, stream)) return launch_status();
    int64_t blocks = (rows * cols + 255) / 256;
    const int64_t cap = 32LL * sm_count();
    if (blocks > cap) blocks = cap;
    chain_scalar_kernel<T, PT, ACT><<<(unsigned)blocks, 256, 0, stream>>>(x, bias, res, y, rows, cols, xs, rs, ys, a);
    return launch_status();
}

template <typename T, typename PT>
kop_status_t launch_chain(const void* xv, const void* biasv, const void* rv, void* yv, int64_t rows, int64_t cols,
                          int64_t xs, int64_t rs, int64_t ys, int act, const ChainArgs& a, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    const PT* bias = static_cast<const PT*>(biasv);
    const T* r = static_cast<const T*>(rv);
    T* y = static_cast<T*>(yv);
#define KOP_CHAIN_CASE(A) \
    case A: return launch_chain_a<T, PT, A>(x, bias, r, y, rows, cols, xs, rs, ys, a, stream)
    switch (act) {
        KOP_CHAIN_CASE(kActRelu);
        KOP_CHAIN_CASE(kActLeakyRelu);
        KOP_CHAIN_CASE(kActGeluTanh);
        KOP_CHAIN_CASE(kActGeluErf);
        KOP_CHAIN_CASE(kActSilu);
        KOP_CHAIN_CASE(kActSigmoid);
        KOP_CHAIN_CASE(kActTanh);
        KOP_CHAIN_CASE(kActMish);
        KOP_CHAIN_CASE(kActHardswish);
        KOP_CHAIN_CASE(kActElu);
    default: return launch_chain_a<T, PT, kActIdentity>(x, bias, r, y, rows, cols, xs, rs, ys, a, stream);
    }
#undef KOP_CHAIN_CASE
}

template <typename T, typename PT, int ACT>
kop_status_t launch_bias_act_a(const T* x, const PT* bias, T* y, int64_t rows, int64_t cols, int64_t xs,
                               int64_t ys, float alpha, cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    // without a bias a contiguous tensor is one long row (no per-row tail, no row index)
    if (bias == nullptr && xs == cols && ys == cols && rows * cols / E <= 0x3FFFFFFFLL) {
        cols = rows * cols;
        xs = ys = cols;
        rows = 1;
    }
    const bool vec = vec_ok(x, cols, xs, sizeof(T)) && vec_ok(y, cols, ys, sizeof(T)) && cols / E <= 0x3FFFFFFF &&
                     (bias == nullptr || aligned_to(bias, 16));
    if (vec) {
        const int nvec = (int)(cols / E);
        // a CTA is one tile of one row, sized to the row (32 to 256 threads); rows too short for that, or whose
        // last tile would be mostly empty, take tiles that cross rows
        int threads = ((nvec + 3) / 4 + 31) / 32 * 32;
        if (threads > 256) threads = 256;
        const int tiles = (nvec + 4 * threads - 1) / (4 * threads);
        if (nvec < 128 || ((int64_t)tiles * 4 * threads - nvec) * 4 > nvec) {
            const int64_t total = rows * nvec, grid = (total + 1023) / 1024;
            if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
            if (bias != nullptr) bias_act_kernel<T, PT, ACT, true, true><<<(unsigned)grid, 256, 0, stream>>>(x, bias, y, nvec, 1, total, xs, ys, alpha);
            else bias_act_kernel<T, PT, ACT, true, false><<<(unsigned)grid, 256, 0, stream>>>(x, bias, y, nvec, 1, total, xs, ys, alpha);
            return launch_status();
        }
        const int64_t grid = rows * tiles;
        if (grid > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        if (bias != nullptr) bias_act_kernel<T, PT, ACT, false, true><<<(unsigned)grid, threads, 0, stream>>>(x, bias, y, nvec, tiles, 0, xs, ys, alpha);
        else bias_act_kernel<T, PT, ACT, false, false><<<(unsigned)grid, threads, 0, stream>>>(x, bias, y, nvec, tiles, 0, xs, ys, alpha);
        return launch_status();
    }
    if (launch_span<T, PT, ACT, false>(x, bias, static_cast<const T*>(nullptr), y, rows, cols, xs, 0, ys,
                                       ChainArgs{1.0f, 0.0f, 0.0f, 0.0f, alpha}, stream))
        return launch_status();
    int64_t blocks = (rows * cols + 255) / 256;
    const int64_t cap = 32LL * sm_count();
    if (blocks > cap) blocks = cap;
    bias_act_scalar_kernel<T, PT, ACT><<<(unsigned)blocks, 256, 0, stream>>>(x, bias, y, rows, cols, xs, ys, alpha);
    return launch_status();
}

template <typename T, typename PT>
kop_status_t launch_bias_act(const void* xv, const void* biasv, void* yv, int64_t rows, int64_t cols, int64_t xs,
                             int64_t ys, int act, float alpha, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    const PT* bias = static_cast<const PT*>(biasv);
    T* y = static_cast<T*>(yv);
#define KOP_ACT_CASE(A) \
    case A: return launch_bias_act_a<T, PT, A>(x, bias, y, rows, cols, xs, ys, alpha, stream)
    switch (act) {
        KOP_ACT_CASE(kActRelu);
        KOP_ACT_CASE(kActLeakyRelu);
        KOP_ACT_CASE(kActGeluTanh);
        KOP_ACT_CASE(kActGeluErf);
        KOP_ACT_CASE(kActSilu);
        KOP_ACT_CASE(kActSigmoid);
        KOP_ACT_CASE(kActTanh);
        KOP_ACT_CASE(kActMish);
        KOP_ACT_CASE(kActHardswish);
        KOP_ACT_CASE(kActElu);
    default: return launch_bias_act_a<T, PT, kActIdentity>(x, bias, y, rows, cols, xs, ys, alpha, stream);
    }
#undef KOP_ACT_CASE
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

kop_status_t bias_act_entry(const void* x, const void* bias, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                            int64_t y_row_stride, int act, float alpha, kop_dtype_t dtype, kop_dtype_t pdtype,
                            kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (act < 0 || act >= kActCount) return KOP_ERR_BAD_SHAPE;
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, cols, rows)) != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (bias && !aligned_to(bias, elem_size(pdtype)))) return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, cols, esz, true)) return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
#define KOP_BA_GO(T, PT) launch_bias_act<T, PT>(x, bias, y, rows, cols, x_row_stride, y_row_stride, act, alpha, s)
    return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_BA_GO);
#undef KOP_BA_GO
}

kop_status_t chain_entry(const void* x, const void* bias, const void* residual, void* y, int64_t rows, int64_t cols,
                         int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride, float scale,
                         float residual_scale, float clamp_lo, float clamp_hi, int act, float alpha, kop_dtype_t dtype,
                         kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (act < 0 || act >= kActCount || !(clamp_lo <= clamp_hi)) return KOP_ERR_BAD_SHAPE;
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if (residual != nullptr && (st = check_row_stride(res_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, cols, rows)) != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (residual && !aligned_to(residual, esz)) ||
        (bias && !aligned_to(bias, elem_size(pdtype))))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, cols, esz, true) ||
        (residual && !alias_ok(residual, res_row_stride, y, y_row_stride, rows, cols, esz, true)))
        return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    const ChainArgs a{scale, residual_scale, clamp_lo, clamp_hi, alpha};
#define KOP_CH_GO(T, PT) launch_chain<T, PT>(x, bias, residual, y, rows, cols, x_row_stride, res_row_stride, y_row_stride, act, a, s)
    return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_CH_GO);
#undef KOP_CH_GO
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_bias_act(const void* x, const float* bias, void* y, int64_t rows, int64_t cols,
                                     int64_t x_row_stride, int64_t y_row_stride, int act, float alpha,
                                     kop_dtype_t dtype, kop_stream_t stream)
{
    return kop::bias_act_entry(x, bias, y, rows, cols, x_row_stride, y_row_stride, act, alpha, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_bias_act_ex(const void* x, const void* bias, void* y, int64_t rows, int64_t cols,
                                        int64_t x_row_stride, int64_t y_row_stride, int act, float alpha,
                                        kop_dtype_t dtype, kop_dtype_t param_dtype, kop_stream_t stream)
{
    return kop::bias_act_entry(x, bias, y, rows, cols, x_row_stride, y_row_stride, act, alpha, dtype, param_dtype, stream);
}

extern "C" kop_status_t kop_epilogue_chain(const void* x, const float* bias, const void* residual, void* y,
                                           int64_t rows, int64_t cols, int64_t x_row_stride, int64_t res_row_stride,
                                           int64_t y_row_stride, float scale, float residual_scale, float clamp_lo,
                                           float clamp_hi, int act, float alpha, kop_dtype_t dtype,
                                           kop_stream_t stream)
{
    return kop::chain_entry(x, bias, residual, y, rows, cols, x_row_stride, res_row_stride, y_row_stride, scale,
                            residual_scale, clamp_lo, clamp_hi, act, alpha, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_epilogue_chain_ex(const void* x, const void* bias, const void* residual, void* y,
                                              int64_t rows, int64_t cols, int64_t x_row_stride, int64_t res_row_stride,
                                              int64_t y_row_stride, float scale, float residual_scale, float clamp_lo,
                                              float clamp_hi, int act, float alpha, kop_dtype_t dtype,
                                              kop_dtype_t param_dtype, kop_stream_t stream)
{
    return kop::chain_entry(x, bias, residual, y, rows, cols, x_row_stride, res_row_stride, y_row_stride, scale,
                            residual_scale, clamp_lo, clamp_hi, act, alpha, dtype, param_dtype, stream);
}
