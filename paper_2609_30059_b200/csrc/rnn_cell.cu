// kop_lstm_cell, kop_gru_cell: the gate arithmetic of one LSTM / GRU step, after the two preserved GEMMs: the
// gate tensors and biases are summed, the gates activated and the state updated, with every tensor read or
// written once. A thread owns four hidden units of one row (16-byte loads of fp32 data, 8-byte loads of
// 16-bit data): its gate vectors and the state vector are in flight together, and the CTAs are short-lived.
// The kernels are bound by load latency and the special-function unit together (for the LSTM eight
// operations a hidden unit with exp2 / reciprocal sigmoids), so bf16 data takes every gate from the
// hardware tanh (five operations) and 16-bit data keeps threads small for more resident warps.
#include "kop_common.cuh"

#include <type_traits>

namespace kop {
namespace {

// One 32-bit word of a tensor: one fp32 value or two 16-bit values.
template <typename T>
struct Word;
template <>
struct Word<float> {
    static constexpr int kN = 1;
    __device__ __forceinline__ static void unpack(uint32_t w, float* f) { f[0] = __uint_as_float(w); }
    __device__ __forceinline__ static uint32_t pack(const float* f) { return __float_as_uint(f[0]); }
};
template <>
struct Word<__nv_bfloat16> {
    static constexpr int kN = 2;
    __device__ __forceinline__ static void unpack(uint32_t w, float* f)
    {
        f[0] = __uint_as_float(w << 16);
        f[1] = __uint_as_float(w & 0xFFFF0000u);
    }
    __device__ __forceinline__ static uint32_t pack(const float* f)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(f[0], f[1]);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};
template <>
struct Word<__half> {
    static constexpr int kN = 2;
    __device__ __forceinline__ static void unpack(uint32_t w, float* f)
    {
        const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&w));
        f[0] = v.x;
        f[1] = v.y;
    }
    __device__ __forceinline__ static uint32_t pack(const float* f)
    {
        __half2 h = __floats2half2_rn(f[0], f[1]);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};

template <int W>
__device__ __forceinline__ void ld_words(const void* p, uint32_t (&w)[W])
{
    if (W == 4)
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[W - 2]), "=r"(w[W - 1]) : "l"(p));
    else
        asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(p));
}
template <int W>
__device__ __forceinline__ void st_words(void* p, const uint32_t (&w)[W])
{
    if (W == 4)
        asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                     :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[W - 2]), "r"(w[W - 1]) : "memory");
    else
        asm volatile("st.global.L1::no_allocate.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(w[0]), "r"(w[1]) : "memory");
}

// fp32 data: tanhf and 1 / (1 + 2^(-x log2 e)); fp16: the same sigmoid with the hardware tanh (2^-11
// relative); bf16: both from the hardware tanh, sigmoid(x) = 0.5 + 0.5 tanh(x / 2), one special-function
// operation per gate.
template <typename T>
__device__ __forceinline__ float tanh_dev(float v) { return sizeof(T) == 2 ? tanh_approx(v) : tanhf(v); }
template <typename T>
__device__ __forceinline__ float sigmoid_dev(float v)
{
    if (std::is_same<T, __nv_bfloat16>::value) return fmaf(tanh_approx(0.5f * v), 0.5f, 0.5f);
    return rcp_approx(1.0f + ex2_approx(-v * kLog2e));
}

// Rows are laid end to end over the grid, so a short row does not leave part of a CTA idle. Returns false for
// a thread past the end. kCtaInRow: units_per_row is a multiple of the CTA size (row index uniform in a CTA).
template <bool kCtaInRow>
__device__ __forceinline__ bool locate(int units_per_row, int64_t total_units, int64_t* row, int* u)
{
    if (kCtaInRow) {
        const unsigned ctas_per_row = (unsigned)units_per_row / blockDim.x;
        const unsigned r = blockIdx.x / ctas_per_row;
        *row = r;
        *u = (int)((blockIdx.x - r * ctas_per_row) * blockDim.x + threadIdx.x);
    } else if (total_units <= 0xFFFFFFFFLL) {
        const unsigned idx = blockIdx.x * blockDim.x + threadIdx.x;
        if (idx >= (unsigned)total_units) return false;
        const unsigned r = idx / (unsigned)units_per_row;
        *row = r;
        *u = (int)(idx - r * (unsigned)units_per_row);
    } else {
        const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        if (idx >= total_units) return false;
        *row = idx / units_per_row;
        *u = (int)(idx - *row * units_per_row);
    }
    return true;
}

// a[0..E) += bias[0..E) with the widest aligned loads (bias + offset is aligned for them on the vector paths)
template <int E>
__device__ __forceinline__ void add_bias(float (&a)[E], const float* __restrict__ b)
{
    if (E % 4 == 0) {
#pragma unroll
        for (int q = 0; q < E / 4; ++q) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(b) + q);
            a[4 * q + 0] += v.x;
            a[4 * q + 1] += v.y;
            a[4 * q + 2] += v.z;
            a[4 * q + 3] += v.w;
        }
    } else if (E == 2) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(b));
        a[0] += v.x;
        a[E - 1] += v.y;
    } else {
        a[0] += __ldg(b);
    }
}

template <typename T, int WW, int E>
__device__ __forceinline__ void unpack_words(const uint32_t (&w)[WW], float (&f)[E])
{
#pragma unroll
    for (int q = 0; q < WW; ++q) Word<T>::unpack(w[q], &f[q * Word<T>::kN]);
}

// W = words per thread and tensor (4: 16-byte loads, 2: 8-byte loads, 0: one element, no alignment needed).
template <typename T, int W, bool kCtaInRow>
__global__ void __launch_bounds__(128)
lstm_cell_kernel(const T* __restrict__ gates, const T* __restrict__ gates2, const float* __restrict__ bias,
                 const T* __restrict__ c_prev, T* __restrict__ h_out, T* __restrict__ c_out, int64_t hidden,
                 int units_per_row, int64_t total_units)
{
    constexpr int N = Word<T>::kN;
    constexpr int WW = W == 0 ? 1 : W;
    constexpr int E = W == 0 ? 1 : W * N;
    int64_t row;
    int u;                                                   // vector (or element) of hidden units in this row
    if (!locate<kCtaInRow>(units_per_row, total_units, &row, &u)) return;
    const int64_t j = (int64_t)u * E;
    const T* g = gates + row * 4 * hidden + j;
    const T* g2 = gates2 != nullptr ? gates2 + row * 4 * hidden + j : nullptr;
    float a[4][E], c[E];
    if (W != 0) {
        uint32_t raw[4][WW], raw2[4][WW], rc[WW];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            ld_words<WW>(g + k * hidden, raw[k]);
            if (g2 != nullptr) ld_words<WW>(g2 + k * hidden, raw2[k]);
        }
        ld_words<WW>(c_prev + row * hidden + j, rc);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int q = 0; q < WW; ++q) Word<T>::unpack(raw[k][q], &a[k][q * N]);
            if (g2 != nullptr) {
#pragma unroll
                for (int q = 0; q < WW; ++q) {
                    float f[N];
                    Word<T>::unpack(raw2[k][q], f);
#pragma unroll
                    for (int e = 0; e < N; ++e) a[k][q * N + e] += f[e];
                }
            }
        }
#pragma unroll
        for (int q = 0; q < WW; ++q) Word<T>::unpack(rc[q], &c[q * N]);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k)
            a[k][0] = Elem<T>::load1(g + k * hidden) + (g2 != nullptr ? Elem<T>::load1(g2 + k * hidden) : 0.0f);
        c[0] = Elem<T>::load1(c_prev + row * hidden + j);
    }
    if (bias != nullptr) {
#pragma unroll
        for (int k = 0; k < 4; ++k) add_bias<E>(a[k], bias + k * hidden + j);
    }
    float h[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const float cn = fmaf(sigmoid_dev<T>(a[1][e]), c[e], sigmoid_dev<T>(a[0][e]) * tanh_dev<T>(a[2][e]));
        c[e] = cn;
        h[e] = sigmoid_dev<T>(a[3][e]) * tanh_dev<T>(cn);
    }
    if (W != 0) {
        uint32_t wc[WW], wh[WW];
#pragma unroll
        for (int q = 0; q < WW; ++q) {
            wc[q] = Word<T>::pack(&c[q * N]);
            wh[q] = Word<T>::pack(&h[q * N]);
        }
        st_words<WW>(c_out + row * hidden + j, wc);
        st_words<WW>(h_out + row * hidden + j, wh);
    } else {
        Elem<T>::store1(c_out + row * hidden + j, c[0]);
        Elem<T>::store1(h_out + row * hidden + j, h[0]);
    }
}

// GRU: r = sigmoid(gi_r + gh_r), z = sigmoid(gi_z + gh_z), n = tanh(gi_n + r gh_n), h' = n + z (h - n).
template <typename T, int W, bool kCtaInRow>
__global__ void __launch_bounds__(128, W == 4 ? 8 : 16)
gru_cell_kernel(const T* __restrict__ gi, const T* __restrict__ gh, const float* __restrict__ bias_i,
                const float* __restrict__ bias_h, const T* __restrict__ h_prev, T* __restrict__ h_out, int64_t hidden,
                int units_per_row, int64_t total_units)
{
    constexpr int N = Word<T>::kN;
    constexpr int WW = W == 0 ? 1 : W;
    constexpr int E = W == 0 ? 1 : W * N;
    int64_t row;
    int u;
    if (!locate<kCtaInRow>(units_per_row, total_units, &row, &u)) return;
    const int64_t j = (int64_t)u * E;
    const T* pi = gi + row * 3 * hidden + j;
    const T* ph = gh + row * 3 * hidden + j;
    float xi[3][E], xh[3][E], h[E];
    if (W != 0) {
        uint32_t ri[3][WW], rh[3][WW], rp[WW];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            ld_words<WW>(pi + k * hidden, ri[k]);
            ld_words<WW>(ph + k * hidden, rh[k]);
        }
        ld_words<WW>(h_prev + row * hidden + j, rp);
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            unpack_words<T, WW, E>(ri[k], xi[k]);
            unpack_words<T, WW, E>(rh[k], xh[k]);
        }
        unpack_words<T, WW, E>(rp, h);
    } else {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            xi[k][0] = Elem<T>::load1(pi + k * hidden);
            xh[k][0] = Elem<T>::load1(ph + k * hidden);
        }
        h[0] = Elem<T>::load1(h_prev + row * hidden + j);
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        if (bias_i != nullptr) add_bias<E>(xi[k], bias_i + k * hidden + j);
        if (bias_h != nullptr) add_bias<E>(xh[k], bias_h + k * hidden + j);
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const float r = sigmoid_dev<T>(xi[0][e] + xh[0][e]);
        const float z = sigmoid_dev<T>(xi[1][e] + xh[1][e]);
        const float n = tanh_dev<T>(fmaf(r, xh[2][e], xi[2][e]));
        h[e] = fmaf(z, h[e] - n, n);
    }
    if (W != 0) {
        uint32_t wh[WW];
#pragma unroll
        for (int q = 0; q < WW; ++q) wh[q] = Word<T>::pack(&h[q * N]);
        st_words<WW>(h_out + row * hidden + j, wh);
    } else {
        Elem<T>::store1(h_out + row * hidden + j, h[0]);
    }
}

template <typename T, int W>
kop_status_t launch_gru_w(const T* gi, const T* gh, const float* bi, const float* bh, const T* hp, T* ho, int64_t rows,
                          int64_t hidden, cudaStream_t stream)
{
    const int64_t units = W == 0 ? hidden : hidden / (W * Word<T>::kN);
    if (units > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    const int threads = 128;
    const int64_t total = rows * units, ctas = (total + threads - 1) / threads;
    if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    if (units % threads == 0)
        gru_cell_kernel<T, W, true><<<(unsigned)ctas, threads, 0, stream>>>(gi, gh, bi, bh, hp, ho, hidden, (int)units, total);
    else
        gru_cell_kernel<T, W, false><<<(unsigned)ctas, threads, 0, stream>>>(gi, gh, bi, bh, hp, ho, hidden, (int)units, total);
    return launch_status();
}

template <typename T>
kop_status_t launch_gru(const void* gi, const void* gh, const float* bias_i, const float* bias_h, const void* h_prev,
                        void* h_out, int64_t rows, int64_t hidden, cudaStream_t stream)
{
    const T* pi = static_cast<const T*>(gi);
    const T* ph = static_cast<const T*>(gh);
    const T* hp = static_cast<const T*>(h_prev);
    T* ho = static_cast<T*>(h_out);
    const auto all_aligned = [&](int bytes) {
        return aligned_to(gi, bytes) && aligned_to(gh, bytes) && aligned_to(h_prev, bytes) && aligned_to(h_out, bytes);
    };
    const bool bias16 = (bias_i == nullptr || aligned_to(bias_i, 16)) && (bias_h == nullptr || aligned_to(bias_h, 16));
    const bool ok4 = hidden % (4 * Word<T>::kN) == 0 && all_aligned(16) && bias16;
    const bool ok2 = hidden % (2 * Word<T>::kN) == 0 && all_aligned(8) && bias16;
    // seven loads a thread: 16-byte loads win for every data type (measured), unlike the LSTM's nine to
    // thirteen, where 16-bit data does better with smaller threads
    const int w = ok4 ? 4 : ok2 ? 2 : 0;
    if (w == 4) return launch_gru_w<T, 4>(pi, ph, bias_i, bias_h, hp, ho, rows, hidden, stream);
    if (w == 2) return launch_gru_w<T, 2>(pi, ph, bias_i, bias_h, hp, ho, rows, hidden, stream);
    return launch_gru_w<T, 0>(pi, ph, bias_i, bias_h, hp, ho, rows, hidden, stream);
}

template <typename T, int W>
kop_status_t launch_lstm_w(const T* g, const T* g2, const float* bias, const T* cp, T* ho, T* co, int64_t rows,
                           int64_t hidden, cudaStream_t stream)
{
    const int64_t units = W == 0 ? hidden : hidden / (W * Word<T>::kN);
    if (units > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    const int threads = 128;
    const int64_t total = rows * units, ctas = (total + threads - 1) / threads;
    if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    if (units % threads == 0)
        lstm_cell_kernel<T, W, true><<<(unsigned)ctas, threads, 0, stream>>>(g, g2, bias, cp, ho, co, hidden, (int)units, total);
    else
        lstm_cell_kernel<T, W, false><<<(unsigned)ctas, threads, 0, stream>>>(g, g2, bias, cp, ho, co, hidden, (int)units, total);
    return launch_status();
}

template <typename T>
kop_status_t launch_lstm(const void* gates, const void* gates2, const float* bias, const void* c_prev, void* h_out,
                         void* c_out, int64_t rows, int64_t hidden, cudaStream_t stream)
{
    const T* g = static_cast<const T*>(gates);
    const T* g2 = static_cast<const T*>(gates2);
    const T* cp = static_cast<const T*>(c_prev);
    T* ho = static_cast<T*>(h_out);
    T* co = static_cast<T*>(c_out);
    const auto all_aligned = [&](int bytes) {
        return aligned_to(gates, bytes) && aligned_to(c_prev, bytes) && aligned_to(h_out, bytes) &&
               aligned_to(c_out, bytes) && (gates2 == nullptr || aligned_to(gates2, bytes));
    };
    const bool bias16 = bias == nullptr || aligned_to(bias, 16);
    const bool ok4 = hidden % (4 * Word<T>::kN) == 0 && all_aligned(16) && bias16;
    const bool ok2 = hidden % (2 * Word<T>::kN) == 0 && all_aligned(8) && bias16;
    // 16-bit data: 8-byte loads (four hidden units a thread) halve the registers and the special-function
    // work of a thread, and the extra resident warps hide the loads better than wider loads do
    const int w = sizeof(T) == 2 ? (ok2 ? 2 : 0) : (ok4 ? 4 : ok2 ? 2 : 0);
    if (w == 4) return launch_lstm_w<T, 4>(g, g2, bias, cp, ho, co, rows, hidden, stream);
    if (w == 2) return launch_lstm_w<T, 2>(g, g2, bias, cp, ho, co, rows, hidden, stream);
    return launch_lstm_w<T, 0>(g, g2, bias, cp, ho, co, rows, hidden, stream);
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_lstm_cell(const void* gates, const void* gates2, const float* bias, const void* c_prev,
                                      void* h_out, void* c_out, int64_t rows, int64_t hidden, kop_dtype_t dtype,
                                      kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, hidden);
    if (st != KOP_OK) return st;
    if (hidden > kMaxElems / 4 || (rows > 0 && 4 * hidden > kMaxElems / rows)) return KOP_ERR_BAD_SHAPE;
    if (rows == 0) return KOP_OK;
    if (!gates || !c_prev || !h_out || !c_out) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(gates, esz) || !aligned_to(c_prev, esz) || !aligned_to(h_out, esz) || !aligned_to(c_out, esz) ||
        (gates2 && !aligned_to(gates2, esz)) || (bias && !aligned_to(bias, 4)))
        return KOP_ERR_MISALIGNED;
    // c_out may be c_prev exactly (the state updated in place); otherwise the outputs overlap nothing
    const auto disjoint = [esz](const void* a, int64_t na, const void* b, int64_t nb) {
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
        return a0 + (uintptr_t)(na * esz) <= b0 || b0 + (uintptr_t)(nb * esz) <= a0;
    };
    const int64_t n = rows * hidden;
    if ((c_out != c_prev && !disjoint(c_prev, n, c_out, n)) || !disjoint(c_prev, n, h_out, n) ||
        !disjoint(c_out, n, h_out, n) || !disjoint(gates, 4 * n, h_out, n) || !disjoint(gates, 4 * n, c_out, n) ||
        (gates2 && (!disjoint(gates2, 4 * n, h_out, n) || !disjoint(gates2, 4 * n, c_out, n))))
        return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_lstm<float>(gates, gates2, bias, c_prev, h_out, c_out, rows, hidden, s)
           : dtype == KOP_BF16 ? launch_lstm<__nv_bfloat16>(gates, gates2, bias, c_prev, h_out, c_out, rows, hidden, s)
                               : launch_lstm<__half>(gates, gates2, bias, c_prev, h_out, c_out, rows, hidden, s);
}

extern "C" kop_status_t kop_gru_cell(const void* gi, const void* gh, const float* bias_i, const float* bias_h,
                                     const void* h_prev, void* h_out, int64_t rows, int64_t hidden, kop_dtype_t dtype,
                                     kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, hidden);
    if (st != KOP_OK) return st;
    if (hidden > kMaxElems / 3 || (rows > 0 && 3 * hidden > kMaxElems / rows)) return KOP_ERR_BAD_SHAPE;
    if (rows == 0) return KOP_OK;
    if (!gi || !gh || !h_prev || !h_out) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(gi, esz) || !aligned_to(gh, esz) || !aligned_to(h_prev, esz) || !aligned_to(h_out, esz) ||
        (bias_i && !aligned_to(bias_i, 4)) || (bias_h && !aligned_to(bias_h, 4)))
        return KOP_ERR_MISALIGNED;
    // h_out may be h_prev exactly (the state updated in place); otherwise it overlaps no input
    const auto disjoint = [esz](const void* a, int64_t na, const void* b, int64_t nb) {
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
        return a0 + (uintptr_t)(na * esz) <= b0 || b0 + (uintptr_t)(nb * esz) <= a0;
    };
    const int64_t n = rows * hidden;
    if ((h_out != h_prev && !disjoint(h_prev, n, h_out, n)) || !disjoint(gi, 3 * n, h_out, n) ||
        !disjoint(gh, 3 * n, h_out, n))
        return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_gru<float>(gi, gh, bias_i, bias_h, h_prev, h_out, rows, hidden, s)
           : dtype == KOP_BF16 ? launch_gru<__nv_bfloat16>(gi, gh, bias_i, bias_h, h_prev, h_out, rows, hidden, s)
                               : launch_gru<__half>(gi, gh, bias_i, bias_h, h_prev, h_out, rows, hidden, s);
}
