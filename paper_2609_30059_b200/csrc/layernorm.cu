// kop_bias_gelu_residual_layernorm: v = residual + gelu_tanh(x + bias); y = LayerNorm(v) in one
// HBM pass. A CTA owns a row; each thread keeps its share of v in fp32 registers, so the mean
// and the centred second moment are both exact two-sweep sums over registers (no E[v^2]-mu^2
// cancellation, no Welford merge needed) while x and residual are read from HBM once.
#include "kop_common.cuh"

namespace kop {
namespace {

// 0.5 u (1 + tanh(k0 (u + 0.044715 u^3))). bf16 rows use the hardware tanh (abs error ~2^-11,
// below the 2^-9 relative step of the bf16 store); fp32 rows use the accurate tanhf.
template <bool kFastTanh>
__device__ __forceinline__ float gelu_tanh(float u)
{
    const float k0 = 0.7978845608028654f;          // sqrt(2/pi)
    const float k1 = 0.7978845608028654f * 0.044715f;
    const float inner = u * fmaf(k1, u * u, k0);
    const float t = kFastTanh ? tanh_approx(inner) : tanhf(inner);
    const float hu = 0.5f * u;
    return fmaf(hu, t, hu);
}

// Two-wide version on packed fp32 pairs (fma.rn.f32x2 and friends: one issue slot per two
// elements), returning residual + gelu(x + bias).
template <bool kFastTanh>
__device__ __forceinline__ float2 gelu_residual2(float2 x, float2 b, float2 r)
{
    const float k0 = 0.7978845608028654f, k1 = 0.7978845608028654f * 0.044715f;
    const float2 u = __fadd2_rn(x, b);
    const float2 p = __ffma2_rn(make_float2(k1, k1), __fmul2_rn(u, u), make_float2(k0, k0));
    const float2 inner = __fmul2_rn(u, p);
    const float2 t = kFastTanh ? make_float2(tanh_approx(inner.x), tanh_approx(inner.y))
                               : make_float2(tanhf(inner.x), tanhf(inner.y));
    const float2 hu = __fmul2_rn(make_float2(0.5f, 0.5f), u);
    return __ffma2_rn(hu, t, __fadd2_rn(hu, r));
}

// The error-function form, 0.5 u (1 + erf(u / sqrt 2)), with erf_fast (absolute error of a few 1e-7, far inside every data
// type's tolerance; the library erff is about three times the instructions).
__device__ __forceinline__ float gelu_erf(float u) { return 0.5f * u * (1.0f + erf_fast(u * 0.7071067811865476f)); }

// What precedes the normalisation: kProBiasGeluResidual: v = residual + gelu(x + bias) with the tanh-form
// GELU (the benchmark segment); kProBiasErfGeluResidual: the same with the error-function GELU;
// kProResidual: v = x + residual; kProNone: v = x. The unused operands are never loaded.
enum { kProBiasGeluResidual = 0, kProResidual = 1, kProNone = 2, kProBiasErfGeluResidual = 3 };
__host__ __device__ constexpr bool pro_has_residual(int pro) { return pro != kProNone; }
__host__ __device__ constexpr bool pro_has_bias(int pro) { return pro == kProBiasGeluResidual || pro == kProBiasErfGeluResidual; }
template <int PRO, bool kFastTanh>
__device__ __forceinline__ float2 prologue2(float2 x, float2 b, float2 r)
{
    if (PRO == kProBiasGeluResidual) return gelu_residual2<kFastTanh>(x, b, r);
    if (PRO == kProBiasErfGeluResidual) {
        const float2 u = __fadd2_rn(x, b);
        return __fadd2_rn(r, make_float2(gelu_erf(u.x), gelu_erf(u.y)));
    }
    if (PRO == kProResidual) return __fadd2_rn(x, r);
    return x;
}
// The prologue on one 16-byte vector of x and of the residual, P packed pairs out. 16-bit data never gets unpacked
// where an addition is the first thing that happens to it: x + bias and residual + (...) are mixed-precision
// adds straight from the packed words (same values bit for bit, a third fewer instructions in the prologue).
template <typename T, int PRO, bool kFastTanh>
__device__ __forceinline__ void prologue_vec(const Vec16& rx, const Vec16& rr, const float2 (&bb)[Elem<T>::kPerVec / 2],
                                             float2 (&out)[Elem<T>::kPerVec / 2])
{
    constexpr int P = Elem<T>::kPerVec / 2;
    if constexpr (Elem<T>::kMixedAdd && PRO != kProNone) {
        if constexpr (PRO == kProResidual) {
            float2 fx[P];
            Elem<T>::unpack2(rx, fx);
#pragma unroll
            for (int q = 0; q < P; ++q) out[q] = Elem<T>::add_widen2(rr.w[q], fx[q]);
        } else {
            const float k0 = 0.7978845608028654f, k1 = 0.7978845608028654f * 0.044715f;
#pragma unroll
            for (int q = 0; q < P; ++q) {
                const float2 u = Elem<T>::add_widen2(rx.w[q], bb[q]);
                if constexpr (PRO == kProBiasGeluResidual) {
                    const float2 p = __ffma2_rn(make_float2(k1, k1), __fmul2_rn(u, u), make_float2(k0, k0));
                    const float2 inner = __fmul2_rn(u, p);
                    const float2 t = kFastTanh ? make_float2(tanh_approx(inner.x), tanh_approx(inner.y))
                                               : make_float2(tanhf(inner.x), tanhf(inner.y));
                    const float2 hu = __fmul2_rn(make_float2(0.5f, 0.5f), u);
                    out[q] = __ffma2_rn(hu, t, Elem<T>::add_widen2(rr.w[q], hu));
                } else {
                    out[q] = Elem<T>::add_widen2(rr.w[q], make_float2(gelu_erf(u.x), gelu_erf(u.y)));
                }
            }
        }
    } else {
        float2 fx[P], fr[P];
        Elem<T>::unpack2(rx, fx);
        Elem<T>::unpack2(rr, fr);
#pragma unroll
        for (int q = 0; q < P; ++q) out[q] = prologue2<PRO, kFastTanh>(fx[q], bb[q], fr[q]);
    }
}

template <int PRO, bool kFastTanh>
__device__ __forceinline__ float prologue1(float x, float b, float r)
{
    if (PRO == kProBiasGeluResidual) return r + gelu_tanh<kFastTanh>(x + b);
    if (PRO == kProBiasErfGeluResidual) return r + gelu_erf(x + b);
    if (PRO == kProResidual) return x + r;
    return x;
}

// CTA per row, row in registers as fp32 pairs. kFull: the row is exactly blockDim.x * VPT vectors
// (no tail predicates). kWide: the eight fp32 parameters that go with a bf16 vector are fetched
// with one 256-bit load per lane, so a warp touches each 128-byte line once (two 128-bit loads
// per lane would walk every line twice and double the L1 wavefronts, which bound this kernel).
template <typename T, typename PT, int VPT, bool kFull, bool kWide, int PRO>
__global__ void __launch_bounds__(max_threads_for(VPT * Elem<T>::kPerVec), VPT * Elem<T>::kPerVec >= 32 ? 2 : 1)
ln_block_kernel(const T* __restrict__ x, const T* __restrict__ res, const PT* __restrict__ bias,
                const PT* __restrict__ gamma, const PT* __restrict__ beta, T* __restrict__ y,
                float* __restrict__ mean, float* __restrict__ rstd, int nvec, int64_t x_stride,
                int64_t r_stride, int64_t y_stride, float eps, float inv_hidden)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;                       // fp32 pairs per vector
    constexpr bool kFast = sizeof(T) == 2;
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    const T* rr = res + row * r_stride;
    T* yr = y + row * y_stride;

    Vec16 rx[VPT], rres[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        if (kFull || v < nvec) {
            rx[k] = ld_stream(xr + (int64_t)v * E);
            if (pro_has_residual(PRO)) rres[k] = ld_stream(rr + (int64_t)v * E);
            else rres[k] = Vec16{{0u, 0u, 0u, 0u}};
        } else {
            rx[k] = Vec16{{0u, 0u, 0u, 0u}};
            rres[k] = Vec16{{0u, 0u, 0u, 0u}};
        }
    }
    float2 val[VPT][P];
    float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        float2 bb[P], fx[P];
        if (pro_has_bias(PRO) && (kFull || v < nvec)) load_params<E, kWide>(bias + (int64_t)v * E, bb);
        else {
#pragma unroll
            for (int q = 0; q < P; ++q) bb[q] = make_float2(0.0f, 0.0f);
        }
        prologue_vec<T, PRO, kFast>(rx[k], rres[k], bb, fx);
#pragma unroll
        for (int q = 0; q < P; ++q) {
            float2 t = fx[q];
            if (!kFull && v >= nvec) t = make_float2(0.0f, 0.0f);
            val[k][q] = t;
            sum2 = __fadd2_rn(sum2, t);
        }
    }
    const float mu = block_sum(sum2.x + sum2.y, red_a) * inv_hidden;
    const float2 nmu = make_float2(-mu, -mu);
    float2 ss2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
#pragma unroll
        for (int q = 0; q < P; ++q) {
            float2 d = __fadd2_rn(val[k][q], nmu);
            if (!kFull && v >= nvec) d = make_float2(0.0f, 0.0f);
            val[k][q] = d;
            ss2 = __ffma2_rn(d, d, ss2);
        }
    }
    const float var = block_sum(ss2.x + ss2.y, red_b) * inv_hidden;
    const float rs = rsqrtf(var + eps);
    if (threadIdx.x == 0) {
        if (mean != nullptr) mean[row] = mu;
        if (rstd != nullptr) rstd[row] = rs;
    }
    const float2 rs2 = make_float2(rs, rs);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        if (kFull || v < nvec) {
            float2 g[P], b[P], o[P];
            load_params<E, kWide>(gamma + (int64_t)v * E, g);
            load_params<E, kWide>(beta + (int64_t)v * E, b);
#pragma unroll
            for (int q = 0; q < P; ++q) o[q] = __ffma2_rn(__fmul2_rn(val[k][q], rs2), g[q], b[q]);
            st_stream(yr + (int64_t)v * E, Elem<T>::pack2(o));
        }
    }
}

// Two rows per CTA. The fp32 parameter vectors are three times the bytes of a bf16 row, and at
// one row per CTA their L1 wavefronts (not HBM) bound the kernel (with the parameter loads stubbed
// out the kernel runs at the speed of a plain two-reads-one-write stream). Each thread therefore
// fetches its bias / gamma / beta once and applies them to the same columns of two rows, which
// halves that traffic; both rows' reductions share the two barriers. The row must be exactly
// blockDim.x * VPT vectors; `rows` may be odd (the last CTA then skips its second row). Capped at 64 registers
// (four 256-thread CTAs per SM): at the 76 the compiler takes by itself three fit, and the benchmark shape ran
// 5 % slower (rows of 5120: 12 %); a cap of 48 spills and loses 25 %. With 32 values a thread and row (plain LayerNorm,
// CTAs of at most 160 threads) the cap is four CTAs' worth of a 160-thread CTA, 102 registers; for its 192- to 256-thread
// CTAs three per SM, 85 registers.
template <typename T, typename PT, int VPT, bool kWide, int kMaxThreads, int PRO>
__global__ void __launch_bounds__(kMaxThreads, VPT * Elem<T>::kPerVec == 32 ? (kMaxThreads <= 160 ? 4 : 3) : 1024 / kMaxThreads)
ln_pair_kernel(const T* __restrict__ x, const T* __restrict__ res, const PT* __restrict__ bias,
               const PT* __restrict__ gamma, const PT* __restrict__ beta, T* __restrict__ y,
               float* __restrict__ mean, float* __restrict__ rstd, int64_t rows, int64_t x_stride,
               int64_t r_stride, int64_t y_stride, float eps, float inv_hidden)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;
    constexpr bool kFast = sizeof(T) == 2;
    __shared__ float red_a[2][32], red_b[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * 2;
    const bool two = row0 + 1 < rows;

    Vec16 rx[2][VPT], rres[2][VPT];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int64_t v = (int64_t)k * blockDim.x + threadIdx.x;
            if (r == 0 || two) {
                rx[r][k] = ld_stream(x + (row0 + r) * x_stride + v * E);
                if (pro_has_residual(PRO)) rres[r][k] = ld_stream(res + (row0 + r) * r_stride + v * E);
                else rres[r][k] = Vec16{{0u, 0u, 0u, 0u}};
            } else {
                rx[r][k] = Vec16{{0u, 0u, 0u, 0u}};
                rres[r][k] = Vec16{{0u, 0u, 0u, 0u}};
            }
        }
    float2 val[2][VPT][P];
    float2 sum2[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int64_t v = (int64_t)k * blockDim.x + threadIdx.x;
        float2 bb[P];
        if (pro_has_bias(PRO)) load_params<E, kWide>(bias + v * E, bb);
        else {
#pragma unroll
            for (int q = 0; q < P; ++q) bb[q] = make_float2(0.0f, 0.0f);
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            prologue_vec<T, PRO, kFast>(rx[r][k], rres[r][k], bb, val[r][k]);
#pragma unroll
            for (int q = 0; q < P; ++q) sum2[r] = __fadd2_rn(sum2[r], val[r][k][q]);
        }
    }
    float mu[2], rs[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const float s = warp_sum(sum2[r].x + sum2[r].y);
        if (lane == 0) red_a[r][warp] = s;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) mu[r] = warp_sum(lane < nw ? red_a[r][lane] : 0.0f) * inv_hidden;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const float2 nmu = make_float2(-mu[r], -mu[r]);
        float2 ss2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < VPT; ++k)
#pragma unroll
            for (int q = 0; q < P; ++q) {
                const float2 d = __fadd2_rn(val[r][k][q], nmu);
                val[r][k][q] = d;
                ss2 = __ffma2_rn(d, d, ss2);
            }
        const float s = warp_sum(ss2.x + ss2.y);
        if (lane == 0) red_b[r][warp] = s;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        rs[r] = rsqrtf(warp_sum(lane < nw ? red_b[r][lane] : 0.0f) * inv_hidden + eps);
        if (threadIdx.x == 0 && (r == 0 || two)) {
            if (mean != nullptr) mean[row0 + r] = mu[r];
            if (rstd != nullptr) rstd[row0 + r] = rs[r];
        }
    }
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int64_t v = (int64_t)k * blockDim.x + threadIdx.x;
        float2 g[P], b[P];
        load_params<E, kWide>(gamma + v * E, g);
        load_params<E, kWide>(beta + v * E, b);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (r == 0 || two) {
                const float2 rs2 = make_float2(rs[r], rs[r]);
                float2 o[P];
#pragma unroll
                for (int q = 0; q < P; ++q) o[q] = __ffma2_rn(__fmul2_rn(val[r][k][q], rs2), g[q], b[q]);
                st_stream(y + (row0 + r) * y_stride + v * E, Elem<T>::pack2(o));
            }
        }
    }
}

// Short rows (at most L * 4 vectors): L lanes of a warp per row (L = 2 .. 32), 32 / L rows per warp, eight warps
// per CTA, the row in registers; both reductions are butterflies over the row's lanes, with no barrier.
template <typename T, typename PT, int L, int PRO>
__global__ void __launch_bounds__(256)
ln_group_kernel(const T* __restrict__ x, const T* __restrict__ res, const PT* __restrict__ bias,
                const PT* __restrict__ gamma, const PT* __restrict__ beta, T* __restrict__ y,
                float* __restrict__ mean, float* __restrict__ rstd, int64_t rows, int nvec, int64_t x_stride,
                int64_t r_stride, int64_t y_stride, float eps, float inv_hidden)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;
    constexpr int VPL = 4;
    constexpr bool kFast = sizeof(T) == 2;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t row = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * (32 / L) + lane / L;
    const bool live = row < rows;
    const int64_t r = live ? row : 0;
    const T* xr = x + r * x_stride;
    const T* rr = res + r * r_stride;
    Vec16 rx[VPL], rres[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        rx[k] = Vec16{{0u, 0u, 0u, 0u}};
        rres[k] = Vec16{{0u, 0u, 0u, 0u}};
        if (live && v < nvec) {
            rx[k] = ld_stream(xr + (int64_t)v * E);
            if (pro_has_residual(PRO)) rres[k] = ld_stream(rr + (int64_t)v * E);
        }
    }
    float2 val[VPL][P];
    float2 sum2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        const bool in = live && v < nvec;
        float2 bb[P], fx[P];
        if (pro_has_bias(PRO) && in) load_params<E, false>(bias + (int64_t)v * E, bb);
        else {
#pragma unroll
            for (int q = 0; q < P; ++q) bb[q] = make_float2(0.0f, 0.0f);
        }
        prologue_vec<T, PRO, kFast>(rx[k], rres[k], bb, fx);
#pragma unroll
        for (int q = 0; q < P; ++q) {
            float2 t = fx[q];
            if (!in) t = make_float2(0.0f, 0.0f);
            val[k][q] = t;
            sum2 = __fadd2_rn(sum2, t);
        }
    }
    float sum = sum2.x + sum2.y;
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    const float mu = sum * inv_hidden;
    const float2 nmu = make_float2(-mu, -mu);
    float2 ss2 = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const bool in = live && k * L + sub < nvec;
#pragma unroll
        for (int q = 0; q < P; ++q) {
            float2 d = __fadd2_rn(val[k][q], nmu);
            if (!in) d = make_float2(0.0f, 0.0f);
            val[k][q] = d;
            ss2 = __ffma2_rn(d, d, ss2);
        }
    }
    float ss = ss2.x + ss2.y;
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    const float rs = rsqrtf(ss * inv_hidden + eps);
    if (sub == 0 && live) {
        if (mean != nullptr) mean[row] = mu;
        if (rstd != nullptr) rstd[row] = rs;
    }
    const float2 rs2 = make_float2(rs, rs);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + sub;
        if (live && v < nvec) {
            float2 g[P], b[P], o[P];
            load_params<E, false>(gamma + (int64_t)v * E, g);
            load_params<E, false>(beta + (int64_t)v * E, b);
#pragma unroll
            for (int q = 0; q < P; ++q) o[q] = __ffma2_rn(__fmul2_rn(val[k][q], rs2), g[q], b[q]);
            st_stream(y + r * y_stride + (int64_t)v * E, Elem<T>::pack2(o));
        }
    }
}

// Rows beyond one CTA's registers, vector loads, three sweeps (sum; centred squares, walking backwards over
// what the first sweep left in the L2; output, forwards again). v is recomputed from the inputs in each
// sweep, and y is written only in the last one by the thread that read the same position, so exact aliasing
// stays safe.
template <typename T, typename PT, int PRO>
__global__ void __launch_bounds__(512)
ln_long_kernel(const T* __restrict__ x, const T* __restrict__ res, const PT* __restrict__ bias,
               const PT* __restrict__ gamma, const PT* __restrict__ beta, T* __restrict__ y,
               float* __restrict__ mean, float* __restrict__ rstd, int nvec, int64_t x_stride, int64_t r_stride,
               int64_t y_stride, float eps, float inv_hidden)
{
    constexpr int E = Elem<T>::kPerVec, P = E / 2, U = 4;
    constexpr bool kFast = sizeof(T) == 2;
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    const T* rr = res + row * r_stride;
    T* yr = y + row * y_stride;
    const int step = U * blockDim.x;
    const int nbatch = (nvec + step - 1) / step;

    // the U vectors of batch b that belong to this thread, as v = prologue(x, bias, residual); false past the end
    const uint64_t keep = l2_policy_keep(), drop = l2_policy_drop();
    auto load_batch = [&](int b, float2 (&val)[U][P], bool (&in)[U], uint64_t policy) {
        Vec16 rx[U], rres[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            in[k] = v < nvec;
            rx[k] = Vec16{{0u, 0u, 0u, 0u}};
            rres[k] = Vec16{{0u, 0u, 0u, 0u}};
            if (in[k]) {
                rx[k] = ld_stream_hint(xr + (int64_t)v * E, policy);
                if (pro_has_residual(PRO)) rres[k] = ld_stream_hint(rr + (int64_t)v * E, policy);
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            float2 bb[P];
            if (pro_has_bias(PRO) && in[k]) load_params<E, false>(bias + (int64_t)v * E, bb);
            else {
#pragma unroll
                for (int q = 0; q < P; ++q) bb[q] = make_float2(0.0f, 0.0f);
            }
            prologue_vec<T, PRO, kFast>(rx[k], rres[k], bb, val[k]);
        }
    };

    float2 sum2 = make_float2(0.0f, 0.0f);
    for (int b = 0; b < nbatch; ++b) {
        float2 val[U][P];
        bool in[U];
        load_batch(b, val, in, keep);
#pragma unroll
        for (int k = 0; k < U; ++k)
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (in[k]) sum2 = __fadd2_rn(sum2, val[k][q]);
    }
    const float mu = block_sum(sum2.x + sum2.y, red_a) * inv_hidden;
    const float2 nmu = make_float2(-mu, -mu);
    float2 ss2 = make_float2(0.0f, 0.0f);
    for (int b = nbatch - 1; b >= 0; --b) {
        float2 val[U][P];
        bool in[U];
        load_batch(b, val, in, keep);
#pragma unroll
        for (int k = 0; k < U; ++k)
#pragma unroll
            for (int q = 0; q < P; ++q) {
                const float2 d = __fadd2_rn(val[k][q], nmu);
                if (in[k]) ss2 = __ffma2_rn(d, d, ss2);
            }
    }
    const float rs = rsqrtf(block_sum(ss2.x + ss2.y, red_b) * inv_hidden + eps);
    if (threadIdx.x == 0) {
        if (mean != nullptr) mean[row] = mu;
        if (rstd != nullptr) rstd[row] = rs;
    }
    const float2 rs2 = make_float2(rs, rs);
    for (int b = 0; b < nbatch; ++b) {
        float2 val[U][P];
        bool in[U];
        load_batch(b, val, in, drop);
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            if (in[k]) {
                float2 g[P], be[P], o[P];
                load_params<E, false>(gamma + (int64_t)v * E, g);
                load_params<E, false>(beta + (int64_t)v * E, be);
#pragma unroll
                for (int q = 0; q < P; ++q) o[q] = __ffma2_rn(__fmul2_rn(__fadd2_rn(val[k][q], nmu), rs2), g[q], be[q]);
                st_stream_hint(yr + (int64_t)v * E, Elem<T>::pack2(o), drop);
            }
        }
    }
}

// Any hidden size / alignment: scalar loads, v recomputed in each of three sweeps.
template <typename T, typename PT, int PRO, bool kFast>
__device__ __forceinline__ float ln_value(const T* xr, const T* rr, const PT* bias, int64_t j)
{
    const float xv = Elem<T>::load1(xr + j);
    const float rv = pro_has_residual(PRO) ? Elem<T>::load1(rr + j) : 0.0f;
    const float bv = pro_has_bias(PRO) ? param1(bias, j) : 0.0f;
    return prologue1<PRO, kFast>(xv, bv, rv);
}

template <typename T, typename PT, int PRO>
__global__ void __launch_bounds__(256)
ln_generic_kernel(const T* __restrict__ x, const T* __restrict__ res, const PT* __restrict__ bias,
                  const PT* __restrict__ gamma, const PT* __restrict__ beta, T* __restrict__ y,
                  float* __restrict__ mean, float* __restrict__ rstd, int64_t hidden, int64_t x_stride,
                  int64_t r_stride, int64_t y_stride, float eps, float inv_hidden)
{
    constexpr bool kFast = sizeof(T) == 2;
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const T* xr = x + row * x_stride;
    const T* rr = res + row * r_stride;
    T* yr = y + row * y_stride;
    float sum = 0.0f;
    for (int64_t j = threadIdx.x; j < hidden; j += blockDim.x)
        sum += ln_value<T, PT, PRO, kFast>(xr, rr, bias, j);
    const float mu = block_sum(sum, red_a) * inv_hidden;
    float ss = 0.0f;
    for (int64_t j = threadIdx.x; j < hidden; j += blockDim.x) {
        const float d =
            ln_value<T, PT, PRO, kFast>(xr, rr, bias, j) - mu;
        ss = fmaf(d, d, ss);
    }
    const float rs = rsqrtf(block_sum(ss, red_b) * inv_hidden + eps);
    if (threadIdx.x == 0) {
        if (mean != nullptr) mean[row] = mu;
        if (rstd != nullptr) rstd[row] = rs;
    }
    for (int64_t j = threadIdx.x; j < hidden; j += blockDim.x) {
        const float d =
            ln_value<T, PT, PRO, kFast>(xr, rr, bias, j) - mu;
        Elem<T>::store1(yr + j, fmaf(d * rs, param1(gamma, j), param1(beta, j)));
    }
}

template <typename T, typename PT, int PRO>
kop_status_t launch_ln(const void* xv, const void* rv, const void* biasv, const void* gammav,
                       const void* betav, void* yv, float* mean, float* rstd, int64_t rows,
                       int64_t hidden, int64_t xs, int64_t rs, int64_t ys, float eps,
                       cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    const T* r = static_cast<const T*>(rv);
    T* y = static_cast<T*>(yv);
    const PT* bias = static_cast<const PT*>(biasv);
    const PT* gamma = static_cast<const PT*>(gammav);
    const PT* beta = static_cast<const PT*>(betav);
    constexpr int E = Elem<T>::kPerVec;
    const float inv_hidden = (float)(1.0 / (double)hidden);
    if (rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    const bool vec = vec_ok(x, hidden, xs, sizeof(T)) && (!pro_has_residual(PRO) || vec_ok(r, hidden, rs, sizeof(T))) &&
                     vec_ok(y, hidden, ys, sizeof(T)) && (!pro_has_bias(PRO) || aligned_to(bias, 16)) &&
                     aligned_to(gamma, 16) && aligned_to(beta, 16);
    const int64_t nvec64 = hidden / E;
    // rows of at most 128 vectors: lanes-per-row kernel (bf16 rows of 64 / 256 / 512 columns ran at 0.5 / 1.9 /
    // 3.8 TB/s with a CTA per row, 5 - 6 TB/s this way)
    // (16-bit rows of 512 columns and up that can go two to a CTA do better there: the row-pair kernel fetches
    // the fp32 parameters once for two rows, and those loads, not HBM, bound the lanes-per-row kernel on 16-bit
    // data: 4.9 - 5.0 TB/s against 6.2)
    const bool pair_ok = vec && (nvec64 % (16 / E)) == 0 && ((nvec64 / (16 / E)) % 32) == 0 &&
                         nvec64 / (16 / E) >= (sizeof(T) == 2 ? 32 : 128) && nvec64 / (16 / E) <= 320 &&
                         rows >= 8 * (int64_t)sm_count();
    if (vec && nvec64 <= 128 && !pair_ok) {
        const int nvec = (int)nvec64;
        const int lanes = nvec > 64 ? 32 : nvec > 32 ? 16 : nvec > 16 ? 8 : nvec > 8 ? 4 : 2;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const unsigned grid = (unsigned)((rows + rows_per_cta - 1) / rows_per_cta);
#define KOP_LN_GROUP(L)                                                                                           \
    ln_group_kernel<T, PT, L, PRO><<<grid, 256, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, rows, nvec, xs, rs, \
                                                             ys, eps, inv_hidden)
        switch (lanes) {
        case 32: KOP_LN_GROUP(32); break;
        case 16: KOP_LN_GROUP(16); break;
        case 8: KOP_LN_GROUP(8); break;
        case 4: KOP_LN_GROUP(4); break;
        default: KOP_LN_GROUP(2); break;
        }
#undef KOP_LN_GROUP
        return launch_status();
    }
    if (vec && hidden <= kMaxRegisterRow) {
        const int nvec = (int)nvec64;
        // 32 values per thread (hidden 4096 -> 128-thread CTAs, eight 16-byte loads in flight per
        // thread and ~8 CTAs per SM); short rows use fewer, rows beyond 512 threads' worth use 64.
        const bool wide = sizeof(PT) == 4 && E == 8 && (!pro_has_bias(PRO) || aligned_to(bias, 32)) && aligned_to(gamma, 32) &&
                          aligned_to(beta, 32);
        // Rows of up to 5120 elements that split evenly into 16 values per thread (from 512 elements for 16-bit data,
        // 2048 for fp32) go two per CTA
        // (parameters fetched once per pair) once there are enough pairs to fill the GPU. Longer rows do
        // better one per CTA with 32 values a thread (bf16 [8192, 8192]: 86 us against 106 us; 6144: 66
        // against 90), where the pair kernel's 384- to 512-thread CTAs leave one CTA per SM.
        if constexpr (PRO == kProNone && sizeof(T) == 2) {
            // Plain LayerNorm of 16-bit rows of 2048 to 5120 columns: row pairs with 32 values a thread, CTAs of 64 to
            // 160 threads at up to 102 registers, four to an SM. With one input stream the 256-thread pairs of 16
            // values left too few bytes in flight (bf16 rows of 2048 / 3072 / 4096 / 5120 columns, fp32 parameters:
            // 5.9 / 5.5 / 5.4 / 5.1 TB/s; this way 6.1 / 5.9 / 5.9 / 5.8, with 16-bit parameters 6.0 / 5.9 / 6.0 / 5.9).
            // The same shape with 192 to 256 threads (6144 to 8192 columns) at three CTAs per SM (85 registers, a few
            // spilled words): 6144 / 8192 columns 5.2 / 5.1 with one row per CTA, 5.8 / 5.4 this way (at two CTAs per SM
            // and 128 registers it loses: 4.5 / 5.0).
            if (nvec % 4 == 0 && (nvec / 4) % 32 == 0 && nvec / 4 > 160 && nvec / 4 <= 256 && rows >= 8 * (int64_t)sm_count()) {
                const int threads4 = nvec / 4;
                const unsigned grid = (unsigned)((rows + 1) / 2);
                if (wide)
                    ln_pair_kernel<T, PT, 32 / E, true, 256, PRO><<<grid, threads4, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, rows, xs, rs, ys, eps, inv_hidden);
                else
                    ln_pair_kernel<T, PT, 32 / E, false, 256, PRO><<<grid, threads4, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, rows, xs, rs, ys, eps, inv_hidden);
                return launch_status();
            }
            if (nvec % 4 == 0 && (nvec / 4) % 32 == 0 && nvec / 4 >= 64 && nvec / 4 <= 160 && rows >= 8 * (int64_t)sm_count()) {
                const int threads4 = nvec / 4;
                const unsigned grid = (unsigned)((rows + 1) / 2);
                if (wide)
                    ln_pair_kernel<T, PT, 32 / E, true, 160, PRO><<<grid, threads4, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, rows, xs, rs, ys, eps, inv_hidden);
                else
                    ln_pair_kernel<T, PT, 32 / E, false, 160, PRO><<<grid, threads4, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, rows, xs, rs, ys, eps, inv_hidden);
                return launch_status();
            }
        }
        {
            const int vpt2 = 16 / E;
            const int threads2 = nvec / vpt2;
            // (plain LayerNorm with 16-bit parameters is the exception: one input stream and two half-size parameter
            // vectors leave nothing for the pair to save, and 128-thread CTAs with 32 values a thread, eight to an SM,
            // run bf16 rows of 4096 / 5120 columns at 5.9 / 5.6 TB/s against 5.6 / 5.2)
            if (pair_ok && !(PRO == kProNone && sizeof(PT) == 2 && nvec64 / (16 / E) >= 128)) {
                const unsigned grid = (unsigned)((rows + 1) / 2);
#define KOP_LN_PAIR(W, MT)                                                                              \
    ln_pair_kernel<T, PT, 16 / E, W, MT, PRO><<<grid, threads2, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, \
                                                                    rows, xs, rs, ys, eps, inv_hidden)
                if (threads2 <= 256) { if (wide) KOP_LN_PAIR(true, 256); else KOP_LN_PAIR(false, 256); }
                else { if (wide) KOP_LN_PAIR(true, 512); else KOP_LN_PAIR(false, 512); }
#undef KOP_LN_PAIR
                return launch_status();
            }
        }
        int vals = 32;
        if (hidden <= 1024) vals = 16;
        if (hidden <= 256) vals = 8;
        if ((nvec + vals / E - 1) / (vals / E) > max_threads_for(vals)) vals = 64;
        const int vpt = vals / E;
        const int threads = ((nvec + vpt - 1) / vpt + 31) / 32 * 32;
        const bool full = (nvec % vpt) == 0 && (nvec / vpt) == threads;
#define KOP_LN_LAUNCH(V, F, W)                                                                    \
    ln_block_kernel<T, PT, V, F, W, PRO><<<(unsigned)rows, threads, 0, stream>>>(x, r, bias, gamma, beta, y, mean, \
                                                                        rstd, nvec, xs, rs, ys, eps, inv_hidden)
#define KOP_LN(V)                                             \
    do {                                                      \
        if (full && wide) KOP_LN_LAUNCH(V, true, true);       \
        else if (full) KOP_LN_LAUNCH(V, true, false);         \
        else if (wide) KOP_LN_LAUNCH(V, false, true);         \
        else KOP_LN_LAUNCH(V, false, false);                  \
    } while (0)
        switch (vals) {
        case 8: KOP_LN(8 / E); break;
        case 16: KOP_LN(16 / E); break;
        case 32: KOP_LN(32 / E); break;
        default: KOP_LN(64 / E); break;
        }
#undef KOP_LN_LAUNCH
#undef KOP_LN
        return launch_status();
    }
    if (vec && nvec64 <= 0x7FFFFFFF) {
        ln_long_kernel<T, PT, PRO><<<(unsigned)rows, 512, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd, (int)nvec64,
                                                                      xs, rs, ys, eps, inv_hidden);
        return launch_status();
    }
    ln_generic_kernel<T, PT, PRO><<<(unsigned)rows, 256, 0, stream>>>(x, r, bias, gamma, beta, y, mean, rstd,
                                                             hidden, xs, rs, ys, eps, inv_hidden);
    return launch_status();
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

// One validated entry for every LayerNorm variant. `pro` is one of the kPro* values; pdtype is KOP_F32 or, for
// 16-bit data, the data type itself (bias / gamma / beta then hold elements of that type).
kop_status_t ln_entry(int pro, const void* x, const void* residual, const void* bias, const void* gamma,
                      const void* beta, void* y, float* mean, float* rstd, int64_t rows, int64_t hidden,
                      int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride, float eps, kop_dtype_t dtype,
                      kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!dtype_ok(dtype) || !dtype_ok(pdtype) || (pdtype != KOP_F32 && pdtype != dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    if (pro < 0 || pro > 3) return KOP_ERR_BAD_SHAPE;
    const bool has_res = pro_has_residual(pro), has_bias = pro_has_bias(pro);
    kop_status_t st = check_rows_cols(rows, hidden);
    if (st != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || (has_res && !residual) || (has_bias && !bias) || !gamma || !beta || !y) return KOP_ERR_NULL_POINTER;
    if ((st = check_row_stride(x_row_stride, hidden, rows)) != KOP_OK) return st;
    if (has_res && (st = check_row_stride(res_row_stride, hidden, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, hidden, rows)) != KOP_OK) return st;
    if (!(eps >= 0.0f)) return KOP_ERR_BAD_SHAPE;
    const int esz = elem_size(dtype), psz = elem_size(pdtype);
    if (!aligned_to(x, esz) || (has_res && !aligned_to(residual, esz)) || !aligned_to(y, esz) ||
        (has_bias && !aligned_to(bias, psz)) || !aligned_to(gamma, psz) || !aligned_to(beta, psz) ||
        (mean && !aligned_to(mean, 4)) || (rstd && !aligned_to(rstd, 4)))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, hidden, esz, true) ||
        (has_res && !alias_ok(residual, res_row_stride, y, y_row_stride, rows, hidden, esz, true)))
        return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    if (!has_res) {                                          // never loaded; keep the pointer arithmetic valid
        residual = x;
        res_row_stride = x_row_stride;
    }
#define KOP_LN_GO(T, PT, PRO) \
    return launch_ln<T, PT, PRO>(x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden, x_row_stride, \
                                 res_row_stride, y_row_stride, eps, s)
#define KOP_LN_TYPES(PRO)                                                         \
    do {                                                                          \
        if (dtype == KOP_F32) KOP_LN_GO(float, float, PRO);                       \
        if (dtype == KOP_BF16) {                                                  \
            if (pdtype == KOP_F32) KOP_LN_GO(__nv_bfloat16, float, PRO);          \
            KOP_LN_GO(__nv_bfloat16, __nv_bfloat16, PRO);                         \
        }                                                                         \
        if (pdtype == KOP_F32) KOP_LN_GO(__half, float, PRO);                     \
        KOP_LN_GO(__half, __half, PRO);                                           \
    } while (0)
    switch (pro) {
    case kProBiasGeluResidual: KOP_LN_TYPES(kProBiasGeluResidual);
    case kProResidual: KOP_LN_TYPES(kProResidual);
    case kProNone: KOP_LN_TYPES(kProNone);
    default: KOP_LN_TYPES(kProBiasErfGeluResidual);
    }
#undef KOP_LN_TYPES
#undef KOP_LN_GO
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_bias_gelu_residual_layernorm(
    const void* x, const void* residual, const float* bias, const float* gamma, const float* beta,
    void* y, float* mean, float* rstd, int64_t rows, int64_t hidden, int64_t x_row_stride,
    int64_t res_row_stride, int64_t y_row_stride, float eps, kop_dtype_t dtype, kop_stream_t stream)
{
    return kop::ln_entry(kop::kProBiasGeluResidual, x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden,
                         x_row_stride, res_row_stride, y_row_stride, eps, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_bias_erfgelu_residual_layernorm(
    const void* x, const void* residual, const float* bias, const float* gamma, const float* beta,
    void* y, float* mean, float* rstd, int64_t rows, int64_t hidden, int64_t x_row_stride,
    int64_t res_row_stride, int64_t y_row_stride, float eps, kop_dtype_t dtype, kop_stream_t stream)
{
    return kop::ln_entry(kop::kProBiasErfGeluResidual, x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden,
                         x_row_stride, res_row_stride, y_row_stride, eps, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_residual_layernorm(const void* x, const void* residual, const float* gamma,
                                               const float* beta, void* y, float* mean, float* rstd,
                                               int64_t rows, int64_t hidden, int64_t x_row_stride,
                                               int64_t res_row_stride, int64_t y_row_stride, float eps,
                                               kop_dtype_t dtype, kop_stream_t stream)
{
    return kop::ln_entry(residual ? kop::kProResidual : kop::kProNone, x, residual, nullptr, gamma, beta, y, mean, rstd,
                         rows, hidden, x_row_stride, res_row_stride, y_row_stride, eps, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_layernorm_ex(const void* x, const void* residual, const void* bias, const void* gamma,
                                         const void* beta, void* y, float* mean, float* rstd, int64_t rows,
                                         int64_t hidden, int64_t x_row_stride, int64_t res_row_stride,
                                         int64_t y_row_stride, float eps, int prologue, kop_dtype_t dtype,
                                         kop_dtype_t param_dtype, kop_stream_t stream)
{
    return kop::ln_entry(prologue, x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden, x_row_stride,
                         res_row_stride, y_row_stride, eps, dtype, param_dtype, stream);
}
