// Shared host validation helpers and device building blocks of libkop (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kop.h"

namespace kop {

// ------------------------------------------------------------------------------------------
// Host side: static validation (the paper's Gate 1 analogue). Pure integer checks, no CUDA call.
// ------------------------------------------------------------------------------------------

inline bool dtype_ok(kop_dtype_t d) { return d == KOP_F32 || d == KOP_BF16 || d == KOP_F16; }
inline int elem_size(kop_dtype_t d) { return d == KOP_F32 ? 4 : 2; }
inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
// Parameter vectors are fp32 or stored in the data type (a 16-bit model keeps its biases and norm weights in that type).
inline bool param_dtype_ok(kop_dtype_t dtype, kop_dtype_t pdtype)
{
    return dtype_ok(dtype) && dtype_ok(pdtype) && (pdtype == KOP_F32 || pdtype == dtype);
}

// CALL(T, PT) for the C++ types behind (dtype, pdtype); the caller has checked param_dtype_ok. CALL is a
// function-like macro that expands to an expression of type kop_status_t.
#define KOP_DISPATCH_TYPES(dtype, pdtype, CALL)                                                              \
    ((dtype) == KOP_F32    ? CALL(float, float)                                                              \
     : (dtype) == KOP_BF16 ? ((pdtype) == KOP_F32 ? CALL(__nv_bfloat16, float) : CALL(__nv_bfloat16, __nv_bfloat16)) \
                           : ((pdtype) == KOP_F32 ? CALL(__half, float) : CALL(__half, __half)))

// Largest product / offset we accept: keeps every byte offset inside int64.
constexpr int64_t kMaxElems = (int64_t)1 << 46;

inline kop_status_t check_rows_cols(int64_t rows, int64_t cols)
{
    if (rows < 0 || cols <= 0) return KOP_ERR_BAD_SHAPE;
    if (rows > kMaxElems || cols > kMaxElems) return KOP_ERR_BAD_SHAPE;
    return KOP_OK;
}

inline kop_status_t check_row_stride(int64_t stride, int64_t cols, int64_t rows)
{
    if (stride < cols) return KOP_ERR_BAD_STRIDE;
    if (stride > kMaxElems) return KOP_ERR_BAD_STRIDE;
    // rows * stride must not overflow what we can address
    if (rows > 0 && stride > kMaxElems / (rows > 0 ? rows : 1)) return KOP_ERR_BAD_SHAPE;
    return KOP_OK;
}

// Byte span [lo, hi) touched by a strided 2-D tensor.
inline void span_of(const void* base, int64_t rows, int64_t cols, int64_t stride, int esz,
                    uintptr_t* lo, uintptr_t* hi)
{
    *lo = reinterpret_cast<uintptr_t>(base);
    *hi = *lo + (rows > 0 ? (uintptr_t)(((rows - 1) * stride + cols) * esz) : 0);
}

// Output `out` may be exactly `in` (same base and stride) or disjoint from it.
inline bool alias_ok(const void* in, int64_t in_stride, const void* out, int64_t out_stride,
                     int64_t rows, int64_t cols, int esz, bool exact_allowed)
{
    if (rows == 0) return true;
    if (in == out) return exact_allowed && in_stride == out_stride;
    uintptr_t a0, a1, b0, b1;
    span_of(in, rows, cols, in_stride, esz, &a0, &a1);
    span_of(out, rows, cols, out_stride, esz, &b0, &b1);
    return a1 <= b0 || b1 <= a0;
}

// True when a [rows, cols] tensor can be read with 16-byte vectors row by row.
inline bool vec_ok(const void* base, int64_t cols, int64_t stride, int esz)
{
    const int per = 16 / esz;
    return aligned_to(base, 16) && (cols % per) == 0 && (stride % per) == 0;
}

// Checks that the current device is a B200-class part (compute capability 10.x); the library is
// compiled for sm_100a only. Result is cached per device ordinal.
kop_status_t check_device();

// SM count of the current device (valid after check_device() succeeded on it; 148 otherwise).
int sm_count();

// Maps the last launch error (non-sticky peek) to a status.
inline kop_status_t launch_status()
{
    return cudaGetLastError() == cudaSuccess ? KOP_OK : KOP_ERR_CUDA;
}

inline cudaStream_t as_stream(kop_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }

// ------------------------------------------------------------------------------------------
// Device side
// ------------------------------------------------------------------------------------------
#ifdef __CUDACC__

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Row-in-registers kernels keep `vals` fp32 values per thread; the CTA size they may be launched
// with shrinks as that count grows so the row always fits the register file without spills.
constexpr int max_threads_for(int vals) { return vals <= 16 ? 1024 : (vals <= 32 ? 512 : 256); }
// Longest row (in elements) a single CTA can hold in registers under max_threads_for().
constexpr int64_t kMaxRegisterRow = 16384;

struct __align__(16) Vec16 {
    uint32_t w[4];
};

// Streaming 128-bit global load: data tensors are touched exactly once, so they bypass L1
// allocation and leave L1 to the small parameter vectors that every row re-reads.
// (Not .nc: outputs may alias inputs exactly, so the location is not read-only.)
__device__ __forceinline__ Vec16 ld_stream(const void* p)
{
    Vec16 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3])
                 : "l"(p));
    return v;
}

// 128-bit global store of a result that this kernel never reads back.
__device__ __forceinline__ void st_stream(void* p, const Vec16& v)
{
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3])
                 : "memory");
}

// L2 eviction policies for the kernels that read a row twice: the first sweep asks the L2 to keep what it reads
// (evict_last), the second sweep and the output stores mark their lines as the first to go (evict_first), so that
// the rows in flight, not the finished ones, occupy the L2.
__device__ __forceinline__ uint64_t l2_policy_keep()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_drop()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ Vec16 ld_stream_hint(const void* p, uint64_t policy)
{
    Vec16 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3])
                 : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ void st_stream_hint(void* p, const Vec16& v, uint64_t policy)
{
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;"
                 :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "l"(policy)
                 : "memory");
}

__device__ __forceinline__ float4 ldg_f4(const float* p)
{
    return __ldg(reinterpret_cast<const float4*>(p));
}

// Read-only 256-bit load (sm_100): eight consecutive floats per lane in one request. `p` must be
// 32-byte aligned.
struct __align__(32) Float8 {
    float f[8];
};
__device__ __forceinline__ Float8 ldg_f8(const float* p)
{
    Float8 r;
    asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.f[0]), "=f"(r.f[1]), "=f"(r.f[2]), "=f"(r.f[3]), "=f"(r.f[4]), "=f"(r.f[5]),
                   "=f"(r.f[6]), "=f"(r.f[7])
                 : "l"(p));
    return r;
}

// The E fp32 parameters that belong to one data vector, as E/2 packed pairs. kWide (E == 8 only)
// uses one 256-bit load; otherwise E/4 128-bit loads.
template <int E, bool kWide>
__device__ __forceinline__ void load_params(const float* p, float2 (&out)[E / 2])
{
    if constexpr (kWide && E == 8) {
        const Float8 t = ldg_f8(p);
#pragma unroll
        for (int q = 0; q < 4; ++q) out[q] = make_float2(t.f[2 * q], t.f[2 * q + 1]);
    } else {
#pragma unroll
        for (int q = 0; q < E / 4; ++q) {
            const float4 t = ldg_f4(p + 4 * q);
            out[2 * q] = make_float2(t.x, t.y);
            out[2 * q + 1] = make_float2(t.z, t.w);
        }
    }
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Element traits: how many elements a 16-byte vector holds and how to widen / narrow them.
template <typename T>
struct Elem;

template <>
struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ __forceinline__ static void unpack(const Vec16& v, float (&f)[4])
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) f[i] = __uint_as_float(v.w[i]);
    }
    __device__ __forceinline__ static Vec16 pack(const float (&f)[4])
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) v.w[i] = __float_as_uint(f[i]);
        return v;
    }
    __device__ __forceinline__ static void unpack2(const Vec16& v, float2 (&f)[2])
    {
        f[0] = make_float2(__uint_as_float(v.w[0]), __uint_as_float(v.w[1]));
        f[1] = make_float2(__uint_as_float(v.w[2]), __uint_as_float(v.w[3]));
    }
    __device__ __forceinline__ static Vec16 pack2(const float2 (&f)[2])
    {
        Vec16 v;
        v.w[0] = __float_as_uint(f[0].x);
        v.w[1] = __float_as_uint(f[0].y);
        v.w[2] = __float_as_uint(f[1].x);
        v.w[3] = __float_as_uint(f[1].y);
        return v;
    }
    static constexpr bool kMixedAdd = false;
    __device__ __forceinline__ static float load1(const float* p) { return *p; }
    __device__ __forceinline__ static void store1(float* p, float f) { *p = f; }
    __device__ __forceinline__ static Vec16 fill_neg_inf()
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) v.w[i] = 0xFF800000u;
        return v;
    }
};

template <>
struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    // bf16 is the top half of an fp32: widening is a shift / mask of the packed word.
    __device__ __forceinline__ static void unpack(const Vec16& v, float (&f)[8])
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(v.w[i] << 16);
            f[2 * i + 1] = __uint_as_float(v.w[i] & 0xFFFF0000u);
        }
    }
    // Round to nearest even, two values per cvt.
    __device__ __forceinline__ static Vec16 pack(const float (&f)[8])
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            v.w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        return v;
    }
    __device__ __forceinline__ static void unpack2(const Vec16& v, float2 (&f)[4])
    {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            f[i] = make_float2(__uint_as_float(v.w[i] << 16), __uint_as_float(v.w[i] & 0xFFFF0000u));
    }
    __device__ __forceinline__ static Vec16 pack2(const float2 (&f)[4])
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[i].x, f[i].y);
            v.w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        return v;
    }
    // widen(w) + c for both halves of a packed word with the mixed-precision add of this target (the 16-bit
    // operand is widened exactly inside the instruction, one rounding: bit-identical to unpacking first). It
    // replaces the two mask / shift instructions plus a packed add by two adds.
    static constexpr bool kMixedAdd = true;
    __device__ __forceinline__ static float2 add_widen2(uint32_t w, float2 c)
    {
        float2 r;
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; add.rn.f32.bf16 %0, lo, %3; add.rn.f32.bf16 %1, hi, %4; }"
            : "=f"(r.x), "=f"(r.y) : "r"(w), "f"(c.x), "f"(c.y));
        return r;
    }
    __device__ __forceinline__ static void unpack_pair(uint32_t w, float2& f)
    {
        f = make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    }
    __device__ __forceinline__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    __device__ __forceinline__ static void store1(__nv_bfloat16* p, float f) { *p = __float2bfloat16_rn(f); }
    __device__ __forceinline__ static Vec16 fill_neg_inf()
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) v.w[i] = 0xFF80FF80u;
        return v;
    }
};

template <>
struct Elem<__half> {
    static constexpr int kPerVec = 8;
    __device__ __forceinline__ static void unpack(const Vec16& v, float (&f)[8])
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&v.w[i]));
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
    // Round to nearest even, two values per cvt; values beyond 65504 become infinity, as IEEE requires.
    __device__ __forceinline__ static Vec16 pack(const float (&f)[8])
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 h = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
            v.w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        return v;
    }
    __device__ __forceinline__ static void unpack2(const Vec16& v, float2 (&f)[4])
    {
#pragma unroll
        for (int i = 0; i < 4; ++i) f[i] = __half22float2(*reinterpret_cast<const __half2*>(&v.w[i]));
    }
    __device__ __forceinline__ static Vec16 pack2(const float2 (&f)[4])
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 h = __floats2half2_rn(f[i].x, f[i].y);
            v.w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        return v;
    }
    static constexpr bool kMixedAdd = true;
    __device__ __forceinline__ static float2 add_widen2(uint32_t w, float2 c)
    {
        float2 r;
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; add.rn.f32.f16 %0, lo, %3; add.rn.f32.f16 %1, hi, %4; }"
            : "=f"(r.x), "=f"(r.y) : "r"(w), "f"(c.x), "f"(c.y));
        return r;
    }
    __device__ __forceinline__ static void unpack_pair(uint32_t w, float2& f)
    {
        f = __half22float2(*reinterpret_cast<const __half2*>(&w));
    }
    __device__ __forceinline__ static float load1(const __half* p) { return __half2float(*p); }
    __device__ __forceinline__ static void store1(__half* p, float f) { *p = __float2half_rn(f); }
    __device__ __forceinline__ static Vec16 fill_neg_inf()
    {
        Vec16 v;
#pragma unroll
        for (int i = 0; i < 4; ++i) v.w[i] = 0xFC00FC00u;
        return v;
    }
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// A row of any length and alignment as head elements (up to the first 16-byte boundary), whole 16-byte vectors
// and tail elements: at most 2 (E - 1) edge elements outside the vectors.
template <typename T>
struct RowSplit {
    int head, nvec, tail;
    __device__ __forceinline__ int edges() const { return head + tail; }
    // column of edge element i (0 .. head + tail - 1)
    __device__ __forceinline__ int edge_col(int i) const
    {
        return i < head ? i : head + nvec * Elem<T>::kPerVec + (i - head);
    }
};

template <typename T>
__device__ __forceinline__ RowSplit<T> row_split(const T* row, int64_t cols)
{
    constexpr int E = Elem<T>::kPerVec;
    RowSplit<T> r;
    int head = (int)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(row) & 15u)) & 15u) / (unsigned)sizeof(T));
    if ((int64_t)head > cols) head = (int)cols;
    r.head = head;
    r.nvec = (int)((cols - head) / E);
    r.tail = (int)(cols - head) - r.nvec * E;
    return r;
}

// Block-wide sum / max with ONE barrier: every warp publishes its partial in `slots` (>= 32
// floats of shared memory, a different array for each back-to-back reduction so no second
// barrier is needed), then every thread folds the published partials in slot order. The
// result is identical in all threads and does not depend on scheduling.
__device__ __forceinline__ float block_sum(float v, float* slots)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    if (nw == 1) return v;
    if (lane == 0) slots[warp] = v;
    __syncthreads();
    float t = lane < nw ? slots[lane] : 0.0f;
    return warp_sum(t);
}
__device__ __forceinline__ float block_max(float v, float* slots)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    if (nw == 1) return v;
    if (lane == 0) slots[warp] = v;
    __syncthreads();
    float t = lane < nw ? slots[lane] : -INFINITY;
    return warp_max(t);
}


// Rows shorter than a CTA's tile: the vectors of a [rows, nvec] tensor are numbered row after row and a CTA
// takes a run of them whatever rows they fall in. Position of vector g (g < rows * nvec).
__device__ __forceinline__ void flat_position(int64_t g, int nvec, int64_t* row, int* v)
{
    if (g <= 0xFFFFFFFFLL) {                                 // one 32-bit division
        const unsigned r = (unsigned)g / (unsigned)nvec;
        *row = r;
        *v = (int)((unsigned)g - r * (unsigned)nvec);
    } else {
        const int64_t r = g / nvec;
        *row = r;
        *v = (int)(g - r * nvec);
    }
}

// Parameter vectors stored in a 16-bit data type: the eight that go with one data vector are one 16-byte
// load (half the bytes and L1 wavefronts of fp32 parameters). kWide has no meaning here.
template <int E, bool kWide, typename PT>
__device__ __forceinline__ void load_params(const PT* p, float2 (&out)[E / 2])
{
    static_assert(E == 8 && sizeof(PT) == 2, "16-bit parameters go with 16-bit data");
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    Elem<PT>::unpack2(Vec16{{t.x, t.y, t.z, t.w}}, out);
}
// Four consecutive parameters as fp32 (16-byte aligned for fp32, 8-byte for 16-bit parameters).
__device__ __forceinline__ float4 ldg_p4(const float* p) { return ldg_f4(p); }
__device__ __forceinline__ float4 ldg_p4(const __nv_bfloat16* p)
{
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xFFFF0000u), __uint_as_float(t.y << 16),
                       __uint_as_float(t.y & 0xFFFF0000u));
}
__device__ __forceinline__ float4 ldg_p4(const __half* p)
{
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&t.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&t.y));
    return make_float4(a.x, a.y, b.x, b.y);
}
// One parameter as fp32.
__device__ __forceinline__ float param1(const float* p, int64_t j) { return __ldg(p + j); }
__device__ __forceinline__ float param1(const __nv_bfloat16* p, int64_t j) { return Elem<__nv_bfloat16>::load1(p + j); }
__device__ __forceinline__ float param1(const __half* p, int64_t j) { return Elem<__half>::load1(p + j); }

// erf(x) by the rational-times-Gaussian form of Abramowitz and Stegun 7.1.26 (absolute error below 1.5e-7 in exact
// arithmetic, a few 1e-7 with the hardware reciprocal and exponential): one reciprocal, one ex2 and eight FMA-pipe
// instructions where the library erff costs about twenty-five with a branch. GELU multiplies it by u / 2, so the
// result stays well inside the fp32 tolerance; NaN and infinities come out as erff gives them.
__device__ __forceinline__ float erf_fast(float x)
{
    const float ax = fabsf(x);
    float t;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, ax, 1.0f)));
    float p = fmaf(1.061405429f, t, -1.453152027f);
    p = fmaf(p, t, 1.421413741f);
    p = fmaf(p, t, -0.284496736f);
    p = fmaf(p, t, 0.254829592f);
    p *= t;
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-ax * ax * 1.4426950408889634f));
    return copysignf(fmaf(-p, e, 1.0f), x);
}

// ---- thread-block clusters: distributed shared memory between the CTAs of a cluster ----------------------
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ void store_to_cluster_cta(float* local_slot, uint32_t cta, float v)
{
    const uint32_t la = (uint32_t)__cvta_generic_to_shared(local_slot);
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(cta));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}

__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// A block-reduced value (the same in every thread of the CTA) summed over the CTAs of a cluster: every CTA writes
// its value into slot [rank] of every CTA's `slots`, one hardware cluster barrier, and each CTA adds the slots in
// rank order (a fixed order: the same result in every CTA and from run to run). Every thread of every CTA of
// the cluster must call it; `slots` holds at least csize floats and is used for one call only.
__device__ __forceinline__ float cluster_sum(float v, float* slots, uint32_t rank, uint32_t csize)
{
    if (threadIdx.x < csize) store_to_cluster_cta(&slots[rank], threadIdx.x, v);
    cluster_barrier();
    float r = 0.0f;
    for (uint32_t i = 0; i < csize; ++i) r += slots[i];
    return r;
}

#endif  // __CUDACC__

}  // namespace kop
