// kop_reduce_rows: sum / mean / max (+ argmax) / min (+ argmin) / logsumexp of every row in one read-only
// pass. Rows beyond 16 KB get a CTA each (batches of four 16-byte vectors per thread in flight, one-barrier
// block merge); shorter rows get 4 to 32 lanes of a warp each, sixteen vectors a lane where the row has them,
// so that the butterfly merge (the per-row cost) has two to five steps and no barrier. Per-thread partial results
// are merged in a fixed order, so results do not depend on scheduling; max / min and their indices are exact
// (first position on ties; a NaN outranks every number and the first NaN's position is reported).
#include <climits>

#include "kop_common.cuh"

namespace kop {
namespace {

enum { kOpSum = 0, kOpMean = 1, kOpMax = 2, kOpMin = 3, kOpLse = 4 };

// Partial result of a set of elements. Which fields are live depends on OP (dead ones fold away).
template <int OP>
struct Acc {
    float a;        // sum / mean: the sum. max / min: the best value. logsumexp: the running maximum m
    float s;        // logsumexp: sum of exp(x - m)
    int idx;        // max / min: position of the best value
    int nan_idx;    // max / min / logsumexp: position of the first NaN, INT_MAX if none
    // max / min on the vector path: the first vector that holds the thread's best value (or its first NaN) and
    // that vector's number; the element position is looked up once, after the sweep (resolve())
    Vec16 best_raw;
    int best_vec;

    __device__ __forceinline__ void init()
    {
        a = (OP == kOpMax || OP == kOpLse) ? -INFINITY : (OP == kOpMin ? INFINITY : 0.0f);
        s = 0.0f;
        idx = INT_MAX;
        nan_idx = INT_MAX;
        best_vec = -1;
    }
    // elements must arrive in increasing position within a thread (first occurrence wins by strict compare)
    __device__ __forceinline__ void add(float v, int j)
    {
        if (OP == kOpSum || OP == kOpMean) {
            a += v;
        } else if (OP == kOpMax || OP == kOpMin) {
            if (v != v) nan_idx = min(nan_idx, j);
            if (OP == kOpMax ? v > a : v < a) {
                a = v;
                idx = j;
            } else if (idx == INT_MAX && v == a) {     // the very first element equal to the identity (+-inf)
                idx = j;
            }
        }
    }
    // logsumexp takes a whole batch: one rescale per batch instead of per element
    template <int N>
    __device__ __forceinline__ void add_batch_lse(const float (&v)[N], int count)
    {
        float bm = -INFINITY;
#pragma unroll
        for (int e = 0; e < N; ++e)
            if (e < count) {
                bm = fmaxf(bm, v[e]);
                if (v[e] != v[e]) nan_idx = 0;
            }
        const float m2 = fmaxf(a, bm);
        const float off = m2 == -INFINITY ? 0.0f : m2;          // all -inf so far: avoid inf - inf
        float t = 0.0f;
#pragma unroll
        for (int e = 0; e < N; ++e)
            if (e < count) t += ex2_approx((v[e] - off) * kLog2e);
        s = s * ex2_approx((a - off) * kLog2e) + t;
        a = m2;
    }
    // Vector path of max / min: `ve` is the vector's extreme, NaN if it holds a NaN. A NaN outranks every
    // number and then sticks; otherwise strict improvement, so the first vector with the best value is kept.
    __device__ __forceinline__ void add_vector_extreme(float ve, const Vec16& raw, int vec)
    {
        const bool take = best_vec < 0 || ((ve != ve) ? !(a != a) : (OP == kOpMax ? ve > a : ve < a));
        if (take) {
            a = ve;
            best_vec = vec;
            best_raw = raw;
        }
    }
    template <typename T>
    __device__ __forceinline__ void resolve()
    {
        constexpr int E = Elem<T>::kPerVec;
        if (best_vec < 0) return;
        float f[E];
        Elem<T>::unpack(best_raw, f);
        const bool is_nan = a != a;
        int e0 = E - 1;
#pragma unroll
        for (int e = E - 1; e >= 0; --e)
            if (is_nan ? f[e] != f[e] : f[e] == a) e0 = e;
        if (is_nan) {
            nan_idx = best_vec * E + e0;
            a = OP == kOpMax ? -INFINITY : INFINITY;           // back to the identity: the NaN lives in nan_idx
            idx = INT_MAX;
        } else {
            idx = best_vec * E + e0;
        }
    }
    __device__ __forceinline__ void merge(const Acc& o)
    {
        if (OP == kOpSum || OP == kOpMean) {
            a += o.a;
        } else if (OP == kOpMax || OP == kOpMin) {
            nan_idx = min(nan_idx, o.nan_idx);
            const bool better = OP == kOpMax ? o.a > a : o.a < a;
            if (better || (o.a == a && o.idx < idx)) {
                a = o.a;
                idx = o.idx;
            }
        } else {
            nan_idx = min(nan_idx, o.nan_idx);
            const float m2 = fmaxf(a, o.a);
            const float off = m2 == -INFINITY ? 0.0f : m2;
            s = s * ex2_approx((a - off) * kLog2e) + o.s * ex2_approx((o.a - off) * kLog2e);
            a = m2;
        }
    }
    __device__ __forceinline__ Acc shuffled(int o) const
    {
        Acc r;
        r.a = __shfl_xor_sync(0xFFFFFFFFu, a, o);
        r.s = OP == kOpLse ? __shfl_xor_sync(0xFFFFFFFFu, s, o) : 0.0f;
        r.idx = (OP == kOpMax || OP == kOpMin) ? __shfl_xor_sync(0xFFFFFFFFu, idx, o) : INT_MAX;
        r.nan_idx = (OP >= kOpMax) ? __shfl_xor_sync(0xFFFFFFFFu, nan_idx, o) : INT_MAX;
        return r;
    }
    __device__ __forceinline__ float value(float inv_cols) const
    {
        if (OP == kOpSum) return a;
        if (OP == kOpMean) return a * inv_cols;
        if (nan_idx != INT_MAX) return __int_as_float(0x7FC00000);
        if (OP == kOpLse) return (a == INFINITY || a == -INFINITY) ? a : a + lg2_approx(s) * kLn2;
        return a;
    }
    __device__ __forceinline__ int position() const { return nan_idx != INT_MAX ? nan_idx : idx; }
};

// Lanes must merge in the same order on both sides of a butterfly to agree bit for bit (fp32 sums): the
// lower lane's partial is always the left operand.
template <int OP, int L = 32>
__device__ __forceinline__ Acc<OP> warp_merge(Acc<OP> acc)
{
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) {
        Acc<OP> other = acc.shuffled(o);
        if ((threadIdx.x & o) == 0) {
            acc.merge(other);
        } else {
            other.merge(acc);
            acc = other;
        }
    }
    return acc;
}

// Largest (kMax) or smallest element of a vector, NaN if any element is NaN: NaN-propagating min / max
// instructions, two elements at a time for the 16-bit types.
__device__ __forceinline__ float ext_nan(float a, float b, bool want_max)
{
    float r;
    if (want_max) asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    else asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
template <typename T, bool kMax>
__device__ __forceinline__ float vec_ext_nan(const Vec16& v);
template <>
__device__ __forceinline__ float vec_ext_nan<float, true>(const Vec16& v)
{
    return ext_nan(ext_nan(__uint_as_float(v.w[0]), __uint_as_float(v.w[1]), true),
                   ext_nan(__uint_as_float(v.w[2]), __uint_as_float(v.w[3]), true), true);
}
template <>
__device__ __forceinline__ float vec_ext_nan<float, false>(const Vec16& v)
{
    return ext_nan(ext_nan(__uint_as_float(v.w[0]), __uint_as_float(v.w[1]), false),
                   ext_nan(__uint_as_float(v.w[2]), __uint_as_float(v.w[3]), false), false);
}
template <>
__device__ __forceinline__ float vec_ext_nan<__nv_bfloat16, true>(const Vec16& v)
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(v.w);
    const __nv_bfloat162 m = __hmax2_nan(__hmax2_nan(h[0], h[1]), __hmax2_nan(h[2], h[3]));
    return ext_nan(__low2float(m), __high2float(m), true);
}
template <>
__device__ __forceinline__ float vec_ext_nan<__nv_bfloat16, false>(const Vec16& v)
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(v.w);
    const __nv_bfloat162 m = __hmin2_nan(__hmin2_nan(h[0], h[1]), __hmin2_nan(h[2], h[3]));
    return ext_nan(__low2float(m), __high2float(m), false);
}
template <>
__device__ __forceinline__ float vec_ext_nan<__half, true>(const Vec16& v)
{
    const __half2* h = reinterpret_cast<const __half2*>(v.w);
    const __half2 m = __hmax2_nan(__hmax2_nan(h[0], h[1]), __hmax2_nan(h[2], h[3]));
    return ext_nan(__low2float(m), __high2float(m), true);
}
template <>
__device__ __forceinline__ float vec_ext_nan<__half, false>(const Vec16& v)
{
    const __half2* h = reinterpret_cast<const __half2*>(v.w);
    const __half2 m = __hmin2_nan(__hmin2_nan(h[0], h[1]), __hmin2_nan(h[2], h[3]));
    return ext_nan(__low2float(m), __high2float(m), false);
}

template <typename T, int OP>
__device__ __forceinline__ void add_vector(Acc<OP>& acc, const Vec16& raw, int j0)
{
    constexpr int E = Elem<T>::kPerVec;
    if (OP == kOpMax || OP == kOpMin) {
        // only the vector's extreme is looked at here (a handful of instructions per 16 bytes)
        acc.add_vector_extreme(vec_ext_nan<T, OP == kOpMax>(raw), raw, j0 / E);
        return;
    }
    float f[E];
    Elem<T>::unpack(raw, f);
    if (OP == kOpLse) {
        const float vm = vec_ext_nan<T, true>(raw);
        if (vm != vm) acc.nan_idx = 0;
        const float m2 = fmaxf(acc.a, vm);                        // fmaxf drops a NaN operand
        const float off = m2 == -INFINITY ? 0.0f : m2;            // all -inf so far: avoid inf - inf
        const float noff = -off * kLog2e;
        float t = 0.0f;
#pragma unroll
        for (int e = 0; e < E; ++e) t += ex2_approx(fmaf(f[e], kLog2e, noff));
        acc.s = acc.s * ex2_approx(fmaf(acc.a, kLog2e, noff)) + t;
        acc.a = m2;
    } else {
#pragma unroll
        for (int e = 0; e < E; ++e) acc.add(f[e], j0 + e);
    }
}

// logsumexp over a batch of U vectors: the batch maximum on the packed values, one rescale of the running sum
// for the whole batch (U * E + 1 special-function operations instead of U * (E + 1)), two partial sums to
// halve the chain of dependent adds. Vectors past the end of the row must hold -inf.
template <typename T, int U>
__device__ __forceinline__ void add_vectors_lse(Acc<kOpLse>& acc, const Vec16 (&raw)[U])
{
    constexpr int E = Elem<T>::kPerVec;
    float bm = vec_ext_nan<T, true>(raw[0]);
#pragma unroll
    for (int k = 1; k < U; ++k) bm = ext_nan(bm, vec_ext_nan<T, true>(raw[k]), true);
    if (bm != bm) acc.nan_idx = 0;
    const float m2 = fmaxf(acc.a, bm);                            // fmaxf drops a NaN operand
    const float off = m2 == -INFINITY ? 0.0f : m2;                // all -inf so far: avoid inf - inf
    const float noff = -off * kLog2e;
    float t0 = 0.0f, t1 = 0.0f;
#pragma unroll
    for (int k = 0; k < U; ++k) {
        float f[E];
        Elem<T>::unpack(raw[k], f);
#pragma unroll
        for (int e = 0; e < E; e += 2) {
            t0 += ex2_approx(fmaf(f[e], kLog2e, noff));
            t1 += ex2_approx(fmaf(f[e + 1], kLog2e, noff));
        }
    }
    acc.s = fmaf(acc.s, ex2_approx(fmaf(acc.a, kLog2e, noff)), t0 + t1);
    acc.a = m2;
}

template <typename T, int OP>
__device__ __forceinline__ void write_result(const Acc<OP>& acc, float* out, int32_t* index, int64_t row, float inv_cols)
{
    out[row] = acc.value(inv_cols);
    if ((OP == kOpMax || OP == kOpMin) && index != nullptr) index[row] = acc.position();
}

// The vector sweep of one row by `nthreads` threads (a CTA or a warp), U loads in flight per thread.
template <typename T, int OP, int U>
__device__ __forceinline__ void sweep_vectors(Acc<OP>& acc, const T* xr, int nvec, int tid, int nthreads)
{
    constexpr int E = Elem<T>::kPerVec;
    for (int base = 0; base < nvec; base += U * nthreads) {
        Vec16 raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * nthreads + tid;
            if (OP == kOpLse) raw[k] = Elem<T>::fill_neg_inf();
            if (v < nvec) raw[k] = ld_stream(xr + (int64_t)v * E);
        }
        if constexpr (OP == kOpLse) {
            add_vectors_lse<T, U>(acc, raw);
        } else {
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int v = base + k * nthreads + tid;
                if (v < nvec) add_vector<T, OP>(acc, raw[k], v * E);
            }
        }
    }
    if (OP == kOpMax || OP == kOpMin) acc.template resolve<T>();
}

// A row of any length and alignment by `nthreads` threads: the aligned 16-byte vectors between the first boundary
// and the last (positions counted from the row's start), then the at most 2 (E - 1) edge elements before and after
// them, one to a thread at a time, merged in as a partial result of their own.
template <typename T, int OP, int U>
__device__ __forceinline__ void sweep_row(Acc<OP>& acc, const T* xr, int cols, int tid, int nthreads)
{
    const RowSplit<T> sp = row_split<T>(xr, cols);
    sweep_vectors<T, OP, U>(acc, xr + sp.head, sp.nvec, tid, nthreads);
    if (OP == kOpMax || OP == kOpMin) {
        if (acc.idx != INT_MAX) acc.idx += sp.head;
        if (acc.nan_idx != INT_MAX) acc.nan_idx += sp.head;
    }
    if (tid < sp.edges()) {
        Acc<OP> edge;
        edge.init();
        for (int i = tid; i < sp.edges(); i += nthreads) {
            const int j = sp.edge_col(i);
            const float v = Elem<T>::load1(xr + j);
            if constexpr (OP == kOpLse) {
                const float one[1] = {v};
                edge.template add_batch_lse<1>(one, 1);
            } else {
                edge.add(v, j);
            }
        }
        acc.merge(edge);
    }
}

// One CTA per row.
template <typename T, int OP>
__global__ void __launch_bounds__(256)
reduce_row_block_kernel(const T* __restrict__ x, float* __restrict__ out, int32_t* __restrict__ index, int cols,
                        int64_t stride, float inv_cols)
{
    constexpr int U = 4;
    __shared__ float sa[8], ss[8];
    __shared__ int si[8], sn[8];
    const T* xr = x + (int64_t)blockIdx.x * stride;
    Acc<OP> acc;
    acc.init();
    sweep_row<T, OP, U>(acc, xr, cols, threadIdx.x, blockDim.x);
    acc = warp_merge<OP>(acc);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if (lane == 0) {
        sa[warp] = acc.a;
        ss[warp] = acc.s;
        si[warp] = acc.idx;
        sn[warp] = acc.nan_idx;
    }
    __syncthreads();
    if (warp == 0) {
        Acc<OP> t;
        t.init();
        if (lane < nw) {
            t.a = sa[lane];
            t.s = ss[lane];
            t.idx = si[lane];
            t.nan_idx = sn[lane];
        }
        t = warp_merge<OP>(t);
        if (lane == 0) write_result<T, OP>(t, out, index, blockIdx.x, inv_cols);
    }
}

// L lanes per row (L = 4 .. 32, a power of two), 32 / L rows per warp, eight warps per CTA: a short row does
// not pay for a full warp's five butterfly steps, and a lane still has up to four loads in flight. Lanes
// whose row is past the end sweep nothing but take part in the shuffles.
template <typename T, int OP, int L>
__global__ void __launch_bounds__(256)
reduce_row_group_kernel(const T* __restrict__ x, float* __restrict__ out, int32_t* __restrict__ index, int64_t rows,
                        int cols, int64_t stride, float inv_cols)
{
    constexpr int kRowsPerWarp = 32 / L;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t row = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * kRowsPerWarp + lane / L;
    const bool live = row < rows;
    const T* xr = x + (live ? row : 0) * stride;
    const int n = live ? cols : 0;
    Acc<OP> acc;
    acc.init();
    sweep_row<T, OP, 4>(acc, xr, n, sub, L);
    acc = warp_merge<OP, L>(acc);
    if (sub == 0 && live) write_result<T, OP>(acc, out, index, row, inv_cols);
}

template <typename T, int OP>
kop_status_t launch_reduce_op(const T* x, float* out, int32_t* index, int64_t rows, int cols, int64_t stride,
                              cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    const float inv_cols = (float)(1.0 / (double)cols);
    const int64_t row_bytes = (int64_t)cols * sizeof(T);
    // Rows up to 16 KB: lanes-per-row kernel, measured against a CTA per row on 537 MB of bf16, max + argmax:
    // rows of 256 / 1024 / 2048 / 8192 columns 346 -> 88, 267 -> 91, 150 -> 90, 94 -> 90 us. Longer rows: a CTA each.
    if (row_bytes > 16384) {
        const int nvec = cols / E;
        int threads = ((nvec + 15) / 16 + 31) / 32 * 32;     // four batches of four vectors per thread if they fit
        if (threads > 256) threads = 256;
        if (threads < 64) threads = 64;
        reduce_row_block_kernel<T, OP><<<(unsigned)rows, threads, 0, stream>>>(x, out, index, cols, stride, inv_cols);
    } else {
        // sixteen vectors a lane where the row is long enough: fewer lanes and merge steps beat more lanes with
        // fewer batches each (four vectors a lane: 102 - 113 us on the rows above)
        const int64_t units = cols / E;
        const int lanes = units >= 512 ? 32 : units >= 256 ? 16 : units >= 128 ? 8 : 4;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
#define KOP_REDUCE_GROUP(L) \
    reduce_row_group_kernel<T, OP, L><<<(unsigned)ctas, 256, 0, stream>>>(x, out, index, rows, cols, stride, inv_cols)
        switch (lanes) {
        case 32: KOP_REDUCE_GROUP(32); break;
        case 16: KOP_REDUCE_GROUP(16); break;
        case 8: KOP_REDUCE_GROUP(8); break;
        default: KOP_REDUCE_GROUP(4); break;
        }
#undef KOP_REDUCE_GROUP
    }
    return launch_status();
}

template <typename T>
kop_status_t launch_reduce(const void* xv, float* out, int32_t* index, int64_t rows, int64_t cols, int64_t stride,
                           int op, cudaStream_t stream)
{
    const T* x = static_cast<const T*>(xv);
    switch (op) {
    case kOpSum: return launch_reduce_op<T, kOpSum>(x, out, index, rows, (int)cols, stride, stream);
    case kOpMean: return launch_reduce_op<T, kOpMean>(x, out, index, rows, (int)cols, stride, stream);
    case kOpMax: return launch_reduce_op<T, kOpMax>(x, out, index, rows, (int)cols, stride, stream);
    case kOpMin: return launch_reduce_op<T, kOpMin>(x, out, index, rows, (int)cols, stride, stream);
    default: return launch_reduce_op<T, kOpLse>(x, out, index, rows, (int)cols, stride, stream);
    }
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_reduce_rows(const void* x, float* out, int32_t* index, int64_t rows, int64_t cols,
                                        int64_t x_row_stride, int op, kop_dtype_t dtype, kop_stream_t stream)
{
    using namespace kop;
    if (!dtype_ok(dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (op < 0 || op > 4 || cols > 0x7FFFFFFFLL || rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if (rows == 0) return KOP_OK;
    if (!x || !out) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(out, 4) || (index && !aligned_to(index, 4))) return KOP_ERR_MISALIGNED;
    {
        uintptr_t a0, a1;
        span_of(x, rows, cols, x_row_stride, esz, &a0, &a1);
        const uintptr_t b0 = reinterpret_cast<uintptr_t>(out), b1 = b0 + (uintptr_t)rows * 4;
        if (!(a1 <= b0 || b1 <= a0)) return KOP_ERR_BAD_ALIAS;
        if (index) {
            const uintptr_t c0 = reinterpret_cast<uintptr_t>(index), c1 = c0 + (uintptr_t)rows * 4;
            if (!(a1 <= c0 || c1 <= a0) || !(b1 <= c0 || c1 <= b0)) return KOP_ERR_BAD_ALIAS;
        }
    }
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    return dtype == KOP_F32 ? launch_reduce<float>(x, out, index, rows, cols, x_row_stride, op, s)
           : dtype == KOP_BF16 ? launch_reduce<__nv_bfloat16>(x, out, index, rows, cols, x_row_stride, op, s)
                               : launch_reduce<__half>(x, out, index, rows, cols, x_row_stride, op, s);
}
