// kop_softmax_scale_bias: y = softmax_j(x * scale + bias) per row, one HBM pass.
//
// The row lives in registers between the load and the store: a warp owns a row when it is short
// (each lane holds VPL 16-byte vectors), a whole CTA owns it when it is long. The exponent runs
// in the base-2 domain: t = x * (scale*log2e) + bias*log2e is one FMA, the row max is taken on t,
// and exp(z - max z) = 2^(t - max t) is one ex2.approx. Rows shorter than 32 vectors take 2 to 8 lanes of
// a warp each; rows beyond 32 KB (vocabulary-sized) are read twice, the second time backwards out of the
// L2 (a cluster of up to 8 CTAs holding such a row in registers, with the maximum and the sum combined
// through distributed shared memory, was measured too: 2.4 - 3.7 TB/s against 3.9 - 4.2 TB/s, the cluster
// barriers serialise what short-lived CTAs overlap). Rows that are not whole aligned vectors (197 or 77
// attention keys, a 50257-wide vocabulary) are split into head elements up to the first 16-byte boundary,
// aligned vectors and tail elements inside the same three kernels; only a causal mask on such rows, or x and
// y rows at different offsets from a boundary, go to a scalar three-sweep kernel with the same arithmetic.
#include "kop_common.cuh"

namespace kop {
namespace {

// ---- warp per row, one row per warp ---------------------------------------------------------------
// (A grid-stride version with the bias held in registers across rows measured 8 % slower on
// [131072, 512] fp32: many short-lived CTAs at different phases overlap loads, math and stores better
// than a few resident warps that each serialise them.)
// kFull: the row is exactly L * VPL vectors (no tail predicates); kBias: bias != NULL. L: lanes per row (32, or
// 2 .. 16 for rows of fewer than 32 vectors, 32 / L rows per warp: attention scores and class logits of 64 to
// 256 columns would leave most of a warp idle otherwise).
// kLog: the log form of the output. kCausal: row r sees columns 0 .. (r mod period) + cols - period only (`causal`
// carries the period, cols - period and ceil(2^64 / period) for the remainder); later columns count as -inf, and a
// row's vectors beyond its last visible column are not read.
struct SmCausal {
    int period, base;
    unsigned long long magic;
};

// kRagged: rows that are not whole aligned vectors (`nvec` then carries the row length in elements): a row is split
// into head elements up to the first 16-byte boundary, whole vectors and tail elements; every lane holds at most one
// of the edge elements (L >= 16 covers the 14 that 16-bit data can have) next to its vectors, the bias is read per
// element, the edge results are stored one by one. x and y rows must sit at the same offset from a 16-byte boundary.
template <typename T, typename PT, int VPL, bool kFull, bool kBias, int L = 32, bool kLog = false, bool kCausal = false,
          bool kRagged = false>
__global__ void __launch_bounds__(256)
softmax_warp_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y,
                    int64_t rows, int nvec, int64_t x_stride, int64_t y_stride, float scale,
                    SmCausal causal = SmCausal{0, 0, 0ull})
{
    static_assert(!kRagged || (!kFull && !kCausal && L >= 8), "ragged rows: predicated vectors, no causal mask");
    constexpr int KE = kRagged ? (2 * (Elem<T>::kPerVec - 1) + L - 1) / L : 1;      // edge elements a lane holds at most
    constexpr int E = Elem<T>::kPerVec;
    const int lane = L == 32 ? (threadIdx.x & 31) : (threadIdx.x & (L - 1));
    int64_t row = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * (32 / L) + (threadIdx.x & 31) / L;
    if (L == 32 && row >= rows) return;                      // whole warps leave together
    // narrower groups: a group past the end reads the last row again and stores nothing, so that its lanes
    // still take part in the shuffles
    const bool live = row < rows;
    if (!live) row = rows - 1;
    const float s2 = scale * kLog2e;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    int head = 0, edge_col[KE];                              // ragged rows: first vector's column, this lane's edge columns
#pragma unroll
    for (int q = 0; q < KE; ++q) edge_col[q] = -1;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, nvec);
        head = sp.head;
#pragma unroll
        for (int q = 0; q < KE; ++q)
            if (lane + q * L < sp.edges()) edge_col[q] = sp.edge_col(lane + q * L);
        nvec = sp.nvec;
        xr += head;
        yr += head;
    }
    int last = 0;
    if (kCausal) {
        // row / period by multiply-shift (exact for row < 2^64 / period; a period of 1 has no 64-bit reciprocal)
        const unsigned long long q = causal.period == 1 ? (unsigned long long)row : __umul64hi((unsigned long long)row, causal.magic);
        last = (int)((unsigned long long)row - q * (unsigned)causal.period) + causal.base;
    }
    Vec16 raw[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + lane;
        if ((kFull || v < nvec) && (!kCausal || v * E <= last)) raw[k] = ld_stream(xr + (int64_t)v * E);
        else raw[k] = Vec16{{0u, 0u, 0u, 0u}};
    }
    float t[VPL][E];
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + lane;
        float f[E];
        Elem<T>::unpack(raw[k], f);
        const int vis = kCausal ? last - v * E : 0;          // elements 0 .. vis of this vector are visible
#pragma unroll
        for (int q = 0; q < E / 4; ++q) {
            float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
            if constexpr (kRagged) {
                if (kBias && v < nvec) {
                    const int j = head + v * E + 4 * q;
                    b = make_float4(param1(bias, j), param1(bias, j + 1), param1(bias, j + 2), param1(bias, j + 3));
                }
            } else {
                if (kBias && (kFull || v < nvec)) b = ldg_p4(bias + (int64_t)v * E + 4 * q);
            }
            const float bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = 4 * q + c;
                t[k][e] = ((kFull || v < nvec) && (!kCausal || e <= vis)) ? fmaf(f[e], s2, bb[c] * kLog2e) : -INFINITY;
                m = fmaxf(m, t[k][e]);
            }
        }
    }
    float te[KE];                                            // this lane's edge elements
#pragma unroll
    for (int q = 0; q < KE; ++q) te[q] = -INFINITY;
    if constexpr (kRagged) {
#pragma unroll
        for (int q = 0; q < KE; ++q) {
            if (edge_col[q] >= 0) {
                const float b = kBias ? param1(bias, edge_col[q]) * kLog2e : 0.0f;
                te[q] = fmaf(Elem<T>::load1(xr - head + edge_col[q]), s2, b);
            }
            m = fmaxf(m, te[q]);
        }
    }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    float s = 0.0f;
    if constexpr (kRagged) {
#pragma unroll
        for (int q = 0; q < KE; ++q) {
            const float d = te[q] - m;
            const float p = ex2_approx(d);
            s += p;
            te[q] = kLog ? d : p;
        }
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k)
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const float d = t[k][e] - m;
            const float p = ex2_approx(d);
            s += p;
            t[k][e] = kLog ? d : p;                          // the log form keeps the base-2 exponent
        }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    const float inv = 1.0f / s;
    const float lg = lg2_approx(s);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int v = k * L + lane;
        float o[E];
#pragma unroll
        for (int e = 0; e < E; ++e) o[e] = kLog ? (t[k][e] - lg) * kLn2 : t[k][e] * inv;
        if (live && (kFull || v < nvec)) st_stream(yr + (int64_t)v * E, Elem<T>::pack(o));
    }
    if constexpr (kRagged) {
#pragma unroll
        for (int q = 0; q < KE; ++q)
            if (live && edge_col[q] >= 0) Elem<T>::store1(yr - head + edge_col[q], kLog ? (te[q] - lg) * kLn2 : te[q] * inv);
    }
}

// ---- CTA per row, row in registers ---------------------------------------------------------------
// kOpts adds the variants of kop_softmax_opts: `last` is the row's last visible column (causal rows; every
// later column counts as -inf) and log_out selects z - m - ln(sum) instead of exp(z - m) / sum.
struct SmOpts {
    int log_out;
    int64_t period;      // 0: not causal
    int64_t cols;
};
__device__ __forceinline__ int64_t last_visible(const SmOpts& o, int64_t row)
{
    return o.period > 0 ? (row % o.period) + (o.cols - o.period) : o.cols - 1;
}

// kPlain: the row is exactly blockDim.x * VPT vectors and there is no bias (no tail predicates, no bias code); the
// general form tests both at run time.
// kRagged: rows that are not whole aligned vectors, split as in the warp kernel (opts.cols carries the row length),
// one edge element to a thread.
template <typename T, typename PT, int VPT, bool kOpts, bool kPlain, bool kLog = false, bool kRagged = false,
          bool kRagBias = false>                             // kRagBias: ragged or kOpts rows with a bias (its loads compiled in)
__global__ void __launch_bounds__(max_threads_for(VPT * Elem<T>::kPerVec))
softmax_block_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y,
                     int nvec, int64_t x_stride, int64_t y_stride, float scale, SmOpts opts)
{
    static_assert(!kRagged || (!kOpts && !kPlain), "ragged rows: predicated vectors, no causal mask");
    constexpr int E = Elem<T>::kPerVec;
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const int64_t last = kOpts ? last_visible(opts, row) : 0;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    const float s2 = scale * kLog2e;
    int head = 0, edge_col = -1;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, opts.cols);
        head = sp.head;
        nvec = sp.nvec;
        if ((int)threadIdx.x < sp.edges()) edge_col = sp.edge_col(threadIdx.x);
        xr += head;
        yr += head;
    }

    Vec16 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        // a causal row's vectors beyond its last visible column are not read at all
        if (kOpts) raw[k] = Vec16{{0u, 0u, 0u, 0u}};
        if ((kPlain || v < nvec) && (!kOpts || v * E <= (int)last)) raw[k] = ld_stream(xr + (int64_t)v * E);
    }
    float t[VPT][E];
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        float f[E];
        Elem<T>::unpack(raw[k], f);
        const int vis = kOpts ? (int)last - v * E : 0;          // elements 0 .. vis of this vector are visible (rows here are short)
#pragma unroll
        for (int q = 0; q < E / 4; ++q) {
            float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
            if constexpr (kRagged) {
                if (kRagBias && v < nvec) {
                    const int j = head + v * E + 4 * q;
                    b = make_float4(param1(bias, j), param1(bias, j + 1), param1(bias, j + 2), param1(bias, j + 3));
                }
            } else {
                // the causal / log form tests the bias at compile time (kRagBias); the plain general form at run time,
                // where a compile-time variant measured slower on rows with a bias
                if (!kPlain && (!kOpts || kRagBias) && bias != nullptr && v < nvec) b = ldg_p4(bias + (int64_t)v * E + 4 * q);
            }
            const float bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = 4 * q + c;
                const bool keep = (kPlain || v < nvec) && (!kOpts || e <= vis);
                t[k][e] = keep ? fmaf(f[e], s2, bb[c] * kLog2e) : -INFINITY;
                m = fmaxf(m, t[k][e]);
            }
        }
    }
    float te = -INFINITY;                                    // this thread's edge element
    if constexpr (kRagged) {
        if (edge_col >= 0) {
            const float b = kRagBias ? param1(bias, edge_col) * kLog2e : 0.0f;
            te = fmaf(Elem<T>::load1(xr - head + edge_col), s2, b);
        }
        m = fmaxf(m, te);
    }
    m = block_max(m, red_a);
    float s = 0.0f;
    const bool log_out = kLog || (kOpts && opts.log_out != 0);
    if constexpr (kRagged) {
        const float d = te - m;
        const float p = ex2_approx(d);
        s = p;
        te = log_out ? d : p;
    }
#pragma unroll
    for (int k = 0; k < VPT; ++k)
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const float d = t[k][e] - m;
            const float p = ex2_approx(d);
            s += p;
            t[k][e] = log_out ? d : p;                       // the log form keeps the base-2 exponent
        }
    s = block_sum(s, red_b);
    const float inv = 1.0f / s;
    const float lg = lg2_approx(s);
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = k * blockDim.x + threadIdx.x;
        float o[E];
#pragma unroll
        for (int e = 0; e < E; ++e) o[e] = log_out ? (t[k][e] - lg) * kLn2 : t[k][e] * inv;
        if (kPlain || v < nvec) st_stream(yr + (int64_t)v * E, Elem<T>::pack(o));
    }
    if constexpr (kRagged) {
        if (edge_col >= 0) Elem<T>::store1(yr - head + edge_col, log_out ? (te - lg) * kLn2 : te * inv);
    }
}

// ---- long rows, vector loads, two sweeps ------------------------------------------------------------
// Sweep 1 reads the row once and keeps a running (maximum, sum) per thread, rescaled once per batch of U
// vectors; sweep 2 walks the row backwards (the end of the row is what the first sweep left in L2) and writes
// the result. HBM sees the row about once each way while the rows in flight fit the L2.
// kRagged: rows that are not whole aligned vectors, split as in the warp kernel (opts.cols carries the row length);
// the edge elements go one to a thread, enter its running (maximum, sum) before the first sweep and are stored after
// the second.
template <typename T, typename PT, bool kOpts, bool kBias, bool kLog = false, bool kRagged = false>
__global__ void __launch_bounds__(512)
softmax_twosweep_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y, int nvec,
                        int64_t x_stride, int64_t y_stride, float scale, SmOpts opts)
{
    static_assert(!kRagged || !kOpts, "ragged rows: no causal mask");
    constexpr int E = Elem<T>::kPerVec, U = 4;
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const int64_t last = kOpts ? last_visible(opts, row) : 0;
    const bool log_out = kLog || (kOpts && opts.log_out != 0);
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    const float s2 = scale * kLog2e;
    int head = 0, edge_col = -1;
    if constexpr (kRagged) {
        const RowSplit<T> sp = row_split<T>(xr, opts.cols);
        head = sp.head;
        nvec = sp.nvec;
        if ((int)threadIdx.x < sp.edges()) edge_col = sp.edge_col(threadIdx.x);
        xr += head;
        yr += head;
    }
    const int step = U * blockDim.x;
    const int nbatch = (nvec + step - 1) / step;

    // t[e] = x * scale * log2e + bias * log2e for the elements of vector v, -inf where masked
    auto logits2 = [&](const Vec16& raw, int v, float (&t)[E]) {
        float f[E];
        Elem<T>::unpack(raw, f);
#pragma unroll
        for (int q = 0; q < E / 4; ++q) {
            float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
            if constexpr (kRagged) {
                if (kBias) {
                    const int64_t j = head + (int64_t)v * E + 4 * q;
                    b = make_float4(param1(bias, j), param1(bias, j + 1), param1(bias, j + 2), param1(bias, j + 3));
                }
            } else {
                if (kBias) b = ldg_p4(bias + (int64_t)v * E + 4 * q);
            }
            const float bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = 4 * q + c;
                const bool keep = !kOpts || (int64_t)v * E + e <= last;
                t[e] = keep ? fmaf(f[e], s2, bb[c] * kLog2e) : -INFINITY;
            }
        }
    };

    const uint64_t keep = l2_policy_keep(), drop = l2_policy_drop();
    float m = -INFINITY, s = 0.0f;
    float te = -INFINITY;                                    // this thread's edge element
    if constexpr (kRagged) {
        if (edge_col >= 0) {
            const float b = kBias ? param1(bias, edge_col) * kLog2e : 0.0f;
            te = fmaf(Elem<T>::load1(xr - head + edge_col), s2, b);
            if (te != -INFINITY) {                           // a NaN enters too and reaches the sum through ex2
                m = te;
                s = 1.0f;
            }
        }
    }
    for (int b = 0; b < nbatch; ++b) {
        Vec16 raw[U];
        float t[U][E];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            if (v < nvec) raw[k] = ld_stream_hint(xr + (int64_t)v * E, keep);
        }
        float bm = -INFINITY;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = b * step + k * blockDim.x + threadIdx.x;
            if (v < nvec) {
                logits2(raw[k], v, t[k]);
            } else {
#pragma unroll
                for (int e = 0; e < E; ++e) t[k][e] = -INFINITY;
            }
#pragma unroll
            for (int e = 0; e < E; ++e) bm = fmaxf(bm, t[k][e]);
        }
        if (bm > -INFINITY) {
            const float m2 = fmaxf(m, bm);
            float acc = s * ex2_approx(m - m2);              // m = -inf before the first finite batch: s * 0
#pragma unroll
            for (int k = 0; k < U; ++k)
#pragma unroll
                for (int e = 0; e < E; ++e) acc += ex2_approx(t[k][e] - m2);
            s = acc;
            m = m2;
        }
    }
    const float M = block_max(m, red_a);
    s = block_sum(m == -INFINITY ? 0.0f : s * ex2_approx(m - M), red_b);
    const float inv = 1.0f / s;
    const float lg = lg2_approx(s);
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
                float t[E], o[E];
                logits2(raw[k], v, t);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float d = t[e] - M;
                    o[e] = log_out ? (d - lg) * kLn2 : ex2_approx(d) * inv;
                }
                st_stream_hint(yr + (int64_t)v * E, Elem<T>::pack(o), drop);
            }
        }
    }
    if constexpr (kRagged) {
        if (edge_col >= 0) {
            const float d = te - M;
            Elem<T>::store1(yr - head + edge_col, log_out ? (d - lg) * kLn2 : ex2_approx(d) * inv);
        }
    }
}

// ---- any length, any alignment: scalar loads, three sweeps over the row ----------------------------
template <typename T, typename PT, bool kOpts>
__global__ void __launch_bounds__(256)
softmax_generic_kernel(const T* __restrict__ x, const PT* __restrict__ bias, T* __restrict__ y,
                       int64_t cols, int64_t x_stride, int64_t y_stride, float scale, SmOpts opts)
{
    __shared__ float red_a[32], red_b[32];
    const int64_t row = blockIdx.x;
    const int64_t last = kOpts ? last_visible(opts, row) : cols - 1;
    const bool log_out = kOpts && opts.log_out != 0;
    const T* xr = x + row * x_stride;
    T* yr = y + row * y_stride;
    const float s2 = scale * kLog2e;
    float m = -INFINITY;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float b = bias != nullptr ? param1(bias, j) * kLog2e : 0.0f;
        if (j <= last) m = fmaxf(m, fmaf(Elem<T>::load1(xr + j), s2, b));
    }
    m = block_max(m, red_a);
    float s = 0.0f;
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float b = bias != nullptr ? param1(bias, j) * kLog2e : 0.0f;
        if (j <= last) s += ex2_approx(fmaf(Elem<T>::load1(xr + j), s2, b) - m);
    }
    s = block_sum(s, red_b);
    const float inv = 1.0f / s;
    const float lg = lg2_approx(s);
    // The last sweep reads x[j] and writes y[j] in the same thread, so exact aliasing stays safe.
    for (int64_t j = threadIdx.x; j < cols; j += blockDim.x) {
        const float b = bias != nullptr ? param1(bias, j) * kLog2e : 0.0f;
        const float d = j <= last ? fmaf(Elem<T>::load1(xr + j), s2, b) - m : -INFINITY;
        Elem<T>::store1(yr + j, log_out ? (d - lg) * kLn2 : ex2_approx(d) * inv);
    }
}

template <typename T, typename PT>
kop_status_t launch_softmax(const void* xv, const void* biasv, void* yv, int64_t rows, int64_t cols,
                            int64_t xs, int64_t ys, float scale, cudaStream_t stream, bool with_opts = false,
                            SmOpts opts = SmOpts{0, 0, 0})
{
    const T* x = static_cast<const T*>(xv);
    const PT* bias = static_cast<const PT*>(biasv);
    T* y = static_cast<T*>(yv);
    constexpr int E = Elem<T>::kPerVec;
    const bool vec = vec_ok(x, cols, xs, sizeof(T)) && vec_ok(y, cols, ys, sizeof(T)) &&
                     (bias == nullptr || aligned_to(bias, 16));
    const int64_t nvec64 = cols / E;
    // log-softmax without a causal mask: the plain kernels with the log form of the output (no per-element test of the
    // visible range; bf16 rows of 1024 - 8192 columns 4.3 - 4.6 TB/s through the general form)
    const bool log_only = with_opts && opts.period == 0 && opts.log_out != 0;
    // causal rows without the log form on short rows: the lanes-per-row / warp-per-row kernels with the visible range
    // worked out per row (attention scores of 256 / 512 keys ran at 2.0 / 3.8 TB/s through the CTA-per-row form)
    const bool causal_short = with_opts && opts.period != 0 && opts.log_out == 0 && rows < (1LL << 53);
    SmCausal cz{0, 0, 0ull};
    if (causal_short) {
        cz.period = (int)opts.period;
        cz.base = (int)(opts.cols - opts.period);
        cz.magic = opts.period > 1 ? (~0ull) / (unsigned long long)opts.period + 1ull : 0ull;
    }
    if (vec && nvec64 < 32 && (!with_opts || log_only || causal_short)) {                  // fewer than 32 vectors: 2 to 8 lanes per row, four vectors each
        const int nvec = (int)nvec64;
        const int lanes = nvec > 16 ? 8 : nvec > 8 ? 4 : 2;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        const unsigned grid = (unsigned)ctas;
        const bool full = nvec == lanes * 4;
#define KOP_SM_GROUP_L(F, B, L)                                                                                                  \
    do {                                                                                                                         \
        if (causal_short) softmax_warp_kernel<T, PT, 4, false, B, L, false, true><<<grid, 256, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale, cz); \
        else if (log_only) softmax_warp_kernel<T, PT, 4, F, B, L, true><<<grid, 256, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale); \
        else softmax_warp_kernel<T, PT, 4, F, B, L><<<grid, 256, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale);           \
    } while (0)
#define KOP_SM_GROUP(L)                                                         \
    do {                                                                        \
        if (full && bias != nullptr) KOP_SM_GROUP_L(true, true, L);             \
        else if (full) KOP_SM_GROUP_L(true, false, L);                          \
        else if (bias != nullptr) KOP_SM_GROUP_L(false, true, L);               \
        else KOP_SM_GROUP_L(false, false, L);                                   \
    } while (0)
        if (lanes == 8) KOP_SM_GROUP(8);
        else if (lanes == 4) KOP_SM_GROUP(4);
        else KOP_SM_GROUP(2);
#undef KOP_SM_GROUP_L
#undef KOP_SM_GROUP
        return launch_status();
    }
    if (vec && nvec64 <= 32 * 4 && (!with_opts || log_only || causal_short)) {
        const int nvec = (int)nvec64;
        const int vpl = (nvec + 31) / 32;
        const int threads = 256;
        const int64_t ctas = (rows + 7) / 8;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        const unsigned grid = (unsigned)ctas;
        const int vp = vpl <= 1 ? 1 : (vpl <= 2 ? 2 : 4);
        const bool full = nvec == 32 * vp;
#define KOP_SM_WARP_L(V, F, B)                                                                                                   \
    do {                                                                                                                         \
        if (causal_short) softmax_warp_kernel<T, PT, V, false, B, 32, false, true><<<grid, threads, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale, cz); \
        else if (log_only) softmax_warp_kernel<T, PT, V, F, B, 32, true><<<grid, threads, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale); \
        else softmax_warp_kernel<T, PT, V, F, B><<<grid, threads, 0, stream>>>(x, bias, y, rows, nvec, xs, ys, scale);          \
    } while (0)
#define KOP_SM_WARP(V)                                                         \
    do {                                                                       \
        if (full && bias != nullptr) KOP_SM_WARP_L(V, true, true);             \
        else if (full) KOP_SM_WARP_L(V, true, false);                          \
        else if (bias != nullptr) KOP_SM_WARP_L(V, false, true);               \
        else KOP_SM_WARP_L(V, false, false);                                   \
    } while (0)
        if (vp == 1) KOP_SM_WARP(1);
        else if (vp == 2) KOP_SM_WARP(2);
        else KOP_SM_WARP(4);
#undef KOP_SM_WARP_L
#undef KOP_SM_WARP
        return launch_status();
    }
    if (rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
    // rows up to 32 KB stay in one CTA's registers; longer ones take the two-sweep kernel (fp32 rows of 8192 columns:
    // 5.1 TB/s in two sweeps, 6.5 in registers with 32 values a thread; of 16384 columns 5.7 either way; bf16 rows of
    // 16384 columns: 4.7 in registers against 4.0)
    if (vec && cols <= kMaxRegisterRow && cols * (int64_t)sizeof(T) <= 32768) {
        const int nvec = (int)nvec64;
        // Per-thread vector count: 16 values per thread while the CTA stays within 1024 threads
        // keeps many CTAs resident; longer rows double the count (and halve the CTA limit).
        // (32 values a thread from 2048 columns: bf16 rows of 2048 / 4096 / 8192 / 16384 columns 5.1 / 5.0 / 4.8 / 3.8 TB/s
        // with 16, 6.1 / 5.9 / 5.4 / 4.7 with 32; 64 values a thread: 3.8 / 3.5 at 8192 / 16384)
        int vpt = (cols >= 2048 ? 32 : 16) / E;
        while (vpt * E < 64 && (nvec + vpt - 1) / vpt > max_threads_for(vpt * E)) vpt *= 2;
        const int threads = ((nvec + vpt - 1) / vpt + 31) / 32 * 32;
        // exact rows without a bias take the predicate-free variant (bf16 rows of 2048 / 4096 / 8192 columns 6.1 / 5.9 / 5.4
        // to 6.5 / 6.4 / 5.8 TB/s, fp32 1024 - 4096 columns 5.6 to 6.5); a compile-time bias variant measured 10 - 16 %
        // slower than the form that tests the pointer at run time (bf16 8192 columns, fp32 bias: 5.1 to 4.5), so rows
        // with a bias keep that form
        const bool full = nvec % vpt == 0 && nvec / vpt == threads;
        if (!full && bias == nullptr && (!with_opts || log_only)) {
            // rows that do not fill the CTA exactly, without a bias: the split-row variant, which has no bias code at all
            // (the general form keeps the bias loads as predicated-off instructions: fp32 rows of 1000 columns 5.2 TB/s
            // there, 6.4 here)
#define KOP_SM_BLOCK_NB(V)                                                                                                         \
    do {                                                                                                                          \
        if (log_only) softmax_block_kernel<T, PT, V, false, false, true, true, false><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, 0, xs, ys, scale, opts); \
        else softmax_block_kernel<T, PT, V, false, false, false, true, false><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, 0, xs, ys, scale, opts); \
    } while (0)
            switch (vpt * E) {
            case 16: KOP_SM_BLOCK_NB(16 / E); break;
            case 32: KOP_SM_BLOCK_NB(32 / E); break;
            default: KOP_SM_BLOCK_NB(64 / E); break;
            }
#undef KOP_SM_BLOCK_NB
            return launch_status();
        }
#define KOP_SM_BLOCK_L(V, O, P) \
    softmax_block_kernel<T, PT, V, O, P><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts)
#define KOP_SM_BLOCK(V)                                                          \
    do {                                                                         \
        if (with_opts && !log_only && bias != nullptr) softmax_block_kernel<T, PT, V, true, false, false, false, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts); \
        else if (with_opts && !log_only) KOP_SM_BLOCK_L(V, true, false);         \
        else if (log_only && full && bias == nullptr) softmax_block_kernel<T, PT, V, false, true, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts); \
        else if (log_only) softmax_block_kernel<T, PT, V, false, false, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts); \
        else if (full && bias == nullptr) KOP_SM_BLOCK_L(V, false, true);        \
        else KOP_SM_BLOCK_L(V, false, false);                                    \
    } while (0)
        switch (vpt * E) {
        case 16: KOP_SM_BLOCK(16 / E); break;
        case 32: KOP_SM_BLOCK(32 / E); break;
        default: KOP_SM_BLOCK(64 / E); break;
        }
#undef KOP_SM_BLOCK
#undef KOP_SM_BLOCK_L
        return launch_status();
    }
    if (vec && nvec64 <= 0x7FFFFFFF) {
        const int nvec = (int)nvec64;
        // 256-thread CTAs up to about 100 KB a row, 512 beyond (bf16 rows of 32000 / 50264 columns 4.9 / 4.7 TB/s with 512
        // threads, 5.6 / 5.1 with 256; fp32 12288 columns 5.1 / 6.2; but bf16 128256 columns 5.2 / 4.6 and fp32 32000 / 65536
        // columns 6.0 / 5.4 with 512 against 5.6 / 4.6)
        const int threads = cols * (int64_t)sizeof(T) <= 112 * 1024 ? 256 : 512;
#define KOP_SM_TWO(O, B) softmax_twosweep_kernel<T, PT, O, B><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts)
        if (log_only) {
            if (bias != nullptr) softmax_twosweep_kernel<T, PT, false, true, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts);
            else softmax_twosweep_kernel<T, PT, false, false, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, nvec, xs, ys, scale, opts);
        } else if (with_opts) { if (bias != nullptr) KOP_SM_TWO(true, true); else KOP_SM_TWO(true, false); }
        else { if (bias != nullptr) KOP_SM_TWO(false, true); else KOP_SM_TWO(false, false); }
#undef KOP_SM_TWO
        return launch_status();
    }
    // rows that are not whole aligned vectors, x and y rows at the same offset from a 16-byte boundary, no causal mask:
    // head elements, aligned vectors, tail elements (attention scores of 197 or 77 keys, a 50257-wide vocabulary)
    const bool ragged = !vec && (!with_opts || log_only) &&
                        (reinterpret_cast<uintptr_t>(x) - reinterpret_cast<uintptr_t>(y)) % 16 == 0 &&
                        ((xs - ys) * (int64_t)sizeof(T)) % 16 == 0 && cols <= 0x7FFFFFFFLL;
    if (ragged && nvec64 <= 32 * 4) {
        // 8 lanes a row up to 32 vectors, a warp beyond; two or four vectors a lane (fp32 rows of 197 columns: 54 us a
        // warp a row, 58 with 16 lanes; bf16 rows of 77: 29 us with 8 lanes, 33 with 16)
        const int lanes = nvec64 <= 32 ? 8 : 32;
        const int vp = (nvec64 <= 16 || (nvec64 > 32 && nvec64 <= 64)) ? 2 : 4;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const int64_t ctas = (rows + rows_per_cta - 1) / rows_per_cta;
        if (ctas > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;
        const unsigned grid = (unsigned)ctas;
#define KOP_SM_RAG_B(V, L, B)                                                                                          \
    do {                                                                                                               \
        if (log_only) softmax_warp_kernel<T, PT, V, false, B, L, true, false, true><<<grid, 256, 0, stream>>>(x, bias, y, rows, (int)cols, xs, ys, scale); \
        else softmax_warp_kernel<T, PT, V, false, B, L, false, false, true><<<grid, 256, 0, stream>>>(x, bias, y, rows, (int)cols, xs, ys, scale); \
    } while (0)
    // the bias as a compile-time variant: tested at run time its element loads stay in the code as predicated-off
    // instructions (1.6 load instructions an element on rows without a bias)
#define KOP_SM_RAG(V, L)                        \
    do {                                        \
        if (bias != nullptr) KOP_SM_RAG_B(V, L, true); \
        else KOP_SM_RAG_B(V, L, false);         \
    } while (0)
        if (lanes == 8 && vp == 2) KOP_SM_RAG(2, 8);
        else if (lanes == 8) KOP_SM_RAG(4, 8);
        else if (vp == 2) KOP_SM_RAG(2, 32);
        else KOP_SM_RAG(4, 32);
#undef KOP_SM_RAG
#undef KOP_SM_RAG_B
        return launch_status();
    }
    if (ragged && cols <= kMaxRegisterRow && cols * (int64_t)sizeof(T) <= 32768) {
        const int nvec = (int)nvec64;                        // a row has this many whole vectors, or one fewer
        int vpt = (cols >= 2048 ? 32 : 16) / E;
        while (vpt * E < 64 && (nvec + vpt - 1) / vpt > max_threads_for(vpt * E)) vpt *= 2;
        const int threads = ((nvec + vpt - 1) / vpt + 31) / 32 * 32;
#define KOP_SM_BLOCK_RAG_B(V, B)                                                                                                  \
    do {                                                                                                                          \
        if (log_only) softmax_block_kernel<T, PT, V, false, false, true, true, B><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, 0, xs, ys, scale, opts); \
        else softmax_block_kernel<T, PT, V, false, false, false, true, B><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, 0, xs, ys, scale, opts); \
    } while (0)
#define KOP_SM_BLOCK_RAG(V)                              \
    do {                                                 \
        if (bias != nullptr) KOP_SM_BLOCK_RAG_B(V, true); \
        else KOP_SM_BLOCK_RAG_B(V, false);               \
    } while (0)
        switch (vpt * E) {
        case 16: KOP_SM_BLOCK_RAG(16 / E); break;
        case 32: KOP_SM_BLOCK_RAG(32 / E); break;
        default: KOP_SM_BLOCK_RAG(64 / E); break;
        }
#undef KOP_SM_BLOCK_RAG
#undef KOP_SM_BLOCK_RAG_B
        return launch_status();
    }
    if (ragged) {
        const int threads = cols * (int64_t)sizeof(T) <= 112 * 1024 ? 256 : 512;
#define KOP_SM_TWO_RAG(B, G) softmax_twosweep_kernel<T, PT, false, B, G, true><<<(unsigned)rows, threads, 0, stream>>>(x, bias, y, 0, xs, ys, scale, opts)
        if (log_only) { if (bias != nullptr) KOP_SM_TWO_RAG(true, true); else KOP_SM_TWO_RAG(false, true); }
        else { if (bias != nullptr) KOP_SM_TWO_RAG(true, false); else KOP_SM_TWO_RAG(false, false); }
#undef KOP_SM_TWO_RAG
        return launch_status();
    }
    if (with_opts) softmax_generic_kernel<T, PT, true><<<(unsigned)rows, 256, 0, stream>>>(x, bias, y, cols, xs, ys, scale, opts);
    else softmax_generic_kernel<T, PT, false><<<(unsigned)rows, 256, 0, stream>>>(x, bias, y, cols, xs, ys, scale, opts);
    return launch_status();
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

// One validation and dispatch routine for the three softmax entry points. with_opts selects the kernels that carry
// the log-output / causal options (kop_softmax_scale_bias never pays for them).
kop_status_t softmax_entry(const void* x, const void* bias, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                           int64_t y_row_stride, float scale, bool with_opts, int log_output, int64_t causal_period,
                           kop_dtype_t dtype, kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(rows, cols);
    if (st != KOP_OK) return st;
    if (with_opts && (causal_period < 0 || causal_period > cols)) return KOP_ERR_BAD_SHAPE;
    if (rows == 0) return KOP_OK;                       // empty: nothing to validate further or launch
    if (x == nullptr || y == nullptr) return KOP_ERR_NULL_POINTER;
    if ((st = check_row_stride(x_row_stride, cols, rows)) != KOP_OK) return st;
    if ((st = check_row_stride(y_row_stride, cols, rows)) != KOP_OK) return st;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (bias != nullptr && !aligned_to(bias, elem_size(pdtype))))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, x_row_stride, y, y_row_stride, rows, cols, esz, true)) return KOP_ERR_BAD_ALIAS;
    if ((st = check_device()) != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    const SmOpts opts{log_output != 0, causal_period, cols};
#define KOP_SM_GO(T, PT) launch_softmax<T, PT>(x, bias, y, rows, cols, x_row_stride, y_row_stride, scale, s, with_opts, opts)
    return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_SM_GO);
#undef KOP_SM_GO
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_softmax_scale_bias(const void* x, const float* bias, void* y,
                                               int64_t rows, int64_t cols, int64_t x_row_stride,
                                               int64_t y_row_stride, float scale,
                                               kop_dtype_t dtype, kop_stream_t stream)
{
    return kop::softmax_entry(x, bias, y, rows, cols, x_row_stride, y_row_stride, scale, false, 0, 0, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_softmax_opts(const void* x, const float* bias, void* y, int64_t rows, int64_t cols,
                                         int64_t x_row_stride, int64_t y_row_stride, float scale, int log_output,
                                         int64_t causal_period, kop_dtype_t dtype, kop_stream_t stream)
{
    // no option set: the kernels of kop_softmax_scale_bias
    return kop::softmax_entry(x, bias, y, rows, cols, x_row_stride, y_row_stride, scale,
                              log_output != 0 || causal_period != 0, log_output, causal_period, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_softmax_ex(const void* x, const void* bias, void* y, int64_t rows, int64_t cols,
                                       int64_t x_row_stride, int64_t y_row_stride, float scale, int log_output,
                                       int64_t causal_period, kop_dtype_t dtype, kop_dtype_t param_dtype,
                                       kop_stream_t stream)
{
    // no options asked for: the kernels of kop_softmax_scale_bias
    return kop::softmax_entry(x, bias, y, rows, cols, x_row_stride, y_row_stride, scale,
                              log_output != 0 || causal_period != 0, log_output, causal_period, dtype, param_dtype, stream);
}
