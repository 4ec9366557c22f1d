// kop_affine_relu_pool2d: per-channel affine (folded BatchNorm), optional ReLU and windowed max / average
// pooling over NCHW planes in one pass: the activation is never written to memory, only the pooled map is.
//
// A CTA owns a band of output rows of one (n, c) plane. The input rows the band needs are contiguous in
// memory, so they are fetched once with flat 16-byte loads, turned into fp32 activations and parked in a
// shared-memory tile that already contains the padding (-inf for max, 0 for average): the windows are then
// read from shared memory without bounds checks, and overlapping windows cost no extra HBM traffic (only
// the kh - sh halo rows between bands are read twice). Bands are sized to about 24 KB of tile so that
// several CTAs share an SM and overlap their phases.
#include <algorithm>

#include "kop_common.cuh"

namespace kop {
namespace {

// A per-channel parameter vector in fp32 or in a 16-bit type, read once per plane: the type is a runtime tag (no
// second set of kernel instances for the parameter type; the load is outside every inner loop).
struct ParamVec {
    const void* p;
    int tag;                                                 // kop_dtype_t of the vector
    __device__ __forceinline__ float at(int64_t j) const
    {
        if (tag == KOP_F32) return __ldg(static_cast<const float*>(p) + j);
        if (tag == KOP_BF16) return Elem<__nv_bfloat16>::load1(static_cast<const __nv_bfloat16*>(p) + j);
        return Elem<__half>::load1(static_cast<const __half*>(p) + j);
    }
};

constexpr int kPoolThreads = 256;
constexpr int kPoolTileBytes = 24 * 1024;       // preferred tile size
constexpr int kPoolTileMax = 46 * 1024;         // static + dynamic shared memory stays under the 48 KB default

// max that returns NaN when either operand is NaN: one instruction
__device__ __forceinline__ float max_keep_nan(float m, float a)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(m), "f"(a));
    return r;
}

// i / d for 0 <= i < 2^22 without an integer division: float estimate, one-step fix-up
__device__ __forceinline__ int div_small(int i, int d, float inv_d)
{
    int q = (int)((float)i * inv_d);
    const int r = i - q * d;
    q += (r >= d) ? 1 : 0;
    q -= (r < 0) ? 1 : 0;
    return q;
}

// affine, then ReLU as one NaN-propagating max (relu_floor = 0) or nothing (relu_floor = -inf)
__device__ __forceinline__ float act_of(float v, float sc, float sf, float relu_floor)
{
    return max_keep_nan(fmaf(v, sc, sf), relu_floor);
}

// Tile geometry shared by host and device: image column 0 sits at tile column `lead` (the left padding
// rounded up to four floats, so that staged rows start 16-byte aligned and take 128-bit shared-memory
// stores); a tile row holds lead + W + pw floats, rounded up to four.
__host__ __device__ __forceinline__ int pool_lead(int pw) { return (pw + 3) / 4 * 4; }
__host__ __device__ __forceinline__ int pool_row_floats(int W, int pw) { return (pool_lead(pw) + W + pw + 3) / 4 * 4; }

// One window out of the tile: the max (NaN-propagating) or the average of kh x kw cells starting at `win`.
template <int MODE, int KS>
__device__ __forceinline__ float window_value(const float* win, int Ws, int kh, int kw, float inv_area)
{
    float res = MODE == 0 ? -INFINITY : 0.0f;
    if (KS) {
#pragma unroll
        for (int di = 0; di < (KS ? KS : 1); ++di)
#pragma unroll
            for (int dj = 0; dj < (KS ? KS : 1); ++dj) {
                const float a = win[di * Ws + dj];
                res = MODE == 0 ? max_keep_nan(res, a) : res + a;
            }
    } else {
        for (int di = 0; di < kh; ++di)
            for (int dj = 0; dj < kw; ++dj) {
                const float a = win[di * Ws + dj];
                res = MODE == 0 ? max_keep_nan(res, a) : res + a;
            }
    }
    return MODE == 1 ? res * inv_area : res;
}

// MODE 0 max, 1 average. KS / ST: compile-time square window and stride (0 = use the runtime values).
// Consecutive threads take consecutive outputs: their windows start sw floats apart in shared memory (a
// 2-way bank conflict at stride 2 instead of the 8-way one of a vector of outputs per thread), and a warp's
// 32 scalar stores still make one contiguous run.
// kRowMap: a warp takes whole rows (lanes along the row), so no index is ever divided; used when rows are
// long enough to keep most lanes busy. Otherwise threads walk the band's flat index range.
template <typename T, int MODE, int KS, int ST, bool kVecIn, bool kRowMap>
__global__ void __launch_bounds__(kPoolThreads)
pool2d_tile_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                   T* __restrict__ y, int C, int H, int W, int OH, int OW, int kh_, int kw_, int sh_, int sw_,
                   int ph, int pw, int band_rows, int bands, int relu_flag, float inv_area)
{
    constexpr int E = Elem<T>::kPerVec;
    extern __shared__ __align__(16) float tile[];
    const float relu = relu_flag ? 0.0f : -INFINITY;
    const int kh = KS ? KS : kh_, kw = KS ? KS : kw_, sh = ST ? ST : sh_, sw = ST ? ST : sw_;
    const int64_t plane = blockIdx.x / bands;
    const int band = (int)(blockIdx.x - plane * bands);
    const int c = (int)(plane % C);
    const float sc = scale.p != nullptr ? scale.at(c) : 1.0f;
    const float sf = shift.p != nullptr ? shift.at(c) : 0.0f;
    const float pad = MODE == 0 ? -INFINITY : 0.0f;

    const int oh0 = band * band_rows;
    const int oh1 = min(OH, oh0 + band_rows);
    const int t0 = oh0 * sh - ph;                            // first tile row, in image coordinates (may be < 0)
    const int trows = (oh1 - 1 - oh0) * sh + kh;             // tile rows
    const int lead = pool_lead(pw), Ws = pool_row_floats(W, pw);
    const int i0 = max(t0, 0), i1 = min(t0 + trows, H);      // image rows present in the tile

    // 1. padding cells only: whole rows above / below the image, then the pw cells left and right of the rest
    const int top = i0 - t0, bottom = t0 + trows - i1;       // padding rows in the tile (each 0 .. ph)
    for (int k = threadIdx.x; k < (top + bottom) * Ws; k += kPoolThreads) {
        const int r = k < top * Ws ? 0 : (i1 - t0) - top;    // rows [0, top) and [i1 - t0, trows)
        tile[r * Ws + k] = pad;
    }
    for (int k = threadIdx.x; k < (i1 - i0) * 2 * pw; k += kPoolThreads) {
        const int r = k / (2 * pw), m = k - r * 2 * pw;
        tile[(top + r) * Ws + (m < pw ? lead - pw + m : lead + W + m - pw)] = pad;
    }
    // 2. the band's input rows: one contiguous run of (i1 - i0) * W elements
    const T* xp = x + (plane * H + i0) * (int64_t)W;
    const int n_in = (i1 - i0) * W;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (kVecIn && kRowMap) {
        const int wv = W / E, nrows = i1 - i0;
        constexpr int NW = kPoolThreads / 32;
        for (int cv = lane; cv < wv; cv += 32) {
            const T* src = xp + warp * W + cv * E;
            float* dst_f = tile + (top + warp) * Ws + lead + cv * E;
#pragma unroll 2
            for (int r = warp; r < nrows; r += NW, src += NW * W, dst_f += NW * Ws) {
                float f[E];
                Elem<T>::unpack(ld_stream(src), f);
                float4* dst = reinterpret_cast<float4*>(dst_f);
#pragma unroll
                for (int q = 0; q < E / 4; ++q)
                    dst[q] = make_float4(act_of(f[4 * q], sc, sf, relu), act_of(f[4 * q + 1], sc, sf, relu),
                                         act_of(f[4 * q + 2], sc, sf, relu), act_of(f[4 * q + 3], sc, sf, relu));
            }
        }
    } else if (kVecIn) {
        const float inv_w = 1.0f / (float)W;
        for (int v = threadIdx.x; v < n_in / E; v += kPoolThreads) {
            float f[E];
            Elem<T>::unpack(ld_stream(xp + (int64_t)v * E), f);
            const int idx = v * E;
            const int r = div_small(idx, W, inv_w), cc = idx - r * W;   // W % E == 0: a vector stays inside one row
            float4* dst = reinterpret_cast<float4*>(tile + (top + r) * Ws + lead + cc);     // 16-byte aligned
#pragma unroll
            for (int q = 0; q < E / 4; ++q)
                dst[q] = make_float4(act_of(f[4 * q], sc, sf, relu), act_of(f[4 * q + 1], sc, sf, relu),
                                     act_of(f[4 * q + 2], sc, sf, relu), act_of(f[4 * q + 3], sc, sf, relu));
        }
    } else {
        // rows that are not whole vectors (odd widths, bases off a boundary): the run as head elements up to the first
        // 16-byte boundary, aligned vectors whose elements may continue in the next row, and tail elements
        int head = (int)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(xp) & 15u)) & 15u) / (unsigned)sizeof(T));
        if (head > n_in) head = n_in;
        const int nv = (n_in - head) / E, tail0 = head + nv * E;
        const float inv_w = 1.0f / (float)W;
        for (int k = threadIdx.x; k < head + (n_in - tail0); k += kPoolThreads) {
            const int idx = k < head ? k : tail0 + (k - head);
            const int r = div_small(idx, W, inv_w), cc = idx - r * W;
            tile[(top + r) * Ws + lead + cc] = act_of(Elem<T>::load1(xp + idx), sc, sf, relu);
        }
        const T* xm = xp + head;
#pragma unroll 2
        for (int v = threadIdx.x; v < nv; v += kPoolThreads) {
            float f[E];
            Elem<T>::unpack(ld_stream(xm + (int64_t)v * E), f);
            const int idx = head + v * E;
            const int r = div_small(idx, W, inv_w);
            int cc = idx - r * W;
            float* dst = tile + (top + r) * Ws + lead + cc;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                *dst++ = act_of(f[e], sc, sf, relu);
                if (++cc == W) {
                    cc = 0;
                    dst += Ws - W;
                }
            }
        }
    }
    __syncthreads();
    // 3. windows out of the tile; the band's outputs are one contiguous run of (oh1 - oh0) * OW elements
    T* yp = y + (plane * OH + oh0) * (int64_t)OW;
    const int n_out = (oh1 - oh0) * OW;
    const float inv_ow = 1.0f / (float)OW;
    const float* origin = tile + (lead - pw);
    if (kRowMap) {
        constexpr int NW = kPoolThreads / 32;
        const int orows = oh1 - oh0;
        for (int ocol = lane; ocol < OW; ocol += 32) {
            const float* win = origin + warp * sh * Ws + ocol * sw;
            T* dst = yp + warp * OW + ocol;
#pragma unroll 2
            for (int orow = warp; orow < orows; orow += NW, win += NW * sh * Ws, dst += NW * OW) {
                Elem<T>::store1(dst, window_value<MODE, KS>(win, Ws, kh, kw, inv_area));
            }
        }
    } else {
        for (int o = threadIdx.x; o < n_out; o += kPoolThreads) {
            const int orow = div_small(o, OW, inv_ow), ocol = o - orow * OW;
            Elem<T>::store1(yp + o, window_value<MODE, KS>(origin + orow * sh * Ws + ocol * sw, Ws, kh, kw, inv_area));
        }
    }
}

// ---- strip kernel: the two stride-2 windows CNNs use (3x3 pad 1, 2x2 pad 0), no shared memory ----------
// A thread owns eight input columns (four outputs) of a band of output rows and walks down the rows: per
// input row two 16-byte loads (one for bf16) plus, for 3x3, the single halo element to its left (a scalar
// load that hits L1), the affine / ReLU on the nine values, the four horizontal window reductions, and per
// output row the vertical combination of three (two) such rows, the lowest of which is carried over to
// the next output row. About four instructions per input element, no index arithmetic inside the loop,
// every load and store of a warp a contiguous run.
template <typename T, int MODE>
__device__ __forceinline__ float pool_op(float a, float b) { return MODE == 0 ? max_keep_nan(a, b) : a + b; }

// Eight consecutive elements of the data type as floats: one 256-bit load for fp32 (a lane then uses whole
// 32-byte sectors; two 128-bit loads would fetch every sector twice, L1 allocation being off), one 128-bit
// load for bf16.
__device__ __forceinline__ void load8(const float* p, float (&f)[8])
{
    uint32_t w[8];
    asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(w[e]);
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&f)[8])
{
    Elem<__nv_bfloat16>::unpack(ld_stream(p), f);
}

__device__ __forceinline__ void load8(const __half* p, float (&f)[8])
{
    Elem<__half>::unpack(ld_stream(p), f);
}

// The raw values of one row for one thread: its eight columns and, for the first / last lane of a warp, the halo
// element that no neighbour lane holds. All loads are issued here, before anything is computed.
template <typename T>
struct StripRowRaw {
    float f[8];
    float edge;
};
template <typename T>
__device__ __forceinline__ void strip_load_s1(const T* __restrict__ row, int seg, int segs, int lane, StripRowRaw<T>& r)
{
    load8(row, r.f);
    r.edge = 0.0f;
    if (lane == 0 && seg > 0) r.edge = Elem<T>::load1(row - 1);
    if (lane == 31 && seg < segs - 1) r.edge = Elem<T>::load1(row + 8);
}

// The stride-2 kernel's loads: only a left halo exists there.
template <typename T, int KS>
__device__ __forceinline__ void strip_load_s2(const T* __restrict__ row, int seg, int lane, StripRowRaw<T>& r)
{
    load8(row, r.f);
    r.edge = 0.0f;
    if (KS == 3 && lane == 0 && seg > 0) r.edge = Elem<T>::load1(row - 1);
}

// Horizontal reductions of one input row for this thread's four outputs. KS == 3: windows of columns
// (2j-1, 2j, 2j+1) relative to the thread's first column, v[0] being the halo, which is the left
// neighbour lane's last column (a shuffle; lane 0 of a warp loads it); KS == 2: (2j, 2j+1). Rows outside
// the image are loaded from a clamped row and overridden with padding, so the warp stays converged for
// the shuffle. Called by all 32 lanes.
template <typename T, int MODE, int KS>
__device__ __forceinline__ void strip_row(const StripRowRaw<T>& raw, bool row_ok, int seg, int lane, float sc,
                                          float sf, float relu, float (&h)[4])
{
    const float pad = MODE == 0 ? -INFINITY : 0.0f;
    float v[9];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[1 + e] = row_ok ? act_of(raw.f[e], sc, sf, relu) : pad;
    if (KS == 3) {
        float left = __shfl_up_sync(0xFFFFFFFFu, v[8], 1);
        if (lane == 0) left = row_ok ? act_of(raw.edge, sc, sf, relu) : pad;
        v[0] = seg > 0 ? left : pad;
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = pool_op<T, MODE>(pool_op<T, MODE>(v[2 * j], v[2 * j + 1]), v[2 * j + 2]);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) h[j] = pool_op<T, MODE>(v[2 * j + 1], v[2 * j + 2]);
    }
}

template <typename T>
__device__ __forceinline__ void store4(T* dst, const float (&o)[4]);
template <>
__device__ __forceinline__ void store4<float>(float* dst, const float (&o)[4])
{
    st_stream(dst, Elem<float>::pack(o));
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* dst, const float (&o)[4])
{
    const __nv_bfloat162 a = __floats2bfloat162_rn(o[0], o[1]), b = __floats2bfloat162_rn(o[2], o[3]);
    uint2 w;
    w.x = *reinterpret_cast<const uint32_t*>(&a);
    w.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(dst) = w;                   // four outputs = 8 bytes, 8-byte aligned (OW % 4 == 0)
}

template <>
__device__ __forceinline__ void store4<__half>(__half* dst, const float (&o)[4])
{
    const __half2 a = __floats2half2_rn(o[0], o[1]), b = __floats2half2_rn(o[2], o[3]);
    uint2 w;
    w.x = *reinterpret_cast<const uint32_t*>(&a);
    w.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(dst) = w;
}

// R: output rows per trip, all 2 R row loads issued before the first is used (R = 2 measured slower for every data
// type: bf16 3x3 4.4 to 3.6 TB/s, 2x2 5.5 to 5.0).
template <typename T, int MODE, int KS, int R>
__global__ void __launch_bounds__(256)
pool2d_strip_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                    T* __restrict__ y, int64_t strips, int C, int H, int W, int OH, int OW, int segs, int bands,
                    int band_rows, int relu_flag, float inv_area)
{
    const int64_t g_raw = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = g_raw < strips;                       // surplus threads of the last CTA shadow the last strip
    const int64_t g = live ? g_raw : strips - 1;
    const int lane = threadIdx.x & 31;
    const int seg = (int)(g % segs);
    const int64_t rest = g / segs;
    const int band = (int)(rest % bands);
    const int64_t plane = rest / bands;
    const int c = (int)(plane % C);
    const float sc = scale.p != nullptr ? scale.at(c) : 1.0f;
    const float sf = shift.p != nullptr ? shift.at(c) : 0.0f;
    const float relu = relu_flag ? 0.0f : -INFINITY;
    constexpr int P = KS == 3 ? 1 : 0;
    const int oh0 = band * band_rows, oh1 = min(OH, oh0 + band_rows);
    const T* col = x + plane * H * (int64_t)W + seg * 8;            // this strip's first column, row 0
    T* out = y + (plane * OH + oh0) * (int64_t)OW + seg * 4;

    float carry[4];
    if (KS == 3) {
        const int i = 2 * oh0 - P;
        StripRowRaw<T> r0;
        strip_load_s2<T, KS>(col + (int64_t)max(i, 0) * W, seg, lane, r0);
        strip_row<T, MODE, KS>(r0, i >= 0, seg, lane, sc, sf, relu, carry);
    }
    // every lane runs band_rows trips so that the shuffles stay warp-wide; trips past a short last band are idle
    for (int t = 0; t < band_rows; t += R, out += (int64_t)R * OW) {
        StripRowRaw<T> ra[R], rb[R];                                  // all rows' loads first, then the arithmetic
        int i2s[R];
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const int oi = min(oh0 + t + k, OH - 1);
            const int i1 = 2 * oi - P + (KS == 3 ? 1 : 0);            // the two rows first needed by this output row
            i2s[k] = i1 + 1;
            strip_load_s2<T, KS>(col + (int64_t)i1 * W, seg, lane, ra[k]);
            strip_load_s2<T, KS>(col + (int64_t)min(i1 + 1, H - 1) * W, seg, lane, rb[k]);
        }
#pragma unroll
        for (int k = 0; k < R; ++k) {
            float a[4], b[4], o[4];
            strip_row<T, MODE, KS>(ra[k], true, seg, lane, sc, sf, relu, a);
            strip_row<T, MODE, KS>(rb[k], i2s[k] < H, seg, lane, sc, sf, relu, b);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float r = pool_op<T, MODE>(a[j], b[j]);
                if (KS == 3) {
                    r = pool_op<T, MODE>(carry[j], r);
                    carry[j] = b[j];
                }
                o[j] = MODE == 1 ? r * inv_area : r;
            }
            if (live && oh0 + t + k < oh1) store4<T>(out + (int64_t)k * OW, o);
        }
    }
}

// ---- the strip walk for stride-2 windows on rows of any width and alignment -----------------------------------
// Widths that are not whole 8-column segments (55, 27, 147, 71, 35: the pooling layers of AlexNet-, SqueezeNet- and
// Inception-style networks, 3 x 3 / stride 2 without padding) start every row at another offset from a 16-byte
// boundary. A thread still owns four outputs and the nine (eight) input columns under them, but fetches them as the
// aligned 16-byte vectors that cover them (three for fp32, two for 16-bit data) and picks its elements by the
// offset, which is the same for all threads of a row, so the selection is a warp-uniform switch over register
// moves. Every thread loads its own halo column: no shuffles, so threads past the end leave and short bands stop.
// The first and last 16 bytes of the tensor are read element by element where a whole vector would cross its end.
template <typename T>
__device__ __forceinline__ Vec16 window_vector(uintptr_t q, uintptr_t xb, uintptr_t xe)
{
    if (q >= xb && q + 16 <= xe) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(q));
        return Vec16{{t.x, t.y, t.z, t.w}};
    }
    Vec16 v{{0u, 0u, 0u, 0u}};
    constexpr int E = Elem<T>::kPerVec;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const uintptr_t a = q + e * sizeof(T);
        if (a >= xb && a + sizeof(T) <= xe) {
            if constexpr (sizeof(T) == 4) v.w[e] = *reinterpret_cast<const uint32_t*>(a);
            else v.w[e / 2] |= (uint32_t)(*reinterpret_cast<const unsigned short*>(a)) << (16 * (e & 1));
        }
    }
    return v;
}

// The nine elements that start at p, widened: r[0 .. 8].
template <typename T>
__device__ __forceinline__ void window9(const T* p, uintptr_t xb, uintptr_t xe, float (&r)[9])
{
    const uintptr_t addr = reinterpret_cast<uintptr_t>(p), base = addr & ~(uintptr_t)15;
    const int s = (int)((addr - base) / sizeof(T));
    if constexpr (sizeof(T) == 4) {
        const Vec16 a = window_vector<T>(base, xb, xe), b = window_vector<T>(base + 16, xb, xe),
                    c = window_vector<T>(base + 32, xb, xe);
        const uint32_t w[12] = {a.w[0], a.w[1], a.w[2], a.w[3], b.w[0], b.w[1], b.w[2], b.w[3], c.w[0], c.w[1], c.w[2], c.w[3]};
        switch (s) {
        case 0:
#pragma unroll
            for (int e = 0; e < 9; ++e) r[e] = __uint_as_float(w[e]);
            break;
        case 1:
#pragma unroll
            for (int e = 0; e < 9; ++e) r[e] = __uint_as_float(w[e + 1]);
            break;
        case 2:
#pragma unroll
            for (int e = 0; e < 9; ++e) r[e] = __uint_as_float(w[e + 2]);
            break;
        default:
#pragma unroll
            for (int e = 0; e < 9; ++e) r[e] = __uint_as_float(w[e + 3]);
            break;
        }
    } else {
        const Vec16 a = window_vector<T>(base, xb, xe), b = window_vector<T>(base + 16, xb, xe);
        const uint32_t w[8] = {a.w[0], a.w[1], a.w[2], a.w[3], b.w[0], b.w[1], b.w[2], b.w[3]};
        uint32_t u[5];
        switch (s >> 1) {
        case 0:
#pragma unroll
            for (int i = 0; i < 5; ++i) u[i] = w[i];
            break;
        case 1:
#pragma unroll
            for (int i = 0; i < 5; ++i) u[i] = w[i + 1];
            break;
        case 2:
#pragma unroll
            for (int i = 0; i < 5; ++i) u[i] = w[i + 2];
            break;
        default:
#pragma unroll
            for (int i = 0; i < 5; ++i) u[i] = w[i + 3];
            break;
        }
        if (s & 1) {
#pragma unroll
            for (int i = 0; i < 4; ++i) u[i] = __funnelshift_r(u[i], u[i + 1], 16);
            u[4] >>= 16;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f;
            Elem<T>::unpack_pair(u[i], f);
            r[2 * i] = f.x;
            r[2 * i + 1] = f.y;
        }
        float2 f;
        Elem<T>::unpack_pair(u[4], f);
        r[8] = f.x;
    }
}

// 3 x 3 windows; ST: stride 1 or 2; P: padding 0 or 1 (both directions). A thread's nine elements start at column
// 4 ST seg - P; with padding the columns from W on are padding too (the last window of a row reaches one).
template <typename T, int MODE, int ST, int P>
__global__ void __launch_bounds__(256)
pool2d_strip_any_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift, T* __restrict__ y, int64_t strips,
                        int64_t x_elems, int C, int H, int W, int OH, int OW, int segs, int bands, int band_rows,
                        int relu_flag, float inv_area)
{
    constexpr int KS = 3;
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= strips) return;
    const int seg = (int)(g % segs);
    const int64_t rest = g / segs;
    const int band = (int)(rest % bands);
    const int64_t plane = rest / bands;
    const int c = (int)(plane % C);
    const float sc = scale.p != nullptr ? scale.at(c) : 1.0f;
    const float sf = shift.p != nullptr ? shift.at(c) : 0.0f;
    const float relu = relu_flag ? 0.0f : -INFINITY;
    const float pad = MODE == 0 ? -INFINITY : 0.0f;
    const uintptr_t xb = reinterpret_cast<uintptr_t>(x), xe = xb + (uintptr_t)x_elems * sizeof(T);
    const int oh0 = band * band_rows, oh1 = min(OH, oh0 + band_rows);
    const int c0 = seg * 4 * ST - P;                                  // this strip's first column (the halo with padding)
    const T* col = x + plane * H * (int64_t)W + c0;
    T* out = y + (plane * OH + oh0) * (int64_t)OW + seg * 4;
    const int nout = min(4, OW - seg * 4);
    const int nvalid = W - c0;                                        // elements of the nine that are image columns

    // horizontal windows of input row i for this thread's four outputs
    auto hrow = [&](int i, float (&h)[4]) {
        const bool row_ok = i >= 0 && i < H;
        float v[9];
        window9<T>(col + (int64_t)min(max(i, 0), H - 1) * W, xb, xe, v);
#pragma unroll
        for (int e = 0; e < 9; ++e) v[e] = (row_ok && (P == 0 || e < nvalid)) ? act_of(v[e], sc, sf, relu) : pad;
        if (P == 1 && seg == 0) v[0] = pad;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            h[j] = pool_op<T, MODE>(pool_op<T, MODE>(v[ST * j], v[ST * j + 1]), v[ST * j + 2]);
    };
    float hs[KS][4];
#pragma unroll
    for (int i = 0; i < KS - ST; ++i) hrow(ST * oh0 - P + i, hs[i]);
    for (int oh = oh0; oh < oh1; ++oh, out += OW) {
#pragma unroll
        for (int i = KS - ST; i < KS; ++i) hrow(ST * oh - P + i, hs[i]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float r = pool_op<T, MODE>(pool_op<T, MODE>(hs[0][j], hs[1][j]), hs[2][j]);
            if (j < nout) Elem<T>::store1(out + j, MODE == 1 ? r * inv_area : r);
        }
#pragma unroll
        for (int i = 0; i < KS - ST; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) hs[i][j] = hs[i + ST][j];
    }
}

// ---- the same strip walk for 3x3 windows at stride 1 (pad 1): eight outputs per thread and row ----------------
// A thread owns eight columns and produces the eight outputs above them: per input row one vector load, the left
// and right halo values from the neighbour lanes by shuffle (the first / last lane of a warp loads its own; at the
// image edge it is padding), eight horizontal window reductions; the horizontal results of the two rows above are
// carried in registers, so every input row is loaded once per band. No shared memory, no barrier, loads of the
// next rows in flight while the current ones are combined.
template <typename T, int MODE>
__device__ __forceinline__ void strip_row_s1(const StripRowRaw<T>& raw, bool row_ok, int seg, int segs, int lane,
                                             float sc, float sf, float relu, float (&h)[8])
{
    const float pad = MODE == 0 ? -INFINITY : 0.0f;
    float v[10];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[1 + e] = row_ok ? act_of(raw.f[e], sc, sf, relu) : pad;
    const float edge = row_ok ? act_of(raw.edge, sc, sf, relu) : pad;
    float left = __shfl_up_sync(0xFFFFFFFFu, v[8], 1);
    float right = __shfl_down_sync(0xFFFFFFFFu, v[1], 1);
    if (lane == 0) left = edge;
    if (lane == 31) right = edge;
    v[0] = seg > 0 ? left : pad;
    v[9] = seg < segs - 1 ? right : pad;
#pragma unroll
    for (int j = 0; j < 8; ++j) h[j] = pool_op<T, MODE>(pool_op<T, MODE>(v[j], v[j + 1]), v[j + 2]);
}

template <typename T>
__device__ __forceinline__ void store8(T* dst, const float (&o)[8])
{
    if constexpr (sizeof(T) == 4) {
        const float a[4] = {o[0], o[1], o[2], o[3]}, b[4] = {o[4], o[5], o[6], o[7]};
        st_stream(dst, Elem<float>::pack(a));
        st_stream(dst + 4, Elem<float>::pack(b));
    } else {
        st_stream(dst, Elem<T>::pack(o));
    }
}

// R: input rows loaded per trip (all R loads are issued before the first is used).
template <typename T, int MODE, int R>
__global__ void __launch_bounds__(256)
pool2d_strip_s1_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                       T* __restrict__ y, int64_t strips, int C, int H, int W, int segs, int bands, int band_rows,
                       int relu_flag, float inv_area)
{
    const int64_t g_raw = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = g_raw < strips;                       // surplus threads of the last CTA shadow the last strip
    const int64_t g = live ? g_raw : strips - 1;
    const int lane = threadIdx.x & 31;
    const int seg = (int)(g % segs);
    const int64_t rest = g / segs;
    const int band = (int)(rest % bands);
    const int64_t plane = rest / bands;
    const int c = (int)(plane % C);
    const float sc = scale.p != nullptr ? scale.at(c) : 1.0f;
    const float sf = shift.p != nullptr ? shift.at(c) : 0.0f;
    const float relu = relu_flag ? 0.0f : -INFINITY;
    const int oh0 = band * band_rows, oh1 = min(H, oh0 + band_rows);      // OH == H, OW == W
    const T* col = x + plane * H * (int64_t)W + seg * 8;
    T* out = y + (plane * H + oh0) * (int64_t)W + seg * 8;

    float up[8], mid[8];
    {
        StripRowRaw<T> a, b;
        strip_load_s1<T>(col + (int64_t)max(oh0 - 1, 0) * W, seg, segs, lane, a);
        strip_load_s1<T>(col + (int64_t)oh0 * W, seg, segs, lane, b);
        strip_row_s1<T, MODE>(a, oh0 >= 1, seg, segs, lane, sc, sf, relu, up);
        strip_row_s1<T, MODE>(b, true, seg, segs, lane, sc, sf, relu, mid);
    }
    // every lane runs the same number of trips so that the shuffles stay warp-wide; rows past the band are idle
    for (int t = 0; t < band_rows; t += R, out += (int64_t)R * W) {
        StripRowRaw<T> raw[R];
#pragma unroll
        for (int k = 0; k < R; ++k) strip_load_s1<T>(col + (int64_t)min(oh0 + t + k + 1, H - 1) * W, seg, segs, lane, raw[k]);
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const int i2 = oh0 + t + k + 1;
            float low[8], o[8];
            strip_row_s1<T, MODE>(raw[k], i2 < H, seg, segs, lane, sc, sf, relu, low);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float r = pool_op<T, MODE>(pool_op<T, MODE>(up[j], mid[j]), low[j]);
                o[j] = MODE == 1 ? r * inv_area : r;
                up[j] = mid[j];
                mid[j] = low[j];
            }
            if (live && oh0 + t + k < oh1) store8<T>(out + (int64_t)k * W, o);
        }
    }
}

// Small planes (up to 32 x 32: 28 x 28, 14 x 14, 7 x 7 ...), any window geometry: a CTA per plane would leave most
// of its threads idle and most of its 16-byte loads ragged. Consecutive planes are contiguous, so a CTA takes a
// run of G planes (G a multiple of the vector length: every run starts on a 16-byte boundary) as one flat
// array: 16-byte loads across plane boundaries, the activations parked in shared memory as fp32 with each
// plane's scale / shift, then one thread per output over the whole run, windows read from shared memory with
// bounds checks, outputs (contiguous for the run) stored by consecutive threads.
// KS: 3 or 2 for square windows of that size (taps unrolled), 0 for any window.
// kFixed (stride-1 windows, where outputs are as many as inputs and their index arithmetic was most of the kernel):
// thread t keeps one output position of the plane for the whole run (see the output loop).
template <typename T, int MODE, int KS, bool kFixed>
__global__ void __launch_bounds__(kPoolThreads, kFixed ? 6 : 0)
pool2d_planes_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                     T* __restrict__ y, int64_t planes, int G, int Gp, int C, int H, int W, int OH, int OW, int kh, int kw,
                     int sh, int sw, int ph, int pw, float relu_floor, float inv_area)
{
    constexpr int E = Elem<T>::kPerVec;
    extern __shared__ __align__(16) float planes_smem[];
    const int nthreads = kFixed ? (int)blockDim.x : kPoolThreads;    // the fixed-position CTA is trimmed to whole passes
    const int plane = H * W, oplane = OH * OW;
    float* act = planes_smem;
    float* sc_s = act + G * plane;
    float* sf_s = sc_s + G;
    const int64_t p0 = (int64_t)blockIdx.x * G;
    const int g_here = (int)(planes - p0 < G ? planes - p0 : G);
    const int elems = g_here * plane;
    const T* xc = x + p0 * plane;
    for (int g = threadIdx.x; g < g_here; g += nthreads) {
        const int c = (int)((p0 + g) % C);
        sc_s[g] = scale.p != nullptr ? scale.at(c) : 1.0f;
        sf_s[g] = shift.p != nullptr ? shift.at(c) : 0.0f;
    }
    __syncthreads();
    const float inv_plane = 1.0f / (float)plane;
    const int nvec = elems / E;
    constexpr int U = 4;                                     // loads in flight per thread
    for (int base = 0; base < nvec; base += U * nthreads) {
        Vec16 raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * nthreads + threadIdx.x;
            if (v < nvec) raw[k] = ld_stream(xc + (int64_t)v * E);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * nthreads + threadIdx.x;
            if (v < nvec) {
                float f[E];
                Elem<T>::unpack(raw[k], f);
                const int i0 = v * E;
                int pl = div_small(i0, plane, inv_plane);
                int rem = i0 - pl * plane;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    f[e] = act_of(f[e], sc_s[pl], sf_s[pl], relu_floor);
                    if (++rem == plane) {
                        rem = 0;
                        ++pl;
                    }
                }
                float4* dst = reinterpret_cast<float4*>(act + i0);
#pragma unroll
                for (int q = 0; q < E / 4; ++q) dst[q] = make_float4(f[4 * q], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
            }
        }
    }
    for (int i = nvec * E + threadIdx.x; i < elems; i += nthreads) {     // the tensor's last run may end inside a vector
        const int pl = i / plane;
        act[i] = act_of(Elem<T>::load1(xc + i), sc_s[pl], sf_s[pl], relu_floor);
    }
    __syncthreads();
    const float inv_oplane = 1.0f / (float)oplane, inv_ow = 1.0f / (float)OW;
    T* yc = y + p0 * oplane;
    const int n_out = g_here * oplane;
    if constexpr (kFixed) {
        // Plane slot t / oplane of each pass of Gp planes, position t % oplane. The window geometry is worked out
        // once: clamped tap offsets (a clamped tap repeats an element of the same window, which leaves a maximum
        // unchanged and is masked out of a sum), so a pass costs the taps and a store, with no index division and no
        // bounds predicate per output. The CTA is trimmed to the warps that have a position.
        const int slot = (int)threadIdx.x / oplane;
        const int r = (int)threadIdx.x - slot * oplane;
        if (slot >= Gp) return;
        const int oi = r / OW, oj = r - oi * OW;
        const int i_lo = oi * sh - ph, j_lo = oj * sw - pw;
        int off[KS ? KS : 1][KS ? KS : 1];
        unsigned rm[KS ? KS : 1], cm[KS ? KS : 1];
#pragma unroll
        for (int d = 0; d < KS; ++d) {
            rm[d] = (unsigned)(i_lo + d) < (unsigned)H ? 0xFFFFFFFFu : 0u;
            cm[d] = (unsigned)(j_lo + d) < (unsigned)W ? 0xFFFFFFFFu : 0u;
        }
#pragma unroll
        for (int di = 0; di < KS; ++di)
#pragma unroll
            for (int dj = 0; dj < KS; ++dj)
                off[di][dj] = min(max(i_lo + di, 0), H - 1) * W + min(max(j_lo + dj, 0), W - 1);
        const float* a = act + slot * plane;
        T* yo = yc + threadIdx.x;
        const int a_step = Gp * plane, o_step = Gp * oplane;
        for (int g = slot; g < g_here; g += Gp, a += a_step, yo += o_step) {
            float res;
            if (MODE == 0) {
                res = a[off[0][0]];
#pragma unroll
                for (int di = 0; di < KS; ++di)
#pragma unroll
                    for (int dj = 0; dj < KS; ++dj)
                        if (di + dj > 0) res = max_keep_nan(res, a[off[di][dj]]);
            } else {
                res = 0.0f;
#pragma unroll
                for (int di = 0; di < KS; ++di) {
                    float rs = __uint_as_float(__float_as_uint(a[off[di][0]]) & cm[0]);
#pragma unroll
                    for (int dj = 1; dj < KS; ++dj) rs += __uint_as_float(__float_as_uint(a[off[di][dj]]) & cm[dj]);
                    res += __uint_as_float(__float_as_uint(rs) & rm[di]);
                }
                res *= inv_area;
            }
            Elem<T>::store1(yo, res);
        }
    } else {
    for (int o = threadIdx.x; o < n_out; o += nthreads) {
        const int g = div_small(o, oplane, inv_oplane);
        const int r = o - g * oplane;
        const int oi = div_small(r, OW, inv_ow), oj = r - oi * OW;
        const float* a = act + g * plane;
        const int i_lo = oi * sh - ph, j_lo = oj * sw - pw;
        float res = MODE == 0 ? -INFINITY : 0.0f;
        if (KS) {
            bool col_ok[KS ? KS : 1];
#pragma unroll
            for (int dj = 0; dj < KS; ++dj) col_ok[dj] = (unsigned)(j_lo + dj) < (unsigned)W;
            const float* win = a + i_lo * W + j_lo;
#pragma unroll
            for (int di = 0; di < KS; ++di) {
                const bool row_ok = (unsigned)(i_lo + di) < (unsigned)H;
#pragma unroll
                for (int dj = 0; dj < KS; ++dj) {
                    // an excluded tap counts as the identity (-inf / 0) and its address is never formed
                    const float t = (row_ok && col_ok[dj]) ? win[di * W + dj] : (MODE == 0 ? -INFINITY : 0.0f);
                    res = MODE == 0 ? max_keep_nan(res, t) : res + t;
                }
            }
        } else {
            for (int di = 0; di < kh; ++di) {
                const int i = i_lo + di;
                if (i < 0 || i >= H) continue;
                for (int dj = 0; dj < kw; ++dj) {
                    const int j = j_lo + dj;
                    if (j < 0 || j >= W) continue;
                    res = MODE == 0 ? max_keep_nan(res, a[i * W + j]) : res + a[i * W + j];
                }
            }
        }
        Elem<T>::store1(yc + o, MODE == 0 ? res : res * inv_area);
    }
    }
}

// ---- 2 x 2 windows at stride 2 without padding: nothing is shared between windows ------------------------------
// Every output reads its own four inputs, two adjacent elements in each of two rows, so no tile is needed: a thread
// per output (two outputs a thread for bytes in flight), one load of a pair per row when the pairs are aligned
// (even width, plane rows starting on a pair boundary), and consecutive threads take consecutive outputs, so a
// warp's two loads cover a contiguous run of input rows between them (the first the even rows, the second the odd
// ones; the read-only path keeps the shared sectors in L1) and its stores are contiguous. The output index is taken
// apart with multiply-shift divisions by the two invariant divisors (exact while index * divisor < 2^40).
struct MagicDiv {
    uint64_t m;                                              // ceil(2^40 / d)
    int d;
    __device__ __forceinline__ int div(int n) const { return (int)(((uint64_t)(unsigned)n * m) >> 40); }
};

template <typename T, int MODE, bool kPair>
__global__ void __launch_bounds__(256)
pool2d_k2s2_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift, T* __restrict__ y, int total, MagicDiv by_c,
                   int H, int W, MagicDiv by_oplane, MagicDiv by_ow, float relu_floor, float inv_area)
{
    constexpr int U = sizeof(T) == 4 ? 2 : 4;                // outputs per thread: 16 bytes of loads in flight each
    const bool identity = scale.p == nullptr && relu_floor == -INFINITY;
    const int o0 = (int)blockIdx.x * (U * 256) + (int)threadIdx.x;
    float v[U][4];
    int pl[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 256;
        pl[u] = 0;
        if (o < total) {
            const int p = by_oplane.div(o), r = o - p * by_oplane.d;
            const int oi = by_ow.div(r), oj = r - oi * by_ow.d;
            pl[u] = p;
            const T* top = x + ((int64_t)p * H + 2 * oi) * W + 2 * oj;
            if constexpr (kPair) {
                if constexpr (sizeof(T) == 4) {
                    const float2 a = __ldg(reinterpret_cast<const float2*>(top));
                    const float2 b = __ldg(reinterpret_cast<const float2*>(top + W));
                    v[u][0] = a.x, v[u][1] = a.y, v[u][2] = b.x, v[u][3] = b.y;
                } else {
                    const uint32_t a = __ldg(reinterpret_cast<const uint32_t*>(top));
                    const uint32_t b = __ldg(reinterpret_cast<const uint32_t*>(top + W));
                    float2 fa[1], fb[1];
                    Elem<T>::unpack_pair(a, fa[0]);
                    Elem<T>::unpack_pair(b, fb[0]);
                    v[u][0] = fa[0].x, v[u][1] = fa[0].y, v[u][2] = fb[0].x, v[u][3] = fb[0].y;
                }
            } else {
                v[u][0] = Elem<T>::load1(top), v[u][1] = Elem<T>::load1(top + 1);
                v[u][2] = Elem<T>::load1(top + W), v[u][3] = Elem<T>::load1(top + W + 1);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 256;
        if (o < total) {
            if (!identity) {
                const int c = pl[u] - by_c.div(pl[u]) * by_c.d;
                const float sc = scale.p != nullptr ? scale.at(c) : 1.0f, sf = shift.p != nullptr ? shift.at(c) : 0.0f;
#pragma unroll
                for (int e = 0; e < 4; ++e) v[u][e] = act_of(v[u][e], sc, sf, relu_floor);
            }
            float res;
            if (MODE == 0) res = max_keep_nan(max_keep_nan(v[u][0], v[u][1]), max_keep_nan(v[u][2], v[u][3]));
            else res = ((v[u][0] + v[u][1]) + (v[u][2] + v[u][3])) * inv_area;
            Elem<T>::store1(y + o, res);
        }
    }
}

// The same for K x K windows at stride K without padding (K = 3, 4): K * K element loads an output; consecutive threads
// take consecutive outputs, so the K loads of an input row by a warp cover a contiguous run between them.
template <typename T, int MODE, int K>
__global__ void __launch_bounds__(256)
pool2d_kksk_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift, T* __restrict__ y, int total, MagicDiv by_c,
                   int H, int W, MagicDiv by_oplane, MagicDiv by_ow, float relu_floor, float inv_area)
{
    constexpr int U = 2;                                     // outputs per thread
    const bool identity = scale.p == nullptr && relu_floor == -INFINITY;
    const int o0 = (int)blockIdx.x * (U * 256) + (int)threadIdx.x;
    float v[U][K * K];
    int pl[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 256;
        pl[u] = 0;
        if (o < total) {
            const int p = by_oplane.div(o), r = o - p * by_oplane.d;
            const int oi = by_ow.div(r), oj = r - oi * by_ow.d;
            pl[u] = p;
            const T* top = x + ((int64_t)p * H + K * oi) * W + K * oj;
#pragma unroll
            for (int di = 0; di < K; ++di)
#pragma unroll
                for (int dj = 0; dj < K; ++dj) v[u][di * K + dj] = Elem<T>::load1(top + (int64_t)di * W + dj);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 256;
        if (o < total) {
            if (!identity) {
                const int c = pl[u] - by_c.div(pl[u]) * by_c.d;
                const float sc = scale.p != nullptr ? scale.at(c) : 1.0f, sf = shift.p != nullptr ? shift.at(c) : 0.0f;
#pragma unroll
                for (int e = 0; e < K * K; ++e) v[u][e] = act_of(v[u][e], sc, sf, relu_floor);
            }
            float res = v[u][0];
#pragma unroll
            for (int e = 1; e < K * K; ++e) res = MODE == 0 ? max_keep_nan(res, v[u][e]) : res + v[u][e];
            Elem<T>::store1(y + o, MODE == 0 ? res : res * inv_area);
        }
    }
}

// The same for widths that are a multiple of four: a thread takes two adjacent outputs at a time, one load of four
// elements per row (16 bytes of fp32, 8 of 16-bit data) and one store of the pair, which halves the index arithmetic
// and the memory instructions per output (what bounded the 16-bit path above).
template <typename T, int MODE>
__global__ void __launch_bounds__(256)
pool2d_k2s2_quad_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift, T* __restrict__ y, int units, MagicDiv by_c,
                        int H, int W, MagicDiv by_uplane, MagicDiv by_uw, float relu_floor, float inv_area)
{
    constexpr int U = sizeof(T) == 4 ? 2 : 4;
    const bool identity = scale.p == nullptr && relu_floor == -INFINITY;
    const int q0 = (int)blockIdx.x * (U * 256) + (int)threadIdx.x;
    float v[U][8];                                           // row 2i: elements 0..3, row 2i + 1: elements 4..7
    int pl[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int q = q0 + u * 256;
        pl[u] = 0;
        if (q < units) {
            const int p = by_uplane.div(q), r = q - p * by_uplane.d;
            const int oi = by_uw.div(r), oj2 = r - oi * by_uw.d;
            pl[u] = p;
            const T* top = x + ((int64_t)p * H + 2 * oi) * W + 4 * oj2;
            if constexpr (sizeof(T) == 4) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(top));
                const float4 b = __ldg(reinterpret_cast<const float4*>(top + W));
                v[u][0] = a.x, v[u][1] = a.y, v[u][2] = a.z, v[u][3] = a.w;
                v[u][4] = b.x, v[u][5] = b.y, v[u][6] = b.z, v[u][7] = b.w;
            } else {
                const uint2 a = __ldg(reinterpret_cast<const uint2*>(top));
                const uint2 b = __ldg(reinterpret_cast<const uint2*>(top + W));
                float2 f;
                Elem<T>::unpack_pair(a.x, f);
                v[u][0] = f.x, v[u][1] = f.y;
                Elem<T>::unpack_pair(a.y, f);
                v[u][2] = f.x, v[u][3] = f.y;
                Elem<T>::unpack_pair(b.x, f);
                v[u][4] = f.x, v[u][5] = f.y;
                Elem<T>::unpack_pair(b.y, f);
                v[u][6] = f.x, v[u][7] = f.y;
            }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int q = q0 + u * 256;
        if (q < units) {
            if (!identity) {
                const int c = pl[u] - by_c.div(pl[u]) * by_c.d;
                const float sc = scale.p != nullptr ? scale.at(c) : 1.0f, sf = shift.p != nullptr ? shift.at(c) : 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) v[u][e] = act_of(v[u][e], sc, sf, relu_floor);
            }
            float r0, r1;
            if (MODE == 0) {
                r0 = max_keep_nan(max_keep_nan(v[u][0], v[u][1]), max_keep_nan(v[u][4], v[u][5]));
                r1 = max_keep_nan(max_keep_nan(v[u][2], v[u][3]), max_keep_nan(v[u][6], v[u][7]));
            } else {
                r0 = ((v[u][0] + v[u][1]) + (v[u][4] + v[u][5])) * inv_area;
                r1 = ((v[u][2] + v[u][3]) + (v[u][6] + v[u][7])) * inv_area;
            }
            if constexpr (sizeof(T) == 4) {
                *reinterpret_cast<float2*>(y + 2 * (int64_t)q) = make_float2(r0, r1);
            } else {
                T two[2];
                Elem<T>::store1(&two[0], r0);
                Elem<T>::store1(&two[1], r1);
                *reinterpret_cast<uint32_t*>(y + 2 * (int64_t)q) = *reinterpret_cast<const uint32_t*>(two);
            }
        }
    }
}

// ---- the window is the whole plane (global average / max pooling): a reduction per plane --------------------------
// L lanes per plane (L = 2 .. 32, a power of two chosen from the plane's size), 32 / L planes per warp, eight warps per
// CTA; a lane sweeps its share of the plane in batches of four 16-byte vectors (scalars when planes are not whole
// aligned vectors), activates and accumulates in fp32, and a butterfly over the plane's lanes finishes it. The sum is
// a fixed order (lane-sequential, then the butterfly): bit-identical from run to run.
// VB: bytes per load (16, 8, 4 or one element: the widest that divides a plane's bytes and the tensor's alignment).
// A load lands as raw words and is widened when it is used, so that a batch in flight costs its bytes in registers.
template <int VB>
struct RawUnit {
    uint32_t w[VB >= 4 ? VB / 4 : 1];
};

template <typename T, int VB>
__device__ __forceinline__ RawUnit<VB> load_raw(const T* p)
{
    RawUnit<VB> r;
    if constexpr (VB == 16) {
        const Vec16 v = ld_stream(p);
        r.w[0] = v.w[0], r.w[1] = v.w[1], r.w[2] = v.w[2], r.w[3] = v.w[3];
    } else if constexpr (VB == 8) {
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
        r.w[0] = t.x, r.w[1] = t.y;
    } else if constexpr (VB == 4) {
        r.w[0] = __ldg(reinterpret_cast<const uint32_t*>(p));
    } else {
        r.w[0] = __ldg(reinterpret_cast<const unsigned short*>(p));
    }
    return r;
}

template <typename T, int VB>
__device__ __forceinline__ void widen_raw(const RawUnit<VB>& r, float (&f)[VB / (int)sizeof(T)])
{
    if constexpr (VB == 16) {
        Elem<T>::unpack(Vec16{{r.w[0], r.w[1], r.w[2], r.w[3]}}, f);
    } else if constexpr (sizeof(T) == 4) {
#pragma unroll
        for (int i = 0; i < VB / 4; ++i) f[i] = __uint_as_float(r.w[i]);
    } else if constexpr (VB >= 4) {
#pragma unroll
        for (int i = 0; i < VB / 4; ++i) {
            float2 a;
            Elem<T>::unpack_pair(r.w[i], a);
            f[2 * i] = a.x, f[2 * i + 1] = a.y;
        }
    } else {
        float2 a;
        Elem<T>::unpack_pair(r.w[0], a);                     // the value sits in the low half
        f[0] = a.x;
    }
}

template <typename T, int MODE, int VB, int L>
__global__ void __launch_bounds__(256)
pool2d_global_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift, T* __restrict__ y, int planes, int plane,
                     MagicDiv by_c, float relu_floor, float inv_area)
{
    constexpr int EV = VB / (int)sizeof(T);                  // elements per load
    constexpr int U = VB >= 16 ? 4 : (VB == 8 ? 8 : 16);     // loads in flight per lane: 64 bytes (32 for 2-byte loads)
    constexpr int kPerWarp = 32 / L;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int p = ((int)blockIdx.x * 8 + ((int)threadIdx.x >> 5)) * kPerWarp + lane / L;
    const bool live = p < planes;
    const bool identity = scale.p == nullptr && relu_floor == -INFINITY;
    float sc = 1.0f, sf = 0.0f;
    if (live && !identity) {
        const int c = p - by_c.div(p) * by_c.d;
        sc = scale.p != nullptr ? scale.at(c) : 1.0f;
        sf = shift.p != nullptr ? shift.at(c) : 0.0f;
    }
    const T* xp = x + (int64_t)(live ? p : 0) * plane;
    float acc = MODE == 0 ? -INFINITY : 0.0f;
    const int n = live ? plane / EV : 0;                     // loads this plane's lanes share
    for (int base = 0; base < n; base += U * L) {
        RawUnit<VB> raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * L + sub;
            if (v < n) raw[k] = load_raw<T, VB>(xp + (int64_t)v * EV);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * L + sub;
            if (v < n) {
                float f[EV];
                widen_raw<T, VB>(raw[k], f);
#pragma unroll
                for (int e = 0; e < EV; ++e) {
                    const float a = identity ? f[e] : act_of(f[e], sc, sf, relu_floor);
                    acc = MODE == 0 ? max_keep_nan(acc, a) : acc + a;
                }
            }
        }
    }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        // the lower lane's term first on both sides, so that the two lanes agree bit for bit
        acc = MODE == 0 ? max_keep_nan(acc, other) : ((lane & o) ? other + acc : acc + other);
    }
    if (live && sub == 0) Elem<T>::store1(y + p, MODE == 0 ? acc : acc * inv_area);
}

// ---- walk kernel: 2x2 / 3x3 windows at stride 1 or 2, any width, any alignment --------------------------------
// What the strip kernel above does in registers for its two aligned stride-2 cases, done out of a shared-memory tile
// for everything else with these windows: stride 1, widths that are not whole vectors, rows that do not start on a
// 16-byte boundary, small planes. A CTA takes either a band of output rows of one plane or a run of whole small
// planes (always a contiguous piece of memory): flat 16-byte loads (scalar head / tail where the piece does not
// start or end on a vector), fp32 activations parked in a tile that already holds the padding, every plane's row
// 16-byte aligned. Then each thread owns four adjacent outputs of a row and walks down the output rows: per input
// row one or two 128-bit shared-memory loads (plus the single left-halo float when the window is padded), the
// KS - ST rows shared by consecutive windows kept in registers, vertical combination first (one operation per
// column), then the four horizontal windows. No index division inside the walk, about five arithmetic
// instructions and well under one shared-memory load per output.
template <int KS, int ST>
struct WalkGeom {
    static constexpr int kCols = 3 * ST + KS;          // input columns under four adjacent windows
};

// Tile geometry (host and device): image column 0 at tile column `lead`; a tile row is long enough for the
// last group's reads (groups of four outputs, the last one possibly ragged) plus a vector of slack.
__host__ __device__ __forceinline__ int walk_row_floats(int W, int OW, int pw, int KS, int ST)
{
    const int lead = pool_lead(pw), OG = (OW + 3) / 4;
    const int need_data = lead + W + pw, need_read = lead - pw + 4 * OG * ST - ST + KS + 3;
    return ((need_data > need_read ? need_data : need_read) + 3) / 4 * 4;
}

template <typename T, int MODE, int KS, int ST, bool kPadW>
__global__ void __launch_bounds__(kPoolThreads)
pool2d_walk_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                   T* __restrict__ y, int64_t planes, int np, int C, int H, int W, int OH, int OW, int ph,
                   int band_rows, int bands, int chunks, int relu_flag, float inv_area)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int NV = WalkGeom<KS, ST>::kCols;
    constexpr int pw = kPadW ? 1 : 0;
    extern __shared__ __align__(16) float tile[];
    const float relu = relu_flag ? 0.0f : -INFINITY;
    const float pad = MODE == 0 ? -INFINITY : 0.0f;
    const int lead = pool_lead(pw), Ws = walk_row_floats(W, OW, pw, KS, ST);

    // what this CTA owns: planes [p0, p0 + nq), output rows [oh0, oh1) of each
    int64_t p0;
    int nq, oh0, oh1;
    if (np > 1) {
        p0 = (int64_t)blockIdx.x * np;
        nq = (int)(planes - p0 < np ? planes - p0 : np);
        oh0 = 0;
        oh1 = OH;
    } else {
        p0 = blockIdx.x / bands;
        const int band = (int)(blockIdx.x - p0 * bands);
        nq = 1;
        oh0 = band * band_rows;
        oh1 = min(OH, oh0 + band_rows);
    }
    const int t0 = oh0 * ST - ph;                            // first tile row in image coordinates (may be < 0)
    const int trows = (oh1 - 1 - oh0) * ST + KS;
    const int i0 = max(t0, 0), i1 = min(t0 + trows, H);      // image rows present
    const int top = i0 - t0, nrows = i1 - i0;
    const int PS = ((np > 1 ? (OH - 1) * ST + KS : (band_rows - 1) * ST + KS)) * Ws;      // floats per plane in the tile
    float* sc_s = tile + np * PS;                            // per-plane scale / shift behind the tiles
    float* sf_s = sc_s + np;
    for (int q = threadIdx.x; q < nq; q += kPoolThreads) {
        const int c = (int)((p0 + q) % C);
        sc_s[q] = scale.p != nullptr ? scale.at(c) : 1.0f;
        sf_s[q] = shift.p != nullptr ? shift.at(c) : 0.0f;
    }
    // 1. padding cells: rows above / below the image, then the pw cells left and right of the image rows
    {
        const int bottom = trows - top - nrows;
        const int per_plane = (top + bottom) * Ws;
        for (int k = threadIdx.x; k < nq * per_plane; k += kPoolThreads) {
            const int q = k / per_plane, m = k - q * per_plane;
            tile[q * PS + (m < top * Ws ? m : m + nrows * Ws)] = pad;
        }
        if (kPadW) {
            for (int k = threadIdx.x; k < nq * nrows * 2; k += kPoolThreads) {
                const int q = k / (nrows * 2), m = k - q * nrows * 2;
                const int r = m >> 1;
                tile[q * PS + (top + r) * Ws + ((m & 1) ? lead + W : lead - 1)] = pad;
            }
        }
    }
    __syncthreads();                                         // scale / shift visible
    // 2. the input: one contiguous piece of nq * nrows * W elements (nq > 1 only with whole planes: nrows == H)
    {
        const T* xp = x + (p0 * H + i0) * (int64_t)W;
        const int n_in = nq * nrows * W;
        const int plane_in = nrows * W;
        const float inv_w = 1.0f / (float)W, inv_plane = 1.0f / (float)plane_in;
        const int head_raw = (int)(((16 - (reinterpret_cast<uintptr_t>(xp) & 15)) & 15) / sizeof(T));
        const int head = head_raw < n_in ? head_raw : n_in;
        const int nvec = (n_in - head) / E;
        auto put = [&](int idx, float v) {                   // one element by flat index (head, tail)
            const int q = nq > 1 ? div_small(idx, plane_in, inv_plane) : 0;
            const int rem = idx - q * plane_in;
            const int r = div_small(rem, W, inv_w);
            tile[q * PS + (top + r) * Ws + lead + (rem - r * W)] = act_of(v, sc_s[q], sf_s[q], relu);
        };
        for (int i = threadIdx.x; i < head; i += kPoolThreads) put(i, Elem<T>::load1(xp + i));
        for (int i = head + nvec * E + threadIdx.x; i < n_in; i += kPoolThreads) put(i, Elem<T>::load1(xp + i));
        constexpr int U = 4;
        for (int base = 0; base < nvec; base += U * kPoolThreads) {
            Vec16 raw[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int v = base + k * kPoolThreads + threadIdx.x;
                if (v < nvec) raw[k] = ld_stream(xp + head + (int64_t)v * E);
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int v = base + k * kPoolThreads + threadIdx.x;
                if (v < nvec) {
                    float f[E];
                    Elem<T>::unpack(raw[k], f);
                    const int idx = head + v * E;
                    int q = nq > 1 ? div_small(idx, plane_in, inv_plane) : 0;
                    const int rem = idx - q * plane_in;
                    int r = div_small(rem, W, inv_w);
                    int cc = rem - r * W;
                    if (((W | head) & 3) == 0) {
                        // rows are whole groups of four and the piece starts on one: a group never leaves its row
#pragma unroll
                        for (int h = 0; h < E / 4; ++h) {
                            const float sc = sc_s[q], sf = sf_s[q];
                            *reinterpret_cast<float4*>(tile + q * PS + (top + r) * Ws + lead + cc) =
                                make_float4(act_of(f[4 * h], sc, sf, relu), act_of(f[4 * h + 1], sc, sf, relu),
                                            act_of(f[4 * h + 2], sc, sf, relu), act_of(f[4 * h + 3], sc, sf, relu));
                            cc += 4;
                            if (cc == W) {
                                cc = 0;
                                if (++r == nrows) {
                                    r = 0;
                                    ++q;
                                }
                            }
                        }
                    } else {
                        // element by element with a running destination: rows and planes wrap rarely
                        float* d = tile + q * PS + (top + r) * Ws + lead + cc;
                        float sc = sc_s[q], sf = sf_s[q];
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            *d++ = act_of(f[e], sc, sf, relu);
                            if (++cc == W) {
                                cc = 0;
                                d += Ws - W;
                                if (++r == nrows) {
                                    r = 0;
                                    ++q;
                                    d += PS - nrows * Ws;
                                    if (e + 1 < E) {
                                        sc = sc_s[q];
                                        sf = sf_s[q];
                                    }
                                }
                            }
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
    // 3. walks: unit u = (chunk of output rows, plane, group of four outputs); consecutive threads take
    // consecutive groups, so shared-memory reads and global stores of a warp run along rows
    const int OG = (OW + 3) / 4;
    const int walkers = nq * OG;
    const int orows = oh1 - oh0;
    const int rpc = (orows + chunks - 1) / chunks;           // output rows per chunk
    const float inv_walkers = 1.0f / (float)walkers, inv_og = 1.0f / (float)OG;
    const bool vec_out = (OW & 3) == 0 && (reinterpret_cast<uintptr_t>(y) & (4 * sizeof(T) - 1)) == 0;
    for (int u = threadIdx.x; u < walkers * chunks; u += kPoolThreads) {
        const int chunk = div_small(u, walkers, inv_walkers);
        const int w = u - chunk * walkers;
        const int q = div_small(w, OG, inv_og), g = w - q * OG;
        const int r_lo = chunk * rpc, r_hi = min(orows, r_lo + rpc);
        if (r_lo >= r_hi) continue;
        const float* src = tile + q * PS + r_lo * ST * Ws + (lead - pw) + 4 * g * ST;
        T* dst = y + ((p0 + q) * OH + oh0 + r_lo) * (int64_t)OW + 4 * g;
        float rows[KS][NV];
        auto load_row = [&](const float* p, float (&v)[NV]) {
            // p is one float short of a 16-byte boundary when the window is padded, on one otherwise
            constexpr int first = kPadW ? 1 : 0;
            if (kPadW) v[0] = p[0];
#pragma unroll
            for (int b = first; b < NV; b += 4) {
                const float4 t = *reinterpret_cast<const float4*>(p + b);
                v[b] = t.x;
                if (b + 1 < NV) v[b + 1] = t.y;
                if (b + 2 < NV) v[b + 2] = t.z;
                if (b + 3 < NV) v[b + 3] = t.w;
            }
        };
#pragma unroll
        for (int i = 0; i < KS - ST; ++i) load_row(src + i * Ws, rows[i]);
        src += (KS - ST) * Ws;
        for (int r = r_lo; r < r_hi; ++r, src += ST * Ws, dst += OW) {
#pragma unroll
            for (int i = 0; i < ST; ++i) load_row(src + i * Ws, rows[KS - ST + i]);
            float colv[NV], o[4];
#pragma unroll
            for (int cidx = 0; cidx < NV; ++cidx) {
                float a = rows[0][cidx];
#pragma unroll
                for (int i = 1; i < KS; ++i) a = pool_op<T, MODE>(a, rows[i][cidx]);
                colv[cidx] = a;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float a = colv[j * ST];
#pragma unroll
                for (int d = 1; d < KS; ++d) a = pool_op<T, MODE>(a, colv[j * ST + d]);
                o[j] = MODE == 1 ? a * inv_area : a;
            }
            if (vec_out) store4<T>(dst, o);
            else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (4 * g + j < OW) Elem<T>::store1(dst + j, o[j]);
            }
#pragma unroll
            for (int i = 0; i < KS - ST; ++i)
#pragma unroll
                for (int cidx = 0; cidx < NV; ++cidx) rows[i][cidx] = rows[i + ST][cidx];
        }
    }
}

// Any geometry (rows too wide for the tile): one thread per output, window read from global memory.
template <typename T>
__global__ void __launch_bounds__(256)
pool2d_direct_kernel(const T* __restrict__ x, ParamVec scale, ParamVec shift,
                     T* __restrict__ y, int64_t total, int C, int H, int W, int OH, int OW, int kh, int kw, int sh,
                     int sw, int ph, int pw, int mode, int relu, float inv_area)
{
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int oj = (int)(o % OW);
        const int oi = (int)((o / OW) % OH);
        const int64_t plane = o / ((int64_t)OW * OH);
        const int c = (int)(plane % C);
        const float sc = scale.p != nullptr ? scale.at(c) : 1.0f;
        const float sf = shift.p != nullptr ? shift.at(c) : 0.0f;
        const T* xp = x + plane * H * (int64_t)W;
        float res = mode == 0 ? -INFINITY : 0.0f;
        for (int di = 0; di < kh; ++di) {
            const int i = oi * sh - ph + di;
            if (i < 0 || i >= H) continue;
            for (int dj = 0; dj < kw; ++dj) {
                const int j = oj * sw - pw + dj;
                if (j < 0 || j >= W) continue;
                const float a = act_of(Elem<T>::load1(xp + (int64_t)i * W + j), sc, sf, relu ? 0.0f : -INFINITY);
                res = mode == 0 ? max_keep_nan(res, a) : res + a;
            }
        }
        Elem<T>::store1(y + o, mode == 0 ? res : res * inv_area);
    }
}

template <typename T, int MODE, int KS, int ST>
void launch_tile(bool vin, bool rowmap, unsigned grid, size_t smem, cudaStream_t stream, const T* x,
                 ParamVec scale, ParamVec shift, T* y, int C, int H, int W, int OH, int OW, int kh, int kw,
                 int sh, int sw, int ph, int pw, int band_rows, int bands, int relu, float inv_area)
{
#define KOP_POOL_GO(VI, RM)                                                                                         \
    pool2d_tile_kernel<T, MODE, KS, ST, VI, RM><<<grid, kPoolThreads, smem, stream>>>(                               \
        x, scale, shift, y, C, H, W, OH, OW, kh, kw, sh, sw, ph, pw, band_rows, bands, relu, inv_area)
    if (vin && rowmap) KOP_POOL_GO(true, true);
    else if (vin) KOP_POOL_GO(true, false);
    else if (rowmap) KOP_POOL_GO(false, true);
    else KOP_POOL_GO(false, false);
#undef KOP_POOL_GO
}

template <typename T>
kop_status_t launch_pool(const void* xv, ParamVec scale, ParamVec shift, void* yv, int64_t N, int64_t C,
                         int H, int W, int OH, int OW, int kh, int kw, int sh, int sw, int ph, int pw, int mode,
                         int relu, cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    const T* x = static_cast<const T*>(xv);
    T* y = static_cast<T*>(yv);
    const float inv_area = (float)(1.0 / ((double)kh * kw));
    const int64_t planes = N * C;
    // the window is the plane: a reduction per plane (as windows 7 x 7 / 14 x 14 / 28 x 28 / 56 x 56 fp32 planes ran at 2.4 /
    // 2.4 / 1.1 / 0.7 TB/s, a thread looping over the plane per output; this way 4.5 / 6.6 / 6.3 / 6.0, bf16 2.7 / 5.4 / 5.9 / 5.5)
    if (kh == H && kw == W && ph == 0 && pw == 0 && planes < (1LL << 31) - 256 && (int64_t)H * W < (1 << 30) &&
        planes * C < (1LL << 40) && planes < (1LL << 24) * C) {
        const int plane = H * W;
        const int pbytes = plane * (int)sizeof(T);
        const int vb = (pbytes % 16 == 0 && aligned_to(x, 16)) ? 16
                       : (pbytes % 8 == 0 && aligned_to(x, 8)) ? 8
                       : (pbytes % 4 == 0 && aligned_to(x, 4)) ? 4 : (int)sizeof(T);
        const int units = pbytes / vb, per_lane = vb >= 16 ? 4 : (vb == 8 ? 8 : 16);
        int L = 2;
        while (L < 32 && L * per_lane < units) L *= 2;
        const MagicDiv by_c{((1ULL << 40) + (uint64_t)C - 1) / (uint64_t)C, (int)C};
        const int per_cta = 8 * (32 / L);
        const unsigned blocks = (unsigned)((planes + per_cta - 1) / per_cta);
        const float floor_v = relu ? 0.0f : -INFINITY;
        const float inv_plane = (float)(1.0 / ((double)H * W));
#define KOP_GLOBAL_L(M, V, LL) \
    pool2d_global_kernel<T, M, V, LL><<<blocks, 256, 0, stream>>>(x, scale, shift, y, (int)planes, plane, by_c, floor_v, inv_plane)
#define KOP_GLOBAL_V(M, V)                        \
    do {                                          \
        if (L == 2) KOP_GLOBAL_L(M, V, 2);        \
        else if (L == 4) KOP_GLOBAL_L(M, V, 4);   \
        else if (L == 8) KOP_GLOBAL_L(M, V, 8);   \
        else if (L == 16) KOP_GLOBAL_L(M, V, 16); \
        else KOP_GLOBAL_L(M, V, 32);              \
    } while (0)
#define KOP_GLOBAL(M)                                            \
    do {                                                         \
        if (vb == 16) KOP_GLOBAL_V(M, 16);                       \
        else if (vb == 8) KOP_GLOBAL_V(M, 8);                    \
        else if (vb == 4) KOP_GLOBAL_V(M, 4);                    \
        else KOP_GLOBAL_V(M, (int)sizeof(T));                    \
    } while (0)
        if (mode == 0) KOP_GLOBAL(0);
        else KOP_GLOBAL(1);
#undef KOP_GLOBAL_V
#undef KOP_GLOBAL
#undef KOP_GLOBAL_L
        return launch_status();
    }
    // the strip kernel: stride-2 3x3 (pad 1) or 2x2 (pad 0) windows over rows of whole 8-column segments
    const bool k3 = kh == 3 && kw == 3 && ph == 1 && pw == 1, k2 = kh == 2 && kw == 2 && ph == 0 && pw == 0;
    if ((k3 || k2) && sh == 2 && sw == 2 && W % 8 == 0 && H % 2 == 0 && aligned_to(x, 32) && aligned_to(y, 16)) {
        const int segs = W / 8;
        // bands of output rows: enough strips for a full complement of resident warps per SM, at least 4 output rows each
        int band_rows = OH;
        const int64_t want = 64LL * 32 * sm_count();
        while (band_rows > 4 && planes * segs * ((OH + band_rows - 1) / band_rows) < want) band_rows = (band_rows + 1) / 2;
        const int bands = (OH + band_rows - 1) / band_rows;
        const int64_t strips = planes * segs * bands;
        const int64_t blocks = (strips + 255) / 256;
        if (blocks <= 0x7FFFFFFFLL) {
#define KOP_STRIP(MODE, KS)                                                                                       \
    pool2d_strip_kernel<T, MODE, KS, 1><<<(unsigned)blocks, 256, 0, stream>>>(               \
        x, scale, shift, y, strips, (int)C, H, W, OH, OW, segs, bands, band_rows, relu, inv_area)
            if (mode == 0) {
                if (k3) KOP_STRIP(0, 3);
                else KOP_STRIP(0, 2);
            } else {
                if (k3) KOP_STRIP(1, 3);
                else KOP_STRIP(1, 2);
            }
#undef KOP_STRIP
            return launch_status();
        }
    }
    // 3 x 3 windows at stride 2 (with or without padding) or stride 1 (with padding) on rows of any width and alignment
    // that the aligned strip kernels do not take.
    // Planes from 256 elements (fp32 / bf16 TB/s against the runs-of-planes kernel: 17 x 17 3.2 / 1.6 to 3.7 / 1.9,
    // 28 x 28 3.2 / 1.8 to 4.0 / 2.0; 13 x 13 and 15 x 15 fp32 3.1 / 3.2 to 2.7 / 2.8)
    {
        const bool k3p0 = kh == 3 && kw == 3 && ph == 0 && pw == 0;
        // at stride 1 only odd widths (fp32 / bf16: 57 x 57 2.6 / 1.4 to 3.4 / 1.7, 35 x 35 3.1 / 1.5 to 3.3 / 1.6, 17 x 17
        // 2.7 / 1.3 to 3.0 / 1.3; even widths that are not whole segments are faster out of the shared-memory walk:
        // 28 x 28 3.8 / 2.3 against 2.9 / 1.4 here)
        if (((k3p0 || k3) && sh == 2 && sw == 2 && (int64_t)H * W >= 256) ||
            (k3 && sh == 1 && sw == 1 && W % 2 == 1 && (int64_t)H * W >= 256)) {
            const int segs = (OW + 3) / 4;
            int band_rows = OH;
            const int64_t want = 64LL * 32 * sm_count();
            while (band_rows > 4 && planes * segs * ((OH + band_rows - 1) / band_rows) < want) band_rows = (band_rows + 1) / 2;
            const int bands = (OH + band_rows - 1) / band_rows;
            const int64_t strips = planes * segs * bands;
            const int64_t blocks = (strips + 255) / 256;
            if (blocks <= 0x7FFFFFFFLL) {
#define KOP_STRIP_ANY(MODE, ST, P)                                                                     \
    pool2d_strip_any_kernel<T, MODE, ST, P><<<(unsigned)blocks, 256, 0, stream>>>(                     \
        x, scale, shift, y, strips, planes * H * W, (int)C, H, W, OH, OW, segs, bands, band_rows, relu, inv_area)
#define KOP_STRIP_ANY_M(MODE)                         \
    do {                                              \
        if (sh == 1) KOP_STRIP_ANY(MODE, 1, 1);       \
        else if (k3p0) KOP_STRIP_ANY(MODE, 2, 0);     \
        else KOP_STRIP_ANY(MODE, 2, 1);               \
    } while (0)
                if (mode == 0) KOP_STRIP_ANY_M(0);
                else KOP_STRIP_ANY_M(1);
#undef KOP_STRIP_ANY_M
#undef KOP_STRIP_ANY
                return launch_status();
            }
        }
    }
    // 2 x 2 / stride 2 without padding on anything the strip kernel does not take: a thread per output, no tile
    // (fp32 14 x 14 / 7 x 7 / 28 x 28 / 60 x 60 / 57 x 57 planes: 3.6 / 3.7 / 3.3 / 3.3 / 2.4 TB/s out of the shared-memory
    // kernels, 5.1 / 5.5 / 5.1 / 4.4 / 4.4 here; bf16 1.9 / 2.0 / 2.1 / 1.6 / 1.2 to 2.2 / 2.6 / 2.3 / 2.2 / 2.2)
    // (index * ceil(2^40 / divisor) must be exact and fit 64 bits: index * divisor < 2^40 and index / divisor < 2^24)
    if (k2 && sh == 2 && sw == 2 && planes * OH * OW < (1LL << 31) - 1024 && planes < (1LL << 24) && planes * C < (1LL << 40) &&
        planes * OH * OW * std::max((int64_t)OH * OW, (int64_t)1) < (1LL << 40)) {
        const int total = (int)(planes * OH * OW);
        const MagicDiv by_oplane{((1ULL << 40) + (uint64_t)(OH * OW) - 1) / (uint64_t)(OH * OW), OH * OW};
        const MagicDiv by_ow{((1ULL << 40) + (uint64_t)OW - 1) / (uint64_t)OW, OW};
        const MagicDiv by_c{((1ULL << 40) + (uint64_t)C - 1) / (uint64_t)C, (int)C};     // planes * C < 2^40: planes, C < 2^31 / ...
        const int per_cta = 256 * (sizeof(T) == 4 ? 2 : 4);
        const unsigned blocks = (unsigned)((total + per_cta - 1) / per_cta);
        const bool pair = W % 2 == 0 && aligned_to(x, 2 * sizeof(T));
        const float floor_v = relu ? 0.0f : -INFINITY;
        if (W % 4 == 0 && aligned_to(x, 4 * sizeof(T)) && aligned_to(y, 2 * sizeof(T))) {
            // two adjacent outputs a thread (fp32 28 x 28 / 60 x 60 / 4 x 4 planes 5.1 / 4.4 / 3.6 to 5.6 / 5.0 / 5.1 TB/s, bf16
            // 2.3 / 2.2 / 1.8 to 2.6 / 3.0 / 2.4)
            const int units = total / 2, uplane = OH * OW / 2, uw = OW / 2;
            const MagicDiv by_uplane{((1ULL << 40) + (uint64_t)uplane - 1) / (uint64_t)uplane, uplane};
            const MagicDiv by_uw{((1ULL << 40) + (uint64_t)uw - 1) / (uint64_t)uw, uw};
            const unsigned qblocks = (unsigned)((units + per_cta - 1) / per_cta);
            if (mode == 0)
                pool2d_k2s2_quad_kernel<T, 0><<<qblocks, 256, 0, stream>>>(x, scale, shift, y, units, by_c, H, W, by_uplane, by_uw, floor_v, inv_area);
            else
                pool2d_k2s2_quad_kernel<T, 1><<<qblocks, 256, 0, stream>>>(x, scale, shift, y, units, by_c, H, W, by_uplane, by_uw, floor_v, inv_area);
            return launch_status();
        }
#define KOP_K2S2(M, PR) \
    pool2d_k2s2_kernel<T, M, PR><<<blocks, 256, 0, stream>>>(x, scale, shift, y, total, by_c, H, W, by_oplane, by_ow, floor_v, inv_area)
        if (mode == 0) { if (pair) KOP_K2S2(0, true); else KOP_K2S2(0, false); }
        else { if (pair) KOP_K2S2(1, true); else KOP_K2S2(1, false); }
#undef KOP_K2S2
        return launch_status();
    }
    // K x K / stride K without padding, K = 3 or 4: a thread per output as well (same index limits)
    if (kh == kw && sh == kh && sw == kw && (kh == 3 || kh == 4) && ph == 0 && pw == 0 && planes * OH * OW < (1LL << 31) - 1024 &&
        planes < (1LL << 24) && planes * C < (1LL << 40) && planes * OH * OW * std::max((int64_t)OH * OW, (int64_t)1) < (1LL << 40)) {
        const int total = (int)(planes * OH * OW);
        const MagicDiv by_oplane{((1ULL << 40) + (uint64_t)(OH * OW) - 1) / (uint64_t)(OH * OW), OH * OW};
        const MagicDiv by_ow{((1ULL << 40) + (uint64_t)OW - 1) / (uint64_t)OW, OW};
        const MagicDiv by_c{((1ULL << 40) + (uint64_t)C - 1) / (uint64_t)C, (int)C};
        const unsigned blocks = (unsigned)((total + 511) / 512);
        const float floor_v = relu ? 0.0f : -INFINITY;
#define KOP_KKSK(M, K) \
    pool2d_kksk_kernel<T, M, K><<<blocks, 256, 0, stream>>>(x, scale, shift, y, total, by_c, H, W, by_oplane, by_ow, floor_v, inv_area)
        if (mode == 0) { if (kh == 3) KOP_KKSK(0, 3); else KOP_KKSK(0, 4); }
        else { if (kh == 3) KOP_KKSK(1, 3); else KOP_KKSK(1, 4); }
#undef KOP_KKSK
        return launch_status();
    }
    // 3x3 / stride 1 / pad 1 over rows of whole, aligned 8-column segments: the stride-1 strip kernel
    if (k3 && sh == 1 && sw == 1 && W % 8 == 0 && aligned_to(x, 32) && aligned_to(y, 32)) {
        const int segs = W / 8;
        // bands of at least 16 output rows (each band reads two rows of its neighbours again)
        int band_rows = H;
        const int64_t want = 64LL * 32 * sm_count();
        while (band_rows > 16 && planes * segs * ((H + band_rows - 1) / band_rows) < want) band_rows = (band_rows + 1) / 2;
        const int bands = (H + band_rows - 1) / band_rows;
        const int64_t strips = planes * segs * bands;
        const int64_t blocks = (strips + 255) / 256;
        if (blocks <= 0x7FFFFFFFLL) {
            // two input rows per trip (one: fp32 4.4 - 4.7 TB/s, bf16 2.9 - 3.4; two: 4.6 - 5.2 and 3.7 - 4.0; four: slower again)
            if (mode == 0)
                pool2d_strip_s1_kernel<T, 0, 2><<<(unsigned)blocks, 256, 0, stream>>>(x, scale, shift, y, strips, (int)C, H, W, segs, bands, band_rows, relu, inv_area);
            else
                pool2d_strip_s1_kernel<T, 1, 2><<<(unsigned)blocks, 256, 0, stream>>>(x, scale, shift, y, strips, (int)C, H, W, segs, bands, band_rows, relu, inv_area);
            return launch_status();
        }
    }
    // 2x2 / 3x3 windows at stride 1 or 2 that the strip kernel does not take (stride 1, any width or alignment,
    // small planes): the walk kernel, on runs of whole small planes or on bands of output rows of a large one
    // (planes of at most 1024 elements stay with the runs-of-planes kernel below, which copies them flat without
    // padding, unless the stride is 1 and the plane has 512 elements or more: 28 x 28 fp32 3 x 3 / 1 2.4 against 3.7 TB/s
    // here, but 14 x 14 2.4 against 2.2 and the stride-2 windows 3.1 - 3.4 against 2.7 - 3.1)
    const bool small_plane = (int64_t)H * W <= 1024;
    if (kh == kw && sh == sw && (kh == 2 || kh == 3) && (sh == 1 || sh == 2) && pw <= 1 &&
        (!small_plane || (sh == 1 && (int64_t)H * W >= 512))) {
        const int Ws = walk_row_floats(W, OW, pw, kh, sh);
        const int64_t plane_tile = ((int64_t)(OH - 1) * sh + kh) * Ws * 4;        // bytes of one whole padded plane
        const bool all_rows_used = (OH - 1) * sh + kh - ph >= H;                  // else a plane's rows are not one run
        int np = 1, br = OH, bands = 1;
        bool ok = true;
        if (plane_tile <= 12 * 1024 && all_rows_used && planes > 1) {
            np = (int)(32 * 1024 / plane_tile);
            if (np > planes) np = (int)planes;
        } else {
            const int64_t row_bytes = (int64_t)Ws * 4;
            // about 24 KB of tile per band (12 KB and 8 KB tiles were 25 - 45 % slower: more halo rows, shorter walks)
            int64_t b = ((int64_t)kPoolTileBytes / row_bytes - kh) / sh + 1;
            if (b < 1) b = 1;
            if (b > OH) b = OH;
            ok = ((b - 1) * sh + kh) * row_bytes + 8 <= kPoolTileMax;
            bands = (int)((OH + b - 1) / b);
            br = (int)((OH + bands - 1) / bands);                                 // even bands
            bands = (OH + br - 1) / br;
        }
        const int64_t grid = np > 1 ? (planes + np - 1) / np : planes * bands;
        const size_t smem = (size_t)np * (((size_t)(br - 1) * sh + kh) * Ws * 4 + 8);
        if (ok && grid <= 0x7FFFFFFFLL && smem <= (size_t)kPoolTileMax) {
            // one pass of the CTA's threads over (row chunks x planes x groups of four outputs), at least two output
            // rows per chunk where the band has them (the rows shared by consecutive windows stay in registers)
            const int walkers = np * ((OW + 3) / 4);
            int chunks = kPoolThreads / walkers;
            if (chunks > (br + 1) / 2) chunks = (br + 1) / 2;
            if (chunks < 1) chunks = 1;
#define KOP_WALK(M, K, S, P)                                                                                     \
    pool2d_walk_kernel<T, M, K, S, P><<<(unsigned)grid, kPoolThreads, smem, stream>>>(                             \
        x, scale, shift, y, planes, np, (int)C, H, W, OH, OW, ph, br, bands, chunks, relu, inv_area)
#define KOP_WALK_P(M, K, S)            \
    do {                               \
        if (pw) KOP_WALK(M, K, S, true); \
        else KOP_WALK(M, K, S, false);   \
    } while (0)
#define KOP_WALK_KS(M)                                   \
    do {                                                 \
        if (kh == 3 && sh == 1) KOP_WALK_P(M, 3, 1);     \
        else if (kh == 3) KOP_WALK_P(M, 3, 2);           \
        else if (sh == 1) KOP_WALK_P(M, 2, 1);           \
        else KOP_WALK_P(M, 2, 2);                        \
    } while (0)
            if (mode == 0) KOP_WALK_KS(0);
            else KOP_WALK_KS(1);
#undef KOP_WALK_KS
#undef KOP_WALK_P
#undef KOP_WALK
            return launch_status();
        }
    }
    // planes of at most 1024 elements that the strip kernel above does not take: runs of planes per CTA
    // (14 x 14 fp32, 3 x 3 / stride 2: 0.5 TB/s with a CTA per plane, 2.7 TB/s this way; 7 x 7: 0.2 to 2.8)
    if ((int64_t)H * W <= 1024 && aligned_to(x, 16)) {
        const int plane = H * W;
        int G = (6144 / plane) / E * E;
        if (G < E) G = E;
        const int64_t ctas = (planes + G - 1) / G;
        const size_t smem = ((size_t)G * plane + 2 * (size_t)G) * sizeof(float);
        if (ctas <= 0x7FFFFFFFLL && smem <= (size_t)kPoolTileMax && (int64_t)G * plane < (1 << 22)) {
            const float floor_v = relu ? 0.0f : -INFINITY;
            const int ks = (kh == kw && (kh == 2 || kh == 3)) ? kh : 0;
            // stride-1 2 x 2 / 3 x 3 windows with at most a CTA's worth of outputs per plane: one fixed output
            // position per thread, Gp planes per pass (14 x 14 fp32 3 x 3 / 1 max: 2.4 -> 3.5 TB/s, 7 x 7: 2.4 -> 3.1,
            // 4 x 4: 1.9 -> 2.9; at stride 2 the outputs are a quarter of the inputs and the extra registers of the
            // fixed geometry cost more occupancy than the loop saves: 2.9 -> 2.7, so those keep the plain loop)
            const int oplane = OH * OW;
            const bool fixed = ks != 0 && sh == 1 && sw == 1 && oplane <= kPoolThreads;
            const int Gp = fixed ? kPoolThreads / oplane : 0;
            const int threads = fixed ? (Gp * oplane + 31) / 32 * 32 : kPoolThreads;
#define KOP_POOL_PLANES(M, K, F) \
    pool2d_planes_kernel<T, M, K, F><<<(unsigned)ctas, threads, smem, stream>>>(x, scale, shift, y, planes, G, Gp, (int)C, H, W, OH, OW, kh, kw, sh, sw, ph, pw, floor_v, inv_area)
#define KOP_POOL_PLANES_F(M, K)             \
    do {                                    \
        if (fixed) KOP_POOL_PLANES(M, K, true); \
        else KOP_POOL_PLANES(M, K, false);  \
    } while (0)
            if (mode == 0) {
                if (ks == 3) KOP_POOL_PLANES_F(0, 3);
                else if (ks == 2) KOP_POOL_PLANES_F(0, 2);
                else KOP_POOL_PLANES(0, 0, false);
            } else {
                if (ks == 3) KOP_POOL_PLANES_F(1, 3);
                else if (ks == 2) KOP_POOL_PLANES_F(1, 2);
                else KOP_POOL_PLANES(1, 0, false);
            }
#undef KOP_POOL_PLANES_F
#undef KOP_POOL_PLANES
            return launch_status();
        }
    }
    const int64_t row_bytes = (int64_t)pool_row_floats(W, pw) * 4;
    if ((int64_t)kh * row_bytes <= kPoolTileMax) {
        // output rows per band: about kPoolTileBytes of tile, at least one row, then evened out
        int64_t br = ((int64_t)kPoolTileBytes / row_bytes - kh) / sh + 1;
        if (br < 1) br = 1;
        while (br > 1 && ((br - 1) * sh + kh) * row_bytes > kPoolTileMax) --br;
        if (br > OH) br = OH;
        {
            // among band heights down to half of that, take the one whose outputs fill the CTA's passes best
            // (row mapping: whole rows per warp, 8 warps; flat mapping: outputs per pass of 256 threads)
            const bool by_rows = ((aligned_to(x, 16) && W % E == 0) ? W / E : W) >= 20 && OW >= 20;
            const int64_t unit = by_rows ? 1 : OW, pass = by_rows ? kPoolThreads / 32 : kPoolThreads;
            int64_t best = br;
            double best_util = 0.0;
            for (int64_t cand = br; cand >= 1 && cand * 2 >= br; --cand) {
                const int64_t n = cand * unit;
                const double util = (double)n / (double)((n + pass - 1) / pass * pass);
                if (util > best_util + 1e-9) {
                    best_util = util;
                    best = cand;
                }
            }
            br = best;
        }
        const int bands = (int)((OH + br - 1) / br);
        const size_t smem = (size_t)(((br - 1) * sh + kh) * row_bytes);
        const int64_t grid = planes * bands;
        if (grid <= 0x7FFFFFFFLL && smem <= (size_t)kPoolTileMax) {
            // flat vector loads need every band to start on a 16-byte boundary: rows that are whole vectors
            const bool vin = aligned_to(x, 16) && W % E == 0;
            // a warp per row pays off when rows keep most of its lanes busy on both sides
            const bool rowmap = (vin ? W / E : W) >= 20 && OW >= 20;
            const unsigned g = (unsigned)grid;
#define KOP_POOL_ARGS vin, rowmap, g, smem, stream, x, scale, shift, y, (int)C, H, W, OH, OW, kh, kw, sh, sw, ph, pw, (int)br, bands, relu, inv_area
            const bool square = kh == kw && sh == sw;
            if (mode == 0) {
                if (square && kh == 3 && sh == 2) launch_tile<T, 0, 3, 2>(KOP_POOL_ARGS);
                else if (square && kh == 2 && sh == 2) launch_tile<T, 0, 2, 2>(KOP_POOL_ARGS);
                else if (square && kh == 3 && sh == 1) launch_tile<T, 0, 3, 1>(KOP_POOL_ARGS);
                else launch_tile<T, 0, 0, 0>(KOP_POOL_ARGS);
            } else {
                if (square && kh == 3 && sh == 2) launch_tile<T, 1, 3, 2>(KOP_POOL_ARGS);
                else if (square && kh == 2 && sh == 2) launch_tile<T, 1, 2, 2>(KOP_POOL_ARGS);
                else if (square && kh == 3 && sh == 1) launch_tile<T, 1, 3, 1>(KOP_POOL_ARGS);
                else launch_tile<T, 1, 0, 0>(KOP_POOL_ARGS);
            }
#undef KOP_POOL_ARGS
            return launch_status();
        }
    }
    const int64_t total = planes * OH * OW;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = 32LL * sm_count();
    if (blocks > cap) blocks = cap;
    pool2d_direct_kernel<T><<<(unsigned)blocks, 256, 0, stream>>>(x, scale, shift, y, total, (int)C, H, W, OH, OW, kh,
                                                                   kw, sh, sw, ph, pw, mode, relu, inv_area);
    return launch_status();
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

kop_status_t pool_entry(const void* x, const void* scale, const void* shift, void* y, int64_t N, int64_t C, int64_t H,
                        int64_t W, int kh, int kw, int sh, int sw, int ph, int pw, int mode, int relu, kop_dtype_t dtype,
                        kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    if (N < 0 || C <= 0 || H <= 0 || W <= 0) return KOP_ERR_BAD_SHAPE;
    if (kh <= 0 || kw <= 0 || sh <= 0 || sw <= 0 || ph < 0 || pw < 0 || ph > kh / 2 || pw > kw / 2)
        return KOP_ERR_BAD_SHAPE;
    if (mode != 0 && mode != 1) return KOP_ERR_BAD_SHAPE;
    if (C > 0x7FFFFFFF || H > 0x3FFFFFFF || W > 0x3FFFFFFF || N > kMaxElems) return KOP_ERR_BAD_SHAPE;
    if (kh > 0xFFFF || kw > 0xFFFF || H + 2 * (int64_t)ph < kh || W + 2 * (int64_t)pw < kw) return KOP_ERR_BAD_SHAPE;
    if (H > kMaxElems / W || C > kMaxElems / (H * W)) return KOP_ERR_BAD_SHAPE;
    if (N == 0) return KOP_OK;
    if (C * H * W > kMaxElems / N) return KOP_ERR_BAD_SHAPE;
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    if ((scale == nullptr) != (shift == nullptr)) return KOP_ERR_NULL_POINTER;      // both or neither
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (scale && !aligned_to(scale, elem_size(pdtype))) ||
        (shift && !aligned_to(shift, elem_size(pdtype))))
        return KOP_ERR_MISALIGNED;
    const int64_t OH = (H + 2 * (int64_t)ph - kh) / sh + 1, OW = (W + 2 * (int64_t)pw - kw) / sw + 1;
    {
        // the output has another shape: it must not overlap the input at all
        const uintptr_t a0 = reinterpret_cast<uintptr_t>(x), a1 = a0 + (uintptr_t)(N * C * H * W * esz);
        const uintptr_t b0 = reinterpret_cast<uintptr_t>(y), b1 = b0 + (uintptr_t)(N * C * OH * OW * esz);
        if (!(a1 <= b0 || b1 <= a0)) return KOP_ERR_BAD_ALIAS;
    }
    kop_status_t st = check_device();
    if (st != KOP_OK) return st;
    cudaStream_t s = as_stream(stream);
    const ParamVec sc{scale, (int)pdtype}, sf{shift, (int)pdtype};
    return dtype == KOP_F32 ? launch_pool<float>(x, sc, sf, y, N, C, (int)H, (int)W, (int)OH, (int)OW, kh, kw, sh, sw, ph, pw,
                                                 mode, relu != 0, s)
           : dtype == KOP_BF16
               ? launch_pool<__nv_bfloat16>(x, sc, sf, y, N, C, (int)H, (int)W, (int)OH, (int)OW, kh, kw, sh, sw, ph, pw, mode,
                                            relu != 0, s)
               : launch_pool<__half>(x, sc, sf, y, N, C, (int)H, (int)W, (int)OH, (int)OW, kh, kw, sh, sw, ph, pw, mode,
                                     relu != 0, s);
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_affine_relu_pool2d(const void* x, const float* scale, const float* shift, void* y,
                                               int64_t N, int64_t C, int64_t H, int64_t W, int kh, int kw, int sh,
                                               int sw, int ph, int pw, int mode, int relu, kop_dtype_t dtype,
                                               kop_stream_t stream)
{
    return kop::pool_entry(x, scale, shift, y, N, C, H, W, kh, kw, sh, sw, ph, pw, mode, relu, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_affine_relu_pool2d_ex(const void* x, const void* scale, const void* shift, void* y,
                                                  int64_t N, int64_t C, int64_t H, int64_t W, int kh, int kw, int sh,
                                                  int sw, int ph, int pw, int mode, int relu, kop_dtype_t dtype,
                                                  kop_dtype_t param_dtype, kop_stream_t stream)
{
    return kop::pool_entry(x, scale, shift, y, N, C, H, W, kh, kw, sh, sw, ph, pw, mode, relu, dtype, param_dtype, stream);
}
