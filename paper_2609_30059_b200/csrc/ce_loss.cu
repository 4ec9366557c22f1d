// kop_ce_loss_rowwise: loss[i] = logsumexp_j z[i,j] - z[i, label_i] and the mean over rows, with a
// single pass over the logits.
//
// One CTA streams one row. Each thread pulls a batch of 16-byte vectors into registers (all loads
// issued before first use), takes the batch maximum on the packed values, and then adds
// 2^(z*log2e - M) for every element with M the thread's running offset (the online-softmax
// recurrence, applied once per batch rather than once per element: one ex2 per element). The
// per-thread (M, S) pairs are merged across the CTA, lse = (M + log2 S) * ln 2, and thread 0
// subtracts the label logit. The last CTA to finish (a ticket counter in the workspace; nobody
// waits on it) sums loss[] in a fixed order, so the mean is bit-identical run to run.
#include <atomic>

#include "kop_common.cuh"

#ifndef KOP_CE_PACKED
#define KOP_CE_PACKED 1
#endif

namespace kop {
namespace {

// Workspace layout (all 4-byte words): [0] global ticket, [1..3] pad, then per group of
// kGroupRows rows: a ticket, a partial loss sum, a bad-label count, a counted-row count (the last
// only used by the variant with ignore_index).
constexpr int kGroupRows = 256;
static_assert(kGroupRows % 8 == 0, "a warp of the lanes-per-row kernel (up to 8 rows) must stay inside one group");
struct CeWorkspace {
    unsigned int* global_ticket;
    unsigned int* group_ticket;
    float* group_sum;
    int* group_bad;
    int* group_cnt;
};
// Options of kop_ce_loss_rowwise_opts (unused by the plain entry point).
struct CeOpts {
    int32_t ignore_index;
    float smoothing;
    int32_t* counted_rows;
    float* sum_loss;
};
__host__ __device__ inline int64_t ce_groups(int64_t rows) { return (rows + kGroupRows - 1) / kGroupRows; }
__host__ __device__ inline CeWorkspace ce_workspace(void* base, int64_t rows)
{
    const int64_t g = ce_groups(rows);
    unsigned int* w = static_cast<unsigned int*>(base);
    CeWorkspace ws;
    ws.global_ticket = w;
    ws.group_ticket = w + 4;
    ws.group_sum = reinterpret_cast<float*>(w + 4 + g);
    ws.group_bad = reinterpret_cast<int*>(w + 4 + 2 * g);
    ws.group_cnt = reinterpret_cast<int*>(w + 4 + 3 * g);
    return ws;
}
inline size_t ce_workspace_bytes(int64_t rows) { return (size_t)(4 + 4 * ce_groups(rows)) * 4; }
inline size_t ce_workspace_clear_bytes(int64_t rows) { return (size_t)(4 + ce_groups(rows)) * 4; }

template <typename T>
__device__ __forceinline__ float vec_max(const Vec16& v);

template <>
__device__ __forceinline__ float vec_max<float>(const Vec16& v)
{
    return fmaxf(fmaxf(__uint_as_float(v.w[0]), __uint_as_float(v.w[1])),
                 fmaxf(__uint_as_float(v.w[2]), __uint_as_float(v.w[3])));
}
template <>
__device__ __forceinline__ float vec_max<__nv_bfloat16>(const Vec16& v)
{
    // max.bf16x2: two elements per instruction.
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(v.w);
    const __nv_bfloat162 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
    return fmaxf(__low2float(m), __high2float(m));
}

template <>
__device__ __forceinline__ float vec_max<__half>(const Vec16& v)
{
    const __half2* h = reinterpret_cast<const __half2*>(v.w);
    const __half2 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
    return fmaxf(__low2float(m), __high2float(m));
}

__device__ __forceinline__ int warp_sum_int(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// What a whole warp does once its row's ticket `t` is known (the same value in all 32 lanes): nothing unless
// it was the group's last ticket.
template <bool kOpts>
__device__ __forceinline__ void ce_after_ticket(unsigned t, int64_t row, int lane, const int32_t* labels, float* loss,
                                                float* mean_loss, int32_t* bad_label_count, CeWorkspace ws,
                                                int64_t rows, int64_t vocab, CeOpts opts)
{
    const int64_t g = row / kGroupRows;
    const int64_t g0 = g * kGroupRows;
    const int gsize = (int)(rows - g0 < kGroupRows ? rows - g0 : kGroupRows);
    if (t != (unsigned)(gsize - 1)) return;
    __threadfence();
    float acc = 0.0f;
    int bad = 0, cnt = 0;
    for (int i = lane; i < gsize; i += 32) {
        acc += __ldcg(loss + g0 + i);
        const int32_t lab = __ldg(labels + g0 + i);
        const bool ignored = kOpts && lab == opts.ignore_index;
        bad += (!ignored && (lab < 0 || (int64_t)lab >= vocab)) ? 1 : 0;
        cnt += ignored ? 0 : 1;
    }
    acc = warp_sum(acc);
    bad = warp_sum_int(bad);
    if (kOpts) cnt = warp_sum_int(cnt);
    const int64_t ngroups = ce_groups(rows);
    unsigned t2 = 0;
    if (lane == 0) {
        ws.group_sum[g] = acc;
        ws.group_bad[g] = bad;
        if (kOpts) ws.group_cnt[g] = cnt;
        __threadfence();
        t2 = atomicAdd(ws.global_ticket, 1u);
    }
    t2 = __shfl_sync(0xFFFFFFFFu, t2, 0);
    if (t2 != (unsigned)(ngroups - 1)) return;
    __threadfence();
    float tot = 0.0f;
    int64_t nbad = 0, ncnt = 0;
    for (int64_t i = lane; i < ngroups; i += 32) {
        tot += __ldcg(ws.group_sum + i);
        nbad += __ldcg(ws.group_bad + i);
        if (kOpts) ncnt += __ldcg(ws.group_cnt + i);
    }
    tot = warp_sum(tot);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        nbad += __shfl_xor_sync(0xFFFFFFFFu, nbad, o);
        if (kOpts) ncnt += __shfl_xor_sync(0xFFFFFFFFu, ncnt, o);
    }
    if (lane == 0) {
        if (kOpts) {
            // mean over the rows that count; no counted row gives 0 / 0 = NaN, as the definition does
            if (mean_loss != nullptr) *mean_loss = tot / (float)ncnt;
            if (opts.counted_rows != nullptr) *opts.counted_rows = (int32_t)ncnt;
            // reduction "sum": the same fixed-order total before the division (ignored rows added 0)
            if (opts.sum_loss != nullptr) *opts.sum_loss = tot;
        } else if (mean_loss != nullptr) *mean_loss = tot / (float)rows;
        if (bad_label_count != nullptr)
            *bad_label_count = (int32_t)(nbad > 0x7FFFFFFF ? 0x7FFFFFFF : nbad);
    }
}

// Merge the per-thread (M, S) pairs and finish the row; then the mean, without anybody waiting:
// only warp 0 stays. Its lane 0 takes a ticket of the row's group (kGroupRows consecutive rows);
// the warp that draws a group's last ticket sums that group's losses in a fixed lane-strided order
// and takes a global ticket; the warp that draws the last global ticket sums the group partials,
// again in a fixed order. Which CTA does the summing varies, the order of the additions does not,
// so the mean is bit-identical run to run. (A whole-CTA wait on a single ticket held every CTA's
// registers for an extra L2 round trip and cost 12 % on the benchmark shape.)
template <typename T, bool kOpts, bool kSmooth>
__device__ __forceinline__ void ce_finish(float M, float S, float Z, const T* zr, const int32_t* labels,
                                          float* loss, float* mean_loss, int32_t* bad_label_count,
                                          CeWorkspace ws, int64_t row, int64_t rows, int64_t vocab,
                                          CeOpts opts)
{
    __shared__ float red_a[32], red_b[32], red_c[32];
    const float Mb = block_max(M, red_a);
    // A thread that saw nothing has M = -inf and S = 0; keep its term at 0 rather than 0 * 2^nan. A thread that
    // saw only NaNs also has M = -inf, but S = NaN: S * 0 keeps that NaN in the row's sum.
    const float Sb = block_sum(M == -INFINITY ? S * 0.0f : S * ex2_approx(M - Mb), red_b);
    float Zb = 0.0f;
    if (kSmooth) Zb = block_sum(Z, red_c);          // sum of the row's logits, for label smoothing
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    const int64_t g = row / kGroupRows;
    unsigned t = 0;
    if (lane == 0) {
        const float lse = (Mb + log2f(Sb)) * kLn2;
        const int32_t lab = labels[row];
        float l;
        if (kOpts && lab == opts.ignore_index) l = 0.0f;
        else if (lab < 0 || (int64_t)lab >= vocab) l = __int_as_float(0x7FC00000);
        else {
            l = lse - Elem<T>::load1(zr + lab);
            if (kSmooth) l = (1.0f - opts.smoothing) * l + opts.smoothing * (lse - Zb / (float)vocab);
        }
        loss[row] = l;
        __threadfence();
        t = atomicAdd(ws.group_ticket + g, 1u);
    }
    t = __shfl_sync(0xFFFFFFFFu, t, 0);
    ce_after_ticket<kOpts>(t, row, lane, labels, loss, mean_loss, bad_label_count, ws, rows, vocab, opts);
}

// Rows of any length and alignment are split (row_split) into head elements, whole 16-byte vectors and tail
// elements; the edge elements are taken one per thread before the vector sweep.
// Edge element i (0 .. head + tail - 1) of a split row enters a thread's still empty (M, S, Z).
template <typename T, bool kSum>
__device__ __forceinline__ void ce_edge(const T* zr, const RowSplit<T>& sp, int i, float& M, float& S, float& Z)
{
    const int j = sp.edge_col(i);
    const float xj = Elem<T>::load1(zr + j);
    if (kSum) Z += xj;
    const float x2 = xj * kLog2e;
    if (x2 == -INFINITY) return;
    if (x2 > M) {
        // + 1 for this element; (x2 - x2) is 0 for a number and NaN for +inf, where the max-shifted
        // definition has exp(inf - inf): the row becomes NaN as in the vector sweep
        S = S * ex2_approx(M - x2) + (1.0f + (x2 - x2));
        M = x2;
    } else {
        S += ex2_approx(x2 - M);                             // a NaN element: S becomes NaN, M stays
    }
}

// One batch of VPT vectors per thread: loads first (all in flight), then the batch maximum on the
// packed values, then one ex2 per element against the updated running offset.
template <typename T, int VPT, bool kTail, bool kSum>
__device__ __forceinline__ void ce_batch(const T* zr, int base, int nvec, float& M, float& S, float& Z)
{
    constexpr int E = Elem<T>::kPerVec;
    Vec16 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int v = base + k * blockDim.x + threadIdx.x;
        if (kTail) {
            raw[k] = Elem<T>::fill_neg_inf();
            if (v < nvec) raw[k] = ld_stream(zr + (int64_t)v * E);
        } else {
            raw[k] = ld_stream(zr + (int64_t)v * E);
        }
    }
    float cm = vec_max<T>(raw[0]);
#pragma unroll
    for (int k = 1; k < VPT; ++k) cm = fmaxf(cm, vec_max<T>(raw[k]));
    const float cm2 = cm * kLog2e;
    // != rather than >: a batch of nothing but NaNs has a NaN maximum (the packed max drops a NaN only against a
    // number) and must enter, so that its ex2(NaN) terms reach S.
    if (cm2 != -INFINITY) {
        const float newM = fmaxf(M, cm2);
        float s = S * ex2_approx(M - newM);          // M = -inf on the first batch: S * 0
        const float neg = -newM;
#if KOP_CE_PACKED
        float2 s2 = make_float2(s, 0.0f), z2 = make_float2(Z, 0.0f);
        const float2 l2 = make_float2(kLog2e, kLog2e), n2 = make_float2(neg, neg);
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            float2 f[E / 2];
            Elem<T>::unpack2(raw[k], f);
#pragma unroll
            for (int e = 0; e < E / 2; ++e) {
                const float2 t = __ffma2_rn(f[e], l2, n2);
                s2 = __fadd2_rn(s2, make_float2(ex2_approx(t.x), ex2_approx(t.y)));
            }
            if (kSum && (!kTail || base + k * (int)blockDim.x + (int)threadIdx.x < nvec)) {
#pragma unroll
                for (int e = 0; e < E / 2; ++e) z2 = __fadd2_rn(z2, f[e]);
            }
        }
        s = s2.x + s2.y;
        if (kSum) Z = z2.x + z2.y;
#else
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            float f[E];
            Elem<T>::unpack(raw[k], f);
#pragma unroll
            for (int e = 0; e < E; ++e) s += ex2_approx(fmaf(f[e], kLog2e, neg));
            if (kSum && (!kTail || base + k * (int)blockDim.x + (int)threadIdx.x < nvec)) {
                // pairwise first: half the dependent adds on the running sum
#pragma unroll
                for (int e = 0; e < E; e += 2) Z += f[e] + f[e + 1];
            }
        }
#endif
        S = s;
        M = newM;
    }
}

// 256 threads, capped at 32 registers: eight CTAs (2048 threads) per SM. Occupancy is what hides the
// load latency here; a build that drifted to 40 registers (six CTAs) was 6 % slower.
// kOpts: ignore_index handling; kSmooth: additionally the row sum of the logits for label smoothing (one more
// add per element). That variant spills 36 bytes under the same cap and is still 2 - 4 % faster with eight CTAs
// and the spills than with 40 registers and six CTAs.
template <typename T, int VPT, bool kOpts, bool kSmooth>
__global__ void __launch_bounds__(256, 8)
ce_row_kernel(const T* __restrict__ z, const int32_t* __restrict__ labels, float* __restrict__ loss,
              float* __restrict__ mean_loss, int32_t* __restrict__ bad_label_count,
              CeWorkspace ws, int64_t rows, int64_t row_stride, int64_t vocab, CeOpts opts)
{
    const int64_t row = blockIdx.x;
    const T* zr = z + row * row_stride;
    float M = -INFINITY, S = 0.0f, Z = 0.0f;
    RowSplit<T> sp = row_split<T>(zr, vocab);
    // An ignored row is not read at all: it only takes its tickets.
    if (kOpts && __ldg(labels + row) == opts.ignore_index) sp.head = sp.nvec = sp.tail = 0;
    if ((int)threadIdx.x < sp.head + sp.tail) ce_edge<T, kSmooth>(zr, sp, threadIdx.x, M, S, Z);
    // One loop body with bounds predicates on every batch (out-of-range vectors read as -inf). A
    // predicate-free main loop plus a separate tail batch doubled the inlined body, pushed the kernel
    // from 32 to 40 registers (six CTAs per SM instead of eight) and measured 3-6 % slower.
    const int step = VPT * blockDim.x;
    const int nvec = sp.nvec;
    const T* zm = zr + sp.head;
    for (int base = 0; base < nvec; base += step) ce_batch<T, VPT, true, kSmooth>(zm, base, nvec, M, S, Z);
    ce_finish<T, kOpts, kSmooth>(M, S, Z, zr, labels, loss, mean_loss, bad_label_count, ws, row, rows, vocab, opts);
}

// Rows of at most 16 KB (classification heads, small vocabularies): L lanes of a warp per row (L = 4 .. 32),
// 32 / L rows per warp, eight warps per CTA. Each lane sweeps its share in batches of four vectors with the
// same recurrence as above; the row's (maximum, sum) pair is a butterfly over its lanes; the row's first lane
// writes the loss, and the warp draws one ticket for all of its rows (an atomic per row was the cost of rows
// this short), so that whichever warp draws a group's last ticket has all 32 lanes for the group sum, exactly
// as in the CTA-per-row kernel.
template <typename T, int L, bool kOpts, bool kSmooth>
__global__ void __launch_bounds__(256)
ce_group_kernel(const T* __restrict__ z, const int32_t* __restrict__ labels, float* __restrict__ loss,
                float* __restrict__ mean_loss, int32_t* __restrict__ bad_label_count, CeWorkspace ws,
                int64_t rows, int64_t row_stride, int64_t vocab, CeOpts opts)
{
    constexpr int E = Elem<T>::kPerVec, U = 4;
    constexpr int kRowsPerWarp = 32 / L;
    const int lane = threadIdx.x & 31, sub = lane & (L - 1);
    const int64_t warp_row0 = ((int64_t)blockIdx.x * 8 + (threadIdx.x >> 5)) * kRowsPerWarp;
    const int64_t row = warp_row0 + lane / L;
    const bool live = row < rows;
    const T* zr = z + (live ? row : 0) * row_stride;
    RowSplit<T> sp = row_split<T>(zr, vocab);
    // a row past the end and an ignored row are not read
    if (!live || (kOpts && __ldg(labels + row) == opts.ignore_index)) sp.head = sp.nvec = sp.tail = 0;
    const int n = sp.nvec;
    const T* zm = zr + sp.head;
    float M = -INFINITY, S = 0.0f, Z = 0.0f;
    for (int i = sub; i < sp.head + sp.tail; i += L) ce_edge<T, kSmooth>(zr, sp, i, M, S, Z);
    for (int base = 0; base < n; base += U * L) {
        Vec16 raw[U];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int v = base + k * L + sub;
            raw[k] = Elem<T>::fill_neg_inf();
            if (v < n) raw[k] = ld_stream(zm + (int64_t)v * E);
        }
        float cm = vec_max<T>(raw[0]);
#pragma unroll
        for (int k = 1; k < U; ++k) cm = fmaxf(cm, vec_max<T>(raw[k]));
        const float cm2 = cm * kLog2e;
        if (cm2 != -INFINITY) {                              // a NaN maximum enters (see ce_batch)
            const float newM = fmaxf(M, cm2);
            float s = S * ex2_approx(M - newM);
            const float neg = -newM;
#pragma unroll
            for (int k = 0; k < U; ++k) {
                float f[E];
                Elem<T>::unpack(raw[k], f);
#pragma unroll
                for (int e = 0; e < E; ++e) s += ex2_approx(fmaf(f[e], kLog2e, neg));
                if (kSmooth && base + k * L + sub < n) {
#pragma unroll
                    for (int e = 0; e < E; e += 2) Z += f[e] + f[e + 1];
                }
            }
            S = s;
            M = newM;
        }
    }
    // the row's lanes: butterfly merge of (M, S) and of Z
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) {
        const float Mo = __shfl_xor_sync(0xFFFFFFFFu, M, o), So = __shfl_xor_sync(0xFFFFFFFFu, S, o);
        const float M2 = fmaxf(M, Mo);
        const float a = M == -INFINITY ? S * 0.0f : S * ex2_approx(M - M2);       // S * 0 keeps a NaN sum
        const float b = Mo == -INFINITY ? So * 0.0f : So * ex2_approx(Mo - M2);
        // the lower lane's term first on both sides, so that the two lanes agree bit for bit
        S = (lane & o) ? b + a : a + b;
        M = M2;
        if (kSmooth) Z += __shfl_xor_sync(0xFFFFFFFFu, Z, o);
    }
    if (live && sub == 0) {
        const float lse = (M + log2f(S)) * kLn2;
        const int32_t lab = labels[row];
        float l;
        if (kOpts && lab == opts.ignore_index) l = 0.0f;
        else if (lab < 0 || (int64_t)lab >= vocab) l = __int_as_float(0x7FC00000);
        else {
            l = lse - Elem<T>::load1(zr + lab);
            if (kSmooth) l = (1.0f - opts.smoothing) * l + opts.smoothing * (lse - Z / (float)vocab);
        }
        loss[row] = l;
    }
    // One ticket draw per warp, worth all of its rows: a warp's rows are consecutive and kGroupRows is a multiple
    // of every rows-per-warp count, so they share a group. The losses were written by other lanes: the warp
    // barrier orders them before lane 0's fence, which orders them before its ticket.
    if (warp_row0 >= rows) return;                           // the whole warp is past the end
    __syncwarp();
    const int64_t left = rows - warp_row0;
    const unsigned mine = (unsigned)(left < kRowsPerWarp ? left : kRowsPerWarp);
    unsigned t = 0;
    if (lane == 0) {
        __threadfence();
        t = atomicAdd(ws.group_ticket + warp_row0 / kGroupRows, mine) + mine - 1u;
    }
    t = __shfl_sync(0xFFFFFFFFu, t, 0);
    ce_after_ticket<kOpts>(t, warp_row0, lane, labels, loss, mean_loss, bad_label_count, ws, rows, vocab, opts);
}

template <typename T, bool kOpts>
kop_status_t launch_ce(const void* zv, const int32_t* labels, float* loss, float* mean_loss,
                       int32_t* bad, int64_t rows, int64_t vocab, int64_t stride, void* workspace,
                       cudaStream_t stream, CeOpts opts)
{
    const T* z = static_cast<const T*>(zv);
    constexpr int E = Elem<T>::kPerVec;
    const CeWorkspace ws = ce_workspace(workspace, rows);
    if (cudaMemsetAsync(workspace, 0, ce_workspace_clear_bytes(rows), stream) != cudaSuccess) return KOP_ERR_CUDA;
    // every row is split in the kernel into head elements, whole 16-byte vectors and tail elements, so any vocabulary
    // size, row stride and base alignment takes the vector kernels
    const int64_t nvec64 = vocab / E;
    if (vocab * (int64_t)sizeof(T) <= 16384) {
        const int nvec = (int)nvec64;
        // up to 32 vectors a lane (eight batches): bf16 rows of 4096 classes 4.7 TB/s with 16 a lane, 5.8 with 32 (5.7 with
        // 64, 4.9 with 128); fp32 rows of 2048 classes 4.5 / 5.8 / 5.9 / 5.2
        int lanes = 4;
        while (lanes < 32 && lanes * 32 < nvec) lanes *= 2;
        const int64_t rows_per_cta = 8 * (32 / lanes);
        const unsigned grid = (unsigned)((rows + rows_per_cta - 1) / rows_per_cta);
#define KOP_CE_G(L, SM) ce_group_kernel<T, L, kOpts, SM><<<grid, 256, 0, stream>>>(z, labels, loss, mean_loss, bad, ws, rows, stride, vocab, opts)
#define KOP_CE_GROUP(L)                                            \
    do {                                                           \
        if (kOpts && opts.smoothing > 0.0f) KOP_CE_G(L, true);     \
        else KOP_CE_G(L, false);                                   \
    } while (0)
        switch (lanes) {
        case 32: KOP_CE_GROUP(32); break;
        case 16: KOP_CE_GROUP(16); break;
        case 8: KOP_CE_GROUP(8); break;
        default: KOP_CE_GROUP(4); break;
        }
#undef KOP_CE_G
#undef KOP_CE_GROUP
        return launch_status();
    }
    const int threads = 256;
    const int64_t per = (nvec64 + threads - 1) / threads;
    // Batches of at most four vectors per thread: ~50 registers, so five 256-thread CTAs stay
    // resident per SM and their load and exp phases interleave. Larger batches (more bytes in
    // flight per thread, fewer resident warps) measured 5-30 % slower on a 32000-wide bf16 row.
#define KOP_CE_L(V, SM) ce_row_kernel<T, V, kOpts, SM><<<(unsigned)rows, threads, 0, stream>>>(z, labels, loss, mean_loss, bad, ws, rows, stride, vocab, opts)
#define KOP_CE(V)                                                  \
    do {                                                           \
        if (kOpts && opts.smoothing > 0.0f) KOP_CE_L(V, true);     \
        else KOP_CE_L(V, false);                                   \
    } while (0)
    if (per <= 1) KOP_CE(1);
    else if (per <= 2) KOP_CE(2);
    else KOP_CE(4);
#undef KOP_CE
#undef KOP_CE_L
    return launch_status();
}

}  // namespace
}  // namespace kop

extern "C" size_t kop_ce_loss_rowwise_workspace_bytes(int64_t rows, int64_t vocab, kop_dtype_t dtype)
{
    if (rows < 0 || vocab <= 0 || !kop::dtype_ok(dtype)) return 0;
    return kop::ce_workspace_bytes(rows);
}

namespace kop {
namespace {

// Static validation shared by the three cross-entropy entry points (no CUDA call). `done` is set when the call
// has nothing to do (rows == 0). kOwnScratch: the scratch is the library's built-in array, so there is no
// caller workspace to check, but the problem must fit the array.
struct CeArgs {
    const void* logits;
    const int32_t* labels;
    float* loss;
    float* mean_loss;
    int32_t* bad_label_count;
    int32_t* counted_rows;
    float* sum_loss;
    int64_t rows, vocab, row_stride;
    kop_dtype_t dtype;
};
kop_status_t ce_validate(const CeArgs& a, bool own_scratch, int64_t own_scratch_max_rows, const void* workspace,
                         size_t workspace_bytes, bool* done)
{
    *done = false;
    if (!dtype_ok(a.dtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    kop_status_t st = check_rows_cols(a.rows, a.vocab);
    if (st != KOP_OK) return st;
    if (a.rows == 0) {
        *done = true;
        return KOP_OK;
    }
    if (own_scratch && a.rows > own_scratch_max_rows) return KOP_ERR_WORKSPACE_TOO_SMALL;
    if (!a.logits || !a.labels || !a.loss || (!own_scratch && !workspace)) return KOP_ERR_NULL_POINTER;
    if (a.vocab > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;            // labels are int32
    if (a.rows > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;             // one CTA per row
    if ((st = check_row_stride(a.row_stride, a.vocab, a.rows)) != KOP_OK) return st;
    const int esz = elem_size(a.dtype);
    if (!aligned_to(a.logits, esz) || !aligned_to(a.labels, 4) || !aligned_to(a.loss, 4) ||
        (a.mean_loss && !aligned_to(a.mean_loss, 4)) || (a.bad_label_count && !aligned_to(a.bad_label_count, 4)) ||
        (a.counted_rows && !aligned_to(a.counted_rows, 4)) || (a.sum_loss && !aligned_to(a.sum_loss, 4)) ||
        (!own_scratch && !aligned_to(workspace, 16)))
        return KOP_ERR_MISALIGNED;
    if (!own_scratch && workspace_bytes < ce_workspace_bytes(a.rows)) return KOP_ERR_WORKSPACE_TOO_SMALL;
    return KOP_OK;
}

template <bool kOpts>
kop_status_t ce_dispatch(const CeArgs& a, void* workspace, cudaStream_t s, CeOpts opts)
{
    return a.dtype == KOP_F32
               ? launch_ce<float, kOpts>(a.logits, a.labels, a.loss, a.mean_loss, a.bad_label_count, a.rows, a.vocab, a.row_stride, workspace, s, opts)
               : a.dtype == KOP_BF16 ? launch_ce<__nv_bfloat16, kOpts>(a.logits, a.labels, a.loss, a.mean_loss, a.bad_label_count, a.rows, a.vocab, a.row_stride, workspace, s, opts)
               : launch_ce<__half, kOpts>(a.logits, a.labels, a.loss, a.mean_loss, a.bad_label_count, a.rows, a.vocab, a.row_stride, workspace, s, opts);
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_ce_loss_rowwise(const void* logits, const int32_t* labels, float* loss,
                                            float* mean_loss, int32_t* bad_label_count, int64_t rows,
                                            int64_t vocab, int64_t row_stride, void* workspace,
                                            size_t workspace_bytes, kop_dtype_t dtype,
                                            kop_stream_t stream)
{
    using namespace kop;
    const CeArgs a{logits, labels, loss, mean_loss, bad_label_count, nullptr, nullptr, rows, vocab, row_stride, dtype};
    bool done = false;
    kop_status_t st = ce_validate(a, false, 0, workspace, workspace_bytes, &done);
    if (st != KOP_OK || done) return st;
    if ((st = check_device()) != KOP_OK) return st;
    return ce_dispatch<false>(a, workspace, as_stream(stream), CeOpts{0, 0.0f, nullptr, nullptr});
}

extern "C" kop_status_t kop_ce_loss_rowwise_opts(const void* logits, const int32_t* labels, float* loss,
                                                 float* mean_loss, float* sum_loss, int32_t* bad_label_count,
                                                 int32_t* counted_rows, int64_t rows, int64_t vocab,
                                                 int64_t row_stride, int32_t ignore_index,
                                                 float label_smoothing, void* workspace,
                                                 size_t workspace_bytes, kop_dtype_t dtype,
                                                 kop_stream_t stream)
{
    using namespace kop;
    const CeArgs a{logits, labels, loss, mean_loss, bad_label_count, counted_rows, sum_loss, rows, vocab, row_stride, dtype};
    if (dtype_ok(dtype) && check_rows_cols(rows, vocab) == KOP_OK &&
        !(label_smoothing >= 0.0f && label_smoothing < 1.0f))
        return KOP_ERR_BAD_SHAPE;
    bool done = false;
    kop_status_t st = ce_validate(a, false, 0, workspace, workspace_bytes, &done);
    if (st != KOP_OK || done) return st;
    if ((st = check_device()) != KOP_OK) return st;
    return ce_dispatch<true>(a, workspace, as_stream(stream), CeOpts{ignore_index, label_smoothing, counted_rows, sum_loss});
}

// ------------------------------------------------------------------------------------------------
// kop_ce_loss_rowwise_static: the same cross-entropy, for callers that cannot allocate.
//
// Some callers have no way to get scratch memory at the point of the call: a plug-in running inside
// another runtime's operator has no handle on that runtime's memory pool, and a raw cudaMalloc there
// would synchronise the whole device and grow memory behind the pool's back; a serving process that
// fixed its memory plan at start-up may forbid driver allocations afterwards; C callers on a
// latency-critical path cannot afford an allocator round trip per call. For them the ticket / partial
// scratch of the mean reduction lives in a file-scope device array that every GPU loading this
// library holds until the process exits. Its size fixes the largest problem this entry point takes.
namespace kop {
namespace {

constexpr int64_t kStaticMaxRows = (int64_t)1 << 20;                       // 1,048,576 rows
constexpr int64_t kStaticScratchWords = 4 + 4 * (kStaticMaxRows / kGroupRows);   // 16,388 words = 65,552 B
static __device__ __align__(256) unsigned int g_ce_static_scratch[kStaticScratchWords];

// In host code the array's name is only a stand-in for the symbol, not a device address: the address
// the kernel needs comes from cudaGetSymbolAddress, asked once per device with that device current.
constexpr int kStaticMaxDevices = 64;
// Several host threads may make a device's first call together: each looks the address up and stores the same
// value, so relaxed atomics are all the ordering this needs.
std::atomic<void*> g_ce_static_ptr[kStaticMaxDevices];

kop_status_t ce_static_scratch(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return KOP_ERR_CUDA;
    }
    if (dev < 0 || dev >= kStaticMaxDevices) return KOP_ERR_UNSUPPORTED_DEVICE;
    void* p = g_ce_static_ptr[dev].load(std::memory_order_relaxed);
    if (p == nullptr) {
        if (cudaGetSymbolAddress(&p, g_ce_static_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return KOP_ERR_CUDA;
        }
        g_ce_static_ptr[dev].store(p, std::memory_order_relaxed);
    }
    *out = p;
    return KOP_OK;
}

}  // namespace
}  // namespace kop

extern "C" int64_t kop_ce_loss_rowwise_static_max_rows(void) { return kop::kStaticMaxRows; }

extern "C" kop_status_t kop_ce_loss_rowwise_static(const void* logits, const int32_t* labels,
                                                   float* loss, float* mean_loss,
                                                   int32_t* bad_label_count, int64_t rows, int64_t vocab,
                                                   int64_t row_stride, kop_dtype_t dtype,
                                                   kop_stream_t stream)
{
    using namespace kop;
    // All argument checks first, without touching the device: more rows than the built-in scratch holds, NULL or
    // misaligned pointers and bad strides are refused before any CUDA call, as for every other entry point.
    const CeArgs a{logits, labels, loss, mean_loss, bad_label_count, nullptr, nullptr, rows, vocab, row_stride, dtype};
    bool done = false;
    kop_status_t st = ce_validate(a, true, kStaticMaxRows, nullptr, 0, &done);
    if (st != KOP_OK || done) return st;
    if ((st = check_device()) != KOP_OK) return st;
    void* scratch = nullptr;
    if ((st = ce_static_scratch(&scratch)) != KOP_OK) return st;
    // Same clearing of the tickets on `stream`, same kernels as the caller-workspace entry point; only the
    // scratch pointer differs.
    return ce_dispatch<false>(a, scratch, as_stream(stream), CeOpts{0, 0.0f, nullptr, nullptr});
}
