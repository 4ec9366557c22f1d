// kop_groupnorm_act: GroupNorm (InstanceNorm when groups == C) with optional per-channel affine and an
// activation, NCHW, in one HBM pass.
//
// One (image, group) chunk is (C / groups) * H * W contiguous elements. Chunks up to 40 KB stay in the
// registers of a team of threads (8 lanes to 10 warps), whatever the plane size. A longer chunk (100 KB
// for 8 channels of 56x56 fp32) gets a CTA and fits the 227 KB of shared memory a Blackwell CTA can
// have: it is fetched into shared memory once (bulk asynchronous copies requested up front), the
// statistics are accumulated as the parts land, and the normalising sweep re-reads the chunk from
// shared memory instead of HBM.
// With the chunk on chip the statistics are the exact two-pass ones (mean, then squared deviations from
// it). Chunks beyond the shared-memory budget take two sweeps over global memory (the second mostly from
// L2); there, and in the scalar kernel, mean and variance come from one sweep without the
// E[x^2] - mean^2 cancellation: every thread keeps a (count, mean, M2) triple, updated per batch with an
// exact two-sweep computation in registers and merged with the pairwise (Chan) formula.
#include "kop_common.cuh"

#include <algorithm>
#include <atomic>

namespace kop {
namespace {

struct Moments {
    float n, mean, m2;
};

// Pairwise merge: delta = mean_b - mean_a; mean = mean_a + delta n_b / n; M2 = M2_a + M2_b + delta^2 n_a n_b / n.
__device__ __forceinline__ Moments merge(Moments a, Moments b)
{
    const float n = a.n + b.n;
    if (n == 0.0f) return Moments{0.0f, 0.0f, 0.0f};
    const float f = b.n / n;
    const float d = b.mean - a.mean;
    return Moments{n, fmaf(d, f, a.mean), a.m2 + b.m2 + d * d * a.n * f};
}

__device__ __forceinline__ Moments warp_merge(Moments m)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Moments other;
        other.n = __shfl_xor_sync(0xFFFFFFFFu, m.n, o);
        other.mean = __shfl_xor_sync(0xFFFFFFFFu, m.mean, o);
        other.m2 = __shfl_xor_sync(0xFFFFFFFFu, m.m2, o);
        // both lanes of a pair must combine in the same order to agree bit for bit
        const bool low = (threadIdx.x & o) == 0;
        m = low ? merge(m, other) : merge(other, m);
    }
    return m;
}

enum { kActNone = 0, kActRelu = 1, kActSilu = 2 };

// SiLU through ex2.approx and rcp.approx: about 3e-7 relative error, far inside the fp32 gate of 1e-5,
// and a third of the instructions of an IEEE division (this kernel is close to issue-bound on fp32 data).
template <int ACT>
__device__ __forceinline__ float activate(float v)
{
    if (ACT == kActRelu) return v > 0.0f ? v : (v <= 0.0f ? 0.0f : v);       // NaN passes through
    if (ACT == kActSilu) return v * rcp_approx(1.0f + ex2_approx(-v * kLog2e));
    return v;
}

// v / d for 0 <= v < 2^22 without the 20-instruction integer division: float estimate, one-step fix-up.
__device__ __forceinline__ int div_small(int v, int d, float inv_d)
{
    int q = (int)((float)v * inv_d);
    const int r = v - q * d;
    q += (r >= d) ? 1 : 0;
    q -= (r < 0) ? 1 : 0;
    return q;
}

constexpr int kGnThreads = 512;
constexpr int kGnUnroll = 4;
constexpr int kGnCopyVecs = 2048;                        // 32 KB: one bulk copy, one barrier
constexpr int kGnMaxParts = 7;                           // covers the 200 KB staging budget

// y = act((x - mu) * rstd * gamma[c] + beta[c]) for one vector; a vector never straddles two channels.
// (x - mu) first: folding mu into a shift would cost |mu| * rstd ulps when the spread is small.
template <typename T, int ACT, typename PT>
__device__ __forceinline__ void normalize_store(const Vec16& raw, T* dst, int c, const PT* gamma,
                                                const PT* beta, float mu, float rs)
{
    constexpr int P = Elem<T>::kPerVec / 2;
    const float sc = rs * (gamma != nullptr ? param1(gamma, c) : 1.0f);
    const float be = beta != nullptr ? param1(beta, c) : 0.0f;
    const float2 nmu = make_float2(-mu, -mu), sc2 = make_float2(sc, sc), be2 = make_float2(be, be);
    float2 f[P];
    Elem<T>::unpack2(raw, f);
#pragma unroll
    for (int e = 0; e < P; ++e) {
        float2 u = __ffma2_rn(__fadd2_rn(f[e], nmu), sc2, be2);
        if (ACT == kActSilu && sizeof(T) == 2) {
            // 16-bit data: x sigmoid(x) = h + h tanh(h), h = x / 2, one special-function operation an element instead
            // of two (the hardware tanh's 2^-11 relative error is a quarter of a bf16 step, a tenth of the fp16 gate)
            const float2 h = __fmul2_rn(u, make_float2(0.5f, 0.5f));
            u = __ffma2_rn(h, make_float2(tanh_approx(h.x), tanh_approx(h.y)), h);
        } else if (ACT == kActSilu) {
            const float2 a = __fmul2_rn(u, make_float2(-kLog2e, -kLog2e));
            const float2 d = __fadd2_rn(make_float2(ex2_approx(a.x), ex2_approx(a.y)), make_float2(1.0f, 1.0f));
            u = __fmul2_rn(u, make_float2(rcp_approx(d.x), rcp_approx(d.y)));
        } else {
            u = make_float2(activate<ACT>(u.x), activate<ACT>(u.y));
        }
        f[e] = u;
    }
    st_stream(dst, Elem<T>::pack2(f));
}

// Chunks beyond the staging budget: two sweeps over global memory (the second mostly served by L2).
// Self-contained on purpose (it shares only merge / warp_merge / activate with the staged kernel).
template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(kGnThreads)
groupnorm_twosweep_kernel(const T* __restrict__ x, const PT* __restrict__ gamma, const PT* __restrict__ beta,
                          T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd, int nvec,
                          int vec_per_plane, int cpg, int groups, float eps)
{
    constexpr int E = Elem<T>::kPerVec;
    __shared__ float red_n[32], red_mean[32], red_m2[32];
    __shared__ float bc_mean, bc_rstd;

    const int64_t chunk = blockIdx.x;                       // image * groups + group
    const int g = (int)(chunk % groups);
    const T* xc = x + chunk * (int64_t)nvec * E;
    T* yc = y + chunk * (int64_t)nvec * E;

    Moments acc{0.0f, 0.0f, 0.0f};
    for (int base = 0; base < nvec; base += kGnUnroll * kGnThreads) {
        Vec16 raw[kGnUnroll];
        int cnt = 0;
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < nvec) {
                raw[k] = ld_stream(xc + (int64_t)v * E);
                ++cnt;
            } else {
                raw[k] = Vec16{{0u, 0u, 0u, 0u}};
            }
        }
        if (cnt > 0) {
            // exact two-sweep moments of this batch (zero padding adds 0 to the sum and is masked below)
            float f[kGnUnroll][E];
            float s = 0.0f;
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                Elem<T>::unpack(raw[k], f[k]);
#pragma unroll
                for (int e = 0; e < E; ++e) s += f[k][e];
            }
            const float bn = (float)(cnt * E);
            const float bmean = s / bn;
            float m2 = 0.0f;
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                if (k < cnt) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const float d = f[k][e] - bmean;
                        m2 = fmaf(d, d, m2);
                    }
                }
            }
            acc = merge(acc, Moments{bn, bmean, m2});
        }
    }
    // CTA-wide merge in a fixed order: lanes by butterfly, warps by index
    acc = warp_merge(acc);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        red_n[warp] = acc.n;
        red_mean[warp] = acc.mean;
        red_m2[warp] = acc.m2;
    }
    __syncthreads();
    if (warp == 0) {
        constexpr int NW = kGnThreads / 32;
        Moments t = lane < NW ? Moments{red_n[lane], red_mean[lane], red_m2[lane]} : Moments{0.0f, 0.0f, 0.0f};
        t = warp_merge(t);
        if (lane == 0) {
            const float rs = rsqrtf(t.m2 / t.n + eps);
            bc_mean = t.mean;
            bc_rstd = rs;
            if (mean != nullptr) mean[chunk] = t.mean;
            if (rstd != nullptr) rstd[chunk] = rs;
        }
    }
    __syncthreads();
    const float mu = bc_mean, rs = bc_rstd;

    for (int base = 0; base < nvec; base += kGnUnroll * kGnThreads) {
        Vec16 raw[kGnUnroll];
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < nvec) raw[k] = ld_stream(xc + (int64_t)v * E);
        }
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < nvec) {
                const int c = g * cpg + v / vec_per_plane;           // a vector never straddles two channels
                const float ga = gamma != nullptr ? param1(gamma, c) : 1.0f;
                const float be = beta != nullptr ? param1(beta, c) : 0.0f;
                const float sc = rs * ga;
                float f[E];
                Elem<T>::unpack(raw[k], f);
                // (x - mu) first: folding mu into a shift would cost |mu| * rstd ulps when the spread is small
#pragma unroll
                for (int e = 0; e < E; ++e) f[e] = activate<ACT>(fmaf(f[e] - mu, sc, be));
                st_stream(yc + (int64_t)v * E, Elem<T>::pack(f));
            }
        }
    }
}

// ---- staged kernel: the chunk is fetched into shared memory by bulk asynchronous copies --------------
// One thread requests the whole chunk up front as 32 KB copies (cp.async.bulk, global -> shared), each
// completing on its own mbarrier, so the CTA has its entire input in flight from its first cycles and
// the memory system, not the loop structure, sets the pace. All threads then consume the parts in
// order (moments from shared memory as each part lands), merge, and normalise out of shared memory.
__device__ unsigned int g_gn_wait_timeouts;              // CTAs that gave up waiting for a copy

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

// One poll: the thread is suspended until the phase completes or about `hint_ns` nanoseconds pass, so a
// waiting warp costs the SM's schedulers next to nothing.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t done;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return done != 0;
}

// Bounded wait (at most about two seconds): a copy that never lands (it cannot, short of a hardware
// fault) must not hang the GPU.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity)
{
    for (int spin = 0; spin < (1 << 18); ++spin)
        if (mbar_try_wait(bar, parity, 8000u)) return true;
    return false;
}

__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// NT threads per CTA (128, 256 or 512, chosen from the chunk length so short chunks do not pay for idle
// warps). With the chunk in shared memory the statistics are the textbook two-pass ones: the sum is
// accumulated part by part as the copies land, the squared deviations from the exact mean in a second
// sweep over shared memory; both CTA reductions are plain sums (one barrier each, fixed order).
template <typename T, typename PT, int ACT, int NT>
__global__ void __launch_bounds__(NT)
groupnorm_staged_kernel(const T* __restrict__ x, const PT* __restrict__ gamma, const PT* __restrict__ beta,
                        T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd, int nvec,
                        int vec_per_plane, int cpg, int groups, float eps, float inv_count)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;
    constexpr int kPartVecs = kGnUnroll * NT;
    extern __shared__ __align__(128) unsigned char gn_smem[];
    Vec16* stage = reinterpret_cast<Vec16*>(gn_smem);
    __shared__ float slots_a[32], slots_b[32];
    __shared__ __align__(8) uint64_t bars[kGnMaxParts];

    const int64_t chunk = blockIdx.x;                       // image * groups + group
    const int g = (int)(chunk % groups);
    const T* xc = x + chunk * (int64_t)nvec * E;
    T* yc = y + chunk * (int64_t)nvec * E;
    // copies of kGnCopyVecs vectors, one barrier each; kGnMaxParts of them cover the staging budget
    const int nparts = (nvec + kGnCopyVecs - 1) / kGnCopyVecs;

    if (threadIdx.x == 0) {
        for (int p = 0; p < nparts; ++p) mbar_init(bars + p, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int p = 0; p < nparts; ++p) {
            const int v0 = p * kGnCopyVecs;
            const uint32_t bytes = (uint32_t)min(kGnCopyVecs, nvec - v0) * 16u;
            mbar_expect_tx(bars + p, bytes);
            bulk_load(stage + v0, xc + (int64_t)v0 * E, bytes, bars + p);
        }
    }
    __syncthreads();                                        // barriers initialised before anyone polls them

    float2 s2 = make_float2(0.0f, 0.0f);
    for (int p = 0; p < nparts; ++p) {
        // One thread polls the copy's barrier; the rest sleep in the CTA barrier instead of burning the
        // issue slots that co-resident CTAs need for their arithmetic. The vote makes a timeout uniform.
        bool landed = true;
        if (threadIdx.x == 0) landed = mbar_wait_bounded(bars + p, 0);
        if (!__syncthreads_and(landed)) {
            // give the copies one more bounded chance to drain before this CTA's shared memory is released
            if (threadIdx.x == 0) {
                for (int q = p; q < nparts; ++q) mbar_wait_bounded(bars + q, 0);
                atomicAdd(&g_gn_wait_timeouts, 1u);
            }
            return;
        }
        const int end = min(nvec, (p + 1) * kGnCopyVecs);
        for (int base = p * kGnCopyVecs; base < end; base += kPartVecs) {
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                const int v = base + k * NT + threadIdx.x;
                if (v < end) {
                    float2 f[P];
                    Elem<T>::unpack2(stage[v], f);
#pragma unroll
                    for (int e = 0; e < P; ++e) s2 = __fadd2_rn(s2, f[e]);
                }
            }
        }
    }
    const float mu = block_sum(s2.x + s2.y, slots_a) * inv_count;
    const float2 nmu = make_float2(-mu, -mu);
    float2 q2 = make_float2(0.0f, 0.0f);
    for (int base = 0; base < nvec; base += kPartVecs) {
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * NT + threadIdx.x;
            if (v < nvec) {
                float2 f[P];
                Elem<T>::unpack2(stage[v], f);
#pragma unroll
                for (int e = 0; e < P; ++e) {
                    const float2 d = __fadd2_rn(f[e], nmu);
                    q2 = __ffma2_rn(d, d, q2);
                }
            }
        }
    }
    const float rs = rsqrtf(block_sum(q2.x + q2.y, slots_b) * inv_count + eps);
    if (threadIdx.x == 0) {
        if (mean != nullptr) mean[chunk] = mu;
        if (rstd != nullptr) rstd[chunk] = rs;
    }
    const float inv_vpp = 1.0f / (float)vec_per_plane;
    for (int base = 0; base < nvec; base += kPartVecs) {
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * NT + threadIdx.x;
            if (v < nvec)
                normalize_store<T, ACT>(stage[v], yc + (int64_t)v * E, g * cpg + div_small(v, vec_per_plane, inv_vpp),
                                        gamma, beta, mu, rs);
        }
    }
}

// Chunks just beyond one CTA's staging budget (200 KB to 512 KB: GroupNorm on 128 x 128 maps): a thread-block cluster
// of up to 8 CTAs stages the chunk, a slice each, and the two sums are combined over the cluster through
// distributed shared memory, so the chunk is still read from HBM once. The same structure as the staged kernel;
// every CTA runs every cluster barrier whatever happens to its copies.
constexpr int kGnClusterThreads = 512;

template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(kGnClusterThreads)
groupnorm_cluster_kernel(const T* __restrict__ x, const PT* __restrict__ gamma, const PT* __restrict__ beta,
                         T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd, int nvec,
                         int slice_vecs, int csize, int vec_per_plane, int cpg, int groups, float eps, float inv_count)
{
    constexpr int E = Elem<T>::kPerVec;
    constexpr int P = E / 2;
    constexpr int NT = kGnClusterThreads;
    constexpr int kPartVecs = kGnUnroll * NT;
    extern __shared__ __align__(128) unsigned char gn_smem[];
    Vec16* stage = reinterpret_cast<Vec16*>(gn_smem);
    __shared__ float slots_a[32], slots_b[32];
    __shared__ float from_sum[8], from_sq[8], from_bad[8];
    __shared__ __align__(8) uint64_t bars[kGnMaxParts];

    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // "this CTA has started"; waited for below
    const uint32_t rank = cluster_rank();
    const int64_t chunk = blockIdx.x / (unsigned)csize;      // image * groups + group
    const int g = (int)(chunk % groups);
    const int v_lo = (int)rank * slice_vecs;                 // this CTA's slice of the chunk
    const int n_here = max(0, min(slice_vecs, nvec - v_lo));
    const T* xc = x + (chunk * (int64_t)nvec + v_lo) * E;
    T* yc = y + (chunk * (int64_t)nvec + v_lo) * E;
    const int nparts = (n_here + kGnCopyVecs - 1) / kGnCopyVecs;

    if (threadIdx.x == 0) {
        for (int p = 0; p < nparts; ++p) mbar_init(bars + p, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int p = 0; p < nparts; ++p) {
            const int v0 = p * kGnCopyVecs;
            const uint32_t bytes = (uint32_t)min(kGnCopyVecs, n_here - v0) * 16u;
            mbar_expect_tx(bars + p, bytes);
            bulk_load(stage + v0, xc + (int64_t)v0 * E, bytes, bars + p);
        }
    }
    __syncthreads();

    float2 s2 = make_float2(0.0f, 0.0f);
    bool ok = true;                                          // uniform over the CTA
    for (int p = 0; p < nparts && ok; ++p) {
        bool landed = true;
        if (threadIdx.x == 0) landed = mbar_wait_bounded(bars + p, 0);
        ok = __syncthreads_and(landed);
        if (!ok) {
            // give the copies one more bounded chance to drain; this CTA then contributes nothing and the whole
            // cluster writes nothing (it still takes part in both cluster barriers below)
            if (threadIdx.x == 0) {
                for (int q = p; q < nparts; ++q) mbar_wait_bounded(bars + q, 0);
                atomicAdd(&g_gn_wait_timeouts, 1u);
            }
            break;
        }
        const int end = min(n_here, (p + 1) * kGnCopyVecs);
        for (int base = p * kGnCopyVecs; base < end; base += kPartVecs) {
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                const int v = base + k * NT + threadIdx.x;
                if (v < end) {
                    float2 f[P];
                    Elem<T>::unpack2(stage[v], f);
#pragma unroll
                    for (int e = 0; e < P; ++e) s2 = __fadd2_rn(s2, f[e]);
                }
            }
        }
    }
    const float local_sum = block_sum(ok ? s2.x + s2.y : 0.0f, slots_a);
    // every CTA of the cluster has started (arrival at kernel entry): their shared memory may be written now
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // one exchange for the sum and the failure flag: both slots written, one cluster barrier, folded in rank order
    if (threadIdx.x < (unsigned)csize) {
        store_to_cluster_cta(&from_sum[rank], threadIdx.x, local_sum);
        store_to_cluster_cta(&from_bad[rank], threadIdx.x, ok ? 0.0f : 1.0f);
    }
    cluster_barrier();
    float tot = 0.0f, bad = 0.0f;
    for (int i = 0; i < csize; ++i) {
        tot += from_sum[i];
        bad += from_bad[i];
    }
    const float mu = tot * inv_count;
    const float2 nmu = make_float2(-mu, -mu);
    float2 q2 = make_float2(0.0f, 0.0f);
    if (ok) {
        for (int base = 0; base < n_here; base += kPartVecs) {
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                const int v = base + k * NT + threadIdx.x;
                if (v < n_here) {
                    float2 f[P];
                    Elem<T>::unpack2(stage[v], f);
#pragma unroll
                    for (int e = 0; e < P; ++e) {
                        const float2 d = __fadd2_rn(f[e], nmu);
                        q2 = __ffma2_rn(d, d, q2);
                    }
                }
            }
        }
    }
    const float local_sq = block_sum(q2.x + q2.y, slots_b);
    const float rs = rsqrtf(cluster_sum(local_sq, from_sq, rank, (uint32_t)csize) * inv_count + eps);   // last remote access
    if (bad != 0.0f) return;                                 // some CTA of the cluster lost a copy: nothing is written
    if (threadIdx.x == 0 && rank == 0) {
        if (mean != nullptr) mean[chunk] = mu;
        if (rstd != nullptr) rstd[chunk] = rs;
    }
    const float inv_vpp = 1.0f / (float)vec_per_plane;
    for (int base = 0; base < n_here; base += kPartVecs) {
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * NT + threadIdx.x;
            if (v < n_here)
                normalize_store<T, ACT>(stage[v], yc + (int64_t)v * E,
                                        g * cpg + div_small(v_lo + v, vec_per_plane, inv_vpp), gamma, beta, mu, rs);
        }
    }
}

// Few, very large chunks (a batch of one or two images through an image generator's GroupNorm: 32 to 128 chunks of
// megabytes): one CTA per chunk would leave most SMs idle. A cluster of up to 8 CTAs shares the chunk, a slice
// each, in the two-sweep manner (moments in one sweep, output in a second, mostly from the L2); the slices'
// (count, mean, M2) triples are exchanged through distributed shared memory and merged pairwise in rank order.
template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(kGnThreads)
groupnorm_twosweep_cluster_kernel(const T* __restrict__ x, const PT* __restrict__ gamma,
                                  const PT* __restrict__ beta, T* __restrict__ y, float* __restrict__ mean,
                                  float* __restrict__ rstd, int nvec, int slice_vecs, int csize, int vec_per_plane,
                                  int cpg, int groups, float eps)
{
    constexpr int E = Elem<T>::kPerVec;
    __shared__ float red_n[32], red_mean[32], red_m2[32];
    __shared__ float from_n[8], from_mean[8], from_m2[8];
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // "this CTA has started"; waited for below
    const uint32_t rank = cluster_rank();
    const int64_t chunk = blockIdx.x / (unsigned)csize;
    const int g = (int)(chunk % groups);
    const int v_lo = (int)rank * slice_vecs;
    const int n_here = max(0, min(slice_vecs, nvec - v_lo));
    const T* xc = x + (chunk * (int64_t)nvec + v_lo) * E;
    T* yc = y + (chunk * (int64_t)nvec + v_lo) * E;

    Moments acc{0.0f, 0.0f, 0.0f};
    for (int base = 0; base < n_here; base += kGnUnroll * kGnThreads) {
        Vec16 raw[kGnUnroll];
        int cnt = 0;
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < n_here) {
                raw[k] = ld_stream(xc + (int64_t)v * E);
                ++cnt;
            } else {
                raw[k] = Vec16{{0u, 0u, 0u, 0u}};
            }
        }
        if (cnt > 0) {
            float f[kGnUnroll][E];
            float s = 0.0f;
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                Elem<T>::unpack(raw[k], f[k]);
#pragma unroll
                for (int e = 0; e < E; ++e) s += f[k][e];
            }
            const float bn = (float)(cnt * E);
            const float bmean = s / bn;
            float m2 = 0.0f;
#pragma unroll
            for (int k = 0; k < kGnUnroll; ++k) {
                if (k < cnt) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const float d = f[k][e] - bmean;
                        m2 = fmaf(d, d, m2);
                    }
                }
            }
            acc = merge(acc, Moments{bn, bmean, m2});
        }
    }
    acc = warp_merge(acc);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        red_n[warp] = acc.n;
        red_mean[warp] = acc.mean;
        red_m2[warp] = acc.m2;
    }
    __syncthreads();
    // every warp merges the CTA's warp partials for itself (the same order everywhere, so the same triple)
    constexpr int NW = kGnThreads / 32;
    Moments t = lane < NW ? Moments{red_n[lane], red_mean[lane], red_m2[lane]} : Moments{0.0f, 0.0f, 0.0f};
    t = warp_merge(t);
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");     // every CTA of the cluster has started
    if (threadIdx.x < (unsigned)csize) {
        store_to_cluster_cta(&from_n[rank], threadIdx.x, t.n);
        store_to_cluster_cta(&from_mean[rank], threadIdx.x, t.mean);
        store_to_cluster_cta(&from_m2[rank], threadIdx.x, t.m2);
    }
    cluster_barrier();                                       // the only exchange: last remote access before it
    Moments all{0.0f, 0.0f, 0.0f};
    for (int i = 0; i < csize; ++i) all = merge(all, Moments{from_n[i], from_mean[i], from_m2[i]});
    const float mu = all.mean, rs = rsqrtf(all.m2 / all.n + eps);
    if (threadIdx.x == 0 && rank == 0) {
        if (mean != nullptr) mean[chunk] = mu;
        if (rstd != nullptr) rstd[chunk] = rs;
    }
    for (int base = 0; base < n_here; base += kGnUnroll * kGnThreads) {
        Vec16 raw[kGnUnroll];
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < n_here) raw[k] = ld_stream(xc + (int64_t)v * E);
        }
#pragma unroll
        for (int k = 0; k < kGnUnroll; ++k) {
            const int v = base + k * kGnThreads + threadIdx.x;
            if (v < n_here) {
                const int c = g * cpg + (v_lo + v) / vec_per_plane;
                const float ga = gamma != nullptr ? param1(gamma, c) : 1.0f;
                const float be = beta != nullptr ? param1(beta, c) : 0.0f;
                const float sc = rs * ga;
                float f[E];
                Elem<T>::unpack(raw[k], f);
#pragma unroll
                for (int e = 0; e < E; ++e) f[e] = activate<ACT>(fmaf(f[e] - mu, sc, be));
                st_stream(yc + (int64_t)v * E, Elem<T>::pack(f));
            }
        }
    }
}

// Chunks up to 40 KB held in registers. A team of threads owns a chunk: 8 lanes of a warp for chunks of at most 64
// load units, else one to sixteen warps, every thread holding up to eight units. A unit is the widest access
// (16, 8, 4 bytes or one element) that divides the chunk's bytes and the alignment of both tensors, so a chunk of
// 16 channels of 14 x 14 bf16 values moves in 16-byte accesses although no plane is a whole vector; a unit then
// straddles at most two channels (the dispatcher keeps a unit no longer than a plane) and picks gamma / beta per
// element between the two. Exact two-pass statistics out of the registers; the raw words are kept and widened at
// each use, which for 16-bit data halves the registers that a widened copy would take.
template <int VB>
struct GnUnit {
    uint32_t w[VB >= 4 ? VB / 4 : 1];
};

template <typename T, int VB>
__device__ __forceinline__ GnUnit<VB> gn_load(const T* q)
{
    GnUnit<VB> r;
    if constexpr (VB == 16) {
        const Vec16 t = ld_stream(q);
        r.w[0] = t.w[0], r.w[1] = t.w[1], r.w[2] = t.w[2], r.w[3] = t.w[3];
    } else if constexpr (VB == 8) {
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(q));
        r.w[0] = t.x, r.w[1] = t.y;
    } else if constexpr (VB == 4) {
        r.w[0] = __ldg(reinterpret_cast<const uint32_t*>(q));
    } else {
        r.w[0] = __ldg(reinterpret_cast<const unsigned short*>(q));
    }
    return r;
}

template <typename T, int VB>
__device__ __forceinline__ void gn_widen(const GnUnit<VB>& r, float (&f)[VB / (int)sizeof(T)])
{
    if constexpr (sizeof(T) == 4) {
#pragma unroll
        for (int e = 0; e < VB / 4; ++e) f[e] = __uint_as_float(r.w[e]);
    } else if constexpr (VB >= 4) {
#pragma unroll
        for (int i = 0; i < VB / 4; ++i) {
            float2 a;
            Elem<T>::unpack_pair(r.w[i], a);
            f[2 * i] = a.x;
            f[2 * i + 1] = a.y;
        }
    } else {
        float2 a;
        Elem<T>::unpack_pair(r.w[0], a);
        f[0] = a.x;
    }
}

template <typename T, int VB>
__device__ __forceinline__ void gn_store(T* q, const float (&f)[VB / (int)sizeof(T)])
{
    if constexpr (VB == 16) {
        st_stream(q, Elem<T>::pack(f));
    } else if constexpr (sizeof(T) == 4) {
        if constexpr (VB == 8) *reinterpret_cast<float2*>(q) = make_float2(f[0], f[1]);
        else *q = f[0];
    } else if constexpr (VB >= 4) {
        T o[VB / 2];
#pragma unroll
        for (int e = 0; e < VB / 2; ++e) Elem<T>::store1(&o[e], f[e]);
        if constexpr (VB == 8) *reinterpret_cast<uint2*>(q) = *reinterpret_cast<const uint2*>(o);
        else *reinterpret_cast<uint32_t*>(q) = *reinterpret_cast<const uint32_t*>(o);
    } else {
        Elem<T>::store1(q, f[0]);
    }
}

// The activation as the other kernels of this file compute it (16-bit SiLU through one hardware tanh).
template <typename T, int ACT>
__device__ __forceinline__ float gn_activate(float v)
{
    if (ACT == kActSilu && sizeof(T) == 2) {
        const float h = 0.5f * v;
        return fmaf(h, tanh_approx(h), h);
    }
    return activate<ACT>(v);
}

constexpr int kGnRegUnits = 8;                   // units a thread holds at most
constexpr int kGnRegMaxWarps = 16;               // warps of the largest team
constexpr int kGnRegLanes = 8;                   // lanes of a team inside a warp

// Element pair j of a unit plus c; for 16-bit data the add widens its operand itself (exact, one rounding).
template <typename T, int VB>
__device__ __forceinline__ float2 gn_pair_plus(const GnUnit<VB>& r, int j, float2 c)
{
    if constexpr (sizeof(T) == 4)
        return __fadd2_rn(make_float2(__uint_as_float(r.w[2 * j]), __uint_as_float(r.w[2 * j + 1])), c);
    else
        return Elem<T>::add_widen2(r.w[j], c);
}

template <typename T, int ACT>
__device__ __forceinline__ float2 gn_activate2(float2 u)
{
    if (ACT == kActSilu && sizeof(T) == 2) {
        const float2 h = __fmul2_rn(u, make_float2(0.5f, 0.5f));
        return __ffma2_rn(h, make_float2(tanh_approx(h.x), tanh_approx(h.y)), h);
    }
    if (ACT == kActSilu) {
        const float2 a = __fmul2_rn(u, make_float2(-kLog2e, -kLog2e));
        const float2 d = __fadd2_rn(make_float2(ex2_approx(a.x), ex2_approx(a.y)), make_float2(1.0f, 1.0f));
        return __fmul2_rn(u, make_float2(rcp_approx(d.x), rcp_approx(d.y)));
    }
    return make_float2(activate<ACT>(u.x), activate<ACT>(u.y));
}

// kStraddle: a unit may end in the next channel (planes that are not a whole number of units).
template <typename T, typename PT, int VB, int NV, int ACT, bool kStraddle>
__device__ __forceinline__ void gn_reg_normalize(const GnUnit<VB> (&raw)[NV], T* yc, int n, int ts, int tl, int plane,
                                                 float inv_plane, int c_first, const PT* gamma, const PT* beta,
                                                 float mu, float rs)
{
    constexpr int EU = VB / (int)sizeof(T);
    const float2 nmu = make_float2(-mu, -mu);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int u = k * ts + tl;
        if (u < n) {
            const int i0 = u * EU;
            const int cin = div_small(i0, plane, inv_plane);
            const int c = c_first + cin;
            const float sc0 = rs * (gamma != nullptr ? param1(gamma, c) : 1.0f);
            const float be0 = beta != nullptr ? param1(beta, c) : 0.0f;
            float sc1 = sc0, be1 = be0;
            int left = EU;                                   // elements of this unit that belong to channel cin
            if constexpr (kStraddle && EU > 1) {
                left = plane - (i0 - cin * plane);
                if (left < EU) {
                    sc1 = rs * (gamma != nullptr ? param1(gamma, c + 1) : 1.0f);
                    be1 = beta != nullptr ? param1(beta, c + 1) : 0.0f;
                }
            }
            float f[EU];
            if constexpr (EU >= 2) {
#pragma unroll
                for (int j = 0; j < EU / 2; ++j) {
                    const float2 d = gn_pair_plus<T, VB>(raw[k], j, nmu);
                    float2 sc = make_float2(sc0, sc0), be = make_float2(be0, be0);
                    if constexpr (kStraddle) {
                        if (2 * j >= left) sc.x = sc1, be.x = be1;
                        if (2 * j + 1 >= left) sc.y = sc1, be.y = be1;
                    }
                    const float2 o = gn_activate2<T, ACT>(__ffma2_rn(d, sc, be));
                    f[2 * j] = o.x;
                    f[2 * j + 1] = o.y;
                }
            } else {
                gn_widen<T, VB>(raw[k], f);
                f[0] = gn_activate<T, ACT>(fmaf(f[0] - mu, sc0, be0));
            }
            gn_store<T, VB>(yc + i0, f);
        }
    }
}

template <typename T, typename PT, int VB, int NV, int L, bool kStraddle>
__global__ void __launch_bounds__(kGnRegMaxWarps * 32)
groupnorm_reg_kernel(const T* __restrict__ x, const PT* __restrict__ gamma, const PT* __restrict__ beta,
                     T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd, int64_t chunks, int units,
                     int chunk_elems, int plane, int cpg, int groups, float eps, float inv_count, float inv_plane,
                     int act, int tw)
{
    constexpr int EU = VB / (int)sizeof(T);
    __shared__ float slot_a[kGnRegMaxWarps], slot_b[kGnRegMaxWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int team, tl, ts, per_cta;
    if constexpr (L < 32) {
        team = threadIdx.x / L;
        tl = threadIdx.x & (L - 1);
        ts = L;
        per_cta = blockDim.x / L;
    } else {
        team = warp / tw;
        tl = threadIdx.x - team * tw * 32;
        ts = tw * 32;
        per_cta = (blockDim.x >> 5) / tw;
    }
    const int64_t chunk = (int64_t)blockIdx.x * per_cta + team;
    const bool live = chunk < chunks;
    const int n = live ? units : 0;
    const T* xc = x + (live ? chunk : 0) * chunk_elems;
    T* yc = y + (live ? chunk : 0) * chunk_elems;
    GnUnit<VB> raw[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int u = k * ts + tl;
        if (u < n) {
            raw[k] = gn_load<T, VB>(xc + u * EU);
        } else {
#pragma unroll
            for (int i = 0; i < (VB >= 4 ? VB / 4 : 1); ++i) raw[k].w[i] = 0u;
        }
    }
    // a team's sum, the same value in all its threads
    auto team_sum = [&](float v, float* slots) {
        if constexpr (L < 32) {
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            return v;
        } else {
            v = warp_sum(v);
            if (tw == 1) return v;
            if (lane == 0) slots[warp] = v;
            __syncthreads();
            return warp_sum(lane < tw ? slots[team * tw + lane] : 0.0f);
        }
    };
    float s = 0.0f;
    if constexpr (EU >= 2) {
        float2 s2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < NV; ++k)
#pragma unroll
            for (int j = 0; j < EU / 2; ++j) s2 = gn_pair_plus<T, VB>(raw[k], j, s2);    // units past the chunk hold zeros
        s = s2.x + s2.y;
    } else {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            float f[EU];
            gn_widen<T, VB>(raw[k], f);
            s += f[0];
        }
    }
    const float mu = team_sum(s, slot_a) * inv_count;
    float q = 0.0f;
    if constexpr (EU >= 2) {
        const float2 nmu = make_float2(-mu, -mu);
        float2 q2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            if (k * ts + tl < n) {
#pragma unroll
                for (int j = 0; j < EU / 2; ++j) {
                    const float2 d = gn_pair_plus<T, VB>(raw[k], j, nmu);
                    q2 = __ffma2_rn(d, d, q2);
                }
            }
        }
        q = q2.x + q2.y;
    } else {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            if (k * ts + tl < n) {
                float f[EU];
                gn_widen<T, VB>(raw[k], f);
                const float d = f[0] - mu;
                q = fmaf(d, d, q);
            }
        }
    }
    const float rs = rsqrtf(team_sum(q, slot_b) * inv_count + eps);
    if (live && tl == 0) {
        if (mean != nullptr) mean[chunk] = mu;
        if (rstd != nullptr) rstd[chunk] = rs;
    }
    const int c_first = (int)(chunk % groups) * cpg;
    if (act == kActSilu)
        gn_reg_normalize<T, PT, VB, NV, kActSilu, kStraddle>(raw, yc, n, ts, tl, plane, inv_plane, c_first, gamma, beta, mu, rs);
    else if (act == kActRelu)
        gn_reg_normalize<T, PT, VB, NV, kActRelu, kStraddle>(raw, yc, n, ts, tl, plane, inv_plane, c_first, gamma, beta, mu, rs);
    else
        gn_reg_normalize<T, PT, VB, NV, kActNone, kStraddle>(raw, yc, n, ts, tl, plane, inv_plane, c_first, gamma, beta, mu, rs);
}

// Any plane size / alignment: scalar loads, two sweeps over global memory, same moment arithmetic.
template <typename T, typename PT, int ACT>
__global__ void __launch_bounds__(256)
groupnorm_scalar_kernel(const T* __restrict__ x, const PT* __restrict__ gamma, const PT* __restrict__ beta,
                        T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd,
                        int64_t chunk_elems, int64_t plane, int cpg, int groups, float eps)
{
    __shared__ float red_n[32], red_mean[32], red_m2[32];
    __shared__ float bc_mean, bc_rstd;
    const int64_t chunk = blockIdx.x;
    const int g = (int)(chunk % groups);
    const T* xc = x + chunk * chunk_elems;
    T* yc = y + chunk * chunk_elems;
    Moments acc{0.0f, 0.0f, 0.0f};
    for (int64_t j = threadIdx.x; j < chunk_elems; j += blockDim.x)
        acc = merge(acc, Moments{1.0f, Elem<T>::load1(xc + j), 0.0f});
    acc = warp_merge(acc);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if (lane == 0) {
        red_n[warp] = acc.n;
        red_mean[warp] = acc.mean;
        red_m2[warp] = acc.m2;
    }
    __syncthreads();
    if (warp == 0) {
        Moments t = lane < nw ? Moments{red_n[lane], red_mean[lane], red_m2[lane]} : Moments{0.0f, 0.0f, 0.0f};
        t = warp_merge(t);
        if (lane == 0) {
            const float rs = rsqrtf(t.m2 / t.n + eps);
            bc_mean = t.mean;
            bc_rstd = rs;
            if (mean != nullptr) mean[chunk] = t.mean;
            if (rstd != nullptr) rstd[chunk] = rs;
        }
    }
    __syncthreads();
    const float mu = bc_mean, rs = bc_rstd;
    for (int64_t j = threadIdx.x; j < chunk_elems; j += blockDim.x) {
        const int c = g * cpg + (int)(j / plane);
        const float sc = rs * (gamma != nullptr ? param1(gamma, c) : 1.0f);
        const float be = beta != nullptr ? param1(beta, c) : 0.0f;
        Elem<T>::store1(yc + j, activate<ACT>(fmaf(Elem<T>::load1(xc + j) - mu, sc, be)));
    }
}

constexpr size_t kGnStageLimit = 200 * 1024;     // leaves room for the static reduction slots
static_assert(kGnStageLimit <= (size_t)kGnMaxParts * kGnCopyVecs * 16, "one barrier per 32 KB part");
constexpr int kMaxDevices = 64;

// beyond 40 KB (more than ten warps a team) the staged kernel is ahead: bf16 chunks of 49 KB 4.7 against 4.1 TB/s; where
// the staged kernel cannot take the chunk (planes that are not whole vectors) the register kernel goes on to its limit
// of sixteen warps a team, 64 KB (the alternative is the scalar kernel at 0.8 TB/s)
constexpr int64_t kGnRegMaxBytes = 40 * 1024, kGnRegMaxBytesUnstaged = 64 * 1024;

// Launches the register kernel when the chunk fits a team; false when it does not.
template <typename T, typename PT, int VB, bool kStraddle>
bool launch_gn_reg_vb(const T* x, const PT* gamma, const PT* beta, T* y, float* mean, float* rstd, int64_t chunks,
                      int64_t chunk_elems, int64_t plane, int cpg, int groups, float eps, int act, cudaStream_t stream)
{
    const int64_t units = chunk_elems * (int64_t)sizeof(T) / VB;
    const float inv_count = (float)(1.0 / (double)chunk_elems), inv_plane = (float)(1.0 / (double)plane);
#define KOP_GN_REG_GO(NV, L, CTAS, THREADS, TW)                                                                       \
    groupnorm_reg_kernel<T, PT, VB, NV, L, kStraddle><<<(unsigned)(CTAS), (unsigned)(THREADS), 0, stream>>>(         \
        x, gamma, beta, y, mean, rstd, chunks, (int)units, (int)chunk_elems, (int)plane, cpg, groups, eps, inv_count, \
        inv_plane, act, (int)(TW))
    if (units <= kGnRegLanes * kGnRegUnits) {
        constexpr int kThreads = 128, kTeams = kThreads / kGnRegLanes;
        const int64_t ctas = (chunks + kTeams - 1) / kTeams;
        if (ctas > 0x7FFFFFFFLL) return false;
        if (units <= kGnRegLanes * 2) KOP_GN_REG_GO(2, kGnRegLanes, ctas, kThreads, 1);
        else KOP_GN_REG_GO(kGnRegUnits, kGnRegLanes, ctas, kThreads, 1);
        return true;
    }
    // eight units a thread keep the most bytes in flight, four fill the team's last sweep better when the chunk
    // is a small number of warp sweeps (98 units: 38 % of the slots of one warp at eight, 77 % at four)
    const int64_t tw8 = (units + 32 * kGnRegUnits - 1) / (32 * kGnRegUnits);
    const int64_t tw4 = (units + 16 * kGnRegUnits - 1) / (16 * kGnRegUnits);
    bool eight = (double)units / (double)(tw8 * 32 * kGnRegUnits) >= 0.85 * (double)units / (double)(tw4 * 16 * kGnRegUnits);
    if (!eight && tw4 > kGnRegMaxWarps) eight = true;
    const int64_t tw = eight ? tw8 : tw4;
    if (tw > kGnRegMaxWarps) return false;
    const int teams = tw >= 4 ? 1 : 4 / (int)tw;
    const int64_t ctas = (chunks + teams - 1) / teams;
    if (ctas > 0x7FFFFFFFLL) return false;
    if (eight) KOP_GN_REG_GO(kGnRegUnits, 32, ctas, teams * tw * 32, tw);
    else KOP_GN_REG_GO(kGnRegUnits / 2, 32, ctas, teams * tw * 32, tw);
#undef KOP_GN_REG_GO
    return true;
}

template <typename T, typename PT>
bool launch_gn_reg(const T* x, const PT* gamma, const PT* beta, T* y, float* mean, float* rstd, int64_t chunks,
                   int64_t chunk_elems, int64_t plane, int cpg, int groups, float eps, int act, cudaStream_t stream)
{
    constexpr int esz = (int)sizeof(T);
    const int64_t bytes = chunk_elems * esz;
    const bool staged_ok = aligned_to(x, 16) && aligned_to(y, 16) && plane % Elem<T>::kPerVec == 0;
    if (bytes > (staged_ok ? kGnRegMaxBytes : kGnRegMaxBytesUnstaged)) return false;
    int vb = 16;
    while (vb > esz && (bytes % vb != 0 || !aligned_to(x, vb) || !aligned_to(y, vb) || vb / esz > plane)) vb >>= 1;
#define KOP_GN_REG(VB)                                                                                                \
    ((VB) > esz && plane % ((VB) / esz) != 0                                                                          \
         ? launch_gn_reg_vb<T, PT, VB, (VB > esz)>(x, gamma, beta, y, mean, rstd, chunks, chunk_elems, plane, cpg,    \
                                                   groups, eps, act, stream)                                          \
         : launch_gn_reg_vb<T, PT, VB, false>(x, gamma, beta, y, mean, rstd, chunks, chunk_elems, plane, cpg, groups, \
                                              eps, act, stream))
    switch (vb) {
    case 16: return KOP_GN_REG(16);
    case 8: return KOP_GN_REG(8);
    case 4: return KOP_GN_REG(4);
    default:
        if constexpr (esz == 2) return KOP_GN_REG(2);
        else return false;
    }
#undef KOP_GN_REG
}

template <typename T, typename PT, int ACT>
kop_status_t launch_gn_act(const T* x, const PT* gamma, const PT* beta, T* y, float* mean, float* rstd,
                           int64_t chunks, int64_t chunk_elems, int64_t plane, int cpg, int groups, float eps,
                           cudaStream_t stream)
{
    constexpr int E = Elem<T>::kPerVec;
    if (launch_gn_reg<T, PT>(x, gamma, beta, y, mean, rstd, chunks, chunk_elems, plane, cpg, groups, eps, ACT, stream))
        return launch_status();
    const bool vec = aligned_to(x, 16) && aligned_to(y, 16) && (plane % E) == 0 && chunk_elems / E <= 0x7FFFFFFF;
    if (vec) {
        const int nvec = (int)(chunk_elems / E);
        const int vpp = (int)(plane / E);
        const size_t bytes = (size_t)nvec * 16;
        if (bytes <= kGnStageLimit) {
            // the opt-in above 48 KB is per function and per device; one flag per template instance
            static std::atomic<bool> configured[kMaxDevices];
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess) return KOP_ERR_CUDA;
            if (dev < 0 || dev >= kMaxDevices || !configured[dev].load(std::memory_order_acquire)) {
                // only the 512-thread instance ever needs more than the default 48 KB (chunks beyond 32 KB)
                if (cudaFuncSetAttribute(groupnorm_staged_kernel<T, PT, ACT, 512>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kGnStageLimit) != cudaSuccess)
                    return KOP_ERR_CUDA;
                if (dev >= 0 && dev < kMaxDevices) configured[dev].store(true, std::memory_order_release);
            }
            const float inv_count = (float)(1.0 / (double)chunk_elems);
            if (nvec <= 512)
                groupnorm_staged_kernel<T, PT, ACT, 128><<<(unsigned)chunks, 128, bytes, stream>>>(
                    x, gamma, beta, y, mean, rstd, nvec, vpp, cpg, groups, eps, inv_count);
            else if (nvec <= 2048)
                groupnorm_staged_kernel<T, PT, ACT, 256><<<(unsigned)chunks, 256, bytes, stream>>>(
                    x, gamma, beta, y, mean, rstd, nvec, vpp, cpg, groups, eps, inv_count);
            else
                groupnorm_staged_kernel<T, PT, ACT, 512><<<(unsigned)chunks, 512, bytes, stream>>>(
                    x, gamma, beta, y, mean, rstd, nvec, vpp, cpg, groups, eps, inv_count);
        } else if (bytes <= 512 * 1024 && chunks * 8 <= 0x7FFFFFFFLL) {
            // a cluster per chunk, slices of at most 64 KB (three CTAs per SM). Measured against the two-sweep
            // kernel on fp32 chunks of 256 KB: 3.7 against 3.0 TB/s; at 1 MB (six slices of 175 KB, one CTA per
            // SM) it lost, 3.2 against 3.9, and at 98 KB against the single-CTA staged kernel too (4.1 against
            // 5.3): a cluster barrier costs about what a CTA needs for 100 KB, so only this window uses it.
            int csize = (int)((bytes + 64 * 1024 - 1) / (64 * 1024));
            if (csize < 2) csize = 2;
            const int slice_vecs = (nvec + csize - 1) / csize;
            const size_t smem = (size_t)slice_vecs * 16;
            static std::atomic<bool> configured_c[kMaxDevices];
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess) return KOP_ERR_CUDA;
            if (dev < 0 || dev >= kMaxDevices || !configured_c[dev].load(std::memory_order_acquire)) {
                if (cudaFuncSetAttribute(groupnorm_cluster_kernel<T, PT, ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kGnStageLimit) != cudaSuccess)
                    return KOP_ERR_CUDA;
                if (dev >= 0 && dev < kMaxDevices) configured_c[dev].store(true, std::memory_order_release);
            }
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(chunks * csize), 1, 1);
            cfg.blockDim = dim3(kGnClusterThreads, 1, 1);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)csize;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            const float inv_count = (float)(1.0 / (double)chunk_elems);
            if (cudaLaunchKernelEx(&cfg, groupnorm_cluster_kernel<T, PT, ACT>, x, gamma, beta, y, mean, rstd, nvec, slice_vecs,
                                   csize, vpp, cpg, groups, eps, inv_count) != cudaSuccess) {
                (void)cudaGetLastError();
                return KOP_ERR_CUDA;
            }
        } else if (chunks <= (int64_t)sm_count() && bytes >= 1024 * 1024) {
            // too few chunks to fill the GPU: clusters share them, about two CTAs per SM in all
            int csize = (int)((2 * (int64_t)sm_count() + chunks - 1) / chunks);
            if (csize > 8) csize = 8;
            if (csize < 2) csize = 2;
            const int slice_vecs = (nvec + csize - 1) / csize;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(chunks * csize), 1, 1);
            cfg.blockDim = dim3(kGnThreads, 1, 1);
            cfg.dynamicSmemBytes = 0;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)csize;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, groupnorm_twosweep_cluster_kernel<T, PT, ACT>, x, gamma, beta, y, mean, rstd, nvec,
                                   slice_vecs, csize, vpp, cpg, groups, eps) != cudaSuccess) {
                (void)cudaGetLastError();
                return KOP_ERR_CUDA;
            }
        } else {
            groupnorm_twosweep_kernel<T, PT, ACT><<<(unsigned)chunks, kGnThreads, 0, stream>>>(
                x, gamma, beta, y, mean, rstd, nvec, vpp, cpg, groups, eps);
        }
        return launch_status();
    }
    groupnorm_scalar_kernel<T, PT, ACT><<<(unsigned)chunks, 256, 0, stream>>>(x, gamma, beta, y, mean, rstd, chunk_elems,
                                                                          plane, cpg, groups, eps);
    return launch_status();
}

template <typename T, typename PT>
kop_status_t launch_gn(const void* x, const void* gammav, const void* betav, void* y, float* mean, float* rstd,
                       int64_t chunks, int64_t chunk_elems, int64_t plane, int cpg, int groups, float eps, int act,
                       cudaStream_t stream)
{
    const T* xt = static_cast<const T*>(x);
    const PT* gamma = static_cast<const PT*>(gammav);
    const PT* beta = static_cast<const PT*>(betav);
    T* yt = static_cast<T*>(y);
    switch (act) {
    case kActRelu: return launch_gn_act<T, PT, kActRelu>(xt, gamma, beta, yt, mean, rstd, chunks, chunk_elems, plane, cpg, groups, eps, stream);
    case kActSilu: return launch_gn_act<T, PT, kActSilu>(xt, gamma, beta, yt, mean, rstd, chunks, chunk_elems, plane, cpg, groups, eps, stream);
    default: return launch_gn_act<T, PT, kActNone>(xt, gamma, beta, yt, mean, rstd, chunks, chunk_elems, plane, cpg, groups, eps, stream);
    }
}

}  // namespace
}  // namespace kop

namespace kop {
namespace {

kop_status_t gn_entry(const void* x, const void* gamma, const void* beta, void* y, float* mean, float* rstd, int64_t N,
                      int64_t C, int64_t H, int64_t W, int64_t groups, float eps, int act, kop_dtype_t dtype,
                      kop_dtype_t pdtype, kop_stream_t stream)
{
    if (!param_dtype_ok(dtype, pdtype)) return KOP_ERR_UNSUPPORTED_DTYPE;
    if (N < 0 || C <= 0 || H <= 0 || W <= 0 || groups <= 0 || groups > C || C % groups != 0) return KOP_ERR_BAD_SHAPE;
    if (act < 0 || act > 2 || !(eps >= 0.0f)) return KOP_ERR_BAD_SHAPE;
    if (C > 0x7FFFFFFF || H > kMaxElems || W > kMaxElems || N > kMaxElems || H > kMaxElems / W) return KOP_ERR_BAD_SHAPE;
    const int64_t plane = H * W;
    if (C > kMaxElems / plane) return KOP_ERR_BAD_SHAPE;
    if (N == 0) return KOP_OK;
    if (C * plane > kMaxElems / N) return KOP_ERR_BAD_SHAPE;
    if (N * groups > 0x7FFFFFFFLL) return KOP_ERR_BAD_SHAPE;           // one CTA per (image, group)
    if (!x || !y) return KOP_ERR_NULL_POINTER;
    const int esz = elem_size(dtype);
    if (!aligned_to(x, esz) || !aligned_to(y, esz) || (gamma && !aligned_to(gamma, elem_size(pdtype))) ||
        (beta && !aligned_to(beta, elem_size(pdtype))) || (mean && !aligned_to(mean, 4)) || (rstd && !aligned_to(rstd, 4)))
        return KOP_ERR_MISALIGNED;
    if (!alias_ok(x, C * plane, y, C * plane, N, C * plane, esz, true)) return KOP_ERR_BAD_ALIAS;
    kop_status_t st = check_device();
    if (st != KOP_OK) return st;
    const int cpg = (int)(C / groups);
    const int64_t chunk_elems = (int64_t)cpg * plane;
    cudaStream_t s = as_stream(stream);
#define KOP_GN_GO(T, PT) launch_gn<T, PT>(x, gamma, beta, y, mean, rstd, N * groups, chunk_elems, plane, cpg, (int)groups, eps, act, s)
    return KOP_DISPATCH_TYPES(dtype, pdtype, KOP_GN_GO);
#undef KOP_GN_GO
}

}  // namespace
}  // namespace kop

extern "C" kop_status_t kop_groupnorm_act(const void* x, const float* gamma, const float* beta, void* y,
                                          float* mean, float* rstd, int64_t N, int64_t C, int64_t H, int64_t W,
                                          int64_t groups, float eps, int act, kop_dtype_t dtype,
                                          kop_stream_t stream)
{
    return kop::gn_entry(x, gamma, beta, y, mean, rstd, N, C, H, W, groups, eps, act, dtype, KOP_F32, stream);
}

extern "C" kop_status_t kop_groupnorm_act_ex(const void* x, const void* gamma, const void* beta, void* y, float* mean,
                                             float* rstd, int64_t N, int64_t C, int64_t H, int64_t W, int64_t groups,
                                             float eps, int act, kop_dtype_t dtype, kop_dtype_t param_dtype,
                                             kop_stream_t stream)
{
    return kop::gn_entry(x, gamma, beta, y, mean, rstd, N, C, H, W, groups, eps, act, dtype, param_dtype, stream);
}

extern "C" kop_status_t kop_groupnorm_wait_timeouts(unsigned int* host_count)
{
    using namespace kop;
    if (!host_count) return KOP_ERR_NULL_POINTER;
    kop_status_t st = check_device();
    if (st != KOP_OK) return st;
    return cudaMemcpyFromSymbol(host_count, g_gn_wait_timeouts, sizeof(unsigned int)) == cudaSuccess ? KOP_OK
                                                                                                      : KOP_ERR_CUDA;
}
