// Sparse index collection: hidden state x and a threshold t -> the ascending
// list of the entries with |x_k| > t and its length.  Three kernels:
//   sparsify_cluster_kernel (one row, 6144 < n <= 65536): the compaction below spread over a thread-block
//     cluster of 8 CTAs, warp totals exchanged through distributed shared memory (3.4 against 4.9 us at
//     n = 14336; no gain at n = 4096, where the single CTA stays).
//   sparsify_kernel (one row, any n): each warp owns a contiguous segment of x, counts its active entries
//     with __ballot_sync/__popc (the loads of eight groups of 32 entries in flight together), the 32 warp
//     totals are scanned in shared memory, and each warp then writes its indices at its base offset.
//   sparsify_rows_kernel (the small batch, n < 2^16: "active in at least one of B rows"; one CTA, or a
//     cluster of 8 CTAs from n = 6144 up): 16-byte loads,
//     all of a piece's loads in flight together (with B rows, loads that wait for one another cost a round
//     trip each); compaction by warp scans.  For a single row it measured no faster than the kernel above
//     (2.7 against 2.3 us at n = 4096, 5.9 against 5.2 us at n = 14336), which therefore keeps that job.
// The output order is ascending by construction (no atomics, no arrival order).
#include "spqt_common.cuh"

namespace spqt {

constexpr int kSparsifyThreads = 1024;

__device__ __forceinline__ bool is_active(__half v, float t)
{
    // exact widening; NaN compares false and is therefore never active
    return fabsf(__half2float(v)) > t;
}

__global__ void __launch_bounds__(kSparsifyThreads)
sparsify_kernel(const __half* __restrict__ x, int n, float t,
                int32_t* __restrict__ idx, int32_t* __restrict__ count)
{
    __shared__ int warp_total[32];
    __shared__ int warp_base[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Programmatic dependent launch: the block may have been started while the previous kernel of the
    // stream was still draining; nothing above touches global memory, everything below waits for it.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // segment of this warp: a multiple of 32 elements, contiguous, ascending with the warp id
    const int seg = ((n + 32 * 32 - 1) / (32 * 32)) * 32;
    const int begin = min(warp * seg, n), end = min(begin + seg, n);

    // Eight groups of 32 entries at a time: their loads are issued together (addresses clamped into x instead
    // of guarded, so that nothing makes one load wait for another), then one ballot per group.  Up to 64
    // groups per warp (n <= 65536) the lane's activity bits stay in a register for the writing phase.
    const int groups = (end - begin + 31) >> 5;
    const bool in_regs = groups <= 64;
    unsigned long long flags = 0ull;
    int total = 0;
    for (int g0 = 0; g0 < groups; g0 += 8) {
        __half v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (g0 + j < groups) v[j] = x[min(begin + (g0 + j) * 32 + lane, n - 1)];   // (uniform condition)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (g0 + j < groups) {
                const int k = begin + (g0 + j) * 32 + lane;
                const bool p = (k < end) && is_active(v[j], t);
                total += __popc(__ballot_sync(0xffffffffu, p));
                if (p) flags |= 1ull << ((g0 + j) & 63);
            }
        }
    }
    if (lane == 0) warp_total[warp] = total;
    __syncthreads();
    if (warp == 0) {
        int v = warp_total[lane], incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        warp_base[lane] = incl - v;
        if (lane == 31) *count = incl;
    }
    __syncthreads();
    int base = warp_base[warp];
    if (in_regs) {
        for (int g = 0; g < groups; ++g) {
            const bool p = (flags >> g) & 1ull;
            const unsigned mask = __ballot_sync(0xffffffffu, p);
            if (p) idx[base + __popc(mask & ((1u << lane) - 1u))] = begin + g * 32 + lane;
            base += __popc(mask);
        }
        return;
    }
    for (int k0 = begin; k0 < end; k0 += 32) {
        const int k = k0 + lane;
        const bool p = (k < end) && is_active(x[k], t);
        const unsigned mask = __ballot_sync(0xffffffffu, p);
        if (p) idx[base + __popc(mask & ((1u << lane) - 1u))] = k;
        base += __popc(mask);
    }
}

// The same compaction spread over a thread-block cluster of 8 CTAs of 8 warps (n <= 65536): one SM's
// instruction rate is what a single CTA spends most of its time on once n reaches several thousand.  The 64
// warps own consecutive segments of x; every CTA leaves its warps' totals in its own shared memory, the
// cluster synchronises, and each warp adds up the totals of the warps before it, reading the other CTAs'
// tables through distributed shared memory.  A second cluster barrier keeps every CTA's table alive until
// all have read it.  (Hardware barriers that every CTA reaches unconditionally: nothing to time out.)
constexpr int kClusterCtas = 8;
constexpr int kClusterWarps = 8;

__global__ void __launch_bounds__(kClusterWarps * 32)
sparsify_cluster_kernel(const __half* __restrict__ x, int n, float t, int32_t* __restrict__ idx, int32_t* __restrict__ count)
{
    __shared__ int warp_total[kClusterWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int gw = (int)rank * kClusterWarps + warp;      // this warp among the cluster's 64
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int kAll = kClusterCtas * kClusterWarps;
    const int seg = ((n + kAll * 32 - 1) / (kAll * 32)) * 32;   // at most 1024 entries: 32 groups
    const int begin = min(gw * seg, n), end = min(begin + seg, n);
    const int groups = (end - begin + 31) >> 5;
    unsigned flags = 0u;
    int total = 0;
    for (int g0 = 0; g0 < groups; g0 += 8) {
        __half v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (g0 + j < groups) v[j] = x[min(begin + (g0 + j) * 32 + lane, n - 1)];   // (uniform condition)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (g0 + j < groups) {
                const int k = begin + (g0 + j) * 32 + lane;
                const bool p = (k < end) && is_active(v[j], t);
                total += __popc(__ballot_sync(0xffffffffu, p));
                if (p) flags |= 1u << (g0 + j);
            }
        }
    }
    if (lane == 0) warp_total[warp] = total;
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // lane l looks up the totals of warps l and l + 32 of the cluster
    int below = 0, all = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int w = lane + 32 * h;
        unsigned remote;
        const unsigned local = static_cast<unsigned>(__cvta_generic_to_shared(&warp_total[w % kClusterWarps]));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"((unsigned)(w / kClusterWarps)));
        int v;
        asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
        below += (w < gw) ? v : 0;
        all += v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        below += __shfl_xor_sync(0xffffffffu, below, o);
        all += __shfl_xor_sync(0xffffffffu, all, o);
    }
    if (gw == 0 && lane == 0) *count = all;
    int base = below;
    for (int g = 0; g < groups; ++g) {
        const bool p = (flags >> g) & 1u;
        const unsigned mask = __ballot_sync(0xffffffffu, p);
        if (p) idx[base + __popc(mask & ((1u << lane) - 1u))] = begin + g * 32 + lane;
        base += __popc(mask);
    }
    // nobody leaves while another CTA may still be reading its table
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Lane l of a warp holds the 8 columns 256*piece + 8*l .. + 7 of each of the warp's pieces (a warp owns up
// to 8 consecutive pieces of 256 columns: n < 2^16); every row's 8 values arrive with one 16-byte load (plain
// 2-byte loads at a ragged end or when X is not aligned for it), and a piece's loads are all issued before
// the first compare, so that they share one round trip.  Then the usual compaction: totals per warp, a scan
// over the warps, and every lane writes its own active columns behind those of the lanes before it.
// CLUSTER: the same on a thread-block cluster of 8 CTAs of 8 warps (the 64 warps own consecutive runs of
// pieces; warp totals are exchanged through distributed shared memory as in sparsify_cluster_kernel).
template <bool CLUSTER>
__global__ void __launch_bounds__(CLUSTER ? kClusterWarps * 32 : 1024)
sparsify_rows_kernel(const __half* __restrict__ X, int ldx, int batch, int n, float t,
                     int32_t* __restrict__ idx, int32_t* __restrict__ count)
{
    __shared__ int warp_total[32];
    __shared__ int warp_base[32];
    const int lane = threadIdx.x & 31, cta_warp = threadIdx.x >> 5;
    unsigned rank = 0;
    if (CLUSTER) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int warp = CLUSTER ? (int)rank * kClusterWarps + cta_warp : cta_warp;   // among all the warps at work
    constexpr int kAllWarps = CLUSTER ? kClusterCtas * kClusterWarps : 32;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int pieces = (n + 255) >> 8;
    const int pp = (pieces + kAllWarps - 1) / kAllWarps;   // pieces per warp, at most 8
    const bool vec_ok = (reinterpret_cast<uintptr_t>(X) & 15) == 0 && (ldx & 7) == 0;
    const unsigned short* Xs = reinterpret_cast<const unsigned short*>(X);
    // the largest fp16 value not above t (any negative value if t < 0: everything but NaN is active; +inf if t
    // is NaN or +inf: nothing is): |x| > t  <=>  |x| > that value, compared in fp16, two entries at a time
    const __half thr_h = (t != t) ? __ushort_as_half((unsigned short)0x7c00)
                                  : (t < 0.0f ? __float2half_rn(-1.0f) : __float2half_rd(t));
    const __half2 thr_h2 = __half2half2(thr_h);

    unsigned long long flags = 0ull;                   // byte j: activity bits of the lane's 8 columns of piece j
#pragma unroll 1
    for (int j = 0; j < pp; ++j) {
        const int k0 = (warp * pp + j) * 256 + lane * 8;
        const bool have = k0 < n;
        uint4 v[8];
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            v[b] = make_uint4(0u, 0u, 0u, 0u);
            if (have && b < batch) {
                const size_t off = (size_t)b * ldx + k0;
                if (vec_ok && k0 + 8 <= n) {
                    v[b] = __ldg(reinterpret_cast<const uint4*>(Xs + off));
                } else {
                    unsigned short h[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) h[e] = (k0 + e < n) ? __ldg(Xs + off + e) : (unsigned short)0;
                    v[b] = make_uint4(h[0] | ((unsigned)h[1] << 16), h[2] | ((unsigned)h[3] << 16),
                                      h[4] | ((unsigned)h[5] << 16), h[6] | ((unsigned)h[7] << 16));
                }
            }
        }
        unsigned m8 = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            if (b < batch) {   // (uniform)
                const unsigned wds[4] = {v[b].x, v[b].y, v[b].z, v[b].w};
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const unsigned ab = wds[e2] & 0x7fff7fffu;
                    const unsigned gt = __hgt2_mask(*reinterpret_cast<const __half2*>(&ab), thr_h2);   // false for NaN
                    m8 |= ((gt & 1u) | ((gt >> 15) & 2u)) << (2 * e2);
                }
            }
        }
        // columns past n do not exist (with a negative threshold their zeros would count)
        const int left = n - k0;
        if (left < 8) m8 &= (left <= 0) ? 0u : ((1u << left) - 1u);
        flags |= (unsigned long long)m8 << (8 * j);
    }
    int total = __popcll(flags);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    int base;
    if (CLUSTER) {
        if (lane == 0) warp_total[cta_warp] = total;
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        int below = 0, all = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int w = lane + 32 * h;   // lane l looks up the totals of warps l and l + 32 of the cluster
            unsigned remote;
            const unsigned local = static_cast<unsigned>(__cvta_generic_to_shared(&warp_total[w % kClusterWarps]));
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"((unsigned)(w / kClusterWarps)));
            int v;
            asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
            below += (w < warp) ? v : 0;
            all += v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            below += __shfl_xor_sync(0xffffffffu, below, o);
            all += __shfl_xor_sync(0xffffffffu, all, o);
        }
        if (warp == 0 && lane == 0) *count = all;
        base = below;
    } else {
        if (lane == 0) warp_total[warp] = total;
        __syncthreads();
        if (warp == 0) {
            int v = warp_total[lane], incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            warp_base[lane] = incl - v;
            if (lane == 31) *count = incl;
        }
        __syncthreads();
        base = warp_base[warp];
    }
    for (int j = 0; j < pp; ++j) {
        const unsigned m8 = (unsigned)(flags >> (8 * j)) & 0xffu;
        const int c8 = __popc(m8);
        int incl = c8;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int pos = base + incl - c8;
        const int col0 = (warp * pp + j) * 256 + lane * 8;
        // one predicated store per column (a divergent branch per column costs far more than the store)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const unsigned on = (m8 >> e) & 1u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p st.global.u32 [%1], %2;\n\t}" ::"r"(on), "l"(idx + pos), "r"(col0 + e)
                         : "memory");
            pos += (int)on;
        }
        base += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (CLUSTER) {   // nobody leaves while another CTA may still be reading its table
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
}


// One launch of sparsify_rows_kernel: the columns that are active in at least one of `batch` rows (n < 2^16).
spqt_status launch_sparsify_rows(const __half* X, int ldx, int batch, int n, float t, int32_t* idx, int32_t* count,
                                 cudaStream_t stream)
{
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kClusterCtas;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    // from a few thousand columns on, the cluster of 8 CTAs (falls back to the single CTA if it cannot be launched)
    if (n > 6144) {
        cfg.gridDim = dim3(kClusterCtas);
        cfg.blockDim = dim3(kClusterWarps * 32);
        cfg.attrs = g_no_pdl ? attr + 1 : attr;
        cfg.numAttrs = g_no_pdl ? 1 : 2;
        if (cudaLaunchKernelEx(&cfg, sparsify_rows_kernel<true>, X, ldx, batch, n, t, idx, count) == cudaSuccess) {
            count_launch();
            return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
        }
        (void)cudaGetLastError();
    }
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(1024);
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, sparsify_rows_kernel<false>, X, ldx, batch, n, t, idx, count);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

}  // namespace spqt

extern "C" spqt_status spqt_sparsify(const void* x, int n, float t,
                                     int32_t* idx, int32_t* count, void* stream)
{
    using namespace spqt;
    if (n < 0 || !count || (n > 0 && (!x || !idx))) return SPQT_ERR_INVALID_ARG;
    if (!aligned(x, 2) || !aligned(idx, 4) || !aligned(count, 4)) return SPQT_ERR_ALIGNMENT;
    // from a few thousand entries on, the compaction spread over a cluster of 8 CTAs (falls back to the
    // single CTA below if the cluster cannot be launched)
    if (n > 6144 && n <= 65536) {
        cudaLaunchConfig_t cc = {};
        cc.gridDim = dim3(kClusterCtas);
        cc.blockDim = dim3(kClusterWarps * 32);
        cc.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute ca[2];
        ca[0].id = cudaLaunchAttributeClusterDimension;
        ca[0].val.clusterDim.x = kClusterCtas;
        ca[0].val.clusterDim.y = 1;
        ca[0].val.clusterDim.z = 1;
        ca[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        ca[1].val.programmaticStreamSerializationAllowed = 1;
        cc.attrs = ca;
        cc.numAttrs = g_no_pdl ? 1 : 2;
        if (cudaLaunchKernelEx(&cc, sparsify_cluster_kernel, static_cast<const __half*>(x), n, t, idx, count) == cudaSuccess) {
            count_launch();
            return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
        }
        (void)cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(kSparsifyThreads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, sparsify_kernel, static_cast<const __half*>(x), n, t, idx, count);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}
