// Sparse index collection: hidden state x and a threshold t -> the ascending
// list of the entries with |x_k| > t and its length.  A stream compaction built
// on warp ballots: each warp owns a contiguous segment of x, counts its active
// entries with __ballot_sync/__popc, the 32 warp totals are scanned in shared
// memory, and each warp then writes its indices at its base offset.  The output
// order is ascending by construction (no atomics, no arrival order).
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

    int total = 0;
    for (int k0 = begin; k0 < end; k0 += 32) {
        const int k = k0 + lane;
        const bool p = (k < end) && is_active(x[k], t);
        total += __popc(__ballot_sync(0xffffffffu, p));
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
    for (int k0 = begin; k0 < end; k0 += 32) {
        const int k = k0 + lane;
        const bool p = (k < end) && is_active(x[k], t);
        const unsigned mask = __ballot_sync(0xffffffffu, p);
        if (p) idx[base + __popc(mask & ((1u << lane) - 1u))] = k;
        base += __popc(mask);
    }
}

}  // namespace spqt

extern "C" spqt_status spqt_sparsify(const void* x, int n, float t,
                                     int32_t* idx, int32_t* count, void* stream)
{
    using namespace spqt;
    if (n < 0 || !count || (n > 0 && (!x || !idx))) return SPQT_ERR_INVALID_ARG;
    if (!aligned(x, 2) || !aligned(idx, 4) || !aligned(count, 4)) return SPQT_ERR_ALIGNMENT;
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
