// Threshold calibration: the nearest-rank order statistic of |x| over a pool of calibration activations,
// i.e. the threshold that makes a given fraction of the entries inactive.  fp16 has only 2^15
// non-negative bit patterns, and they order like the values, so a histogram over the patterns gives
// the exact order statistic: one pass to count, one small kernel to find the bin of the wanted rank.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kBins = 32768;           // magnitudes 0x0000 .. 0x7fff (0x7c01.. are NaN: never counted)
constexpr int kCalibThreads = 1024;

__global__ void __launch_bounds__(256)
calib_count_kernel(const unsigned short* __restrict__ x, size_t count, unsigned* __restrict__ hist)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) {
        const unsigned mag = x[i] & 0x7fffu;
        if (mag <= 0x7c00u) atomicAdd(hist + mag, 1u);   // NaN entries are not part of the pool
    }
}

// One CTA: thread i owns bins 32 i .. 32 i + 31.  Finds the bin holding the element of rank
// ceil(sparsity * N) (1-based, N = entries counted), writes its value, and zeroes the histogram.
__global__ void __launch_bounds__(kCalibThreads)
calib_select_kernel(unsigned* __restrict__ hist, double sparsity, float* __restrict__ t_out)
{
    __shared__ unsigned long long warp_tot[32];
    __shared__ unsigned long long total_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned h[32];
    unsigned long long mine = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        h[j] = hist[tid * 32 + j];
        hist[tid * 32 + j] = 0u;
        mine += h[j];
    }
    // exclusive prefix over the threads
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned long long v = warp_tot[lane], s = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, s, o);
            if (lane >= o) s += up;
        }
        warp_tot[lane] = s - v;
        if (lane == 31) total_s = s;
    }
    __syncthreads();
    const unsigned long long below = warp_tot[warp] + incl - mine, total = total_s;
    if (total == 0 || !(sparsity > 0.0)) {
        if (tid == 0) *t_out = -1.0f;   // nothing to drop: every entry stays active
        return;
    }
    double r = ceil(sparsity * (double)total - 1e-9);
    if (r < 1.0) r = 1.0;
    if (r > (double)total) r = (double)total;
    const unsigned long long rank = (unsigned long long)r;
    if (below < rank && rank <= below + mine) {
        unsigned long long c = below;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            c += h[j];
            if (c >= rank) {
                *t_out = __half2float(__ushort_as_half((unsigned short)(tid * 32 + j)));
                break;
            }
        }
    }
}

}  // namespace spqt

extern "C" spqt_status spqt_calibrate_threshold(const void* x, size_t count, double sparsity, float* threshold,
                                                void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace spqt;
    if (!threshold || !workspace || (count > 0 && !x)) return SPQT_ERR_INVALID_ARG;
    if (!(sparsity <= 1.0)) return SPQT_ERR_INVALID_ARG;   // also refuses NaN
    if (!aligned(x, 2) || !aligned(threshold, 4) || !aligned(workspace, 4)) return SPQT_ERR_ALIGNMENT;
    if (workspace_bytes < (size_t)kBins * sizeof(unsigned)) return SPQT_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (count > 0) {
        const unsigned blocks = (unsigned)(count < (size_t)256 * 1184 ? (count + 255) / 256 : 1184);
        calib_count_kernel<<<blocks, 256, 0, s>>>(static_cast<const unsigned short*>(x), count, static_cast<unsigned*>(workspace));
        count_launch();
    }
    calib_select_kernel<<<1, kCalibThreads, 0, s>>>(static_cast<unsigned*>(workspace), sparsity, threshold);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}
