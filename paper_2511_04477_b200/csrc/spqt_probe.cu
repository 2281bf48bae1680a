// Measurement aid, not part of the method: how fast this GPU can bring 64-byte blocks into shared
// memory with the copy instruction the GEMV uses (cp.async, 16 bytes per lane, four lanes per block,
// 64-byte L2 granularity), (0) for every block of a buffer, (1) for one randomly chosen half of every
// 128-byte line -- the access pattern of a sparse GEMV at 50 % block density.  The two figures are the
// achievable read and gather rooflines the benchmark prints next to the copy-bandwidth peak.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kProbeWarps = 16;

__device__ __forceinline__ unsigned probe_hash(unsigned x)
{
    x ^= x >> 16; x *= 0x7feb352dU; x ^= x >> 15; x *= 0x846ca68bU; x ^= x >> 16;
    return x;
}

__global__ void __launch_bounds__(kProbeWarps * 32, 1)
probe_kernel(const uint8_t* __restrict__ src, unsigned long long blocks_per_warp, int pattern,
             unsigned long long* __restrict__ moved)
{
    extern __shared__ __align__(16) unsigned char probe_smem[];  // [warps][3 stages][2 KB]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long w = (unsigned long long)blockIdx.x * kProbeWarps + warp;
    const uint8_t* base = src + w * blocks_per_warp * 64;
    const int slot = lane >> 2, part = lane & 3;
    const unsigned long long nsel = pattern == 0 ? blocks_per_warp : blocks_per_warp / 2;
    unsigned long long bytes = 0;
    int stage = 0;
    for (unsigned long long j0 = 0; j0 + 32 <= nsel; j0 += 32) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned long long j = j0 + slot + 8 * u;
            const unsigned long long c = pattern == 0 ? j : 2 * j + (probe_hash((unsigned)(w * 1315423911u + j)) & 1u);
            const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(
                probe_smem + ((warp * 3 + stage) * 2048 + (slot + 8 * u) * 64 + part * 16)));
            asm volatile("cp.async.cg.shared.global.L2::64B [%0], [%1], 16;" ::"r"(dst), "l"(base + c * 64 + part * 16)
                         : "memory");
            if (part == 0) bytes += 64;
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 2;" ::: "memory");
        stage = stage == 2 ? 0 : stage + 1;
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, o);
    if (lane == 0) atomicAdd(moved, bytes);
}

}  // namespace spqt

extern "C" spqt_status spqt_probe_read(const void* buf, size_t bytes, int pattern,
                                       unsigned long long* moved, void* stream)
{
    using namespace spqt;
    if (!buf || !moved || (pattern != 0 && pattern != 1)) return SPQT_ERR_INVALID_ARG;
    if (!aligned(buf, 128) || !aligned(moved, 8)) return SPQT_ERR_ALIGNMENT;
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    const unsigned long long per_warp = bytes / 64 / ((unsigned long long)sms * kProbeWarps);
    if (per_warp < 64) return SPQT_ERR_INVALID_ARG;  // too small to measure anything
    const int smem = kProbeWarps * 3 * 2048;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    probe_kernel<<<sms, kProbeWarps * 32, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(buf), per_warp & ~1ull, pattern, moved);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}
