// Measurement aid, not part of the method: how fast this GPU can bring 64-byte blocks into shared
// memory with the copy instruction the GEMV uses (cp.async, 16 bytes per lane, four lanes per block,
// 64-byte L2 granularity), (0) for every block of a buffer, (1) for one randomly chosen half of every
// 128-byte line -- the access pattern of a sparse GEMV at 50 % block density.  The two figures are the
// achievable read and gather rooflines the benchmark prints next to the copy-bandwidth peak.
//
// A second probe measures the other ceiling of the GEMV loop: the dequantize-FMA arithmetic alone, on
// operands that already sit in shared memory (no copies, no list, no reduction), with the GEMV's own
// device functions.  Its rate, in 2 KB chunks per second, times the bytes a chunk stands for, is the
// bandwidth at which instruction issue alone would saturate.
#include "spqt_common.cuh"

namespace spqt {
constexpr unsigned long long kWaitNs = 1000000000ull;  // (the device header's bounded waits; unused here)
}
#include "spqt_gemv_device.cuh"

namespace spqt {

constexpr int kProbeWarps = 16;
constexpr int kArithStages = 3;          // 2 KB stages a warp cycles through, as in the GEMV
constexpr int kArithWarpBytes = kArithStages * 2048 + 256;   // + the chunk's 32 multiplier pairs

// Every warp runs `chunks` times the eight 512-byte steps of a full 4-bit chunk with groups of 128 rows.
__global__ void __launch_bounds__(kProbeWarps * 32, 1) probe_arith_kernel(int chunks, float* __restrict__ sink)
{
    extern __shared__ __align__(16) unsigned char probe_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned* words = reinterpret_cast<unsigned*>(probe_smem);
    for (int i = threadIdx.x; i < kProbeWarps * kArithWarpBytes / 4; i += blockDim.x) {
        unsigned h = (unsigned)(i + 1) * 2654435761u;
        words[i] = h ^ (h >> 13);       // arbitrary code bytes
    }
    __syncthreads();
    float* mf = reinterpret_cast<float*>(probe_smem + warp * kArithWarpBytes + kArithStages * 2048);
    for (int i = lane; i < 64; i += 32) mf[i] = 0x1p93f * (1.0f + (float)(i >> 1));   // pairs (a, a) * 2^93
    __syncwarp();
    const unsigned base = smem_u32(probe_smem) + warp * kArithWarpBytes;
    const unsigned mult_base = base + kArithStages * 2048;
    const int mslot = lane / 8;
    unsigned long long acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0ull;
    unsigned rc = 0;
#pragma unroll 1
    for (int it = 0; it < chunks; ++it) {
        const unsigned st_addr = base + rc;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const unsigned long long mm = lds_u64(mult_base + 8u * (u * 4 + mslot));
            const uint2 wv = lds_v2(st_addr + lane * 8 + u * 256);
            fma_block8_cum(acc, wv, mm);
        }
        __syncwarp();
        rc = (rc + 2048u == kArithStages * 2048u) ? 0u : rc + 2048u;
    }
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        unpack2(acc[i], lo, hi);
        s += lo + hi;
    }
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

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

extern "C" spqt_status spqt_probe_arith(int chunks_per_warp, float* sink, size_t sink_floats,
                                        unsigned long long* chunks_total, void* stream)
{
    using namespace spqt;
    if (!sink || !chunks_total || chunks_per_warp < 1) return SPQT_ERR_INVALID_ARG;
    if (!aligned(sink, 4)) return SPQT_ERR_ALIGNMENT;
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    if (sink_floats < (size_t)sms * kProbeWarps * 32) return SPQT_ERR_INVALID_ARG;
    const int smem = kProbeWarps * kArithWarpBytes;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(probe_arith_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    probe_arith_kernel<<<sms, kProbeWarps * 32, smem, static_cast<cudaStream_t>(stream)>>>(chunks_per_warp, sink);
    count_launch();
    *chunks_total = (unsigned long long)sms * kProbeWarps * (unsigned long long)chunks_per_warp;
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}
