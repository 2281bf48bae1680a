// Offline conversion: group-wise min/max quantization of fp16 weights and the
// zigzag block layout (groups run down G rows of one column; blocks stored
// row-major over (block-row, column)), plus the inverse of the layout step.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kPackCols = 32;     // columns of one block-row handled by a CTA
constexpr int kPackThreads = 256; // 8 warps, 4 columns each

// One CTA stages a G x 32 tile of W in shared memory with row-contiguous
// (coalesced) reads, then each warp quantizes four columns.  Lane l of a warp
// owns rows l, l+32, ... of the column.
template <int G, int BITS>
__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const __half* __restrict__ W, int n, int ldw,
            uint8_t* __restrict__ codes, __half2* __restrict__ scale_zero)
{
    constexpr int B = G * BITS / 8;
    constexpr int QMAX = (1 << BITS) - 1;
    constexpr int PER_LANE = G / 32;
    __shared__ __align__(16) __half tile[G][kPackCols + 2];
    __shared__ uint8_t q_sm[kPackThreads / 32][G];

    const int r = blockIdx.y;
    const int k0 = blockIdx.x * kPackCols;
    const int tid = threadIdx.x;

    // Stage the tile.  A row of the tile is 64 bytes: four 16-byte loads when W, ldw and the tile allow
    // it (the usual case), else one 2-byte load per weight.
    const bool vec = (reinterpret_cast<uintptr_t>(W) & 15) == 0 && (ldw & 7) == 0 && k0 + kPackCols <= n;
    if (vec) {
        static_assert(kPackCols == 32 && ((kPackCols + 2) * 2) % 4 == 0, "tile rows are copied as 32-bit words");
        for (int e = tid; e < G * 4; e += kPackThreads) {
            const int i = e >> 2, part = e & 3;
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(W + (size_t)(r * G + i) * ldw + k0) + part);
            unsigned* dst = reinterpret_cast<unsigned*>(&tile[i][part * 8]);  // rows start on a 4-byte boundary
            dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
        }
    } else {
        for (int e = tid; e < G * kPackCols; e += kPackThreads) {
            int i = e / kPackCols, c = e % kPackCols;
            int k = k0 + c;
            tile[i][c] = (k < n) ? W[(size_t)(r * G + i) * ldw + k] : __float2half(0.0f);
        }
    }
    __syncthreads();

    const int warp = tid / 32, lane = tid % 32;
    for (int cc = 0; cc < kPackCols / (kPackThreads / 32); ++cc) {
        const int c = warp * (kPackCols / (kPackThreads / 32)) + cc;
        const int k = k0 + c;
        if (k >= n) break;  // uniform across the warp
        float w[PER_LANE];
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int u = 0; u < PER_LANE; ++u) {
            w[u] = __half2float(tile[lane + 32 * u][c]);
            lo = fminf(lo, w[u]);
            hi = fmaxf(hi, w[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        // a zero extreme of either sign counts as +0.0 (x + (+0.0) is x, except that -0.0 becomes +0.0)
        lo = __fadd_rn(lo, 0.0f);
        hi = __fadd_rn(hi, 0.0f);
        // scale = fp16((max - min) / qmax): one IEEE subtract, one IEEE divide, RN-even
        const float s32 = __fdiv_rn(__fsub_rn(hi, lo), (float)QMAX);
        const __half sh = __float2half_rn(s32);
        const float sf = __half2float(sh);
        // w - lo >= 0 exactly, so the rounded quotient needs no lower clamp; round-to-nearest-even
        // conversion and one integer min give the code
        int code[PER_LANE];
#pragma unroll
        for (int u = 0; u < PER_LANE; ++u)
            code[u] = (sf != 0.0f) ? min(__float2int_rn(__fdiv_rn(__fsub_rn(w[u], lo), sf)), QMAX) : 0;
        const size_t blk = (size_t)r * n + k;
        uint8_t* out = codes + blk * B;
        if (BITS == 4) {
            // lane l owns rows l, l+32, ...: byte i pairs rows i and i + G/2, both of the same lane
#pragma unroll
            for (int u = 0; u < PER_LANE / 2; ++u)
                out[lane + 32 * u] = (uint8_t)(code[u] | (code[u + PER_LANE / 2] << 4));
        } else {
#pragma unroll
            for (int u = 0; u < PER_LANE; ++u) q_sm[warp][lane + 32 * u] = (uint8_t)code[u];
            __syncwarp();
            for (int b = lane; b < B; b += 32) {
                unsigned v = 0;
                if (b < G / 4) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) v |= (q_sm[warp][b + u * (G / 4)] & 3u) << (2 * u);
                } else {
                    const int j = b - G / 4;
#pragma unroll
                    for (int u = 0; u < 8; ++u) v |= ((q_sm[warp][j + u * (G / 8)] >> 2) & 1u) << u;
                }
                out[b] = (uint8_t)v;
            }
        }
        if (lane == 0) scale_zero[blk] = __halves2half2(sh, __float2half_rn(lo));  // exact: lo is an fp16 value
        __syncwarp();
    }
}

// 4-bit codes, one THREAD per column: a CTA stages a G x 128 tile with 16-byte loads, then thread c
// walks down column c twice (min/max, then codes), so that nothing crosses lanes and the per-column
// work (scale, offset, stores) is done by all lanes at once.  A thread writes its block with 16-byte
// stores.  Same arithmetic as pack_kernel, bit for bit.  Used for G = 64 when W, ldw and n allow the
// vector loads.
constexpr int kPack4Cols = 128;

template <int G>
__global__ void __launch_bounds__(kPack4Cols)
pack4_kernel(const __half* __restrict__ W, int n, int ldw,
             uint8_t* __restrict__ codes, __half2* __restrict__ scale_zero)
{
    constexpr int B = G / 2;
    constexpr int QMAX = 15;
    constexpr int kStride = kPack4Cols + 8;  // halves per tile row: keeps rows 16-byte aligned
    __shared__ __align__(16) __half tile[G][kStride];

    const int r = blockIdx.y;
    const int k0 = blockIdx.x * kPack4Cols;
    const int tid = threadIdx.x;
    const int cols = min(kPack4Cols, n - k0);  // a multiple of 8 (the host checks n)

    // 16 chunks of 8 halves per tile row
    for (int e = tid; e < G * (kPack4Cols / 8); e += kPack4Cols) {
        const int i = e / (kPack4Cols / 8), part = e % (kPack4Cols / 8);
        if (part * 8 < cols)
            *reinterpret_cast<uint4*>(&tile[i][part * 8]) =
                __ldg(reinterpret_cast<const uint4*>(W + (size_t)(r * G + i) * ldw + k0) + part);
    }
    __syncthreads();
    if (tid >= cols) return;

    // minimum and maximum of the column: exact in fp16
    __half lo_h = tile[0][tid], hi_h = lo_h;
#pragma unroll 8
    for (int i = 1; i < G; ++i) {
        const __half v = tile[i][tid];
        lo_h = __hmin(lo_h, v);
        hi_h = __hmax(hi_h, v);
    }
    // a zero extreme of either sign counts as +0.0
    const float lo = __fadd_rn(__half2float(lo_h), 0.0f), hi = __fadd_rn(__half2float(hi_h), 0.0f);
    // scale = fp16((max - min) / qmax): one IEEE subtract, one IEEE divide, RN-even
    const __half sh = __float2half_rn(__fdiv_rn(__fsub_rn(hi, lo), (float)QMAX));
    const float sf = __half2float(sh);
    const size_t blk = (size_t)r * n + k0 + tid;
    uint4* out = reinterpret_cast<uint4*>(codes + blk * B);
    // byte i = code of row i | code of row i + G/2 << 4; sixteen bytes per store
#pragma unroll 1
    for (int q = 0; q < B / 16; ++q) {
        unsigned wds[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int i = q * 16 + j;
            const float a = __half2float(tile[i][tid]), b = __half2float(tile[i + G / 2][tid]);
            int ca = 0, cb = 0;
            if (sf != 0.0f) {
                // w - lo >= 0 exactly: no lower clamp; round-to-nearest-even conversion and one integer min
                ca = min(__float2int_rn(__fdiv_rn(__fsub_rn(a, lo), sf)), QMAX);
                cb = min(__float2int_rn(__fdiv_rn(__fsub_rn(b, lo), sf)), QMAX);
            }
            wds[j >> 2] |= (unsigned)(ca | (cb << 4)) << (8 * (j & 3));
        }
        out[q] = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    }
    scale_zero[blk] = __halves2half2(sh, __float2half_rn(lo));
}

// One thread per weight: read its code out of the zigzag buffer.
template <int G, int BITS>
__global__ void unpack_kernel(const uint8_t* __restrict__ codes, int m, int n, uint8_t* __restrict__ q)
{
    constexpr int B = G * BITS / 8;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (size_t)m * n) return;
    const int j = (int)(e / n), k = (int)(e % n);
    const int r = j / G, i = j % G;
    const uint8_t* blk = codes + ((size_t)r * n + k) * B;
    int code;
    if (BITS == 4) {
        code = (i < G / 2) ? (blk[i] & 15) : (blk[i - G / 2] >> 4);
    } else {
        const int low2 = (blk[i % (G / 4)] >> (2 * (i / (G / 4)))) & 3;
        const int top1 = (blk[G / 4 + i % (G / 8)] >> (i / (G / 8))) & 1;
        code = low2 | (top1 << 2);
    }
    q[e] = (uint8_t)code;
}

template <int G, int BITS>
static spqt_status launch_pack(const Format& f, const void* W, int ldw, void* codes, void* scale_zero,
                               cudaStream_t s)
{
    // (with G = 128 its 34 KB tile per 128 threads leaves too few warps per SM to hide the division
    // chains, and the warp-per-column kernel below is faster)
    if (BITS == 4 && G == 64 && (reinterpret_cast<uintptr_t>(W) & 15) == 0 && (ldw & 7) == 0 && (f.n & 7) == 0) {
        dim3 grid4((f.n + kPack4Cols - 1) / kPack4Cols, f.R);
        pack4_kernel<G><<<grid4, kPack4Cols, 0, s>>>(
            static_cast<const __half*>(W), f.n, ldw, static_cast<uint8_t*>(codes),
            static_cast<__half2*>(scale_zero));
        count_launch();
        return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
    }
    dim3 grid((f.n + kPackCols - 1) / kPackCols, f.R);
    pack_kernel<G, BITS><<<grid, kPackThreads, 0, s>>>(
        static_cast<const __half*>(W), f.n, ldw, static_cast<uint8_t*>(codes),
        static_cast<__half2*>(scale_zero));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

template <int G, int BITS>
static spqt_status launch_unpack(const Format& f, const void* codes, void* q, cudaStream_t s)
{
    const size_t total = (size_t)f.m * f.n;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    unpack_kernel<G, BITS><<<blocks, 256, 0, s>>>(static_cast<const uint8_t*>(codes), f.m, f.n,
                                                  static_cast<uint8_t*>(q));
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

}  // namespace spqt

extern "C" {

spqt_status spqt_pack(const void* W, int m, int n, int ldw, int bits, int group,
                      void* codes, void* scale_zero, void* stream)
{
    using namespace spqt;
    if (!W || !codes || !scale_zero) return SPQT_ERR_INVALID_ARG;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (ldw < n) return SPQT_ERR_INVALID_ARG;
    if (f.R > 65535) return SPQT_ERR_UNSUPPORTED;
    if (!aligned(W, 2) || !aligned(codes, 16) || !aligned(scale_zero, 16))
        return SPQT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (bits == 4 && group == 128) return launch_pack<128, 4>(f, W, ldw, codes, scale_zero, s);
    if (bits == 4 && group == 64) return launch_pack<64, 4>(f, W, ldw, codes, scale_zero, s);
    if (bits == 3 && group == 128) return launch_pack<128, 3>(f, W, ldw, codes, scale_zero, s);
    return launch_pack<64, 3>(f, W, ldw, codes, scale_zero, s);
}

spqt_status spqt_unpack(const void* codes, int m, int n, int bits, int group, void* q_u8, void* stream)
{
    using namespace spqt;
    if (!codes || !q_u8) return SPQT_ERR_INVALID_ARG;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (((size_t)m * n + 255) / 256 > 0x7fffffffu) return SPQT_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (bits == 4 && group == 128) return launch_unpack<128, 4>(f, codes, q_u8, s);
    if (bits == 4 && group == 64) return launch_unpack<64, 4>(f, codes, q_u8, s);
    if (bits == 3 && group == 128) return launch_unpack<128, 3>(f, codes, q_u8, s);
    return launch_unpack<64, 3>(f, codes, q_u8, s);
}

}  // extern "C"
