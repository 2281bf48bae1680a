// Comparison baseline: the conventional ROW-WISE grouping the paper contrasts its layout with (Sec. 2,
// Sec. 4.1.1: a quantization group is G consecutive weights of one row, which suits a row-parallel GEMV
// but scatters a sparse column over every group it crosses) and a dense 4-bit GEMV over it.  Same
// quantizer as the zigzag layout (min/max, round to nearest, fp16 scale and offset), same byte rule
// inside a block; only the axis of the groups and the block order differ:
//   block (j, g) = the codes of columns g*G .. g*G+G-1 of row j, at byte (j*(n/G) + g) * G/2;
//   scale_zero[j*(n/G) + g] = its (scale, zero) pair.
//
// rowwise_gemv_kernel: row-parallel.  A warp owns a slice of 1024 columns (512 bytes of codes per row),
// lane l bytes 16l..16l+15 of it, i.e. 32 codes of one group; the lane keeps the 32 matching x values in
// registers for the whole launch, already scaled for the conversion-free dequantization (a nibble masked
// in place is an fp32 subnormal; the multiplier carries the matching power of two).  The ceil(n/1024)
// warps that cover a row form a row group; a CTA holds as many row groups as fit into 16 warps.  A row
// group walks over chunks of ROWS rows: the chunk's codes and (scale, zero) pairs arrive through a
// three-stage cp.async ring per warp; per row a lane forms sum(code * x) of its 32 codes, applies its
// group's scale and adds zero * sum(x); the ROWS values are reduced across the warp by a butterfly
// reduce-scatter, across the row group's warps through a ring of shared-memory buffers guarded by
// mbarriers (bounded waits), added by the group's first warp in warp order: bit-reproducible.
#include <cstddef>

#include "spqt_common.cuh"

namespace spqt {
constexpr unsigned long long kWaitNs = 1000000000ull;
}
#include "spqt_gemv_device.cuh"

namespace spqt {

constexpr int kRwWarps = 16;
constexpr int kRwThreads = kRwWarps * 32;
constexpr int kRwDepth = 3;          // chunks in flight per warp
constexpr int kRwStep = 512;         // bytes of one row's codes a warp covers (1024 columns)
constexpr int kRwMaxN = kRwWarps * 1024;
constexpr int kRwParts = 4;          // chunks whose per-warp sums may wait to be added

// ---------------------------------------------------------------- conversion

// One warp per block (row j, group g): lane l owns columns l, l+32, .. of the group.
template <int G>
__global__ void __launch_bounds__(256)
rowwise_pack_kernel(const __half* __restrict__ W, int m, int n, int ldw, uint8_t* __restrict__ codes,
                    __half2* __restrict__ scale_zero)
{
    constexpr int PER = G / 32;
    const int lane = threadIdx.x & 31;
    const int ng = n / G;
    const long long total = (long long)m * ng;
    const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long b = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); b < total; b += warps) {
        const int j = (int)(b / ng), g = (int)(b % ng);
        const __half* src = W + (size_t)j * ldw + (size_t)g * G;
        float w[PER];
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            w[u] = __half2float(src[lane + 32 * u]);
            lo = fminf(lo, w[u]);
            hi = fmaxf(hi, w[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        lo = __fadd_rn(lo, 0.0f);  // a zero extreme of either sign counts as +0.0
        hi = __fadd_rn(hi, 0.0f);
        const __half sh = __float2half_rn(__fdiv_rn(__fsub_rn(hi, lo), 15.0f));
        const float sf = __half2float(sh);
        int c[PER];
#pragma unroll
        for (int u = 0; u < PER; ++u)
            c[u] = (sf != 0.0f) ? min(__float2int_rn(__fdiv_rn(__fsub_rn(w[u], lo), sf)), 15) : 0;
        // byte i = code i | code i+G/2 << 4
        uint8_t* dst = codes + (size_t)b * (G / 2);
        if (G == 128) {
            dst[lane] = (uint8_t)(c[0] | (c[2 % PER] << 4));
            dst[lane + 32] = (uint8_t)(c[1] | (c[3 % PER] << 4));
        } else {
            dst[lane] = (uint8_t)(c[0] | (c[1] << 4));
        }
        if (lane == 0) scale_zero[b] = __halves2half2(sh, __float2half_rn(lo));
    }
}

// ---------------------------------------------------------------- GEMV

template <int G, int ROWS>
struct RwSmem {
    static constexpr int NG = 1024 / G;  // groups of a row inside a warp's slice
    struct Stage {
        alignas(16) unsigned char codes[ROWS][kRwStep];
        alignas(16) unsigned meta[ROWS][NG];
    };
    Stage stage[kRwWarps][kRwDepth];
    float part[kRwParts][kRwWarps][ROWS];   // per-warp sums of a chunk's rows: a ring of kRwParts chunks
    uint64_t full[kRwWarps][kRwParts];      // per row group: every warp of the group has written its sums
    uint64_t empty[kRwWarps][kRwParts];     // per row group: the summing warp has read them
};

// Sums of ROWS values per lane -> one row's sum over the warp in the lanes with (lane & (32/ROWS - 1)) == 0;
// `row` = which row that lane holds.
template <int ROWS>
__device__ __forceinline__ float reduce_rows(const float* v, int lane, int* row)
{
    float r;
    if (ROWS == 8) {
        float a4[4], a2[2], a1[1];
        halve<8>(v, a4, lane, 16);
        halve<4>(a4, a2, lane, 8);
        halve<2>(a2, a1, lane, 4);
        r = a1[0];
        r += __shfl_xor_sync(0xffffffffu, r, 2);
        r += __shfl_xor_sync(0xffffffffu, r, 1);
        *row = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
    } else if (ROWS == 4) {
        float a2[2], a1[1];
        halve<4>(v, a2, lane, 16);
        halve<2>(a2, a1, lane, 8);
        r = a1[0];
        r += __shfl_xor_sync(0xffffffffu, r, 4);
        r += __shfl_xor_sync(0xffffffffu, r, 2);
        r += __shfl_xor_sync(0xffffffffu, r, 1);
        *row = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
    } else {
        float a1[1];
        halve<2>(v, a1, lane, 16);
        r = a1[0];
        r += __shfl_xor_sync(0xffffffffu, r, 8);
        r += __shfl_xor_sync(0xffffffffu, r, 4);
        r += __shfl_xor_sync(0xffffffffu, r, 2);
        r += __shfl_xor_sync(0xffffffffu, r, 1);
        *row = (lane >> 4) & 1;
    }
    return r;
}

template <int G, int ROWS>
__global__ void __launch_bounds__(kRwThreads, 1)
rowwise_gemv_kernel(const uint8_t* __restrict__ codes, const unsigned* __restrict__ meta, int m, int n,
                    const __half* __restrict__ x, __half* __restrict__ y, int Wc, int Rg, int sparse, float thr)
{
    using Smem = RwSmem<G, ROWS>;
    constexpr int B = G / 2, NG = Smem::NG, D = kRwDepth;
    extern __shared__ __align__(16) unsigned char rw_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(rw_raw);
    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    if (threadIdx.x < kRwWarps * kRwParts) {
        mbar_init(&sm.full[0][0] + threadIdx.x, (unsigned)Wc);
        mbar_init(&sm.empty[0][0] + threadIdx.x, 1u);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    if (warp >= Wc * Rg) return;
    const int rg = warp / Wc, cw = warp - rg * Wc;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int ng = n / G;
    const size_t row_bytes = (size_t)n >> 1;
    // this lane's 32 codes: bytes i0 .. i0+15 of block `blk` of the warp's slice; byte t holds the codes of
    // columns c_lo + t (low nibble) and c_lo + t + G/2 (high nibble)
    const int blk = (16 * lane) / B, i0 = (16 * lane) % B;
    const int c_lo = cw * 1024 + blk * G + i0;
    const bool live = c_lo < n;  // n is a multiple of G: a lane's block lies wholly inside or outside the row
    // where this lane copies from (lanes outside the row copy their slice's first bytes and multiply by 0)
    const size_t code_off = (size_t)cw * kRwStep + (live ? (size_t)lane * 16 : 0);
    const int meta_g = (lane < NG && cw * NG + lane < ng) ? cw * NG + lane : cw * NG;

    const unsigned stage0 = smem_u32(&sm.stage[warp][0]);
    constexpr unsigned kStageBytes = (unsigned)sizeof(typename Smem::Stage);
    constexpr unsigned kMetaOff = (unsigned)(ROWS * kRwStep);

    const int chunks = (m + ROWS - 1) / ROWS;
    const int stride = (int)gridDim.x * Rg;
    auto issue = [&](int t, int st) {
        if (t < chunks) {
            const unsigned sa = stage0 + (unsigned)st * kStageBytes;
#pragma unroll
            for (int i = 0; i < ROWS; ++i) {
                const int row = min(t * ROWS + i, m - 1);
                cp_async_16(sa + (unsigned)i * kRwStep + (unsigned)lane * 16u, codes + (size_t)row * row_bytes + code_off);
                if (lane < NG) cp_async_4(sa + kMetaOff + (unsigned)(i * NG + lane) * 4u, meta + (size_t)row * ng + meta_g);
            }
        }
        cp_async_commit();
    };

    int t = (int)blockIdx.x * Rg + rg;
#pragma unroll
    for (int d = 0; d < D; ++d) issue(t + d * stride, d);
    // the lane's 32 values of x, as multipliers (the first chunks are on their way meanwhile)
    unsigned long long xm[16];
    float xs = 0.0f;
    {
        unsigned short xl[16], xh[16];
        if (live && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
            const uint4* pl = reinterpret_cast<const uint4*>(x + c_lo);
            const uint4* ph = reinterpret_cast<const uint4*>(x + c_lo + G / 2);
            const uint4 v[4] = {__ldg(pl), __ldg(pl + 1), __ldg(ph), __ldg(ph + 1)};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const unsigned wl[4] = {v[h].x, v[h].y, v[h].z, v[h].w};
                const unsigned wh[4] = {v[2 + h].x, v[2 + h].y, v[2 + h].z, v[2 + h].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    xl[8 * h + 2 * e] = (unsigned short)(wl[e] & 0xffffu);
                    xl[8 * h + 2 * e + 1] = (unsigned short)(wl[e] >> 16);
                    xh[8 * h + 2 * e] = (unsigned short)(wh[e] & 0xffffu);
                    xh[8 * h + 2 * e + 1] = (unsigned short)(wh[e] >> 16);
                }
            }
        } else {
            const unsigned short* xb = reinterpret_cast<const unsigned short*>(x);
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                xl[t] = live ? __ldg(xb + c_lo + t) : (unsigned short)0;
                xh[t] = live ? __ldg(xb + c_lo + t + G / 2) : (unsigned short)0;
            }
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            // the thresholded call: entries with |x| <= threshold (and NaN) count as zero -- the row-wise
            // layout cannot skip their bytes, only their contribution
            float fl = __half2float(__ushort_as_half(xl[t])), fh = __half2float(__ushort_as_half(xh[t]));
            if (sparse) {
                fl = fabsf(fl) > thr ? fl : 0.0f;
                fh = fabsf(fh) > thr ? fh : 0.0f;
            }
            xs += fl + fh;
            // nibble positions of byte t inside its 32-bit word (after the shift by 16 for bytes 2 and 3):
            // bits 0 and 4 (even byte) or 8 and 12 (odd byte); multiplier = x * 2^(93 - position)
            xm[t] = (t & 1) ? pack2(fl * 0x1p85f, fh * 0x1p81f) : pack2(fl * 0x1p93f, fh * 0x1p89f);
        }
    }
    int st = 0;
    unsigned k = 0;  // chunks this row group has finished
    for (; t < chunks; t += stride) {
        cp_async_wait<D - 1>();
        __syncwarp();
        const unsigned sa = stage0 + (unsigned)st * kStageBytes;
        float val[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            const uint4 wv = lds_v4(sa + (unsigned)i * kRwStep + (unsigned)lane * 16u);
            const unsigned mz = lds_u32(sa + kMetaOff + (unsigned)(i * NG + blk) * 4u);
            const unsigned wd[4] = {wv.x, wv.y, wv.z, wv.w};
            unsigned long long acc[2] = {0ull, 0ull};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const unsigned w = wd[q], v = w >> 16;
                ffma2(acc[q & 1], pack2(__uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000f0u)), xm[4 * q + 0]);
                ffma2(acc[q & 1], pack2(__uint_as_float(w & 0x00000f00u), __uint_as_float(w & 0x0000f000u)), xm[4 * q + 1]);
                ffma2(acc[q & 1], pack2(__uint_as_float(v & 0x0000000fu), __uint_as_float(v & 0x000000f0u)), xm[4 * q + 2]);
                ffma2(acc[q & 1], pack2(__uint_as_float(v & 0x00000f00u), __uint_as_float(v & 0x0000f000u)), xm[4 * q + 3]);
            }
            float p0, p1, p2, p3;
            unpack2(acc[0], p0, p1);
            unpack2(acc[1], p2, p3);
            const float dot = (p0 + p1) + (p2 + p3);  // sum(code * x) * 2^-56
            const float sc = __half2float(__ushort_as_half((unsigned short)(mz & 0xffffu))) * 0x1p56f;  // exact
            const float ze = __half2float(__ushort_as_half((unsigned short)(mz >> 16)));
            val[i] = fmaf(dot, sc, ze * xs);
        }
        __syncwarp();
        issue(t + D * stride, st);
        st = (st + 1 == D) ? 0 : st + 1;

        int row_in_chunk;
        const float r = reduce_rows<ROWS>(val, lane, &row_in_chunk);
        const bool holder = (lane & (32 / ROWS - 1)) == 0;
        if (Wc == 1) {
            const int row = t * ROWS + row_in_chunk;
            if (holder && row < m) y[row] = __float2half_rn(r);
            continue;
        }
        // hand the warp's sums to the row group's first warp through a ring of kRwParts chunks: nobody
        // waits for the slowest warp of a chunk except the one that adds them up
        const unsigned b = k % kRwParts, ph = (k / kRwParts) & 1u;
        if (k >= kRwParts && !mbar_wait(&sm.empty[rg][b], ph ^ 1u)) break;  // (bounded: never hangs)
        if (holder) sm.part[b][warp][row_in_chunk] = r;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.full[rg][b]);
        if (cw == 0) {
            if (!mbar_wait(&sm.full[rg][b], ph)) break;
            if (lane < ROWS) {
                float s = 0.0f;
                for (int w = 0; w < Wc; ++w) s += sm.part[b][rg * Wc + w][lane];
                const int row = t * ROWS + lane;
                if (row < m) y[row] = __float2half_rn(s);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[rg][b]);
        }
        ++k;
    }
    cp_async_wait<0>();
}

// ---------------------------------------------------------------- host side

static spqt_status rowwise_format(int m, int n, int bits, int group)
{
    if (m <= 0 || n <= 0) return SPQT_ERR_INVALID_ARG;
    if (bits != 4) return SPQT_ERR_UNSUPPORTED;
    if (group != 64 && group != 128) return SPQT_ERR_UNSUPPORTED;
    if (n % group != 0) return SPQT_ERR_UNSUPPORTED;
    return SPQT_OK;
}

template <int G, int ROWS>
static spqt_status launch_rowwise(const void* codes, const void* meta, int m, int n, const void* x, void* y,
                                  int Wc, int Rg, int sms, int sparse, float thr, cudaStream_t s)
{
    auto kernel = rowwise_gemv_kernel<G, ROWS>;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(RwSmem<G, ROWS>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    const int chunks = (m + ROWS - 1) / ROWS;
    int P = (chunks + Rg - 1) / Rg;
    if (P > sms) P = sms;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(P);
    cfg.blockDim = dim3(kRwThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, static_cast<const uint8_t*>(codes), static_cast<const unsigned*>(meta),
                                               m, n, static_cast<const __half*>(x), static_cast<__half*>(y), Wc, Rg, sparse, thr);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

template <int G>
static spqt_status dispatch_rowwise(const void* codes, const void* meta, int m, int n, const void* x, void* y, int sparse, float thr,
                                    cudaStream_t s)
{
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    const int Wc = (n + 1023) / 1024;
    int Rg = kRwWarps / Wc;
    if (Wc > 1 && Rg > 8) Rg = 8;
    // the largest chunk of rows that still gives every row group of a full grid a chunk
    const long long groups = (long long)sms * Rg;
    if ((m + 7) / 8 >= groups) return launch_rowwise<G, 8>(codes, meta, m, n, x, y, Wc, Rg, sms, sparse, thr, s);
    if ((m + 3) / 4 >= groups) return launch_rowwise<G, 4>(codes, meta, m, n, x, y, Wc, Rg, sms, sparse, thr, s);
    return launch_rowwise<G, 2>(codes, meta, m, n, x, y, Wc, Rg, sms, sparse, thr, s);
}

}  // namespace spqt

extern "C" {

spqt_status spqt_rowwise_packed_sizes(int m, int n, int bits, int group, size_t* codes_bytes, size_t* scale_zero_bytes)
{
    const spqt_status st = spqt::rowwise_format(m, n, bits, group);
    if (st != SPQT_OK) return st;
    if (codes_bytes) *codes_bytes = (size_t)m * (size_t)n / 2;
    if (scale_zero_bytes) *scale_zero_bytes = (size_t)m * (size_t)(n / group) * 4;
    return SPQT_OK;
}

spqt_status spqt_rowwise_pack(const void* W, int m, int n, int ldw, int bits, int group, void* codes, void* scale_zero,
                              void* stream)
{
    if (!W || !codes || !scale_zero) return SPQT_ERR_INVALID_ARG;
    const spqt_status st = spqt::rowwise_format(m, n, bits, group);
    if (st != SPQT_OK) return st;
    if (ldw < n) return SPQT_ERR_INVALID_ARG;
    if (!spqt::aligned(W, 2) || !spqt::aligned(codes, 16) || !spqt::aligned(scale_zero, 16)) return SPQT_ERR_ALIGNMENT;
    const long long blocks = (long long)m * (n / group);
    long long grid = (blocks + 7) / 8;
    if (grid > 65536) grid = 65536;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (group == 128)
        spqt::rowwise_pack_kernel<128><<<(unsigned)grid, 256, 0, s>>>(static_cast<const __half*>(W), m, n, ldw,
                                                                      static_cast<uint8_t*>(codes), static_cast<__half2*>(scale_zero));
    else
        spqt::rowwise_pack_kernel<64><<<(unsigned)grid, 256, 0, s>>>(static_cast<const __half*>(W), m, n, ldw,
                                                                     static_cast<uint8_t*>(codes), static_cast<__half2*>(scale_zero));
    spqt::count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

static spqt_status rowwise_entry(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                 const void* x, void* y, int sparse, float t, void* stream)
{
    if (!codes || !scale_zero || !x || !y) return SPQT_ERR_INVALID_ARG;
    const spqt_status st = spqt::rowwise_format(m, n, bits, group);
    if (st != SPQT_OK) return st;
    if (n > spqt::kRwMaxN) return SPQT_ERR_UNSUPPORTED;
    if (!spqt::aligned(codes, 16) || !spqt::aligned(scale_zero, 16) || !spqt::aligned(x, 2) || !spqt::aligned(y, 2))
        return SPQT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return group == 128 ? spqt::dispatch_rowwise<128>(codes, scale_zero, m, n, x, y, sparse, t, s)
                        : spqt::dispatch_rowwise<64>(codes, scale_zero, m, n, x, y, sparse, t, s);
}

spqt_status spqt_rowwise_dense_gemv(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                    const void* x, void* y, void* stream)
{
    return rowwise_entry(codes, scale_zero, m, n, bits, group, x, y, 0, 0.0f, stream);
}

spqt_status spqt_rowwise_thresholded_gemv(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                          const void* x, float t, void* y, void* stream)
{
    return rowwise_entry(codes, scale_zero, m, n, bits, group, x, y, 1, t, stream);
}

}  // extern "C"
