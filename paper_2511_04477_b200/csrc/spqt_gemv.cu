// Activation-sparse GEMV over the zigzag layout, and its dense twin.
//
// Work decomposition (the paper's hybrid row/column parallelism): a grid of
// R block-rows x S workers.  Worker w of block-row r takes the even slice
// [w*count/S, (w+1)*count/S) of the ACTIVE index list (load balancing follows
// the active entries, not the matrix columns), streams the code blocks
// (r, idx[i]) with 128-bit loads, dequantizes in registers and accumulates the
// G partial outputs of the block-row in fp32.  Partials of the S workers are
// combined in a fixed order by whichever CTA of the block-row finishes last
// (arrive-only counter: nobody waits), which also adds the offset term and
// rounds to fp16.
//
// Arithmetic: with a = x_k * scale_rk (exact in fp32: 11-bit x 11-bit),
//   y[j] = sum_k a * code_jk  +  sum_k x_k * zero_rk
// and the second sum is one scalar per block-row, hoisted out of the inner loop.
// A 4-bit code is turned into an fp32 operand without any conversion: the
// nibble, masked in place at bit position p of an otherwise zero word, IS the
// fp32 subnormal code * 2^(p-149); the matching multiplier a * 2^(93-p) is an
// exact power-of-two rescale, so each product equals a*code*2^-56 up to the one
// rounding of the FMA.  One logic op and one FMA per weight.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;

static int g_tune_splits = 0;   // 0 = built-in rule
static int g_tune_ctas_per_sm = 0;

__device__ __forceinline__ uint4 ldg_stream_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// acc[0..7] += the eight codes of one 32-bit word, each times a * 2^-56.
// mul[j] = a * 2^(93 - 4j), j = 0..4.
__device__ __forceinline__ void fma_word(float* acc, unsigned w, const float* mul)
{
    const unsigned v = w >> 20;
    acc[0] = fmaf(__uint_as_float(w & 0x0000000fu), mul[0], acc[0]);
    acc[1] = fmaf(__uint_as_float(w & 0x000000f0u), mul[1], acc[1]);
    acc[2] = fmaf(__uint_as_float(w & 0x00000f00u), mul[2], acc[2]);
    acc[3] = fmaf(__uint_as_float(w & 0x0000f000u), mul[3], acc[3]);
    acc[4] = fmaf(__uint_as_float(w & 0x000f0000u), mul[4], acc[4]);
    acc[5] = fmaf(__uint_as_float(v & 0x0000000fu), mul[0], acc[5]);
    acc[6] = fmaf(__uint_as_float(v & 0x000000f0u), mul[1], acc[6]);
    acc[7] = fmaf(__uint_as_float(v & 0x00000f00u), mul[2], acc[7]);
}

// One step of a butterfly reduce-scatter: lanes that differ in bit `bit` hold
// partial sums of the same rows; each keeps one half of its N values and
// receives the partner's partials of that half.
template <int N>
__device__ __forceinline__ void halve(const float* in, float* out, int lane, int bit)
{
    const bool upper = (lane & bit) != 0;
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
        const float keep = upper ? in[i + N / 2] : in[i];
        const float send = upper ? in[i] : in[i + N / 2];
        out[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
    }
}

// 4-bit codes.  A block is B = G/2 bytes; LPB = B/16 lanes share one block, each
// loading 16 bytes = 32 codes, so a warp covers SLOTS = 32/LPB active columns
// per load instruction.  Lane (slot, h): byte 16h + 4c + b of the block holds
// row 16h+4c+b in its low nibble and row 16h+4c+b+G/2 in its high nibble.
template <int G, bool DENSE, int U>
__global__ void __launch_bounds__(kGemvThreads)
gemv_int4_kernel(const uint8_t* __restrict__ codes, const __half* __restrict__ scales,
                 const __half* __restrict__ zeros, int n,
                 const __half* __restrict__ x, const int32_t* __restrict__ idx,
                 const int32_t* __restrict__ count_ptr, __half* __restrict__ y,
                 int* __restrict__ counters, float* __restrict__ partials,
                 float* __restrict__ zpartials)
{
    constexpr int B = G / 2;
    constexpr int LPB = B / 16;
    constexpr int SLOTS = 32 / LPB;
    constexpr int KEEP = 32 / SLOTS;  // values per lane after the in-warp reduce-scatter

    __shared__ float red[kGemvWarps][G];
    __shared__ float zred[kGemvWarps];
    __shared__ int is_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = blockIdx.y, S = gridDim.x, wk = blockIdx.x;
    const int slot = lane / LPB, h = lane % LPB;

    const int count = DENSE ? n : *count_ptr;
    const int lo = (int)(((long long)wk * count) / S);
    const int hi = (int)(((long long)(wk + 1) * count) / S);

    const size_t row_base = (size_t)r * (size_t)n;
    const uint8_t* code_row = codes + row_base * B + 16 * h;
    const __half* s_row = scales + row_base;
    const __half* z_row = zeros + row_base;

    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
    float zs = 0.0f;

    // warps take interleaved chunks of U*SLOTS list entries
    for (int base = lo + warp * (U * SLOTS); base < hi; base += kGemvWarps * U * SLOTS) {
        uint4 wv[U];
        float a[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = base + u * SLOTS + slot;
            const bool ok = i < hi;
            wv[u] = make_uint4(0u, 0u, 0u, 0u);
            a[u] = 0.0f;
            if (ok) {
                const int k = DENSE ? i : __ldg(idx + i);
                wv[u] = ldg_stream_v4(code_row + (size_t)k * B);
                const float xf = __half2float(__ldg(x + k));
                a[u] = xf * __half2float(__ldg(s_row + k));          // exact
                if (h == 0) zs = fmaf(xf, __half2float(__ldg(z_row + k)), zs);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float mul[5];
            mul[0] = a[u] * 0x1p93f;
            mul[1] = a[u] * 0x1p89f;
            mul[2] = a[u] * 0x1p85f;
            mul[3] = a[u] * 0x1p81f;
            mul[4] = a[u] * 0x1p77f;
            fma_word(acc + 0, wv[u].x, mul);
            fma_word(acc + 8, wv[u].y, mul);
            fma_word(acc + 16, wv[u].z, mul);
            fma_word(acc + 24, wv[u].w, mul);
        }
    }

    // in-warp reduce-scatter over the column slots (lane bits above the LPB bits)
    float t16[16], t8[8], t4[4];
    halve<32>(acc, t16, lane, 16);
    halve<16>(t16, t8, lane, 8);
    halve<8>(t8, t4, lane, 4);
    float keep[4];
    int a_base;
    if (LPB == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) keep[i] = t4[i];
        a_base = lane & 0x1c;
    } else {
        float t2[2];
        halve<4>(t4, t2, lane, 2);
        keep[0] = t2[0];
        keep[1] = t2[1];
        a_base = lane & 0x1e;
    }
#pragma unroll
    for (int i = 0; i < KEEP; ++i) {
        const int ai = a_base + i;            // accumulator index = word*8 + nibble
        const int c = ai >> 3, e = ai & 7;
        const int row = 16 * h + 4 * c + (e >> 1) + (e & 1) * (G / 2);
        red[warp][row] = keep[i] * 0x1p56f;   // undo the 2^-56 of the subnormal trick
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) zs += __shfl_xor_sync(0xffffffffu, zs, o);
    if (lane == 0) zred[warp] = zs;
    __syncthreads();

    float* my_part = partials + ((size_t)r * S + wk) * G;
    if (tid < G) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < kGemvWarps; ++w) v += red[w][tid];
        __stcg(my_part + tid, v);
    }
    if (tid == G % kGemvThreads) {  // any one thread other than a row writer when G < threads
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < kGemvWarps; ++w) v += zred[w];
        __stcg(zpartials + (size_t)r * S + wk, v);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(counters + r, 1);
        is_last = (prev == S - 1);
    }
    __syncthreads();
    if (!is_last) return;

    // last CTA of this block-row: combine the S partials in worker order
    __threadfence();
    if (tid < G) {
        float v = 0.0f, zsum = 0.0f;
        const float* p = partials + (size_t)r * S * G + tid;
        const float* zp = zpartials + (size_t)r * S;
        for (int s = 0; s < S; ++s) {
            v += __ldcg(p + (size_t)s * G);
            zsum += __ldcg(zp + s);
        }
        y[(size_t)r * G + tid] = __float2half_rn(v + zsum);
    }
    if (tid == 0) counters[r] = 0;  // leave the workspace ready for the next call
}

struct GemvPlan {
    int S;
};

static GemvPlan plan(const Format& f, int cols_per_cta_iter)
{
    GemvPlan p;
    const int sms = sm_count() > 0 ? sm_count() : 148;
    const int per_sm = g_tune_ctas_per_sm > 0 ? g_tune_ctas_per_sm : 2;
    int S = g_tune_splits > 0 ? g_tune_splits : (sms * per_sm) / f.R;
    const int by_cols = (f.n + cols_per_cta_iter - 1) / cols_per_cta_iter;  // no empty workers when dense
    if (S > by_cols) S = by_cols;
    if (S > max_splits(f.R)) S = max_splits(f.R);
    if (S < 1) S = 1;
    p.S = S;
    return p;
}

template <int G, bool DENSE>
static spqt_status launch_int4(const Format& f, const void* codes, const void* scales,
                               const void* zeros, const void* x, const int32_t* idx,
                               const int32_t* count, void* y, void* workspace, cudaStream_t s)
{
    constexpr int U = 4;
    constexpr int SLOTS = 32 / (G / 32);
    const GemvPlan p = plan(f, kGemvWarps * SLOTS);
    int* counters = static_cast<int*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + counters_bytes(f.R));
    float* zpartials = partials + (size_t)f.R * p.S * G;
    dim3 grid(p.S, f.R);
    gemv_int4_kernel<G, DENSE, U><<<grid, kGemvThreads, 0, s>>>(
        static_cast<const uint8_t*>(codes), static_cast<const __half*>(scales),
        static_cast<const __half*>(zeros), f.n, static_cast<const __half*>(x), idx, count,
        static_cast<__half*>(y), counters, partials, zpartials);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

template <bool DENSE>
static spqt_status gemv_entry(const void* codes, const void* scales, const void* zeros,
                              int m, int n, int bits, int group, const void* x,
                              const int32_t* idx, const int32_t* count, void* y,
                              void* workspace, size_t ws_bytes, void* stream)
{
    if (!codes || !scales || !zeros || !x || !y || !workspace) return SPQT_ERR_INVALID_ARG;
    if (!DENSE && (!idx || !count)) return SPQT_ERR_INVALID_ARG;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (f.R > 65535) return SPQT_ERR_UNSUPPORTED;
    if (!aligned(codes, 16) || !aligned(scales, 16) || !aligned(zeros, 16) || !aligned(x, 2) ||
        !aligned(y, 2) || !aligned(workspace, 16) || (!DENSE && (!aligned(idx, 4) || !aligned(count, 4))))
        return SPQT_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(f)) return SPQT_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (bits == 4 && group == 128)
        return launch_int4<128, DENSE>(f, codes, scales, zeros, x, idx, count, y, workspace, s);
    if (bits == 4 && group == 64)
        return launch_int4<64, DENSE>(f, codes, scales, zeros, x, idx, count, y, workspace, s);
    return SPQT_ERR_UNSUPPORTED;
}

}  // namespace spqt

extern "C" {

spqt_status spqt_sparse_gemv(const void* codes, const void* scales, const void* zeros,
                             int m, int n, int bits, int group,
                             const void* x, const int32_t* idx, const int32_t* count,
                             void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::gemv_entry<false>(codes, scales, zeros, m, n, bits, group, x, idx, count, y,
                                   workspace, workspace_bytes, stream);
}

spqt_status spqt_dense_gemv(const void* codes, const void* scales, const void* zeros,
                            int m, int n, int bits, int group, const void* x,
                            void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::gemv_entry<true>(codes, scales, zeros, m, n, bits, group, x, nullptr, nullptr, y,
                                  workspace, workspace_bytes, stream);
}

spqt_status spqt_set_tuning(int splits_per_block_row, int ctas_per_sm)
{
    if (splits_per_block_row < 0 || ctas_per_sm < 0) return SPQT_ERR_INVALID_ARG;
    spqt::g_tune_splits = splits_per_block_row;
    spqt::g_tune_ctas_per_sm = ctas_per_sm;
    return SPQT_OK;
}

}  // extern "C"
