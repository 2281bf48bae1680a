// Small batch (2..8 decode rows at once: beams, speculative tokens): the sparse product over the UNION
// of the rows' active sets, and its dense twin.  Every active block is fetched once for the whole
// batch and its codes are extracted once; only the FMAs are repeated per row, so the byte and the
// integer-instruction cost per row falls with the batch size.
//
//   sparsify_rows_kernel    (spqt_sparsify.cu) one CTA; "active" = |X[b][k]| > t in at least one row b.
//   gemm_small_kernel       grid (S, R): CTA (s, r) takes the s-th of S equal slices of the union list
//                           for block-row r; its 8 warps take the slice's chunks of 32 entries in turn,
//                           each with three chunk buffers (the next chunks' copies fly during the
//                           arithmetic).  Lane e of a chunk holds entry e: it loads the entry's column,
//                           its (scale, zero) pair and the batch's x values and writes the packed
//                           multiplier pairs of every row; then the warp does the dequantize-FMA work,
//                           four rows per pass.  Partial sums go warp -> CTA (shared memory) -> block-row
//                           (fp32 partials in the workspace, arrive-only counter, the last CTA adds them
//                           in slice order: bit-reproducible).
// Batches of 5..8 rows run as two passes of up to four rows over the same union list.
#include <cstddef>

#include "spqt_common.cuh"

namespace spqt {
constexpr unsigned long long kWaitNs = 1000000000ull;
}
#include "spqt_gemv_device.cuh"

namespace spqt {

constexpr int kSmallWarps = 8;
constexpr int kSmallThreads = kSmallWarps * 32;
constexpr int kSmallRows = 4;      // batch rows per pass at most (a pass of one or two rows keeps two sets of sums)
constexpr int kSmallMaxSplit = 8;  // slices per block-row at most
constexpr int kSmallChunk = 32;    // list entries per chunk
#ifndef SPQT_SMALL_DEPTH
#define SPQT_SMALL_DEPTH 3
#endif
constexpr int kSmallDepth = SPQT_SMALL_DEPTH;     // chunk buffers per warp

template <int G, int BITS, int ROWS>
struct SmallSmem {
    static constexpr int B = G * BITS / 8;
    alignas(16) unsigned char codes[kSmallWarps][kSmallDepth][kSmallChunk * B];
    alignas(16) float mult[kSmallWarps][kSmallChunk][ROWS][2];   // (a, a) * 2^93 per entry and batch row
    alignas(16) unsigned ent[kSmallWarps][kSmallDepth][kSmallChunk][ROWS + 1];  // per entry: its (scale, zero) pair and the words holding the rows' x values
    alignas(16) float red[kSmallWarps][ROWS][G];
    float red_z[kSmallWarps][ROWS];
    int last;
};

// idx == nullptr: the dense product (the list is 0, 1, .., n-1 and count is n).
// CTAs resident per SM: the sums of four rows take 64 registers of a thread, which leaves room for two CTAs.
constexpr int small_ctas_per_sm(int rows) { return rows <= 2 ? 3 : 2; }

template <int G, int BITS, int ROWS>
__global__ void __launch_bounds__(kSmallThreads, small_ctas_per_sm(ROWS))
gemm_small_kernel(const uint8_t* __restrict__ codes, const unsigned* __restrict__ meta, int n,
                  const __half* __restrict__ X, int ldx, int batch,
                  const int32_t* __restrict__ idx, const int32_t* __restrict__ count_ptr,
                  __half* __restrict__ Y, int ldy, float* __restrict__ partials, int* __restrict__ counters)
{
    constexpr int B = G * BITS / 8;
    constexpr int CH = kSmallChunk;
    constexpr int CB = (B % 16 == 0) ? 16 : 8;        // bytes per copy
    constexpr int NC = CH * B / CB / 32;              // copies per lane and chunk
    constexpr int LM = G / 16;                        // arithmetic: lanes per block, 16 codes each
    constexpr int SLM = 32 / LM;                      // blocks per step
    constexpr int MSUBS = CH / SLM;                   // steps per chunk
    constexpr int KEEP = 16 / SLM;
    extern __shared__ __align__(16) unsigned char small_raw[];
    SmallSmem<G, BITS, ROWS>& sm = *reinterpret_cast<SmallSmem<G, BITS, ROWS>*>(small_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int s = blockIdx.x, S = gridDim.x, r = blockIdx.y;
    const int mslot = lane / LM, mh = lane % LM;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int count = idx ? __ldg(count_ptr) : n;
    const int lo = (int)(((long long)s * count) / S), hi = (int)(((long long)(s + 1) * count) / S);
    const size_t row_base = (size_t)r * (size_t)n;
    const uint8_t* row_codes = codes + row_base * B;
    const unsigned* row_meta = meta + row_base;
    const unsigned cbuf = smem_u32(&sm.codes[warp][0][0]);
    const unsigned mbuf = smem_u32(&sm.mult[warp][0][0][0]);
    constexpr unsigned kBufBytes = CH * B;

    unsigned long long acc[ROWS][8];
    float zl[ROWS];
#pragma unroll
    for (int b = 0; b < ROWS; ++b) {
        zl[b] = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[b][i] = 0ull;
    }

    // column of the entry this lane holds in the chunk at list position pos (past the end: the last entry again)
    auto column_at = [&](int pos) -> int {
        const int e = min(pos + lane, hi - 1);
        return idx ? __ldg(idx + e) : e;
    };
    // the chunk's code blocks into one of the warp's buffers, lane after lane
    auto copy_codes = [&](int col, unsigned dst) {
#pragma unroll
        for (int q = 0; q < NC; ++q) {
            const int off = (q * 32 + lane) * CB;
            const int e = off / B, part = off % B;
            const int cu = __shfl_sync(0xffffffffu, col, e);
            const uint8_t* src = row_codes + (size_t)cu * B + part;
            if (CB == 16) cp_async_16_l2_64(dst + off, src);
            else cp_async_8(dst + off, src);
        }
        cp_async_commit();
    };

    // One step: the lane's 16 codes become eight packed operand pairs ONCE (masks and shifts), then every
    // row of the batch multiplies them with its own multiplier pair.
    auto step = [&](unsigned cb, int u) {
        const unsigned ent = (unsigned)(u * SLM + mslot);
        uint2 wv;
        if (BITS == 4) {
            wv = lds_v2(cb + lane * 8 + u * 256);
        } else {
            const unsigned blk = cb + ent * B;
            const unsigned w2 = lds_u32(blk + 4u * mh);
            const unsigned w1 = lds_u32(blk + (G / 4) + 4u * (mh % (LM / 2))) >> (mh / (LM / 2));
            wv.x = (w2 & 0x33333333u) | ((w1 << 2) & 0x44444444u);     // the two planes widened to nibble codes
            wv.y = ((w2 >> 2) & 0x33333333u) | (w1 & 0x44444444u);
        }
        unsigned long long op[8];
        {
            const unsigned w = wv.x, v = wv.x >> 16, w2b = wv.y, v2 = wv.y >> 16;
            // the cumulative values of every half-word (its low 4, 8, 12 and 16 bits), as in the batch-1 kernel
            op[0] = pack2(__uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000ffu));
            op[1] = pack2(__uint_as_float(w & 0x00000fffu), __uint_as_float(w & 0x0000ffffu));
            op[2] = pack2(__uint_as_float(v & 0x0000000fu), __uint_as_float(v & 0x000000ffu));
            op[3] = pack2(__uint_as_float(v & 0x00000fffu), __uint_as_float(v));
            op[4] = pack2(__uint_as_float(w2b & 0x0000000fu), __uint_as_float(w2b & 0x000000ffu));
            op[5] = pack2(__uint_as_float(w2b & 0x00000fffu), __uint_as_float(w2b & 0x0000ffffu));
            op[6] = pack2(__uint_as_float(v2 & 0x0000000fu), __uint_as_float(v2 & 0x000000ffu));
            op[7] = pack2(__uint_as_float(v2 & 0x00000fffu), __uint_as_float(v2));
        }
#pragma unroll
        for (int b = 0; b < ROWS; ++b) {
            const unsigned long long mm = lds_u64(mbuf + 8u * (ent * ROWS + b));
#pragma unroll
            for (int i = 0; i < 8; ++i) ffma2(acc[b][i], op[i], mm);
        }
    };

    // The (scale, zero) pair and the x values of an entry travel like its codes: asynchronous copies into
    // shared memory, one chunk ahead (held in registers across a chunk's arithmetic they made the compiler
    // move the loads next to their use, and every chunk then waited for a round of gathers).  x is fetched as
    // the aligned 4-byte word that holds the value; without that alignment the values are loaded directly.
    const bool xw_ok = (reinterpret_cast<uintptr_t>(X) & 3) == 0 && (ldx & 1) == 0;
    const unsigned ebuf = smem_u32(&sm.ent[warp][0][0][0]);
    constexpr unsigned kEntBytes = CH * (ROWS + 1) * 4;
    auto issue_chunk = [&](int col, unsigned which) {
        const unsigned ed = ebuf + which * kEntBytes + (unsigned)lane * (ROWS + 1) * 4u;
        cp_async_4(ed, row_meta + col);
        if (xw_ok) {
#pragma unroll
            for (int b = 0; b < ROWS; ++b)
                if (b < batch) cp_async_4(ed + 4u * (1 + b), reinterpret_cast<const unsigned*>(X + (size_t)b * ldx + (col & ~1)));
        }
        copy_codes(col, cbuf + which * kBufBytes);   // (commits the group)
    };

    // kSmallDepth buffers per warp: the copies of the next kSmallDepth - 1 chunks fly during a chunk's arithmetic
    const int first = lo + warp * CH, stride = kSmallWarps * CH;
    if (first < hi) {
        constexpr int D = kSmallDepth;
        int cols[D];   // columns of this lane's entry in the chunks at pos, pos + stride, ..
#pragma unroll
        for (int d = 0; d < D; ++d) cols[d] = first + d * stride < hi ? column_at(first + d * stride) : 0;
#pragma unroll
        for (int d = 0; d < D - 1; ++d) {
            if (first + d * stride < hi) issue_chunk(cols[d], (unsigned)d);
            else cp_async_commit();
        }
        unsigned cur = 0;
        for (int pos = first; pos < hi; pos += stride) {
            const unsigned nxt = cur + (D - 1) >= (unsigned)D ? cur + (D - 1) - D : cur + (D - 1);
            if (pos + (D - 1) * stride < hi) issue_chunk(cols[D - 1], nxt);
            else cp_async_commit();
            const int col_after = pos + D * stride < hi ? column_at(pos + D * stride) : 0;
            const int col = cols[0];
            cp_async_wait<D - 1>();   // this chunk's copies have landed (the later chunks' may still fly)
            __syncwarp();
            // lane e: the multiplier pair of every row for its entry
            {
                const bool on = pos + lane < hi;
                const unsigned ea = ebuf + cur * kEntBytes + (unsigned)lane * (ROWS + 1) * 4u;
                const unsigned mz = lds_u32(ea);
                const float sf = __half2float(__ushort_as_half((unsigned short)(mz & 0xffffu)));
                const float zf = __half2float(__ushort_as_half((unsigned short)(mz >> 16)));
#pragma unroll
                for (int b = 0; b < ROWS; ++b) {
                    unsigned short xb = 0;
                    if (on && b < batch) {
                        if (xw_ok) {
                            const unsigned w = lds_u32(ea + 4u * (1 + b));
                            xb = (unsigned short)((col & 1) ? (w >> 16) : (w & 0xffffu));
                        } else {
                            xb = __ldg(reinterpret_cast<const unsigned short*>(X) + (size_t)b * ldx + col);
                        }
                    }
                    const float xf = __half2float(__ushort_as_half(xb));
                    const float am = xf * sf;       // exact
                    zl[b] += xf * zf;               // exact product
                    const unsigned long long aa = pack2(am, am);
                    sts_u64(mbuf + 8u * (lane * ROWS + b), fmul2(aa, pack2(0x1p93f, 0x1p93f)));
                }
            }
            __syncwarp();
            const unsigned cb = cbuf + cur * kBufBytes;
            const int valid = min(CH, hi - pos);
            if (valid == CH) {
#pragma unroll
                for (int u = 0; u < MSUBS; ++u) step(cb, u);
            } else {
                const int nsub = (valid + SLM - 1) / SLM;
#pragma unroll 1
                for (int u = 0; u < nsub; ++u) step(cb, u);
            }
            __syncwarp();
            cur = cur + 1 == (unsigned)D ? 0u : cur + 1;
#pragma unroll
            for (int d = 0; d + 1 < D; ++d) cols[d] = cols[d + 1];
            cols[D - 1] = col_after;
        }
    }
    cp_async_wait<0>();

    // warp -> CTA: reduce-scatter over the block slots, per batch row
#pragma unroll
    for (int b = 0; b < ROWS; ++b) {
        float accf[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) unpack2(acc[b][i], accf[2 * i], accf[2 * i + 1]);
        float t8[8], t4[4], keep[4];
        halve<16>(accf, t8, lane, 16);
        halve<8>(t8, t4, lane, 8);
        uncumulate(t4);
        if (LM == 8) {
#pragma unroll
            for (int i = 0; i < 4; ++i) keep[i] = t4[i];
        } else {
            float t2[2];
            halve<4>(t4, t2, lane, 4);
            keep[0] = t2[0];
            keep[1] = t2[1];
        }
#pragma unroll
        for (int i = 0; i < KEEP; ++i) {
            const int ai = mslot * KEEP + i;  // accumulator index = word*8 + nibble
            const int cw = ai >> 3, e2 = ai & 7;
            const int row = (BITS == 4) ? 8 * mh + 4 * cw + (e2 >> 1) + (e2 & 1) * (G / 2)
                                        : 4 * mh + (e2 >> 1) + (G / 4) * (2 * (e2 & 1) + cw);
            sm.red[warp][b][row] = keep[i] * 0x1p56f;
        }
        float z = zl[b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        if (lane == 0) sm.red_z[warp][b] = z;
    }
    __syncthreads();

    // CTA -> block-row
    float* mine = partials + ((size_t)r * kSmallMaxSplit + s) * kSmallRows * (G + 1);
    for (int i = tid; i < ROWS * (G + 1); i += kSmallThreads) {
        const int b = i / (G + 1), j = i % (G + 1);
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < kSmallWarps; ++w) v += (j < G) ? sm.red[w][b][j] : sm.red_z[w][b];
        if (S == 1) {
            // the only CTA of its block-row: keep the sums in place (warp 0's slot; every element has one writer)
            if (j < G) sm.red[0][b][j] = v;
            else sm.red_z[0][b] = v;
        } else {
            __stcg(mine + i, v);
        }
    }
    if (S == 1) {
        __syncthreads();
        for (int i = tid; i < batch * G; i += kSmallThreads) {
            const int b = i / G, j = i % G;
            Y[(size_t)b * ldy + (size_t)r * G + j] = __float2half_rn(sm.red[0][b][j] + sm.red_z[0][b]);
        }
        return;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sm.last = (atomicAdd(counters + r, 1) == S - 1) ? 1 : 0;
    __syncthreads();
    if (!sm.last) return;
    __threadfence();
    const float* rowp = partials + (size_t)r * kSmallMaxSplit * kSmallRows * (G + 1);
    for (int i = tid; i < batch * G; i += kSmallThreads) {
        const int b = i / G, j = i % G;
        float v = 0.0f, z = 0.0f;
        for (int q = 0; q < S; ++q) {
            v += __ldcg(rowp + ((size_t)q * kSmallRows + b) * (G + 1) + j);
            z += __ldcg(rowp + ((size_t)q * kSmallRows + b) * (G + 1) + G);
        }
        Y[(size_t)b * ldy + (size_t)r * G + j] = __float2half_rn(v + z);
    }
    if (tid == 0) counters[r] = 0;   // ready for the next call
}

inline size_t small_header_bytes(int R) { return (((size_t)R * 4 + 255) / 256) * 256; }
inline size_t small_workspace_bytes(const Format& f)
{
    return small_header_bytes(f.R) + (size_t)f.R * kSmallMaxSplit * kSmallRows * (size_t)(f.group + 1) * sizeof(float);
}

// Slices per block-row: the grid runs in waves of `per_sm` CTAs per SM; a CTA costs a fixed part (set-up,
// reduction, the exchange of partial sums) plus its share of the list.  Pick the split with the lowest
// estimate; ties go to the smaller one.
static int small_split(int R, int n, int sms, int per_sm)
{
    const double slots = (double)per_sm * sms;
    int best = 1;
    double best_t = 0.0;
    for (int S = 1; S <= kSmallMaxSplit; ++S) {
        const double waves = (double)((long long)((R * (double)S + slots - 1) / slots));
        const double t = waves * (4.0 + 1.5 * (double)n / (256.0 * S));
        if (S == 1 || t < best_t - 1e-9) {
            best = S;
            best_t = t;
        }
    }
    return best;
}

template <int G, int BITS, int ROWS>
static spqt_status launch_small_rows(const Format& f, const void* codes, const void* meta, const __half* X, int ldx,
                                     int nb, const int32_t* idx, const int32_t* count, __half* Y, int ldy,
                                     void* workspace, cudaStream_t s)
{
    auto kernel = gemm_small_kernel<G, BITS, ROWS>;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(SmallSmem<G, BITS, ROWS>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(small_split(f.R, f.n, sms, small_ctas_per_sm(ROWS)), f.R);
    cfg.blockDim = dim3(kSmallThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    int* counters = static_cast<int*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + small_header_bytes(f.R));
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, static_cast<const uint8_t*>(codes),
                                               static_cast<const unsigned*>(meta), f.n, X, ldx, nb, idx, count,
                                               Y, ldy, partials, counters);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

template <int G, int BITS>
static spqt_status launch_small(const Format& f, const void* codes, const void* meta, const __half* X, int ldx,
                                int batch, const int32_t* idx, const int32_t* count, __half* Y, int ldy,
                                void* workspace, cudaStream_t s)
{
    for (int b0 = 0; b0 < batch; b0 += kSmallRows) {
        const int nb = batch - b0 < kSmallRows ? batch - b0 : kSmallRows;
        const spqt_status st =
            nb <= 2 ? launch_small_rows<G, BITS, 2>(f, codes, meta, X + (size_t)b0 * ldx, ldx, nb, idx, count, Y + (size_t)b0 * ldy, ldy, workspace, s)
                    : launch_small_rows<G, BITS, 4>(f, codes, meta, X + (size_t)b0 * ldx, ldx, nb, idx, count, Y + (size_t)b0 * ldy, ldy, workspace, s);
        if (st != SPQT_OK) return st;
    }
    return SPQT_OK;
}

static spqt_status small_entry(const void* codes, const void* meta, int m, int n, int bits, int group,
                               const void* X, int ldx, int batch, bool dense, float t, int32_t* idx, int32_t* count,
                               void* Y, int ldy, void* workspace, size_t ws_bytes, void* stream)
{
    if (!codes || !meta || !X || !Y || !workspace) return SPQT_ERR_INVALID_ARG;
    if (!dense && (!idx || !count)) return SPQT_ERR_INVALID_ARG;
    if (batch < 1 || batch > 8 || ldx < n || ldy < m) return SPQT_ERR_INVALID_ARG;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (!aligned(codes, 16) || !aligned(meta, 16) || !aligned(X, 2) || !aligned(Y, 2) || !aligned(workspace, 16) ||
        (!dense && (!aligned(idx, 4) || !aligned(count, 4))))
        return SPQT_ERR_ALIGNMENT;
    if (ws_bytes < small_workspace_bytes(f)) return SPQT_ERR_WORKSPACE;
    if (f.R > 65535) return SPQT_ERR_UNSUPPORTED;
    if (!dense && n > 65535) return SPQT_ERR_UNSUPPORTED;  // the index collection keeps 64 flag bits per lane
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const __half* Xh = static_cast<const __half*>(X);
    if (!dense) {
        const spqt_status st2 = launch_sparsify_rows(Xh, ldx, batch, n, t, idx, count, s);
        if (st2 != SPQT_OK) return st2;
    }
    const int32_t* li = dense ? nullptr : idx;
    const int32_t* lc = dense ? nullptr : count;
    __half* Yh = static_cast<__half*>(Y);
    if (bits == 4 && group == 128) return launch_small<128, 4>(f, codes, meta, Xh, ldx, batch, li, lc, Yh, ldy, workspace, s);
    if (bits == 4 && group == 64) return launch_small<64, 4>(f, codes, meta, Xh, ldx, batch, li, lc, Yh, ldy, workspace, s);
    if (bits == 3 && group == 128) return launch_small<128, 3>(f, codes, meta, Xh, ldx, batch, li, lc, Yh, ldy, workspace, s);
    return launch_small<64, 3>(f, codes, meta, Xh, ldx, batch, li, lc, Yh, ldy, workspace, s);
}

}  // namespace spqt

extern "C" {

spqt_status spqt_gemm_small_workspace(int m, int n, int bits, int group, size_t* workspace_bytes)
{
    spqt::Format f;
    spqt_status st = spqt::make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (workspace_bytes) *workspace_bytes = spqt::small_workspace_bytes(f);
    return SPQT_OK;
}

spqt_status spqt_sparse_gemm_small(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                   const void* X, int ldx, int batch, float t, int32_t* idx, int32_t* count,
                                   void* Y, int ldy, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::small_entry(codes, scale_zero, m, n, bits, group, X, ldx, batch, false, t, idx, count, Y, ldy,
                             workspace, workspace_bytes, stream);
}

spqt_status spqt_dense_gemm_small(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                  const void* X, int ldx, int batch, void* Y, int ldy,
                                  void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::small_entry(codes, scale_zero, m, n, bits, group, X, ldx, batch, true, 0.0f, nullptr, nullptr, Y, ldy,
                             workspace, workspace_bytes, stream);
}

}  // extern "C"
