// The two-level format the paper's implementation builds on (Sec. 2: superblocks of 256 weights split
// into eight blocks of 32, 4-bit codes, a 6-bit scale and a 6-bit minimum per block, a 16-bit scale and
// minimum per superblock), in the zigzag arrangement of Sec. 4.1.2: a superblock is 256 consecutive ROWS
// of one column, superblocks are stored row-major over (block-row, column).  One 144-byte record per
// superblock: 128 bytes of codes (byte i = q_i | q_{i+128} << 4), the sixteen 6-bit fields sc_0..7,
// m_0..7 as a little-endian bit string (12 bytes), d and dmin as fp16.  Dequantized weight of row j of
// block i:  d*sc_i*q_j - dmin*m_i.  The paper fixes neither the rounding rule nor the bit arrangement;
// the rule implemented is stated at kq_pack_kernel, every step a single IEEE fp32 operation.
// Other code widths (Sec. 4.1.3: any width from 2 to 8 bits): the kernels are templates over BITS = 2, 4, 5, 6,
// 8; 2^BITS - 1 replaces 15 in the rule and only the code bytes of a record change -- 8 bits: byte i = q_i (256
// bytes, records of 272); 2 bits: byte i = q_i | q_{i+64} << 2 | q_{i+128} << 4 | q_{i+192} << 6 (64 bytes,
// records of 80); 5 and 6 bits: the low four bits as 4-bit codes, then a plane of the high bits q >> 4, one per
// row (bit j%8 of byte j/8) or two per row arranged like 2-bit codes (records of 176 and 208).  The arithmetic of
// the 2- and 8-bit codes and of the high planes sums cumulative values (per 16-bit half-word the value of its
// first code and of both codes together; per byte of single bits its low 1, 2, .. 8 bits: the cumulative form of
// the main kernel) and takes the differences at the end.
//
//   kq_pack_kernel   a CTA stages a 256 x 32 tile of W; a warp quantizes four columns, lane l owning rows
//                    l, l+32, .. (one row of every block).
//   kq_gemv_kernel   grid (S, R): CTA (s, r) takes the s-th of S slices of the index list (or of all
//                    columns) for block-row r; its 8 warps take the slice's chunks of 16 entries in turn,
//                    two record buffers per warp (cp.async: a record is one contiguous gather of 144 bytes,
//                    metadata included).  Lanes e and e+16 decode the fields of entry e and write the packed
//                    multiplier pairs of its four lane groups; lane t of a 16-lane half owns rows 8t..8t+7
//                    and 128+8t..128+8t+7 of the entry's superblock (blocks t/4 and 4+t/4: one multiplier
//                    pair covers both).  Conversion-free dequantization as in the main kernel.  Partial
//                    sums: warp -> CTA (shared memory) -> block-row (fp32 partials in the workspace,
//                    arrive-only counter, the last CTA adds them in slice order: bit-reproducible).
#include <cstddef>

#include "spqt_common.cuh"

namespace spqt {
constexpr unsigned long long kWaitNs = 1000000000ull;
}
#include "spqt_gemv_device.cuh"

namespace spqt {

constexpr int kKqG = 256;           // rows of a superblock
__host__ __device__ constexpr int kq_code_bytes(int bits) { return kKqG * bits / 8; }
__host__ __device__ constexpr int kq_rec_bytes(int bits) { return kq_code_bytes(bits) + 16; }
__host__ __device__ constexpr int kq_ctas_per_sm(int bits) { return bits >= 5 ? 2 : 3; }   // (registers of a second accumulator set; shared memory of the record buffers)
constexpr int kKqWarps = 8;
constexpr int kKqThreads = kKqWarps * 32;
constexpr int kKqChunk = 16;        // list entries per chunk
constexpr int kKqMaxSplit = 32;     // slices per block-row at most
constexpr int kKqPackCols = 32;

// ---------------------------------------------------------------- conversion
//   per block i:      lo_i = min(min_j w_j, 0),  step_i = (max_j w_j - lo_i) / 15,  neg_i = 0 - lo_i
//                     (zeros of either sign count as +0.0)
//   per superblock:   d = fp16(max_i step_i / 63),  dmin = fp16(max_i neg_i / 63)
//                     sc_i = min(rint(step_i / d), 63),  m_i = min(rint(neg_i / dmin), 63)   (0 if the divisor is 0)
//   per weight:       q_j = clamp(rint((w_j + dmin*m_i) / (d*sc_i)), 0, 15)                   (0 if d*sc_i == 0)
// (15 = 2^BITS - 1 for 4-bit codes; 3 and 255 for the other widths)
template <int BITS>
__global__ void __launch_bounds__(256)
kq_pack_kernel(const __half* __restrict__ W, int n, int ldw, uint8_t* __restrict__ records)
{
    constexpr int kTop = (1 << BITS) - 1, NCB = kq_code_bytes(BITS), REC = kq_rec_bytes(BITS);
    __shared__ __align__(16) __half tile[kKqG][kKqPackCols + 2];
    const int r = blockIdx.y, k0 = blockIdx.x * kKqPackCols, tid = threadIdx.x;
    for (int e = tid; e < kKqG * kKqPackCols; e += 256) {
        const int i = e / kKqPackCols, c = e % kKqPackCols, k = k0 + c;
        tile[i][c] = (k < n) ? W[(size_t)(r * kKqG + i) * ldw + k] : __float2half(0.0f);
    }
    __syncthreads();
    const int warp = tid >> 5, lane = tid & 31;
    for (int cc = 0; cc < 4; ++cc) {
        const int c = warp * 4 + cc, k = k0 + c;
        if (k >= n) break;  // uniform across the warp
        float w[8], step[8], neg[8];
        float step_max = 0.0f, neg_max = 0.0f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            w[u] = __half2float(tile[lane + 32 * u][c]);  // row lane of block u
            float lo = w[u], hi = w[u];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
                hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
            }
            lo = __fadd_rn(fminf(lo, 0.0f), 0.0f);  // a zero of either sign counts as +0.0
            hi = __fadd_rn(hi, 0.0f);
            step[u] = __fdiv_rn(__fsub_rn(hi, lo), (float)kTop);
            neg[u] = __fsub_rn(0.0f, lo);           // (0 - 0 is +0.0)
            step_max = fmaxf(step_max, step[u]);
            neg_max = fmaxf(neg_max, neg[u]);
        }
        const __half dh = __float2half_rn(__fdiv_rn(step_max, 63.0f));
        const __half mh = __float2half_rn(__fdiv_rn(neg_max, 63.0f));
        const float df = __half2float(dh), dminf = __half2float(mh);
        unsigned sc[8], mn[8];
        int q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            sc[u] = (df != 0.0f) ? (unsigned)min(__float2int_rn(__fdiv_rn(step[u], df)), 63) : 0u;
            mn[u] = (dminf != 0.0f) ? (unsigned)min(__float2int_rn(__fdiv_rn(neg[u], dminf)), 63) : 0u;
            const float se = __fmul_rn(df, (float)sc[u]), oe = __fmul_rn(dminf, (float)mn[u]);
            q[u] = (se != 0.0f) ? max(0, min(__float2int_rn(__fdiv_rn(__fadd_rn(w[u], oe), se)), kTop)) : 0;
        }
        uint8_t* rec = records + ((size_t)r * n + k) * REC;
        // this lane holds the codes of rows lane + 32u
        if (BITS == 4) {            // byte i = code of row i | code of row i + 128 << 4
#pragma unroll
            for (int u = 0; u < 4; ++u) rec[lane + 32 * u] = (uint8_t)(q[u] | (q[u + 4] << 4));
        } else if (BITS == 8) {     // byte i = code of row i
#pragma unroll
            for (int u = 0; u < 8; ++u) rec[lane + 32 * u] = (uint8_t)q[u];
        } else if (BITS == 5 || BITS == 6) {
            // the low four bits like 4-bit codes, then the high bits: one per row, bit j % 8 of byte j / 8 (the
            // 32 rows lane + 32u of all lanes are one 32-bit word), or two per row arranged like 2-bit codes
#pragma unroll
            for (int u = 0; u < 4; ++u) rec[lane + 32 * u] = (uint8_t)((q[u] & 15) | ((q[u + 4] & 15) << 4));
            if (BITS == 5) {
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const unsigned bal = __ballot_sync(0xffffffffu, (q[u] >> 4) & 1);
                    if (lane == 0) reinterpret_cast<unsigned*>(rec + 128)[u] = bal;
                }
            } else {
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    rec[128 + lane + 32 * u] = (uint8_t)((q[u] >> 4) | ((q[u + 2] >> 4) << 2) | ((q[u + 4] >> 4) << 4) | ((q[u + 6] >> 4) << 6));
            }
        } else {                    // byte i = codes of rows i, i + 64, i + 128, i + 192, two bits each
#pragma unroll
            for (int u = 0; u < 2; ++u) rec[lane + 32 * u] = (uint8_t)(q[u] | (q[u + 2] << 2) | (q[u + 4] << 4) | (q[u + 6] << 6));
        }
        if (lane == 0) {
            unsigned long long lo64 = 0ull;  // fields 0..9 and the low 4 bits of field 10
            unsigned hi32 = 0u;              // bits 64..95
#pragma unroll
            for (int f = 0; f < 16; ++f) {
                const unsigned long long v = (f < 8) ? sc[f] : mn[f - 8];
                const int b = 6 * f;
                if (b < 64) lo64 |= v << b;
                if (b + 6 > 64) hi32 |= (b >= 64) ? (unsigned)(v << (b - 64)) : (unsigned)(v >> (64 - b));
            }
            unsigned* tail = reinterpret_cast<unsigned*>(rec + NCB);  // records start on 16-byte boundaries
            tail[0] = (unsigned)lo64;
            tail[1] = (unsigned)(lo64 >> 32);
            tail[2] = hi32;
            tail[3] = (unsigned)__half_as_ushort(dh) | ((unsigned)__half_as_ushort(mh) << 16);
        }
    }
}

// ---------------------------------------------------------------- GEMV

template <int BITS>
struct KqSmem {
    alignas(16) unsigned char rec[kKqWarps][2][kKqChunk * kq_rec_bytes(BITS)];  // two record buffers per warp
    alignas(16) float mult[kKqWarps][kKqChunk][4][4];               // per entry and lane group: two packed multiplier pairs
    alignas(16) float red[kKqWarps][kKqG];
    float red_z[kKqWarps][8];
    int last;
};

// 6-bit field f of the 96-bit string w0 | w1 << 32 | w2 << 64
__device__ __forceinline__ unsigned kq_field(unsigned w0, unsigned w1, unsigned w2, int f)
{
    const int b = 6 * f, word = b >> 5;
    const unsigned lo = word == 0 ? w0 : (word == 1 ? w1 : w2);
    const unsigned hi = word == 0 ? w1 : (word == 1 ? w2 : 0u);
    return __funnelshift_r(lo, hi, b & 31) & 63u;
}

// idx == nullptr: the dense product (the list is 0, 1, .., n-1 and count is n).
template <int BITS>
__global__ void __launch_bounds__(kKqThreads, kq_ctas_per_sm(BITS))
kq_gemv_kernel(const uint8_t* __restrict__ records, int n, const __half* __restrict__ x,
               const int32_t* __restrict__ idx, const int32_t* __restrict__ count_ptr,
               __half* __restrict__ y, float* __restrict__ partials, int* __restrict__ counters)
{
    constexpr int CH = kKqChunk, G = kKqG;
    constexpr int REC = kq_rec_bytes(BITS), NCB = kq_code_bytes(BITS), PPR = REC / 16;
    constexpr int NP = CH * REC / 16;            // 16-byte pieces of a chunk
    constexpr int NC = (NP + 31) / 32;           // copies per lane and chunk
    extern __shared__ __align__(16) unsigned char kq_raw[];
    KqSmem<BITS>& sm = *reinterpret_cast<KqSmem<BITS>*>(kq_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int s = blockIdx.x, S = gridDim.x, r = blockIdx.y;
    const int half = lane >> 4, t = lane & 15;   // arithmetic: entry of the step, rows 8t.. and 128+8t..

    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int count = idx ? __ldg(count_ptr) : n;
    const int lo = (int)(((long long)s * count) / S), hi = (int)(((long long)(s + 1) * count) / S);
    const uint8_t* row_rec = records + (size_t)r * (size_t)n * REC;
    const unsigned rbuf = smem_u32(&sm.rec[warp][0][0]);
    const unsigned mbuf = smem_u32(&sm.mult[warp][0][0][0]);
    constexpr unsigned kBufBytes = CH * REC;
    const unsigned short* xb = reinterpret_cast<const unsigned short*>(x);

    unsigned long long acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0ull;
    constexpr bool kHigh = BITS == 5 || BITS == 6;   // a second plane with the bits above the low four
    unsigned long long acch[kHigh ? 8 : 1];          // its sums (cumulative, see the step), same rows as acc
#pragma unroll
    for (int i = 0; i < (kHigh ? 8 : 1); ++i) acch[i] = 0ull;
    float zl[4] = {0.0f, 0.0f, 0.0f, 0.0f};      // x*dmin*m of blocks 4*half .. 4*half+3

    // column of the entry lanes e and e+16 hold in the chunk at list position pos (past the end: the last entry again)
    auto column_at = [&](int pos) -> int {
        const int e = min(pos + t, hi - 1);
        return idx ? __ldg(idx + e) : e;
    };
    auto copy_records = [&](int col, unsigned dst) {
#pragma unroll
        for (int q = 0; q < NC; ++q) {
            const int p = q * 32 + lane;
            const int e = p / PPR, part = p - PPR * e;
            const int cu = __shfl_sync(0xffffffffu, col, e & 15);
            if (p < NP) cp_async_16_l2_64(dst + (unsigned)(e * REC + part * 16), row_rec + (size_t)cu * REC + part * 16);
        }
        cp_async_commit();
    };

    const int first = lo + warp * CH, stride = kKqWarps * CH;
    if (first < hi) {
        int col = column_at(first);
        copy_records(col, rbuf);
        int col_next = first + stride < hi ? column_at(first + stride) : 0;
        unsigned short xv = (first + t < hi) ? __ldg(xb + col) : (unsigned short)0;
        unsigned cur = 0;
        for (int pos = first; pos < hi; pos += stride) {
            const bool more = pos + stride < hi;
            if (more) copy_records(col_next, rbuf + (cur == 0u ? kBufBytes : 0u));
            else cp_async_commit();
            const int col_after = pos + 2 * stride < hi ? column_at(pos + 2 * stride) : 0;
            const unsigned short xv_next = (more && pos + stride + t < hi) ? __ldg(xb + col_next) : (unsigned short)0;
            cp_async_wait<1>();   // this chunk's records have landed (the next chunk's may still fly)
            __syncwarp();
            // lanes e and e+16: the fields of entry e -> multiplier pairs of lane groups 2*half, 2*half+1 and
            // the offset terms of blocks 4*half .. 4*half+3
            {
                const unsigned ra = rbuf + cur + (unsigned)(t * REC) + (unsigned)NCB;
                const uint4 tail = lds_v4(ra);
                const float xf = __half2float(__ushort_as_half(xv));
                const float df = __half2float(__ushort_as_half((unsigned short)(tail.w & 0xffffu)));
                const float dminf = __half2float(__ushort_as_half((unsigned short)(tail.w >> 16)));
#pragma unroll
                for (int g2 = 0; g2 < 2; ++g2) {
                    const int sb = 2 * half + g2;   // lane group: rows of blocks sb (low nibbles) and sb + 4 (high nibbles)
                    const float a_lo = xf * (df * (float)kq_field(tail.x, tail.y, tail.z, sb));       // d*sc is exact
                    const float a_hi = xf * (df * (float)kq_field(tail.x, tail.y, tail.z, sb + 4));
                    if (BITS == 4 || kHigh)
                        sts_pairs(mbuf + 16u * (unsigned)(t * 4 + sb), pack2(a_lo * 0x1p93f, a_hi * 0x1p89f),
                                  pack2(a_lo * 0x1p85f, a_hi * 0x1p81f));
                    else   // one pair: the high rows' codes sit in the same bytes (2 bits, four bits up) or in bytes of their own (8 bits)
                        sts_u64(mbuf + 16u * (unsigned)(t * 4 + sb), pack2(a_lo * 0x1p93f, a_hi * (BITS == 2 ? 0x1p89f : 0x1p93f)));
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    zl[i] += xf * (dminf * (float)kq_field(tail.x, tail.y, tail.z, 8 + 4 * half + i));
            }
            __syncwarp();
            const int valid = min(CH, hi - pos);
            const unsigned cb = rbuf + cur;
            auto step = [&](int u) {
                const unsigned e = (unsigned)(2 * u + half);
                if (BITS == 4 || kHigh) {
                    const uint2 wv = lds_v2(cb + e * REC + (unsigned)t * 8u);
                    unsigned long long m01, m23;
                    lds_pairs(mbuf + 16u * (e * 4u + (unsigned)(t >> 2)), m01, m23);
                    fma_block8(acc, wv, m01, m23);     // the low four bits of every code
                    if (BITS == 6) {
                        // the high two bits, 16 times the weight: a plane laid out like 2-bit codes, summed the same way
                        const unsigned long long mh = fmul2(m01, pack2(16.0f, 16.0f));
                        const uint2 hv = lds_v2(cb + e * REC + 128u + (unsigned)(t & 7) * 8u);
                        const int sh = 2 * (t >> 3);
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
                            const unsigned w = (k ? hv.y : hv.x) >> sh, v = w >> 16;
                            ffma2(acch[4 * k + 0], pack2(__uint_as_float(w & 0x03u), __uint_as_float(w & 0x30u)), mh);
                            ffma2(acch[4 * k + 1], pack2(__uint_as_float(w & 0x0303u), __uint_as_float(w & 0x3030u)), mh);
                            ffma2(acch[4 * k + 2], pack2(__uint_as_float(v & 0x03u), __uint_as_float(v & 0x30u)), mh);
                            ffma2(acch[4 * k + 3], pack2(__uint_as_float(v & 0x0303u), __uint_as_float(v & 0x3030u)), mh);
                        }
                    } else if (BITS == 5) {
                        // the fifth bit of rows 8t.. and 128+8t..: one byte each; position b sums the byte's low b+1 bits
                        const unsigned long long mh = fmul2(m01, pack2(16.0f, 256.0f));   // (a_lo, a_hi) * 16 * 2^93
                        unsigned lb, hb;
                        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(lb) : "r"(cb + e * REC + 128u + (unsigned)t) : "memory");
                        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(hb) : "r"(cb + e * REC + 144u + (unsigned)t) : "memory");
#pragma unroll
                        for (int b = 0; b < 8; ++b) {
                            const unsigned mk = (2u << b) - 1u;
                            ffma2(acch[b], pack2(__uint_as_float(lb & mk), __uint_as_float(hb & mk)), mh);
                        }
                    }
                    return;
                }
                // 2 and 8 bits: per 16-bit half-word the value of its first byte's code and the value of both
                // codes together (second code times 256) are summed; the second code's sum is their difference
                const unsigned long long mm = lds_u64(mbuf + 16u * (e * 4u + (unsigned)(t >> 2)));
                if (BITS == 8) {
                    const uint2 lw = lds_v2(cb + e * REC + (unsigned)t * 8u);           // rows 8t .. 8t+7
                    const uint2 hw = lds_v2(cb + e * REC + 128u + (unsigned)t * 8u);    // rows 128+8t ..
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const unsigned l = k ? lw.y : lw.x, h = k ? hw.y : hw.x, lv = l >> 16, hv = h >> 16;
                        ffma2(acc[4 * k + 0], pack2(__uint_as_float(l & 0xffu), __uint_as_float(h & 0xffu)), mm);
                        ffma2(acc[4 * k + 1], pack2(__uint_as_float(l & 0xffffu), __uint_as_float(h & 0xffffu)), mm);
                        ffma2(acc[4 * k + 2], pack2(__uint_as_float(lv & 0xffu), __uint_as_float(hv & 0xffu)), mm);
                        ffma2(acc[4 * k + 3], pack2(__uint_as_float(lv), __uint_as_float(hv)), mm);
                    }
                } else {
                    // byte i holds rows i, i+64, i+128, i+192: lanes 0..7 use fields 0 and 2 of bytes 8t.., lanes
                    // 8..15 fields 1 and 3 of bytes 8(t-8)..
                    const uint2 wv = lds_v2(cb + e * REC + (unsigned)(t & 7) * 8u);
                    const int sh = 2 * (t >> 3);
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const unsigned w = (k ? wv.y : wv.x) >> sh, v = w >> 16;
                        ffma2(acc[4 * k + 0], pack2(__uint_as_float(w & 0x03u), __uint_as_float(w & 0x30u)), mm);
                        ffma2(acc[4 * k + 1], pack2(__uint_as_float(w & 0x0303u), __uint_as_float(w & 0x3030u)), mm);
                        ffma2(acc[4 * k + 2], pack2(__uint_as_float(v & 0x03u), __uint_as_float(v & 0x30u)), mm);
                        ffma2(acc[4 * k + 3], pack2(__uint_as_float(v & 0x0303u), __uint_as_float(v & 0x3030u)), mm);
                    }
                }
            };
            if (valid == CH) {
#pragma unroll
                for (int u = 0; u < CH / 2; ++u) step(u);   // a full chunk: straight-line code
            } else {
                const int nsub = (valid + 1) >> 1;
#pragma unroll 1
                for (int u = 0; u < nsub; ++u) step(u);
            }
            __syncwarp();
            cur = (cur == 0u) ? kBufBytes : 0u;
            col = col_next;
            col_next = col_after;
            xv = xv_next;
        }
    }
    cp_async_wait<0>();

    // warp -> CTA.  acc[b] = (row 8t+b, row 128+8t+b) of the entries this half-warp handled
    {
        float lo_rows[8], hi_rows[8];
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            unpack2(acc[b], lo_rows[b], hi_rows[b]);
            lo_rows[b] += __shfl_xor_sync(0xffffffffu, lo_rows[b], 16);
            hi_rows[b] += __shfl_xor_sync(0xffffffffu, hi_rows[b], 16);
        }
        if (kHigh) {
            float lh[8], hh[8];
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                unpack2(acch[b], lh[b], hh[b]);
                lh[b] += __shfl_xor_sync(0xffffffffu, lh[b], 16);
                hh[b] += __shfl_xor_sync(0xffffffffu, hh[b], 16);
            }
            if (BITS == 6) {      // pairs, as for 2-bit codes
#pragma unroll
                for (int b = 1; b < 8; b += 2) {
                    lh[b] = (lh[b] - lh[b - 1]) * 0x1p-8f;
                    hh[b] = (hh[b] - hh[b - 1]) * 0x1p-8f;
                }
            } else {              // a chain over the eight bits of a byte
#pragma unroll
                for (int b = 7; b > 0; --b) {
                    lh[b] = (lh[b] - lh[b - 1]) * (1.0f / (float)(1 << b));
                    hh[b] = (hh[b] - hh[b - 1]) * (1.0f / (float)(1 << b));
                }
            }
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                lo_rows[b] += lh[b];
                hi_rows[b] += hh[b];
            }
        } else if (BITS != 4) {   // odd positions hold (first code + 256 * second code) of a half-word
#pragma unroll
            for (int b = 1; b < 8; b += 2) {
                lo_rows[b] = (lo_rows[b] - lo_rows[b - 1]) * 0x1p-8f;
                hi_rows[b] = (hi_rows[b] - hi_rows[b - 1]) * 0x1p-8f;
            }
        }
        if (half == 0) {
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                sm.red[warp][8 * t + b] = lo_rows[b] * 0x1p56f;
                sm.red[warp][128 + 8 * t + b] = hi_rows[b] * 0x1p56f;
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float z = zl[i];
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            if (t == 0) sm.red_z[warp][4 * half + i] = z;
        }
    }
    __syncthreads();

    // CTA -> block-row: G sums and 8 offset terms
    float* mine = partials + ((size_t)r * kKqMaxSplit + s) * (G + 8);
    for (int i = tid; i < G + 8; i += kKqThreads) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < kKqWarps; ++w) v += (i < G) ? sm.red[w][i] : sm.red_z[w][i - G];
        if (S == 1) {
            if (i < G) sm.red[0][i] = v;    // (warp 0's slot; every element has one writer)
            else sm.red_z[0][i - G] = v;
        } else {
            __stcg(mine + i, v);
        }
    }
    if (S == 1) {
        __syncthreads();
        for (int j = tid; j < G; j += kKqThreads) y[(size_t)r * G + j] = __float2half_rn(sm.red[0][j] - sm.red_z[0][j >> 5]);
        return;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) sm.last = (atomicAdd(counters + r, 1) == S - 1) ? 1 : 0;
    __syncthreads();
    if (!sm.last) return;
    __threadfence();
    const float* rowp = partials + (size_t)r * kKqMaxSplit * (G + 8);
    for (int j = tid; j < G; j += kKqThreads) {
        float v = 0.0f, z = 0.0f;
        for (int q = 0; q < S; ++q) {
            v += __ldcg(rowp + (size_t)q * (G + 8) + j);
            z += __ldcg(rowp + (size_t)q * (G + 8) + G + (j >> 5));
        }
        y[(size_t)r * G + j] = __float2half_rn(v - z);
    }
    if (tid == 0) counters[r] = 0;   // ready for the next call
}

// ---------------------------------------------------------------- host side

inline size_t kq_header_bytes(int R) { return (((size_t)R * 4 + 255) / 256) * 256; }
inline size_t kq_workspace_bytes(int R) { return kq_header_bytes(R) + (size_t)R * kKqMaxSplit * (kKqG + 8) * sizeof(float); }

static spqt_status kq_shape(int m, int n)
{
    if (m <= 0 || n <= 0) return SPQT_ERR_INVALID_ARG;
    if (m % kKqG != 0) return SPQT_ERR_UNSUPPORTED;
    if (m / kKqG > 65535) return SPQT_ERR_UNSUPPORTED;
    return SPQT_OK;
}

template <int BITS>
static spqt_status kq_launch(const void* records, int m, int n, const void* x, const int32_t* idx, const int32_t* count,
                             void* y, void* workspace, size_t ws_bytes, void* stream)
{
    if (!records || !x || !y || !workspace) return SPQT_ERR_INVALID_ARG;
    const spqt_status st = kq_shape(m, n);
    if (st != SPQT_OK) return st;
    if (!aligned(records, 16) || !aligned(x, 2) || !aligned(y, 2) || !aligned(workspace, 16) ||
        (idx && (!aligned(idx, 4) || !aligned(count, 4))))
        return SPQT_ERR_ALIGNMENT;
    const int R = m / kKqG;
    if (ws_bytes < kq_workspace_bytes(R)) return SPQT_ERR_WORKSPACE;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(KqSmem<BITS>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kq_gemv_kernel<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    // slices per block-row: fill the resident CTAs of every SM once; never less than a chunk per warp
    int S = (kq_ctas_per_sm(BITS) * sms) / R;
    const int by_work = n / (kKqChunk * kKqWarps);
    if (S > by_work) S = by_work;
    if (S > kKqMaxSplit) S = kKqMaxSplit;
    if (S < 1) S = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, R);
    cfg.blockDim = dim3(kKqThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    int* counters = static_cast<int*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kq_header_bytes(R));
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kq_gemv_kernel<BITS>, static_cast<const uint8_t*>(records), n,
                                               static_cast<const __half*>(x), idx, count, static_cast<__half*>(y), partials, counters);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

}  // namespace spqt

extern "C" {

static bool kq_bits_ok(int bits) { return bits == 2 || bits == 4 || bits == 5 || bits == 6 || bits == 8; }

spqt_status spqt_kqw_packed_sizes(int m, int n, int bits, size_t* records_bytes, size_t* workspace_bytes)
{
    const spqt_status st = spqt::kq_shape(m, n);
    if (st != SPQT_OK) return st;
    if (!kq_bits_ok(bits)) return SPQT_ERR_UNSUPPORTED;
    if (records_bytes) *records_bytes = (size_t)(m / spqt::kKqG) * (size_t)n * spqt::kq_rec_bytes(bits);
    if (workspace_bytes) *workspace_bytes = spqt::kq_workspace_bytes(m / spqt::kKqG);
    return SPQT_OK;
}

spqt_status spqt_kqw_pack(const void* W, int m, int n, int ldw, int bits, void* records, void* stream)
{
    if (!W || !records) return SPQT_ERR_INVALID_ARG;
    const spqt_status st = spqt::kq_shape(m, n);
    if (st != SPQT_OK) return st;
    if (!kq_bits_ok(bits)) return SPQT_ERR_UNSUPPORTED;
    if (ldw < n) return SPQT_ERR_INVALID_ARG;
    if (!spqt::aligned(W, 2) || !spqt::aligned(records, 16)) return SPQT_ERR_ALIGNMENT;
    const dim3 grid((n + spqt::kKqPackCols - 1) / spqt::kKqPackCols, m / spqt::kKqG);
    const cudaStream_t st_ = static_cast<cudaStream_t>(stream);
    const __half* w = static_cast<const __half*>(W);
    uint8_t* rec = static_cast<uint8_t*>(records);
    if (bits == 2) spqt::kq_pack_kernel<2><<<grid, 256, 0, st_>>>(w, n, ldw, rec);
    else if (bits == 4) spqt::kq_pack_kernel<4><<<grid, 256, 0, st_>>>(w, n, ldw, rec);
    else if (bits == 5) spqt::kq_pack_kernel<5><<<grid, 256, 0, st_>>>(w, n, ldw, rec);
    else if (bits == 6) spqt::kq_pack_kernel<6><<<grid, 256, 0, st_>>>(w, n, ldw, rec);
    else spqt::kq_pack_kernel<8><<<grid, 256, 0, st_>>>(w, n, ldw, rec);
    spqt::count_launch();
    return cudaGetLastError() == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

static spqt_status kq_launch_bits(int bits, const void* records, int m, int n, const void* x, const int32_t* idx,
                                  const int32_t* count, void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    if (bits == 2) return spqt::kq_launch<2>(records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
    if (bits == 4) return spqt::kq_launch<4>(records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
    if (bits == 5) return spqt::kq_launch<5>(records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
    if (bits == 6) return spqt::kq_launch<6>(records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
    if (bits == 8) return spqt::kq_launch<8>(records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
    return SPQT_ERR_UNSUPPORTED;
}

spqt_status spqt_kqw_sparse_gemv(const void* records, int m, int n, int bits, const void* x, const int32_t* idx,
                                 const int32_t* count, void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!idx || !count) return SPQT_ERR_INVALID_ARG;
    return kq_launch_bits(bits, records, m, n, x, idx, count, y, workspace, workspace_bytes, stream);
}

spqt_status spqt_kqw_dense_gemv(const void* records, int m, int n, int bits, const void* x, void* y, void* workspace,
                                size_t workspace_bytes, void* stream)
{
    return kq_launch_bits(bits, records, m, n, x, nullptr, nullptr, y, workspace, workspace_bytes, stream);
}

spqt_status spqt_kq_packed_sizes(int m, int n, size_t* records_bytes, size_t* workspace_bytes)
{
    return spqt_kqw_packed_sizes(m, n, 4, records_bytes, workspace_bytes);
}

spqt_status spqt_kq_pack(const void* W, int m, int n, int ldw, void* records, void* stream)
{
    return spqt_kqw_pack(W, m, n, ldw, 4, records, stream);
}

spqt_status spqt_kq_sparse_gemv(const void* records, int m, int n, const void* x, const int32_t* idx, const int32_t* count,
                                void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt_kqw_sparse_gemv(records, m, n, 4, x, idx, count, y, workspace, workspace_bytes, stream);
}

spqt_status spqt_kq_dense_gemv(const void* records, int m, int n, const void* x, void* y, void* workspace,
                               size_t workspace_bytes, void* stream)
{
    return spqt_kqw_dense_gemv(records, m, n, 4, x, y, workspace, workspace_bytes, stream);
}

}  // extern "C"
