// Activation-sparse GEMV over the zigzag layout, and its dense twin (4-bit and 3-bit codes).
//
// Work decomposition (the paper's hybrid row/column parallelism, generalised):
// the R block-rows are laid end to end and cut into P equal pieces, one per CTA,
// P = one persistent CTA per SM.  A piece is a run of (fractions of) block-rows;
// the fraction [u0,u1) of block-row r means the slice [u0*count, u1*count) of
// the ACTIVE index list, so the load follows the active entries, not the matrix
// columns, and every CTA streams the same number of blocks whatever R is.  Each
// (CTA, block-row) segment yields G fp32 partial sums; whichever CTA contributes
// last to a block-row (arrive-only counter: nobody waits on another CTA) adds
// the partials in a fixed order, adds the offset term and rounds to fp16.
//
// Inside a CTA, kWorkers warps each run their own copy pipeline over chunks of
// 32 list entries (chunks are dealt round-robin to the warps); nothing is shared
// between the warps until the end of a segment.  Per chunk, three stages, all
// cp.async into the warp's private shared-memory ring, one commit group per
// iteration:
//   A  the chunk's 32 column numbers (one 4-byte copy per lane);
//   B  once A has landed: the code blocks (16 bytes per lane, the lanes of a
//      block adjacent so that every 32-byte sector crosses once, fetched with
//      64-byte L2 granularity so that an inactive neighbour block is not dragged
//      in) and the 4-byte words holding x_k, scale_rk and zero_rk of the lane's
//      own entry;
//   C  once B has landed: lane l turns its words into a = x_k*scale_rk (exact in
//      fp32) and x_k*zero_rk, the multipliers are dealt out with shuffles, and
//      the warp does the dequantize-FMA work.
// A runs 2*kDepth chunks ahead of C and B kDepth chunks ahead, so kDepth chunks
// (2 KB each) per warp are in flight.  Two more warps, the writers (one per
// hand-over buffer), add the workers' sums at the end of a segment, publish the
// partial and, if this CTA is the last contributor of the block-row, produce y;
// their waits on shared-memory barriers are bounded in wall time (on expiry the
// workspace's status word is set and the kernel returns).
//
// Arithmetic:  y[j] = sum_k a_k * code_jk + sum_k x_k * zero_rk.  A 4-bit code
// becomes an fp32 operand with no conversion: the nibble masked in place at bit
// p of an otherwise zero word IS the fp32 subnormal code*2^(p-149); the matching
// multiplier a*2^(93-p) is an exact power-of-two rescale, so each product is
// a*code*2^-56 up to the single rounding of the FMA.  One logic op and one FMA
// per weight; two FMAs are issued as one packed fma.rn.f32x2.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kWorkers = 18;             // compute warps
constexpr int kWriterWarp = kWorkers;      // first of two writer warps: segment sg goes to writer sg & 1
constexpr int kGemvThreads = (kWorkers + 2) * 32;
constexpr int kChunk = 32;               // list entries per chunk (one per lane)
constexpr int kDepth = 3;                // chunks in flight per warp
constexpr unsigned long long kWaitNs = 1000000000ull;  // bound on every mbarrier wait: one second
constexpr int kMaxFusedN = 32768;        // largest n whose index collection can run inside the GEMV
constexpr int kFusedCols = 8192;         // list entries a CTA keeps in shared memory in that case

static int g_tune_ctas = 0;  // 0 = one CTA per SM
static int g_no_pdl = 0;     // 1 = plain stream-ordered launches

#ifdef SPQT_TRACE
__device__ long long* g_trace;  // time stamps of CTA 0 (debug builds only)
#define SPQT_TRACE_EVENT(cond, slot) do { if ((cond) && blockIdx.x == 0 && g_trace && (slot) < 4096) g_trace[(slot)] = clock64(); } while (0)
#else
#define SPQT_TRACE_EVENT(cond, slot) do { } while (0)
#endif

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ unsigned smem_u32(const void* p)
{
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait for the phase with the given parity; false when the bound
// (wall time, so that a logic error can never hold the GPU) expires.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity)
{
    const unsigned addr = smem_u32(bar);
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
        if (it == 16) t0 = global_ns();
        if (it > 16) {
            __nanosleep(64);
            if (global_ns() - t0 > kWaitNs) return false;
        }
    }
}

__device__ __forceinline__ void cp_async_16(unsigned smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
// the same, asking L2 to fetch no more than the 64 bytes around the address
__device__ __forceinline__ void cp_async_16_l2_64(unsigned smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global.L2::64B [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_8(unsigned smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global.L2::64B [%0], [%1], 8;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_4(unsigned smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global.L2::64B [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_4_ca(unsigned smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Two fp32 lanes in one 64-bit register, the operand form of the packed FMA.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi)
{
    asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// d = a * b + d on both lanes with one instruction
__device__ __forceinline__ void ffma2(unsigned long long& d, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

// acc[0..3] (eight fp32 sums, two per register) += the eight codes of one 32-bit word, each
// times a*2^-56; m01, m23, m40, m12 hold the multipliers a*2^(93-4j) paired as (0,1) (2,3) (4,0) (1,2).
__device__ __forceinline__ void fma_word(unsigned long long* acc, unsigned w, unsigned long long m01,
                                         unsigned long long m23, unsigned long long m40, unsigned long long m12)
{
    const unsigned v = w >> 20;
    ffma2(acc[0], pack2(__uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000f0u)), m01);
    ffma2(acc[1], pack2(__uint_as_float(w & 0x00000f00u), __uint_as_float(w & 0x0000f000u)), m23);
    ffma2(acc[2], pack2(__uint_as_float(w & 0x000f0000u), __uint_as_float(v & 0x0000000fu)), m40);
    ffma2(acc[3], pack2(__uint_as_float(v & 0x000000f0u), __uint_as_float(v & 0x00000f00u)), m12);
}

// acc (32 fp32 sums in 16 registers) += the 32 codes of a lane's 16 bytes, each times a (scaled by 2^-56).
__device__ __forceinline__ void fma_block16(unsigned long long* acc, const uint4& w, float a)
{
    const float m0 = a * 0x1p93f, m1 = a * 0x1p89f, m2 = a * 0x1p85f, m3 = a * 0x1p81f, m4 = a * 0x1p77f;
    const unsigned long long m01 = pack2(m0, m1), m23 = pack2(m2, m3), m40 = pack2(m4, m0), m12 = pack2(m1, m2);
    fma_word(acc + 0, w.x, m01, m23, m40, m12);
    fma_word(acc + 4, w.y, m01, m23, m40, m12);
    fma_word(acc + 8, w.z, m01, m23, m40, m12);
    fma_word(acc + 12, w.w, m01, m23, m40, m12);
}

// 3-bit codes: w2a, w2b are words of the 2-bit plane (byte i, field v = bits 2v..2v+1), w1 the word
// of the 1-bit plane whose byte i, bit u carries the top bit of the code in w2a (u = 2v) or w2b
// (u = 2v+1).  The fields are first widened to four words of eight 4-bit codes, then treated like
// 4-bit codes: word 0/1 = w2a fields v = {0,2} / {1,3}, word 2/3 = the same of w2b (low nibble first).
__device__ __forceinline__ void fma_block3(unsigned long long* acc, unsigned w2a, unsigned w2b, unsigned w1, float a)
{
    const unsigned c0 = (w2a & 0x33333333u) | ((w1 << 2) & 0x44444444u);
    const unsigned c1 = ((w2a >> 2) & 0x33333333u) | (w1 & 0x44444444u);
    const unsigned c2 = (w2b & 0x33333333u) | ((w1 << 1) & 0x44444444u);
    const unsigned c3 = ((w2b >> 2) & 0x33333333u) | ((w1 >> 1) & 0x44444444u);
    fma_block16(acc, make_uint4(c0, c1, c2, c3), a);
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

// ---------------------------------------------------------------- work map

// The piece of CTA c: block-rows r_first..r_last, and of each the slice of the
// active list that belongs to this CTA.  Uniform across the CTA.
constexpr int kSegTable = 16;  // segments of a CTA whose slices are computed once and kept in shared memory

struct Piece {
    int R, P, c, count, r_first, r_last;
    unsigned qc, rc;  // count = qc * P + rc: keeps the slice arithmetic in 32 bits (the host checks R * P < 2^31)
    const int* tab;   // shared memory: [2 * kSegTable] slice begin / end of the first segments, or nullptr

    // the block-rows of the piece do not depend on the count: computed while the count is being fetched
    __device__ __forceinline__ void init_rows(int R_, int P_, int c_)
    {
        R = R_; P = P_; c = c_;
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R;
        r_first = (int)(lo / (unsigned)P);
        r_last = (int)((hi - 1u) / (unsigned)P);
        tab = nullptr;
    }
    __device__ __forceinline__ void set_count(int count_)
    {
        count = count_;
        qc = (unsigned)count / (unsigned)P;
        rc = (unsigned)count - qc * (unsigned)P;
    }
    // floor(u * count / P) for 0 <= u <= P
    __device__ __forceinline__ int scaled(unsigned u) const { return (int)(u * qc + (u * rc) / (unsigned)P); }
    __device__ __forceinline__ void slice_compute(int row, int* a, int* b) const
    {
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R, base = (unsigned)row * (unsigned)P;
        const unsigned u0 = (lo > base ? lo : base) - base;
        const unsigned u1 = (hi < base + (unsigned)P ? hi : base + (unsigned)P) - base;
        *a = scaled(u0);
        *b = scaled(u1);
    }
    __device__ __forceinline__ void slice(int row, int* a, int* b) const
    {
        const int i = row - r_first;
        if (tab != nullptr && i < kSegTable) {
            *a = tab[2 * i];
            *b = tab[2 * i + 1];
        } else {
            slice_compute(row, a, b);
        }
    }
    // Fills the shared-memory table (threads 0..kSegTable-1 each take one segment, so the divisions
    // run side by side) -- call with the whole CTA, followed by a CTA barrier.
    __device__ __forceinline__ void fill_table(int* table, int tid)
    {
        if (tid < kSegTable && r_first + tid <= r_last) slice_compute(r_first + tid, &table[2 * tid], &table[2 * tid + 1]);
        tab = table;
    }
    // contributors to block-row `row`: CTAs first .. first+n-1
    __device__ __forceinline__ void contributors(int row, int* first, int* n) const
    {
        const unsigned f = ((unsigned)row * (unsigned)P) / (unsigned)R;
        const unsigned l = (((unsigned)row + 1u) * (unsigned)P - 1u) / (unsigned)R;
        *first = (int)f;
        *n = (int)(l - f + 1u);
    }
};

// A warp's position in its sequence of chunks: list position `pos` of the
// chunk's first entry inside block-row r (whose slice ends at p1).
struct Cursor {
    int r, pos, p1;
    __device__ __forceinline__ void settle(const Piece& pc, int warp)
    {
        while (r <= pc.r_last && pos >= p1) {
            ++r;
            if (r <= pc.r_last) {
                int p0;
                pc.slice(r, &p0, &p1);
                pos = p0 + warp * kChunk;
            }
        }
    }
    __device__ __forceinline__ void init(const Piece& pc, int warp)
    {
        r = pc.r_first;
        int p0;
        pc.slice(r, &p0, &p1);
        pos = p0 + warp * kChunk;
        settle(pc, warp);
    }
    __device__ __forceinline__ bool valid(const Piece& pc) const { return r <= pc.r_last; }
    __device__ __forceinline__ void advance(const Piece& pc, int warp)
    {
        pos += kWorkers * kChunk;
        if (pos >= p1) settle(pc, warp);
    }
};

// ---------------------------------------------------------------- kernel

template <int G, int BITS>
struct GemvSmem {
    static constexpr int B = G * BITS / 8;
    struct Stage {
        alignas(16) unsigned char codes[kChunk * B];  // block e of the chunk at e*B
        unsigned meta[3][kChunk];                     // words holding x_k, scale_rk, zero_rk of entry e
    };
    Stage stage[kWorkers][kDepth];
    alignas(16) int cols[kWorkers][2 * kDepth][kChunk];  // column numbers of the chunks ahead
    alignas(16) float red[2][kWorkers][G];               // per-warp partial sums of a finished segment
    float red_z[2][kWorkers];                            // and their offset terms
    uint64_t red_full[2], red_empty[2];
    int seg_table[2 * kSegTable];                        // slices of the CTA's first segments
    // fused index collection only
    alignas(16) int load_tot[kMaxFusedN / 256];  // active entries of every 256 entries of x
    int fused_cols[kFusedCols];                   // the part of the index list this CTA reads, when it fits
};

// FUSED: the index collection runs in the kernel's prologue.  Every CTA scans x (each lane tests 8
// entries, popc and warp-shuffle prefix sums; only the totals of every 256 entries cross shared
// memory), keeps the part of the ascending index list that its own slices cover in shared memory (or,
// when that part is too long, writes it to idx_out and reads it back like a list collected by a
// separate launch), and writes an even share of idx_out; CTA 0 writes the count.
template <int G, int BITS, bool DENSE, bool ODD_N, bool FUSED>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const uint8_t* __restrict__ codes, const __half* __restrict__ scales,
                 const __half* __restrict__ zeros, int R, int n,
                 const __half* __restrict__ x, const int32_t* idx_in,
                 const int32_t* count_ptr, __half* __restrict__ y,
                 int* __restrict__ counters, int* __restrict__ status,
                 float* __restrict__ partials, float* __restrict__ zpartials, int max_slots,
                 float thr, int32_t* idx_out, int32_t* count_out)
{
    constexpr int B = G * BITS / 8;
    constexpr int LPB = G / 32;       // lanes that share one block (each owns 32 of its rows)
    constexpr int CB = (B % 16 == 0) ? 16 : 8;   // bytes per copy: 3-bit blocks of 64 rows are only 8-byte aligned
    static_assert(BITS == 3 || BITS == 4, "3- or 4-bit codes");
    constexpr int SLOTS = 32 / LPB;   // blocks per 512-byte warp load
    constexpr int KEEP = 32 / SLOTS;  // values per lane after the in-warp reduce-scatter
    constexpr int SUBS = kChunk / SLOTS;  // 512-byte loads per chunk
    constexpr int D = kDepth;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    GemvSmem<G, BITS>& sm = *reinterpret_cast<GemvSmem<G, BITS>*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = gridDim.x, c = blockIdx.x;
    SPQT_TRACE_EVENT(tid == 0, 3990);
#ifdef SPQT_TRACE
    if (tid == 0 && g_trace && c < 200) g_trace[2000 + c] = (long long)global_ns();
#endif

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.red_full[b], kWorkers);
            mbar_init(&sm.red_empty[b], 1);
        }
    }
    __syncthreads();

    // Programmatic dependent launch: this grid may have been started while the previous kernel of
    // the stream was still draining.  Nothing above touches global memory; everything below waits
    // for that kernel to complete, and lets the next kernel of the stream start early in turn.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    int count = 0;
    if (!FUSED) count = DENSE ? n : *count_ptr;  // in flight while the row range is worked out
    Piece pc;
    pc.init_rows(R, P, c);
    const int32_t* idx = idx_in;
    int need_lo = 0;          // FUSED: first list position held in sm.fused_cols
    bool cols_local = false;  // FUSED: the pipeline reads its column numbers from sm.fused_cols
    if (FUSED) {
        // All loads first (one memory round trip).  A warp load covers 256 entries: lane l holds
        // entries 8l..8l+7.  Masks and counts stay in registers; only the per-load totals go through
        // shared memory, and every warp scans those totals for itself (no second barrier).
        constexpr int kWarps = kGemvThreads / 32;
        constexpr int kMaxLoads = (kMaxFusedN / 256 + kWarps - 1) / kWarps;
        const int nv = (n + 255) / 256;
        const bool vec_ok = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
        uint4 xv[kMaxLoads];
#pragma unroll
        for (int j = 0; j < kMaxLoads; ++j) {
            const int li = warp + j * kWarps;
            const int k0 = li * 256 + lane * 8;
            xv[j] = make_uint4(0u, 0u, 0u, 0u);
            if (li < nv) {
                if (vec_ok && k0 + 8 <= n) {
                    xv[j] = __ldg(reinterpret_cast<const uint4*>(x + k0));
                } else {
                    unsigned short hv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        hv[e] = (k0 + e < n) ? __ldg(reinterpret_cast<const unsigned short*>(x) + k0 + e) : (unsigned short)0;
                    xv[j].x = hv[0] | ((unsigned)hv[1] << 16);
                    xv[j].y = hv[2] | ((unsigned)hv[3] << 16);
                    xv[j].z = hv[4] | ((unsigned)hv[5] << 16);
                    xv[j].w = hv[6] | ((unsigned)hv[7] << 16);
                }
            }
        }
        // the largest fp16 value not above t (any negative value if t < 0: everything but NaN is
        // active; +inf if t is NaN or +inf: nothing is)
        const __half thr_h = (thr != thr) ? __ushort_as_half((unsigned short)0x7c00)
                                          : (thr < 0.0f ? __float2half_rn(-1.0f) : __float2half_rd(thr));
        const __half2 thr_h2 = __half2half2(thr_h);
        unsigned m8[kMaxLoads];   // activity of this lane's 8 entries of load j
        int lane_excl[kMaxLoads]; // active entries of load j in the lanes below
#pragma unroll
        for (int j = 0; j < kMaxLoads; ++j) {
            const int li = warp + j * kWarps;
            m8[j] = 0;
            lane_excl[j] = 0;
            if (li < nv) {  // uniform across the warp
                const int k0 = li * 256 + lane * 8;
                const unsigned wds[4] = {xv[j].x, xv[j].y, xv[j].z, xv[j].w};
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    // |x| > t  <=>  |x| > (largest fp16 value <= t): two entries per compare, in fp16,
                    // exact; the ordered compare is false for NaN
                    const unsigned ab = wds[e2] & 0x7fff7fffu;
                    const unsigned gt = __hgt2_mask(*reinterpret_cast<const __half2*>(&ab), thr_h2);
                    m8[j] |= ((gt & 1u) | ((gt >> 15) & 2u)) << (2 * e2);
                }
                const int left = n - k0;  // entries of this lane that exist
                if (left < 8) m8[j] &= (left <= 0) ? 0u : ((1u << left) - 1u);
                const int c8 = __popc(m8[j]);
                int incl = c8;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += up;
                }
                lane_excl[j] = incl - c8;
                if (lane == 31) sm.load_tot[li] = incl;
            }
        }
        SPQT_TRACE_EVENT(tid == 0, 3991);
        __syncthreads();
        SPQT_TRACE_EVENT(tid == 0, 3992);
        // every warp: exclusive scan of the (at most 128) load totals, four per lane
        int tot4[4], base4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) tot4[q] = (lane * 4 + q < nv) ? sm.load_tot[lane * 4 + q] : 0;
        const int s4 = tot4[0] + tot4[1] + tot4[2] + tot4[3];
        int incl4 = s4;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl4, o);
            if (lane >= o) incl4 += up;
        }
        base4[0] = incl4 - s4;
        base4[1] = base4[0] + tot4[0];
        base4[2] = base4[1] + tot4[1];
        base4[3] = base4[2] + tot4[2];
        count = __shfl_sync(0xffffffffu, incl4, 31);
        SPQT_TRACE_EVENT(tid == 0, 3993);
        pc.set_count(count);
        pc.fill_table(sm.seg_table, tid);
        __syncthreads();
        if (c == 0 && tid == 0) *count_out = count;
        // list positions this CTA will read: the union of its slices.  If that part fits in shared
        // memory the pipeline takes its column numbers from there (no round trip through global
        // memory); idx_out is then written once, an even share of the list per CTA.
        need_lo = count;
        int need_hi = 0;
        for (int r = pc.r_first; r <= pc.r_last; ++r) {
            int p0, p1;
            pc.slice(r, &p0, &p1);
            need_lo = min(need_lo, p0);
            need_hi = max(need_hi, p1);
        }
        cols_local = (need_hi - need_lo) <= kFusedCols;
        SPQT_TRACE_EVENT(tid == 0, 3994);
        const int out_lo = pc.scaled((unsigned)c), out_hi = pc.scaled((unsigned)c + 1u);
#pragma unroll
        for (int j = 0; j < kMaxLoads; ++j) {
            const int li = warp + j * kWarps;
            if (li < nv) {
                // first list position of load li: component li & 3 of lane li >> 2
                const int b0 = __shfl_sync(0xffffffffu, base4[0], li >> 2), b1 = __shfl_sync(0xffffffffu, base4[1], li >> 2);
                const int b2 = __shfl_sync(0xffffffffu, base4[2], li >> 2), b3 = __shfl_sync(0xffffffffu, base4[3], li >> 2);
                const int q = li & 3;
                const int first = (q == 0 ? b0 : q == 1 ? b1 : q == 2 ? b2 : b3) + lane_excl[j];
                const int last = first + __popc(m8[j]);
                const bool mine = last > need_lo && first < need_hi, share = last > out_lo && first < out_hi;
                if (mine || share) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        if ((m8[j] >> e) & 1u) {
                            const int pos = first + __popc(m8[j] & ((1u << e) - 1u));
                            const int col = li * 256 + lane * 8 + e;
                            const bool need = pos >= need_lo && pos < need_hi;
                            if (need && cols_local) sm.fused_cols[pos - need_lo] = col;
                            if ((need && !cols_local) || (pos >= out_lo && pos < out_hi)) idx_out[pos] = col;
                        }
                    }
                }
            }
        }
        __syncthreads();  // the CTA's own writes (shared or global) are visible to its pipeline
        idx = idx_out;
    } else {
        pc.set_count(count);
        pc.fill_table(sm.seg_table, tid);
        __syncthreads();
    }
    SPQT_TRACE_EVENT(tid == 0, 4000);

    if (warp >= kWriterWarp) {
        // ------------------------------------------------------------ writers
        // Two warps, one per hand-over buffer, so that the chains of dependent L2 round trips
        // (store, fence, counter, read back) of consecutive segments overlap.
        constexpr int RPL = G / 32;  // rows per lane
        const int b = warp - kWriterWarp;
        bool ok = true;
        for (int r = pc.r_first + b, sg = b; r <= pc.r_last; r += 2, sg += 2) {
            ok = mbar_wait(&sm.red_full[b], (sg >> 1) & 1);
            if (!ok) break;
            float v[RPL];
#pragma unroll
            for (int i = 0; i < RPL; ++i) v[i] = 0.0f;
            float zpart = 0.0f;
#pragma unroll
            for (int q = 0; q < kWorkers; ++q) {
#pragma unroll
                for (int i = 0; i < RPL; ++i) v[i] += sm.red[b][q][lane * RPL + i];
                zpart += sm.red_z[b][q];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.red_empty[b]);
            int first, nslots;
            pc.contributors(r, &first, &nslots);
            if (nslots == 1) {
                // this CTA holds the whole block-row: no partial, no counter, no fence
#pragma unroll
                for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(v[i] + zpart);
                continue;
            }
            const size_t pslot = (size_t)r * max_slots + (c - first);
#pragma unroll
            for (int i = 0; i < RPL; ++i) __stcg(partials + pslot * G + lane * RPL + i, v[i]);
            if (lane == 0) __stcg(zpartials + pslot, zpart);
            __threadfence();
            __syncwarp();
            int prev = 0;
            if (lane == 0) prev = atomicAdd(counters + r, 1);
            prev = __shfl_sync(0xffffffffu, prev, 0);
            if (prev == nslots - 1) {
                // last contributor of this block-row: combine in slot order
                __threadfence();
                float zsum = 0.0f;
#pragma unroll
                for (int i = 0; i < RPL; ++i) v[i] = 0.0f;
                const float* p = partials + (size_t)r * max_slots * G + lane * RPL;
                const float* zp = zpartials + (size_t)r * max_slots;
                // eight slots' loads in flight at a time; the additions keep the slot order
                for (int s0 = 0; s0 < nslots; s0 += 8) {
                    float pv[8][RPL], pz[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const bool in = s0 + j < nslots;
#pragma unroll
                        for (int i = 0; i < RPL; ++i) pv[j][i] = in ? __ldcg(p + (size_t)(s0 + j) * G + i) : 0.0f;
                        pz[j] = in ? __ldcg(zp + s0 + j) : 0.0f;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
#pragma unroll
                        for (int i = 0; i < RPL; ++i) v[i] += pv[j][i];
                        zsum += pz[j];
                    }
                }
#pragma unroll
                for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(v[i] + zsum);
                if (lane == 0) counters[r] = 0;  // leave the workspace ready for the next call
            }
        }
        SPQT_TRACE_EVENT(lane == 0, 4002);
#ifdef SPQT_TRACE
        if (lane == 0 && g_trace && c < 200) g_trace[2200 + c] = (long long)global_ns();
#endif
        if (!ok && lane == 0) atomicExch(status, 1);
        return;
    }

    // ---------------------------------------------------------------- workers
    const int slot = lane / LPB, h = lane % LPB;
    const unsigned short* xb = reinterpret_cast<const unsigned short*>(x);

    typename GemvSmem<G, BITS>::Stage* my_stage = &sm.stage[warp][0];
    int (*my_cols)[kChunk] = sm.cols[warp];

    Cursor ca, cb;  // stage A / stage B cursors (the consume side walks the segments itself)
    ca.init(pc, warp);
    cb = ca;
    // ring positions of the three stages: chunk number modulo the ring length, kept by wrap-around
    // (the lengths are not powers of two)
    unsigned qa2 = 0, qb1 = 0, qb2 = 0, qc1 = 0, qc2 = 0;  // ..1: modulo D (stages), ..2: modulo 2*D (columns)
    auto wrap = [](unsigned& v, unsigned len) { v = (v + 1 == len) ? 0u : v + 1; };

    // block-row constants of stage B, refreshed when its cursor enters a new block-row
    int b_row = -1;
    unsigned b_par = 0;                       // parity of r*n: which half of a word holds element (r,k)
    const uint8_t* b_codes = nullptr;         // codes of the block-row, this lane's 16-byte part
    const unsigned short* b_scales = nullptr; // scales / zeros of the block-row
    const unsigned short* b_zeros = nullptr;

    // stage A: column numbers of the warp's chunk number qa
    auto issue_a = [&]() {
        if (!DENSE && !(FUSED && cols_local) && ca.valid(pc)) {
            if (ca.pos + lane < ca.p1) cp_async_4(smem_u32(&my_cols[qa2][lane]), idx + ca.pos + lane);
            ca.advance(pc, warp);
            wrap(qa2, 2 * D);
        }
    };
    // stage B: code blocks and metadata words of chunk number qb (its columns have landed)
    auto issue_b = [&]() {
        if (cb.valid(pc)) {
            if (cb.r != b_row) {
                b_row = cb.r;
                const size_t row_base = (size_t)b_row * (size_t)n;
                b_par = (unsigned)(row_base & 1);
                b_codes = codes + row_base * B + (BITS == 4 ? 16 * h : 0);
                b_scales = reinterpret_cast<const unsigned short*>(scales) + row_base;
                b_zeros = reinterpret_cast<const unsigned short*>(zeros) + row_base;
            }
            const int valid = cb.p1 - cb.pos;  // entries of this chunk (>= kChunk when full)
            const int* cols = (FUSED && cols_local) ? &sm.fused_cols[cb.pos - need_lo] : my_cols[qb2];
            typename GemvSmem<G, BITS>::Stage& st = my_stage[qb1];
            const unsigned dst = smem_u32(&st.codes[0]) + lane * 16;
            if (BITS == 4) {
#pragma unroll
                for (int u = 0; u < SUBS; ++u) {
                    const int e = u * SLOTS + slot;
                    if (e < valid) {
                        const unsigned kk = DENSE ? (unsigned)(cb.pos + e) : (unsigned)cols[e];
                        if (DENSE) cp_async_16(dst + u * 512, b_codes + (size_t)kk * B);
                        else cp_async_16_l2_64(dst + u * 512, b_codes + (size_t)kk * B);
                    }
                }
            } else {
                // 3-bit blocks (48 or 24 bytes): the chunk's bytes in copies of CB bytes, lane after lane
                constexpr int NC = kChunk * B / CB / 32;
#pragma unroll
                for (int q = 0; q < NC; ++q) {
                    const int off = (q * 32 + lane) * CB;    // byte offset inside the chunk's stage
                    const int e = off / B, part = off % B;
                    if (e < valid) {
                        const unsigned kk = DENSE ? (unsigned)(cb.pos + e) : (unsigned)cols[e];
                        const uint8_t* src = b_codes + (size_t)kk * B + part;
                        const unsigned d = smem_u32(&st.codes[0]) + off;
                        if (CB == 16) {
                            if (DENSE) cp_async_16(d, src);
                            else cp_async_16_l2_64(d, src);
                        } else {
                            cp_async_8(d, src);
                        }
                    }
                }
            }
            if (lane < valid) {
                // the aligned 4-byte word that holds each fp16 value (index rounded down to even)
                const unsigned kk = DENSE ? (unsigned)(cb.pos + lane) : (unsigned)cols[lane];
                const unsigned mdst = smem_u32(&st.meta[0][lane]);
                const int mo = (int)kk - (int)((kk ^ b_par) & 1u);  // may be -1 only when r*n is odd: still inside the array
                if (!ODD_N || kk != (unsigned)(n - 1)) {
                    cp_async_4_ca(mdst, xb + (kk & ~1u));
                    cp_async_4(mdst + kChunk * 4, b_scales + mo);
                    cp_async_4(mdst + 2 * kChunk * 4, b_zeros + mo);
                } else {
                    // n odd: the word of the last column may reach past the end of an array; fetch directly
                    st.meta[0][lane] = (unsigned)__ldg(xb + kk) << ((kk & 1u) * 16);
                    st.meta[1][lane] = (unsigned)__ldg(b_scales + kk) << (((kk ^ b_par) & 1u) * 16);
                    st.meta[2][lane] = (unsigned)__ldg(b_zeros + kk) << (((kk ^ b_par) & 1u) * 16);
                }
            }
            cb.advance(pc, warp);
            wrap(qb1, D);
            wrap(qb2, 2 * D);
        }
    };

    // fill the pipeline: D chunks of columns, then D chunks of blocks (each needs its columns)
#pragma unroll 1
    for (int s = 0; s < D; ++s) {
        issue_a();
        cp_async_commit();
    }
#pragma unroll 1
    for (int s = 0; s < D; ++s) {
        cp_async_wait<D - 1>();
        __syncwarp();
        issue_b();
        issue_a();
        cp_async_commit();
    }

    unsigned long long acc[16];  // 32 fp32 sums, two per register
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0ull;
    bool ok = true;
#ifdef SPQT_TRACE
    long long tr_wait = 0, tr_issue = 0, tr_math = 0, tr_n = 0;
    SPQT_TRACE_EVENT(lane == 0, 3900 + warp);
#endif

    for (int r = pc.r_first, sg = 0; r <= pc.r_last; ++r, ++sg) {
        int p0, p1;
        pc.slice(r, &p0, &p1);
        const unsigned c_par = (unsigned)(((size_t)r * (size_t)n) & 1);
        float zl = 0.0f;  // this lane's share of sum x_k * zero_rk
        for (int pos = p0 + warp * kChunk; pos < p1; pos += kWorkers * kChunk) {
            // ---- stage C of chunk qc: everything it needs is in commit groups that wait<D-1> covers
#ifdef SPQT_TRACE
            const long long tc0 = clock64();
#endif
            cp_async_wait<D - 1>();
            __syncwarp();
#ifdef SPQT_TRACE
            const long long tc1 = clock64();
#endif
            const typename GemvSmem<G, BITS>::Stage& st = my_stage[qc1];
            const unsigned xw = st.meta[0][lane], sw = st.meta[1][lane], zw = st.meta[2][lane];
            unsigned kk;
            if (DENSE) kk = (unsigned)(pos + lane);
            else if (FUSED && cols_local) kk = (pos + lane < p1) ? (unsigned)sm.fused_cols[pos - need_lo + lane] : 0u;
            else kk = (unsigned)my_cols[qc2][lane];
#ifdef SPQT_TRACE
            const long long tc2 = clock64();
#endif
            float a = 0.0f;
            if (pos + lane < p1) {
                const unsigned xs = (kk & 1u) * 16, ms = ((kk ^ c_par) & 1u) * 16;
                const float xf = __half2float(__ushort_as_half((unsigned short)(xw >> xs)));
                const float sf = __half2float(__ushort_as_half((unsigned short)(sw >> ms)));
                const float zf = __half2float(__ushort_as_half((unsigned short)(zw >> ms)));
                a = xf * sf;  // exact; stays 0 past the end of the slice, where the code bytes are stale
                zl = fmaf(xf, zf, zl);
            }
#pragma unroll
            for (int u = 0; u < SUBS; ++u) {
                const float au = __shfl_sync(0xffffffffu, a, u * SLOTS + slot);
                if (BITS == 4) {
                    const uint4 wv = *reinterpret_cast<const uint4*>(&st.codes[0] + lane * 16 + u * 512);
                    fma_block16(acc, wv, au);
                } else {
                    // lane h of a block: words h and h+LPB of the 2-bit plane, word h of the 1-bit plane
                    const unsigned* blk = reinterpret_cast<const unsigned*>(&st.codes[0] + (u * SLOTS + slot) * B);
                    fma_block3(acc, blk[h], blk[h + LPB], blk[2 * LPB + h], au);
                }
            }
            __syncwarp();  // every lane has read its part of the slots that B and A now refill
            issue_b();
            issue_a();
            cp_async_commit();
            wrap(qc1, D);
            wrap(qc2, 2 * D);
#ifdef SPQT_TRACE
            tr_wait += tc1 - tc0; tr_issue += 0; tr_math += clock64() - tc2; ++tr_n;
#endif
        }

        // ---- end of the segment: in-warp reduce-scatter over the column slots, then hand the
        // per-warp sums to the writer warp
        const int b = sg & 1;
        if (sg >= 2) {
            ok = mbar_wait(&sm.red_empty[b], ((sg >> 1) - 1) & 1);
            if (!ok) break;
        }
        float accf[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            unpack2(acc[i], accf[2 * i], accf[2 * i + 1]);
            acc[i] = 0ull;
        }
        float t16[16], t8[8], t4[4], keep[4];
        halve<32>(accf, t16, lane, 16);
        halve<16>(t16, t8, lane, 8);
        halve<8>(t8, t4, lane, 4);
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
            const int ai = a_base + i;  // accumulator index = word*8 + nibble
            const int cw = ai >> 3, e2 = ai & 7;
            const int row = (BITS == 4)
                                ? 16 * h + 4 * cw + (e2 >> 1) + (e2 & 1) * (G / 2)
                                : 4 * h + (e2 >> 1) + (G / 8) * (cw >> 1) + (G / 4) * ((cw & 1) + 2 * (e2 & 1));
            sm.red[b][warp][row] = keep[i] * 0x1p56f;  // undo the 2^-56 of the subnormal trick
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zl += __shfl_xor_sync(0xffffffffu, zl, o);
        if (lane == 0) sm.red_z[b][warp] = zl;
        __syncwarp();
        SPQT_TRACE_EVENT(tid == 0, 3950 + sg);
        if (lane == 0) mbar_arrive(&sm.red_full[b]);
    }
    cp_async_wait<0>();
    SPQT_TRACE_EVENT(tid == 0, 4001);
#ifdef SPQT_TRACE
    if (blockIdx.x == 0 && lane == 0 && g_trace) {
        g_trace[3000 + warp * 4 + 0] = tr_wait; g_trace[3000 + warp * 4 + 1] = tr_issue;
        g_trace[3000 + warp * 4 + 2] = tr_math; g_trace[3000 + warp * 4 + 3] = tr_n;
    }
#endif
    if (!ok && lane == 0) atomicExch(status, 1);
}

// ---------------------------------------------------------------- host side

struct FusedArgs {
    float t;
    int32_t* idx_out;
    int32_t* count_out;
};

template <int G, int BITS, bool DENSE, bool ODD_N, bool FUSED>
static spqt_status launch_gemv(const Format& f, const void* codes, const void* scales,
                               const void* zeros, const void* x, const int32_t* idx,
                               const int32_t* count, void* y, void* workspace, cudaStream_t s,
                               FusedArgs fa)
{
    auto kernel = gemv_kernel<G, BITS, DENSE, ODD_N, FUSED>;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(GemvSmem<G, BITS>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    int P = g_tune_ctas > 0 ? g_tune_ctas : sms;
    // With few block-rows, a whole number of CTAs per block-row (if that keeps >= 85 % of the SMs
    // busy) gives every CTA a single segment: no CTA then carries two aggregation chains.
    if (g_tune_ctas == 0 && f.R <= P && (P / f.R) * f.R * 100 >= 85 * P) P = (P / f.R) * f.R;
    // no more CTAs than pieces of at least 64 columns of one block-row
    const long long pieces = (long long)f.R * ((f.n + 63) / 64);
    if (P > pieces) P = (int)pieces;
    if (P > kMaxCtas) P = kMaxCtas;
    if (P < 1) P = 1;
    const int slots = max_slots(f.R);
    int* counters = static_cast<int*>(workspace);
    int* status = counters + f.R;
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + header_bytes(f.R));
    float* zpartials = partials + (size_t)f.R * slots * G;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(P);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    const cudaError_t err = cudaLaunchKernelEx(
        &cfg, kernel, static_cast<const uint8_t*>(codes), static_cast<const __half*>(scales),
        static_cast<const __half*>(zeros), f.R, f.n, static_cast<const __half*>(x), idx, count,
        static_cast<__half*>(y), counters, status, partials, zpartials, slots,
        fa.t, fa.idx_out, fa.count_out);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

template <bool DENSE, bool FUSED = false>
static spqt_status gemv_entry(const void* codes, const void* scales, const void* zeros,
                              int m, int n, int bits, int group, const void* x,
                              const int32_t* idx, const int32_t* count, void* y,
                              void* workspace, size_t ws_bytes, void* stream,
                              FusedArgs fa = FusedArgs{0.0f, nullptr, nullptr})
{
    if (!codes || !scales || !zeros || !x || !y || !workspace) return SPQT_ERR_INVALID_ARG;
    if (!DENSE && (!idx || !count)) return SPQT_ERR_INVALID_ARG;
    if (FUSED && n > kMaxFusedN) return SPQT_ERR_UNSUPPORTED;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (!aligned(codes, 16) || !aligned(scales, 16) || !aligned(zeros, 16) || !aligned(x, 4) ||
        !aligned(y, 2) || !aligned(workspace, 16) || (!DENSE && (!aligned(idx, 4) || !aligned(count, 4))))
        return SPQT_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(f)) return SPQT_ERR_WORKSPACE;
    if ((long long)f.R * kMaxCtas >= (1ll << 31)) return SPQT_ERR_UNSUPPORTED;  // the work map is 32-bit
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool odd = (n & 1) != 0;
#define SPQT_DISPATCH(GG, BB)                                                                                      \
    return odd ? launch_gemv<GG, BB, DENSE, true, FUSED>(f, codes, scales, zeros, x, idx, count, y, workspace, s, fa) \
               : launch_gemv<GG, BB, DENSE, false, FUSED>(f, codes, scales, zeros, x, idx, count, y, workspace, s, fa)
    if (bits == 4 && group == 128) { SPQT_DISPATCH(128, 4); }
    if (bits == 4 && group == 64) { SPQT_DISPATCH(64, 4); }
    if (bits == 3 && group == 128) { SPQT_DISPATCH(128, 3); }
    if (bits == 3 && group == 64) { SPQT_DISPATCH(64, 3); }
#undef SPQT_DISPATCH
    return SPQT_ERR_UNSUPPORTED;
}

}  // namespace spqt

// Scratch of the entry point that allocates nothing: one block-row counter array, status word and
// partial-sum area, resident in every device that loads the library until the process exits.
constexpr size_t kStaticScratchBytes = size_t(1) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

#ifdef SPQT_TRACE
extern "C" int spqt_debug_set_trace(void* buf) { return (int)cudaMemcpyToSymbol(spqt::g_trace, &buf, sizeof(buf)); }
#endif

extern "C" {

spqt_status spqt_sparse_gemv(const void* codes, const void* scales, const void* zeros,
                             int m, int n, int bits, int group,
                             const void* x, const int32_t* idx, const int32_t* count,
                             void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::gemv_entry<false>(codes, scales, zeros, m, n, bits, group, x, idx, count, y,
                                   workspace, workspace_bytes, stream);
}

spqt_status spqt_sparsify_gemv(const void* codes, const void* scales, const void* zeros,
                               int m, int n, int bits, int group,
                               const void* x, float t, int32_t* idx, int32_t* count,
                               void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    if (n > spqt::kMaxFusedN) {
        // too long for the in-kernel scan: the same result from the two separate launches
        spqt_status st = spqt_sparsify(x, n, t, idx, count, stream);
        if (st != SPQT_OK) return st;
        return spqt_sparse_gemv(codes, scales, zeros, m, n, bits, group, x, idx, count, y, workspace,
                                workspace_bytes, stream);
    }
    return spqt::gemv_entry<false, true>(codes, scales, zeros, m, n, bits, group, x, idx, count, y,
                                         workspace, workspace_bytes, stream,
                                         spqt::FusedArgs{t, idx, count});
}

spqt_status spqt_dense_gemv(const void* codes, const void* scales, const void* zeros,
                            int m, int n, int bits, int group, const void* x,
                            void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::gemv_entry<true>(codes, scales, zeros, m, n, bits, group, x, nullptr, nullptr, y,
                                  workspace, workspace_bytes, stream);
}

spqt_status spqt_sparse_gemv_static(const void* codes, const void* scales, const void* zeros,
                                    int m, int n, int bits, int group,
                                    const void* x, const int32_t* idx, const int32_t* count,
                                    void* y, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (workspace_bytes(f) > kStaticScratchBytes) return SPQT_ERR_WORKSPACE;  // problem too large for the built-in scratch
    // In host code the array's name is only a handle; the device address has to be asked for,
    // once per device, with that device current.
    static void* scratch_addr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    if (scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return SPQT_ERR_CUDA;
        scratch_addr[dev] = p;
    }
    // The scratch keeps whatever the previous call (or an interrupted one) left: the arrival
    // counters and the status word must start at zero.
    if (cudaMemsetAsync(scratch_addr[dev], 0, header_bytes(f.R), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return SPQT_ERR_CUDA;
    return gemv_entry<false>(codes, scales, zeros, m, n, bits, group, x, idx, count, y,
                             scratch_addr[dev], kStaticScratchBytes, stream);
}

spqt_status spqt_set_tuning(int gemv_ctas, int reserved)
{
    if (gemv_ctas < 0 || reserved < 0 || reserved > 1) return SPQT_ERR_INVALID_ARG;
    spqt::g_tune_ctas = gemv_ctas;
    spqt::g_no_pdl = reserved;
    return SPQT_OK;
}

spqt_status spqt_workspace_status(const void* workspace, int m, int group, int* status_host, void* stream)
{
    if (!workspace || !status_host || m <= 0 || (group != 64 && group != 128) || m % group) return SPQT_ERR_INVALID_ARG;
    const int* word = static_cast<const int*>(workspace) + m / group;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(status_host, word, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return SPQT_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SPQT_ERR_CUDA;
    return SPQT_OK;
}

}  // extern "C"
