// Activation-sparse GEMV over the zigzag layout, and its dense twin (4-bit codes).
//
// Work decomposition (the paper's hybrid row/column parallelism, generalised):
// the R block-rows are laid end to end and cut into P equal pieces, one per CTA,
// P = one persistent CTA per SM.  A piece is a run of (fractions of) block-rows;
// the fraction [u0,u1) of block-row r means the slice
// [u0*count, u1*count) of the ACTIVE index list, so the load follows the active
// entries, not the matrix columns, and every CTA streams the same number of
// blocks whatever R is.  Each (CTA, block-row) segment yields G fp32 partial
// sums; whichever CTA contributes last to a block-row (arrive-only counter:
// nobody waits on another CTA) adds the partials in a fixed order, adds the
// offset term and rounds to fp16.
//
// Inside a CTA the warps are specialised:
//   * producer warps walk the segment in tiles of kTile list entries, gather
//     idx, x, scale and zero for the tile and leave in shared memory the byte
//     offset of every active block, its multiplier a = x_k*scale_rk (exact in
//     fp32) and the tile's offset term sum x_k*zero_rk;
//   * consumer warps stream the code blocks with 16-byte cp.async into a
//     private ring of kStages x 512 B per warp (deep memory-level parallelism,
//     no registers held, no barrier: a lane reads back what it copied) and do
//     the dequantize-FMA work.
//   * one writer warp takes the consumers' per-warp sums at the end of a
//     segment, adds them, publishes the partial and, if its CTA is the last
//     contributor of the block-row, produces y -- so the fence and the global
//     round trip never stall the streaming warps.
// Producers run a tile ahead; tiles are handed over with mbarriers whose waits
// are bounded (on expiry an error word is set and the kernel drains and exits).
//
// Arithmetic:  y[j] = sum_k a_k * code_jk + sum_k x_k * zero_rk.  A 4-bit code
// becomes an fp32 operand with no conversion: the nibble masked in place at bit
// p of an otherwise zero word IS the fp32 subnormal code*2^(p-149); the matching
// multiplier a*2^(93-p) is an exact power-of-two rescale, so each product is
// a*code*2^-56 up to the single rounding of the FMA.  One logic op and one FMA
// per weight; two FMAs are issued as one packed fma.rn.f32x2.
#include "spqt_common.cuh"

namespace spqt {

constexpr int kConsumerWarps = 13;
constexpr int kProducerWarps = 2;
constexpr int kWriterWarp = kConsumerWarps + kProducerWarps;  // one more warp combines and writes partial sums
constexpr int kGemvThreads = (kConsumerWarps + kProducerWarps + 1) * 32;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kSub = 2;                  // 512-byte warp loads per step (one commit / wait per step)
constexpr int kStages = 8;               // ring depth per consumer warp, in steps (x kSub x 512 B)
constexpr int kTile = 1024;              // list entries staged per tile
constexpr int kTileBufs = 4;             // tiles in flight between producers and consumers
constexpr int kTilePerThread = kTile / kProducerThreads;
constexpr unsigned long long kWaitNs = 1000000000ull;  // bound on every mbarrier wait: one second

static int g_tune_ctas = 0;  // 0 = one CTA per SM

#ifdef SPQT_TRACE
__device__ long long* g_trace;  // [role][event] time stamps of CTA 0 (debug builds only)
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

// Non-blocking probe of the same condition.
__device__ __forceinline__ bool mbar_test(uint64_t* bar, unsigned parity)
{
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// Wait until at most `allow` of this thread's copy groups are still in flight
// (rounded down to an encodable count, which only waits longer).
__device__ __forceinline__ void cp_async_wait_at_most(int allow)
{
    if (allow >= kStages - 1) cp_async_wait<kStages - 1>();
    else if (allow >= 4) cp_async_wait<4>();
    else if (allow >= 2) cp_async_wait<2>();
    else if (allow >= 1) cp_async_wait<1>();
    else cp_async_wait<0>();
}

__device__ __forceinline__ void named_barrier_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// d = a * b + d on two fp32 lanes with one instruction
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, float b0, float b1)
{
    unsigned long long a, b, c;
    asm("mov.b64 %0, {%1,%2};" : "=l"(a) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1,%2};" : "=l"(b) : "f"(b0), "f"(b1));
    asm("mov.b64 %0, {%1,%2};" : "=l"(c) : "f"(d0), "f"(d1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(c) : "l"(a), "l"(b));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(d0), "=f"(d1) : "l"(c));
}

// acc[0..7] += the eight codes of one 32-bit word, each times a*2^-56;
// mul[j] = a * 2^(93-4j), j = 0..4.
__device__ __forceinline__ void fma_word(float* acc, unsigned w, const float* mul)
{
    const unsigned v = w >> 20;
    ffma2(acc[0], acc[1], __uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000f0u), mul[0], mul[1]);
    ffma2(acc[2], acc[3], __uint_as_float(w & 0x00000f00u), __uint_as_float(w & 0x0000f000u), mul[2], mul[3]);
    ffma2(acc[4], acc[5], __uint_as_float(w & 0x000f0000u), __uint_as_float(v & 0x0000000fu), mul[4], mul[0]);
    ffma2(acc[6], acc[7], __uint_as_float(v & 0x000000f0u), __uint_as_float(v & 0x00000f00u), mul[1], mul[2]);
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

// Walks the tiles of one CTA's piece, segment by segment.  All members are
// uniform across the CTA; producers and consumers each run their own copy and
// see the same sequence.
struct TileWalk {
    int R, P, c, count;
    int r, r_last;   // current / last block-row of the piece
    int p1;          // end of the current segment's list slice
    int t0, len;     // current tile: first list position, entries
    int tg;          // running tile number (selects buffer and phase)
    bool last_of_segment;

    __device__ __forceinline__ void slice(int row, int* a, int* b) const
    {
        const long long lo = (long long)c * R, hi = lo + R, base = (long long)row * P;
        const long long u0 = (lo > base ? lo : base) - base;
        const long long u1 = (hi < base + P ? hi : base + P) - base;
        *a = (int)((u0 * count) / P);
        *b = (int)((u1 * count) / P);
    }
    __device__ __forceinline__ void set_tile(int start)
    {
        t0 = start;
        len = min(kTile, p1 - t0);
        last_of_segment = (t0 + len >= p1);
    }
    __device__ __forceinline__ void init(int R_, int P_, int c_, int count_)
    {
        R = R_; P = P_; c = c_; count = count_;
        const long long lo = (long long)c * R, hi = lo + R;
        r = (int)(lo / P);
        r_last = (int)((hi - 1) / P);
        tg = 0;
        int p0;
        slice(r, &p0, &p1);
        set_tile(p0);
    }
    __device__ __forceinline__ bool valid() const { return r <= r_last; }
    __device__ __forceinline__ void next()
    {
        ++tg;
        if (!last_of_segment) {
            set_tile(t0 + len);
        } else {
            ++r;
            if (r <= r_last) {
                int p0;
                slice(r, &p0, &p1);
                set_tile(p0);
            }
        }
    }
    // contributors to block-row `row`: CTAs first..last; this CTA's slot among them
    __device__ __forceinline__ void contributors(int row, int* first, int* n) const
    {
        const int f = (int)(((long long)row * P) / R);
        const int l = (int)((((long long)row + 1) * P - 1) / R);
        *first = f;
        *n = l - f + 1;
    }
};

// ---------------------------------------------------------------- kernel

template <int G>
struct GemvSmem {
    static constexpr int B = G / 2;
    alignas(16) unsigned char ring[kConsumerWarps][kStages][kSub * 512];
    alignas(16) unsigned off[kTileBufs][kTile];   // byte offset of the block inside its block-row
    alignas(16) float a[kTileBufs][kTile];        // x_k * scale_rk
    alignas(16) float red[2][kConsumerWarps][G];  // per-warp partial sums of a finished segment
    float red_z[2];                               // its offset term
    float zs_warp[kTileBufs][kProducerWarps];
    float zs_tile[kTileBufs];
    uint64_t full_off[kTileBufs], full_a[kTileBufs], empty[kTileBufs];
    uint64_t red_full[2], red_empty[2];
};

template <int G, bool DENSE>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_int4_kernel(const uint8_t* __restrict__ codes, const __half* __restrict__ scales,
                 const __half* __restrict__ zeros, int R, int n,
                 const __half* __restrict__ x, const int32_t* __restrict__ idx,
                 const int32_t* __restrict__ count_ptr, __half* __restrict__ y,
                 int* __restrict__ counters, int* __restrict__ status,
                 float* __restrict__ partials, float* __restrict__ zpartials, int max_slots)
{
    constexpr int B = G / 2;
    constexpr int LPB = B / 16;       // lanes that share one block
    constexpr int SLOTS = 32 / LPB;   // blocks per warp step
    constexpr int KEEP = 32 / SLOTS;  // values per lane after the in-warp reduce-scatter

    extern __shared__ __align__(16) unsigned char smem_raw[];
    GemvSmem<G>& sm = *reinterpret_cast<GemvSmem<G>*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = gridDim.x, c = blockIdx.x;

    if (tid == 0) {
        for (int b = 0; b < kTileBufs; ++b) {
            mbar_init(&sm.full_off[b], kProducerThreads);
            mbar_init(&sm.full_a[b], kProducerThreads);
            mbar_init(&sm.empty[b], kConsumerWarps);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.red_full[b], kConsumerWarps);
            mbar_init(&sm.red_empty[b], 1);
        }
    }
    __syncthreads();

    const int count = DENSE ? n : *count_ptr;
    SPQT_TRACE_EVENT(tid == 0, 4000);

    if (warp >= kConsumerWarps && warp < kWriterWarp) {
        // ------------------------------------------------------------ producers
        const int pt = tid - kConsumerThreads, pw = warp - kConsumerWarps;
        const unsigned short* xb = reinterpret_cast<const unsigned short*>(x);
        const unsigned short* sb = reinterpret_cast<const unsigned short*>(scales);
        const unsigned short* zb = reinterpret_cast<const unsigned short*>(zeros);

        // column of list entry i of a tile (entries past the tile's end repeat its last one,
        // so that every load below is unconditional and in bounds)
        auto load_cols = [&](const TileWalk& t, int* k) {
            if (t.len > 0) {
#pragma unroll
                for (int u = 0; u < kTilePerThread; ++u) {
                    const int i = min(pt + u * kProducerThreads, t.len - 1);
                    k[u] = DENSE ? (t.t0 + i) : __ldg(idx + t.t0 + i);
                }
            } else {
#pragma unroll
                for (int u = 0; u < kTilePerThread; ++u) k[u] = 0;
            }
        };

        TileWalk w;
        w.init(R, P, c, count);
        int k[kTilePerThread];
        if (w.valid()) load_cols(w, k);
        bool ok = true;
        while (w.valid()) {
            const int buf = w.tg % kTileBufs;
            SPQT_TRACE_EVENT(pt == 0, w.tg * 4 + 0);
            if (w.tg >= kTileBufs) ok = mbar_wait(&sm.empty[buf], ((w.tg / kTileBufs) - 1) & 1);
            if (!ok) break;
            SPQT_TRACE_EVENT(pt == 0, w.tg * 4 + 1);
            const size_t row_base = (size_t)w.r * (size_t)n;
#pragma unroll
            for (int u = 0; u < kTilePerThread; ++u)
                sm.off[buf][pt + u * kProducerThreads] = (unsigned)k[u] * (unsigned)B;
            mbar_arrive(&sm.full_off[buf]);
            SPQT_TRACE_EVENT(pt == 0, w.tg * 4 + 2);
            // all gathers of this tile in flight at once, then the next tile's columns
            unsigned short xr[kTilePerThread], sr[kTilePerThread], zr[kTilePerThread];
#pragma unroll
            for (int u = 0; u < kTilePerThread; ++u) {
                xr[u] = __ldg(xb + k[u]);
                sr[u] = __ldg(sb + row_base + k[u]);
                zr[u] = __ldg(zb + row_base + k[u]);
            }
            TileWalk wn = w;
            wn.next();
            int kn[kTilePerThread];
            if (wn.valid()) load_cols(wn, kn);
            float zs = 0.0f;
#pragma unroll
            for (int u = 0; u < kTilePerThread; ++u) {
                const bool in = pt + u * kProducerThreads < w.len;
                const float xf = in ? __half2float(__ushort_as_half(xr[u])) : 0.0f;
                sm.a[buf][pt + u * kProducerThreads] = xf * __half2float(__ushort_as_half(sr[u]));  // exact
                zs = fmaf(xf, __half2float(__ushort_as_half(zr[u])), zs);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) zs += __shfl_xor_sync(0xffffffffu, zs, o);
            if (lane == 0) sm.zs_warp[buf][pw] = zs;
            named_barrier_sync(2, kProducerThreads);
            if (pt == 0) {
                float t = 0.0f;
#pragma unroll
                for (int q = 0; q < kProducerWarps; ++q) t += sm.zs_warp[buf][q];
                sm.zs_tile[buf] = t;
            }
            mbar_arrive(&sm.full_a[buf]);
            SPQT_TRACE_EVENT(pt == 0, w.tg * 4 + 3);
            w = wn;
#pragma unroll
            for (int u = 0; u < kTilePerThread; ++u) k[u] = kn[u];
        }
        if (!ok && pt == 0) atomicExch(status, 1);
        return;
    }

    if (warp == kWriterWarp) {
        // ------------------------------------------------------------ writer
        constexpr int RPL = G / 32;  // rows per lane
        TileWalk w;
        w.init(R, P, c, count);
        const int r_first = w.r, r_last = w.r_last;
        bool ok = true;
        for (int r = r_first, sg = 0; r <= r_last; ++r, ++sg) {
            const int b = sg & 1;
            ok = mbar_wait(&sm.red_full[b], (sg >> 1) & 1);
            if (!ok) break;
            float v[RPL];
#pragma unroll
            for (int i = 0; i < RPL; ++i) v[i] = 0.0f;
#pragma unroll
            for (int q = 0; q < kConsumerWarps; ++q)
#pragma unroll
                for (int i = 0; i < RPL; ++i) v[i] += sm.red[b][q][lane * RPL + i];
            const float zpart = sm.red_z[b];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.red_empty[b]);
            int first, nslots;
            w.contributors(r, &first, &nslots);
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
                for (int s2 = 0; s2 < nslots; ++s2) {
#pragma unroll
                    for (int i = 0; i < RPL; ++i) v[i] += __ldcg(p + (size_t)s2 * G + i);
                    zsum += __ldcg(zp + s2);
                }
#pragma unroll
                for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(v[i] + zsum);
                if (lane == 0) counters[r] = 0;  // leave the workspace ready for the next call
            }
        }
        if (!ok && lane == 0) atomicExch(status, 1);
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int slot = lane / LPB, h = lane % LPB;
    constexpr unsigned kStepBytes = kSub * 512;
    constexpr unsigned kRingBytes = kStages * kStepBytes;
    constexpr int kStepCols = kSub * SLOTS;               // list entries per step
    constexpr int kStride = kConsumerWarps * kStepCols;   // list entries between two steps of one warp
    const unsigned ring_base = smem_u32(&sm.ring[warp][0][0]) + lane * 16;

    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
    float zacc = 0.0f;  // meaningful in consumer thread 0 only
    bool ok = true;

    // ---- issue side: runs up to kStages steps (and at most kTileBufs-1 tiles) ahead
    TileWalk wi;
    wi.init(R, P, c, count);
    int ie = warp * kStepCols;        // first list entry (within the tile) of the next step to issue
    bool i_open = false;              // current issue tile staged and has steps left for this warp
    const unsigned* i_off = nullptr;  // &off[buf][slot]
    const uint8_t* i_row = nullptr;   // codes of the tile's block-row, this lane's 16-byte part
    unsigned ring_w = 0, ring_r = 0;
    int in_flight = 0;
    int consume_tg = 0;               // tile the consume side is in

    // Move to the next tile in which this warp has a step, if producers have staged it.
    // Only blocks when `must` (nothing in flight, so the consume side cannot go on otherwise).
    auto open_issue_tile = [&](bool must) {
        while (wi.valid() && ie >= wi.len) {
            wi.next();
            ie = warp * kStepCols;
        }
        if (!wi.valid() || wi.tg > consume_tg + (kTileBufs - 1)) return;
        const int buf = wi.tg % kTileBufs;
        const unsigned parity = (wi.tg / kTileBufs) & 1;
        if (must) {
            ok = mbar_wait(&sm.full_off[buf], parity);
            if (!ok) return;
        } else if (!mbar_test(&sm.full_off[buf], parity)) {
            return;
        }
        i_off = &sm.off[buf][slot];
        i_row = codes + (size_t)wi.r * (size_t)n * B + 16 * h;
        i_open = true;
    };
    auto top_up = [&]() {
        while (in_flight < kStages) {
            if (!i_open) {
                open_issue_tile(in_flight == 0);
                if (!i_open) return;
            }
#pragma unroll
            for (int u = 0; u < kSub; ++u) {
#ifdef SPQT_NO_COPY
                if (false) {
#else
                if (ie + u * SLOTS + slot < wi.len) {
#endif
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_base + ring_w + u * 512),
                                 "l"(i_row + i_off[ie + u * SLOTS])
                                 : "memory");
                }
            }
            cp_async_commit();
            ring_w = (ring_w + kStepBytes) & (kRingBytes - 1);
            ++in_flight;
            ie += kStride;
            if (ie >= wi.len) i_open = false;
        }
    };
    // next step's codes and multipliers into registers (its copies have been in flight for kStages steps)
    struct Step {
        uint4 w[kSub];
        float a[kSub];
    };
    auto fetch = [&](const float* a_ptr, int e, Step& st) {
        top_up();
        cp_async_wait_at_most(in_flight - 1);
#pragma unroll
        for (int u = 0; u < kSub; ++u) {
            st.w[u] = *reinterpret_cast<const uint4*>(&sm.ring[warp][0][0] + lane * 16 + ring_r + u * 512);
            st.a[u] = a_ptr[e + u * SLOTS];  // 0 past the tile's end: stale ring data is harmless
        }
        ring_r = (ring_r + kStepBytes) & (kRingBytes - 1);
        --in_flight;
    };
    auto math = [&](const Step& st) {
#ifdef SPQT_NO_MATH
        acc[0] += __uint_as_float(st.w[0].x ^ st.w[1].y) * st.a[0] + st.a[1];
        return;
#endif
#pragma unroll
        for (int u = 0; u < kSub; ++u) {
            float mul[5];
            mul[0] = st.a[u] * 0x1p93f;
            mul[1] = st.a[u] * 0x1p89f;
            mul[2] = st.a[u] * 0x1p85f;
            mul[3] = st.a[u] * 0x1p81f;
            mul[4] = st.a[u] * 0x1p77f;
            fma_word(acc + 0, st.w[u].x, mul);
            fma_word(acc + 8, st.w[u].y, mul);
            fma_word(acc + 16, st.w[u].z, mul);
            fma_word(acc + 24, st.w[u].w, mul);
        }
    };

    // ---- consume side
    TileWalk wc;
    wc.init(R, P, c, count);
    int sg = 0;  // segments finished by this CTA
    for (; wc.valid() && ok; wc.next()) {
        const int buf = wc.tg % kTileBufs;
        consume_tg = wc.tg;
        top_up();
        if (!ok) break;
        // every warp observes every tile's hand-over before releasing it
        ok = mbar_wait(&sm.full_a[buf], (wc.tg / kTileBufs) & 1);
        if (!ok) break;
        if (tid == 0) zacc += sm.zs_tile[buf];
        SPQT_TRACE_EVENT(tid == 0, 1024 + wc.tg * 4 + 0);
        const float* a_ptr = &sm.a[buf][slot];
        int e = warp * kStepCols;
        if (e < wc.len) {
            // two steps in registers: the next one is fetched before this one's arithmetic
            Step s0, s1;
            fetch(a_ptr, e, s0);
            for (;;) {
                e += kStride;
                if (e >= wc.len) { math(s0); break; }
                fetch(a_ptr, e, s1);
                math(s0);
                e += kStride;
                if (e >= wc.len) { math(s1); break; }
                fetch(a_ptr, e, s0);
                math(s1);
            }
        }
        if (!ok) break;
        __syncwarp();
        SPQT_TRACE_EVENT(tid == 0, 1024 + wc.tg * 4 + 1);
        if (lane == 0) mbar_arrive(&sm.empty[buf]);
        if (wc.last_of_segment) {
            // ---- segment epilogue: in-warp reduce-scatter over the column slots,
            // then hand the per-warp sums to the writer warp
            const int b = sg & 1;
            if (sg >= 2) {
                ok = mbar_wait(&sm.red_empty[b], ((sg >> 1) - 1) & 1);
                if (!ok) break;
            }
            float t16[16], t8[8], t4[4], keep[4];
            halve<32>(acc, t16, lane, 16);
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
                const int row = 16 * h + 4 * cw + (e2 >> 1) + (e2 & 1) * (G / 2);
                sm.red[b][warp][row] = keep[i] * 0x1p56f;  // undo the 2^-56 of the subnormal trick
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
            if (tid == 0) {
                sm.red_z[b] = zacc;
                zacc = 0.0f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.red_full[b]);
            ++sg;
        }
        SPQT_TRACE_EVENT(tid == 0, 1024 + wc.tg * 4 + 2);
    }
    cp_async_wait<0>();
    SPQT_TRACE_EVENT(tid == 0, 4001);
    if (!ok && lane == 0) atomicExch(status, 1);
}

// ---------------------------------------------------------------- host side

template <int G, bool DENSE>
static spqt_status launch_int4(const Format& f, const void* codes, const void* scales,
                               const void* zeros, const void* x, const int32_t* idx,
                               const int32_t* count, void* y, void* workspace, cudaStream_t s)
{
    auto kernel = gemv_int4_kernel<G, DENSE>;
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(GemvSmem<G>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SPQT_ERR_CUDA;
        configured[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    int P = g_tune_ctas > 0 ? g_tune_ctas : sms;
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
    kernel<<<P, kGemvThreads, smem, s>>>(
        static_cast<const uint8_t*>(codes), static_cast<const __half*>(scales),
        static_cast<const __half*>(zeros), f.R, f.n, static_cast<const __half*>(x), idx, count,
        static_cast<__half*>(y), counters, status, partials, zpartials, slots);
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
    if ((size_t)n * (size_t)f.B > 0xffffffffull) return SPQT_ERR_UNSUPPORTED;  // 32-bit offsets inside a block-row
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

spqt_status spqt_dense_gemv(const void* codes, const void* scales, const void* zeros,
                            int m, int n, int bits, int group, const void* x,
                            void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::gemv_entry<true>(codes, scales, zeros, m, n, bits, group, x, nullptr, nullptr, y,
                                  workspace, workspace_bytes, stream);
}

spqt_status spqt_set_tuning(int gemv_ctas, int reserved)
{
    if (gemv_ctas < 0 || reserved < 0) return SPQT_ERR_INVALID_ARG;
    spqt::g_tune_ctas = gemv_ctas;
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
