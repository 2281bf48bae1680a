// Activation-sparse GEMV over the zigzag layout, and its dense twin (4-bit and 3-bit codes).
//
// Work decomposition (the paper's hybrid row/column parallelism, generalised):
// the R block-rows are laid end to end and cut into P equal pieces, one per CTA,
// P = one persistent CTA per SM.  A piece is a run of (fractions of) block-rows;
// the fraction [u0,u1) of block-row r means the slice [u0*count, u1*count) of
// the ACTIVE index list, so the load follows the active entries, not the matrix
// columns, and every CTA streams the same number of blocks whatever R is.  Each
// (CTA, block-row) segment yields G fp32 partial sums, published as tagged 64-bit
// words; whichever CTA contributes last to a block-row (arrive-only counter: no
// CTA ever waits for another one to run, only for stores already issued to
// become visible) adds the partials in slot order, adds the offset term and
// rounds to fp16.  A CTA that finds all the other partials present before its own
// sum is ready skips the counter and finishes the block-row directly.  With 2 or 4
// CTAs per block-row the grid is launched as thread-block clusters of that size
// (when the device can hold all of them at once) and the partial sums go through
// the shared memory of the cluster's first CTA instead of global memory.
//
// Inside a CTA, kWorkers warps each run their own copy pipeline over chunks of
// 32 list entries (64 with groups of 64 rows: 2 KB of 4-bit codes either way;
// chunks are dealt round-robin to the warps); nothing is shared
// between the warps until the end of a segment.  Per chunk, three stages, all
// cp.async into the warp's private shared-memory ring, one commit group per
// iteration:
//   A  the chunk's column numbers (one 4-byte copy per lane and entry);
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
#include <cstddef>

#include "spqt_common.cuh"

namespace spqt {

// 12 workers + 2 writers = 14 warps leave 128 registers per thread: measured faster than 18 + 2 at 96
// registers (which spilled) on every shape, and than 10, 11, 13 or 14 workers.
#ifndef SPQT_WORKERS
#define SPQT_WORKERS 12
#endif
#ifndef SPQT_DEPTH
#define SPQT_DEPTH 3
#endif
constexpr int kWorkers = SPQT_WORKERS;   // compute warps
#ifndef SPQT_WRITERS
#define SPQT_WRITERS 2
#endif
constexpr int kWriters = SPQT_WRITERS;     // 1 or 2 writer warps; segment sg goes to writer sg % kWriters
constexpr int kWriterWarp = kWorkers;      // the first of them
constexpr int kGemvThreads = (kWorkers + kWriters) * 32;
// list entries per chunk: 2 KB of 4-bit code blocks for either group size (32 blocks of 128 rows, 64 of 64)
__host__ __device__ constexpr int chunk_entries(int group) { return 32 * (128 / group); }
constexpr int kDepth = SPQT_DEPTH;       // chunks in flight per warp
constexpr unsigned long long kWaitNs = 1000000000ull;  // bound on every mbarrier wait: one second
constexpr int kMaxCluster = 8;           // largest thread-block cluster (CTAs of one block-row) used
constexpr int kMaxFusedN = 32768;        // largest n whose index collection can run inside the GEMV
constexpr int kFusedCols = 16384;        // list entries (16-bit column numbers) a CTA keeps in shared memory in that case

static int g_tune_ctas = 0;  // 0 = one CTA per SM
int g_no_pdl = 0;            // 1 = plain stream-ordered launches (also read by the index-collection launch)
static int g_no_cluster = 0; // 1 = never launch thread-block clusters

#ifdef SPQT_TRACE
__device__ long long* g_trace;  // time stamps of CTA 0 (debug builds only)
#define SPQT_TRACE_EVENT(cond, slot) do { if ((cond) && blockIdx.x == 0 && spqt_tr && (slot) < 4096) spqt_tr[(slot)] = clock64(); } while (0)
#else
#define SPQT_TRACE_EVENT(cond, slot) do { } while (0)
#endif

}  // namespace spqt

#include "spqt_gemv_device.cuh"
#include "spqt_gemv_map.cuh"

namespace spqt {

// ---------------------------------------------------------------- kernel

template <int G, int BITS>
struct GemvSmem {
    static constexpr int B = G * BITS / 8;
    static constexpr int CH = chunk_entries(G);
    struct Stage {
        alignas(16) unsigned char codes[CH * B];  // block e of the chunk at e*B
        unsigned meta[3][CH];                     // words holding x_k, scale_rk, zero_rk of entry e
    };
    Stage stage[kWorkers][kDepth];
    alignas(16) int cols[kWorkers][2 * kDepth][CH];  // column numbers of the chunks ahead
    alignas(16) float red[2][kWorkers][G];               // per-warp partial sums of a finished segment
    float red_z[2][kWorkers];                            // and their offset terms
    uint64_t red_full[2], red_empty[2];
    // thread-block clusters only: partial sums the other CTAs of the cluster store here (CTA rank 0)
    alignas(16) float xred[kMaxCluster][G + 4];
    uint64_t xbar;                                       // counts their arrivals
    // fused index collection only
    alignas(16) int load_tot[kMaxFusedN / 256];  // active entries of every 256 entries of x
    unsigned short fused_cols[kFusedCols];       // the part of the index list this CTA reads, when it fits (n <= 32768)
};

// FUSED: the index collection runs in the kernel's prologue.  Every CTA copies x to shared memory and
// scans it (each lane tests 8 entries in fp16; popc and warp reductions give the number of active
// entries of every 256-entry piece), then expands only the pieces that overlap the list positions its
// own slices cover: into shared memory, or, when that part is too long, into idx_out, from where it
// reads them back like a list collected by a separate launch.  The CTAs that work on block-row 0
// cover the whole list between them and write idx_out; CTA 0 writes the count.
template <int G, int BITS, bool DENSE, bool ODD_N, bool FUSED, bool CLUSTER>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const uint8_t* __restrict__ codes, const __half* __restrict__ scales,
                 const __half* __restrict__ zeros, int R, int n,
                 const __half* __restrict__ x, const int32_t* idx_in,
                 const int32_t* count_ptr, __half* __restrict__ y,
                 int* __restrict__ counters, int* __restrict__ status,
                 unsigned long long* __restrict__ words, float* __restrict__ partials,
                 float* __restrict__ zpartials, int max_slots, unsigned magic_p, unsigned magic_r,
                 int cluster_k, float thr, int32_t* idx_out, int32_t* count_out)
{
    constexpr int B = G * BITS / 8;
    constexpr int LPB = G / 32;       // lanes that share one block (each owns 32 of its rows)
    constexpr int CB = (B % 16 == 0) ? 16 : 8;   // bytes per copy: 3-bit blocks of 64 rows are only 8-byte aligned
    static_assert(BITS == 3 || BITS == 4, "3- or 4-bit codes");
    constexpr int SLOTS = 32 / LPB;   // blocks per 512-byte warp load
    constexpr int KEEP = 32 / SLOTS;  // values per lane after the in-warp reduce-scatter
    constexpr int CH = chunk_entries(G);  // list entries per chunk
    constexpr int EPL = CH / 32;          // entries whose metadata a lane holds
    constexpr int SUBS = CH / SLOTS;      // 512-byte loads per chunk
    constexpr int D = kDepth;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    GemvSmem<G, BITS>& sm = *reinterpret_cast<GemvSmem<G, BITS>*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = gridDim.x, c = blockIdx.x;
#ifdef SPQT_TRACE
    long long* const spqt_tr = g_trace;  // one load: an event is then a clock read and a store
#endif
    SPQT_TRACE_EVENT(tid == 0, 3990);
#ifdef SPQT_TRACE
    if (tid == 0 && g_trace && c < 200) g_trace[2000 + c] = (long long)global_ns();
#endif

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.red_full[b], kWorkers);
            mbar_init(&sm.red_empty[b], 1);
        }
        if (CLUSTER) mbar_init(&sm.xbar, cluster_k - 1);
        if (CLUSTER) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Cluster launch (cluster_k CTAs work on one block-row and CTA rank 0 collects their sums): nobody
    // may touch another CTA's barrier before it is initialised.  Arrive now, wait much later.
    if (CLUSTER) cluster_arrive();

    // Programmatic dependent launch: this grid may have been started while the previous kernel of
    // the stream was still draining.  Nothing above touches global memory; everything below waits
    // for that kernel to complete, and lets the next kernel of the stream start early in turn.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    int count = 0;
    if (!FUSED) count = DENSE ? n : *count_ptr;  // in flight while the row range is worked out
    Piece pc;
    pc.init_rows(R, P, c, magic_p, magic_r);
    const int32_t* idx = idx_in;
    const unsigned short* xb0 = reinterpret_cast<const unsigned short*>(x);
    int need_lo = 0;          // FUSED: first list position held in sm.fused_cols
    bool cols_local = false;  // FUSED: the pipeline reads its column numbers from sm.fused_cols
    if (FUSED) {
        // Three short loops over the 256-entry pieces of x (piece li belongs to warp li % kWarps, lane l
        // holds entries 8l..8l+7): (1) activity mask of the lane's entries and the piece totals, four
        // pieces per warp and round so that their loads share one round trip, (2) every warp sums the
        // totals below its own pieces, (3) the pieces that overlap the list positions this CTA needs are
        // expanded into column numbers.  The per-lane masks wait in shared memory that the pipeline
        // only uses afterwards.
        constexpr int kWarps = kGemvThreads / 32;
        constexpr int kPiecesPerRound = 4;
        unsigned char* pm = reinterpret_cast<unsigned char*>(smem_raw);  // per (piece, lane): activity of its 8 entries
        using Smem = GemvSmem<G, BITS>;
        static_assert(offsetof(Smem, red_z) >= kMaxFusedN / 8,
                      "the prologue's scratch must fit in the part of shared memory it borrows");
        const int nv = (n + 255) / 256;
        for (int i = nv + tid; i < kMaxFusedN / 256; i += kGemvThreads) sm.load_tot[i] = 0;
        const bool vec_ok = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
        // the largest fp16 value not above t (any negative value if t < 0: everything but NaN is
        // active; +inf if t is NaN or +inf: nothing is)
        const __half thr_h = (thr != thr) ? __ushort_as_half((unsigned short)0x7c00)
                                          : (thr < 0.0f ? __float2half_rn(-1.0f) : __float2half_rd(thr));
        const __half2 thr_h2 = __half2half2(thr_h);
        SPQT_TRACE_EVENT(tid == 0, 3991);
#pragma unroll 1
        for (int l0 = warp; l0 < nv; l0 += kPiecesPerRound * kWarps) {
            uint4 xv[kPiecesPerRound];
#pragma unroll
            for (int j = 0; j < kPiecesPerRound; ++j) {
                const int li = l0 + j * kWarps, k0 = li * 256 + lane * 8;
                xv[j] = make_uint4(0u, 0u, 0u, 0u);
                if (li < nv) {  // uniform across the warp
                    if (vec_ok && k0 + 8 <= n) {
                        xv[j] = __ldg(reinterpret_cast<const uint4*>(x + k0));
                    } else {
                        unsigned short hv[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) hv[e] = (k0 + e < n) ? __ldg(xb0 + k0 + e) : (unsigned short)0;
                        xv[j].x = hv[0] | ((unsigned)hv[1] << 16);
                        xv[j].y = hv[2] | ((unsigned)hv[3] << 16);
                        xv[j].z = hv[4] | ((unsigned)hv[5] << 16);
                        xv[j].w = hv[6] | ((unsigned)hv[7] << 16);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kPiecesPerRound; ++j) {
                const int li = l0 + j * kWarps, k0 = li * 256 + lane * 8;
                if (li < nv) {
                    const unsigned wds[4] = {xv[j].x, xv[j].y, xv[j].z, xv[j].w};
                    unsigned m8 = 0;
#pragma unroll
                    for (int e2 = 0; e2 < 4; ++e2) {
                        // |x| > t  <=>  |x| > (largest fp16 value <= t): two entries per compare, in fp16,
                        // exact; the ordered compare is false for NaN
                        const unsigned ab = wds[e2] & 0x7fff7fffu;
                        const unsigned gt = __hgt2_mask(*reinterpret_cast<const __half2*>(&ab), thr_h2);
                        m8 |= (gt & (1u << (2 * e2))) | (gt & (0x20000u << (2 * e2))) >> 16;
                    }
                    const int left = n - k0;  // entries of this lane that exist
                    if (left < 8) m8 &= (left <= 0) ? 0u : ((1u << left) - 1u);
                    pm[li * 32 + lane] = (unsigned char)m8;
                    const unsigned tot = __reduce_add_sync(0xffffffffu, (unsigned)__popc(m8));
                    if (lane == 0) sm.load_tot[li] = (int)tot;
                }
            }
        }
        __syncthreads();
        SPQT_TRACE_EVENT(tid == 0, 3992);
        // (2) every warp for itself: lane l holds the totals of pieces 4l..4l+3; sums over the pieces
        // below a given one come from one warp reduction each
        int tot4[4];
        {
            const int4 t4 = *reinterpret_cast<const int4*>(&sm.load_tot[lane * 4]);  // zero past nv (cleared below)
            tot4[0] = t4.x; tot4[1] = t4.y; tot4[2] = t4.z; tot4[3] = t4.w;
        }
        count = (int)__reduce_add_sync(0xffffffffu, (unsigned)(tot4[0] + tot4[1] + tot4[2] + tot4[3]));
        SPQT_TRACE_EVENT(tid == 0, 3993);
        pc.set_count(count);
        if (c == 0 && tid == 0) *count_out = count;
        // list positions this CTA will read: the union of its slices.  If that part fits in shared
        // memory the pipeline takes its column numbers from there (no round trip through global
        // memory); otherwise they go to idx_out and come back like a list collected by a separate launch.
        // (A piece that spans several block-rows ends the first one and begins the last one: its slices
        // cover the whole list between them.)
        need_lo = 0;
        int need_hi = count;
        if (pc.r_first == pc.r_last) pc.slice(pc.r_first, &need_lo, &need_hi);
        cols_local = (need_hi - need_lo) <= kFusedCols;
        const unsigned need_len = (unsigned)max(need_hi - need_lo, 0);
        const unsigned fc0 = smem_u32(&sm.fused_cols[0]);
        SPQT_TRACE_EVENT(tid == 0, 3994);
        // (3) the pieces that overlap [need_lo, need_hi): prefix sums over the lanes, then one
        // predicated store per entry (a divergent branch per entry would cost far more than the store)
#pragma unroll 1
        for (int li = warp; li < nv; li += kWarps) {
            unsigned below = 0;  // active entries of this lane's pieces that come before piece li
#pragma unroll
            for (int q = 0; q < 4; ++q) below += (lane * 4 + q < li) ? (unsigned)tot4[q] : 0u;
            const int base = (int)__reduce_add_sync(0xffffffffu, below);
            const int q = li & 3;
            const int tsel = q == 0 ? tot4[0] : q == 1 ? tot4[1] : q == 2 ? tot4[2] : tot4[3];
            const int end = base + __shfl_sync(0xffffffffu, tsel, li >> 2);
            if (end <= need_lo || base >= need_hi) continue;  // uniform across the warp
            const unsigned m8 = pm[li * 32 + lane];
            const int c8 = __popc(m8);
            int incl = c8;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            int pos = base + incl - c8;
            const int col0 = li * 256 + lane * 8;
            if (cols_local) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const unsigned on = (m8 >> e) & 1u, d = (unsigned)(pos - need_lo);
                    st_shared_u16_if(on & (d < need_len ? 1u : 0u), fc0 + 2u * d, col0 + e);
                    pos += (int)on;
                }
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const unsigned on = (m8 >> e) & 1u, d = (unsigned)(pos - need_lo);
                    st_global_if(on & (d < need_len ? 1u : 0u), idx_out + pos, col0 + e);
                    pos += (int)on;
                }
            }
        }
        SPQT_TRACE_EVENT(lane == 0, 3960 + warp);
        __syncthreads();  // the CTA's own writes (shared or global) are visible to its pipeline
        idx = idx_out;
    } else {
        pc.set_count(count);
    }
    SPQT_TRACE_EVENT(tid == 0, 4000);
    if (CLUSTER) cluster_wait();  // every CTA of the cluster has initialised its barriers by now

    if (warp >= kWriterWarp) {
        // ------------------------------------------------------------ writers
        // Two warps, one per hand-over buffer, so that the chains of dependent L2 round trips
        // (store, fence, counter, read back) of consecutive segments overlap.
        constexpr int RPL = G / 32;  // rows per lane
        constexpr int kStride = G + 2;  // words per contributing CTA: G sums, the offset term, one of padding
        const int wr = warp - kWriterWarp;
        bool ok = true;
        if (FUSED && cols_local && pc.r_first == 0) {
            // this CTA's slice of block-row 0 is its part of the index list the call returns
            int p0, p1;
            pc.slice(0, &p0, &p1);
            for (int i = p0 + wr * 32 + lane; i < p1; i += 32 * kWriters) idx_out[i] = sm.fused_cols[i - need_lo];
        }
        for (int r = pc.r_first + wr, sg = wr; r <= pc.r_last; r += kWriters, sg += kWriters) {
            const int b = sg & 1;  // hand-over buffer of this segment
            int first, nslots;
            pc.contributors(r, &first, &nslots);
            const int mine = c - first;
            unsigned long long* const row_words = words + (size_t)r * kTagSlots * kStride;
            // A block-row that is not the CTA's first is shared with CTAs that work on it first and are
            // done long before this one.  While the workers are still computing, watch for their words
            // (one word per CTA as a cheap hint, at a low rate).  Once all of them are there, this CTA
            // is the one that finishes the block-row, and nothing remains to be done across CTAs after
            // its own sum.  (On a CTA's first block-row all contributors finish at about the same time
            // and watching would only delay the counter path.)
            constexpr int kSpec = kTagSlots - 1;
            float ov[kSpec][RPL], oz[kSpec];
            bool spec = false;
            if (sg > 0 && nslots > 1 && nslots <= kSpec + 1) {
                unsigned long long t0 = 0;
                for (unsigned it = 0;; ++it) {
                    const unsigned long long hint =
                        lane < nslots - 1 ? ld_word(row_words + (size_t)(lane + (lane >= mine ? 1 : 0)) * kStride + G) : kTagBit;
                    if (__all_sync(0xffffffffu, (hint >> 32) != 0ull)) {
                        unsigned tags = 1u;
#pragma unroll
                        for (int j = 0; j < kSpec; ++j) {
                            const bool in = j < nslots - 1;
                            const unsigned long long* src = row_words + (size_t)(j + (j >= mine ? 1 : 0)) * kStride;
#pragma unroll
                            for (int i = 0; i < RPL; ++i) {
                                const unsigned long long wv = in ? ld_word(src + lane * RPL + i) : kTagBit;
                                ov[j][i] = __uint_as_float((unsigned)wv);
                                tags &= (unsigned)(wv >> 32);
                            }
                            const unsigned long long wz = (in && lane == 0) ? ld_word(src + G) : kTagBit;
                            oz[j] = __uint_as_float((unsigned)wz);
                            tags &= (unsigned)(wz >> 32);
                        }
                        spec = __all_sync(0xffffffffu, tags != 0u);
                        if (spec) break;
                    }
                    if (mbar_test(&sm.red_full[b], (sg >> 1) & 1)) break;  // own sums are ready: stop watching
                    if (it == 64) t0 = global_ns();
                    if (it > 64 && global_ns() - t0 > kWaitNs) break;
                    __nanosleep(100);
                }
                if (spec) {
#pragma unroll
                    for (int j = 0; j < kSpec; ++j) oz[j] = __shfl_sync(0xffffffffu, oz[j], 0);
                }
            }
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
            if (nslots == 1) {
                // this CTA holds the whole block-row: nothing to combine
#pragma unroll
                for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(v[i] + zpart);
                continue;
            }
            float t[RPL], zsum = 0.0f;  // the block-row's sums, always accumulated in slot order
#pragma unroll
            for (int i = 0; i < RPL; ++i) t[i] = 0.0f;
            if (CLUSTER) {
                // The contributors of this block-row are the CTAs of this cluster, in rank order.  The
                // others store their sums into rank 0's shared memory and arrive on its barrier; rank 0
                // adds them in rank order.  Nothing goes through global memory.
                if (mine != 0) {
                    const unsigned dst = cluster_map(smem_u32(&sm.xred[mine][0]), 0u);
#pragma unroll
                    for (int i = 0; i < RPL; ++i) st_cluster_f32(dst + 4u * (lane * RPL + i), v[i]);
                    if (lane == 0) st_cluster_f32(dst + 4u * G, zpart);
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(cluster_map(smem_u32(&sm.xbar), 0u));
                    continue;
                }
                ok = mbar_wait_cluster(&sm.xbar, 0);
                if (!ok) break;
#pragma unroll
                for (int i = 0; i < RPL; ++i) t[i] += v[i];
                zsum += zpart;
                for (int s = 1; s < cluster_k; ++s) {
#pragma unroll
                    for (int i = 0; i < RPL; ++i) t[i] += sm.xred[s][lane * RPL + i];
                    zsum += sm.xred[s][G];
                }
#pragma unroll
                for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(t[i] + zsum);
                continue;
            }
            if (spec) {
#pragma unroll
                for (int s = 0; s < kSpec + 1; ++s) {
                    if (s < nslots) {
                        const int j = s - (s > mine ? 1 : 0);  // position among the other CTAs
#pragma unroll
                        for (int i = 0; i < RPL; ++i) {
                            float pv = v[i];
#pragma unroll
                            for (int jj = 0; jj < kSpec; ++jj) pv = (s != mine && j == jj) ? ov[jj][i] : pv;
                            t[i] += pv;
                        }
                        float pz = zpart;
#pragma unroll
                        for (int jj = 0; jj < kSpec; ++jj) pz = (s != mine && j == jj) ? oz[jj] : pz;
                        zsum += pz;
                    }
                }
            } else if (nslots <= kSpec + 1) {
                // publish this CTA's words (value and tag travel together: no fence), then count arrivals
                unsigned long long* dst = row_words + (size_t)mine * kStride;
#pragma unroll
                for (int i = 0; i < RPL; ++i) st_word(dst + lane * RPL + i, kTagBit | __float_as_uint(v[i]));
                if (lane == 0) st_word(dst + G, kTagBit | __float_as_uint(zpart));
                int prev = 0;
                if (lane == 0) prev = atomicAdd(counters + r, 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev != nslots - 1) continue;
                // last to arrive: every other CTA has issued its stores; wait (bounded) until their
                // words are visible
                float pv[kSpec + 1][RPL], pz[kSpec + 1];
                unsigned long long t0 = 0;
                for (unsigned it = 0;; ++it) {
                    unsigned tags = 1u;
#pragma unroll
                    for (int j = 0; j < kSpec + 1; ++j) {
                        const bool in = j < nslots && j != mine;
                        const unsigned long long* src = row_words + (size_t)j * kStride;
#pragma unroll
                        for (int i = 0; i < RPL; ++i) {
                            const unsigned long long wv = in ? ld_word(src + lane * RPL + i) : kTagBit;
                            pv[j][i] = __uint_as_float((unsigned)wv);
                            tags &= (unsigned)(wv >> 32);
                        }
                        const unsigned long long wz = (in && lane == 0) ? ld_word(src + G) : kTagBit;
                        pz[j] = __uint_as_float((unsigned)wz);
                        tags &= (unsigned)(wz >> 32);
                    }
                    if (__all_sync(0xffffffffu, tags != 0u)) break;
                    if (it == 4) t0 = global_ns();
                    if (it > 4 && global_ns() - t0 > kWaitNs) { ok = false; break; }
                }
                if (!ok) break;
#pragma unroll
                for (int j = 0; j < kSpec + 1; ++j) {
                    const float z0 = __shfl_sync(0xffffffffu, pz[j], 0);
                    if (j < nslots) {
#pragma unroll
                        for (int i = 0; i < RPL; ++i) t[i] += (j == mine) ? v[i] : pv[j][i];
                        zsum += (j == mine) ? zpart : z0;
                    }
                }
            } else {
                // many contributors: plain fp32 partials in a region of their own, a fence, and the
                // counter; the last to arrive reads eight slots at a time
                const size_t pslot = (size_t)r * max_slots + mine;
#pragma unroll
                for (int i = 0; i < RPL; ++i) __stcg(partials + pslot * G + lane * RPL + i, v[i]);
                if (lane == 0) __stcg(zpartials + pslot, zpart);
                __threadfence();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(counters + r, 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev != nslots - 1) continue;
                __threadfence();
                const float* p = partials + (size_t)r * max_slots * G + lane * RPL;
                const float* zp = zpartials + (size_t)r * max_slots;
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
                        if (s0 + j < nslots) {
#pragma unroll
                            for (int i = 0; i < RPL; ++i) t[i] += pv[j][i];
                            zsum += pz[j];
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < RPL; ++i) y[(size_t)r * G + lane * RPL + i] = __float2half_rn(t[i] + zsum);
            // leave the workspace ready for the next call: no tag may stay set
            if (nslots <= kSpec + 1) {
                for (int s = 0; s < nslots; ++s) {
                    unsigned long long* dst = row_words + (size_t)s * kStride;
#pragma unroll
                    for (int i = 0; i < RPL; ++i) st_word(dst + lane * RPL + i, 0ull);
                    if (lane == 0) st_word(dst + G, 0ull);
                }
            }
            // The counter: after the last arrival nobody else touches it, so it is simply cleared.  On the
            // early path the other CTAs' increments may still be under way: a reduction that takes away
            // exactly what they add leaves zero whatever the order (and none of them can see "last").
            if (lane == 0) {
                if (spec) atomicAdd(counters + r, -(nslots - 1));
                else counters[r] = 0;
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
    // Everything the loop touches in shared memory is addressed with 32-bit shared addresses kept in
    // registers (ring positions are byte offsets that wrap), and entries past the end of a slice are
    // handled by clamping the entry number (they re-read the slice's last entry and get weight 0)
    // rather than by branches: the loop is bound by instruction issue.
    using Stage = typename GemvSmem<G, BITS>::Stage;
    constexpr unsigned kStageBytes = (unsigned)sizeof(Stage);
    constexpr unsigned kMetaOff = (unsigned)(CH * B);     // offset of Stage::meta
    constexpr unsigned kColsBytes = CH * 4;               // one chunk of column numbers
    static_assert(offsetof(Stage, meta) == kMetaOff, "stage layout");
    const int slot = lane / LPB, h = lane % LPB;
    const unsigned short* xb = reinterpret_cast<const unsigned short*>(x);
    const unsigned stage_base = smem_u32(&sm.stage[warp][0]);
    const unsigned cols_base = smem_u32(&sm.cols[warp][0][0]);
    const unsigned fused_base = smem_u32(&sm.fused_cols[0]) - 2u * (unsigned)need_lo;  // + 2 * list position
    const bool use_list = !DENSE && !(FUSED && cols_local);  // column numbers come through stage A

    // column number of entry e of a chunk: 32-bit entries in the stage-A ring, 16-bit ones in the list
    // the fused prologue keeps
    auto col_at = [&](unsigned chunk_addr, int e) -> unsigned {
        if (!FUSED || use_list) return lds_u32(chunk_addr + 4u * e);
        return lds_u16(chunk_addr + 2u * e);
    };

    Cursor ca, cb;  // stage A / stage B cursors (the consume side walks the segments itself)
    ca.init(pc, warp, CH);
    cb = ca;
    // Ring positions (byte offsets) of the chunk stage C works on: rc_s in the ring of D stages, rc_c
    // in the ring of 2*D chunks of column numbers, rb_c = D chunks further in that ring.  Stage B
    // refills the stage slot C has just read and takes its columns from rb_c; stage A refills rc_c.
    unsigned rc_s = 0, rc_c = 0, rb_c = D * kColsBytes;
    auto wrap = [](unsigned& v, unsigned step, unsigned len) { v = (v + step == len) ? 0u : v + step; };

    // block-row constants of stage B, refreshed when its cursor enters a new block-row
    int b_row = -1;
    unsigned b_par = 0;                       // parity of r*n: which half of a word holds element (r,k)
    const uint8_t* b_codes = nullptr;         // codes of the block-row, this lane's 16-byte part
    const unsigned short* b_scales = nullptr; // scales / zeros of the block-row
    const unsigned short* b_zeros = nullptr;

    // stage A: column numbers of the warp's next chunk
    auto issue_a = [&](unsigned ring_c) {
        if (use_list && ca.valid(pc)) {
#pragma unroll
            for (int q = 0; q < EPL; ++q) {
                const int e = lane + 32 * q;
                if (ca.pos + e < ca.p1) cp_async_4(cols_base + ring_c + 4u * e, idx + ca.pos + e);
            }
            ca.advance(pc, warp);
        }
    };
    // stage B: code blocks and metadata words of the next chunk (its column numbers have landed)
    // (pre: column numbers of the copies and of the lane's metadata entry, read ahead of time by prep_b,
    // or nullptr to read them here)
    auto issue_b = [&](unsigned ring_s, unsigned ring_c, const unsigned* pre) {
        if (cb.valid(pc)) {
            if (cb.r != b_row) {
                b_row = cb.r;
                const size_t row_base = (size_t)b_row * (size_t)n;
                b_par = ODD_N ? (unsigned)(row_base & 1) : 0u;  // n even: every block-row starts on a word
                b_codes = codes + row_base * B + (BITS == 4 ? 16 * h : 0);
                b_scales = reinterpret_cast<const unsigned short*>(scales) + row_base;
                b_zeros = reinterpret_cast<const unsigned short*>(zeros) + row_base;
            }
            const int vm1 = min(cb.p1 - cb.pos, CH) - 1;  // last entry of this chunk that exists
            // address of the chunk's first column number (unused when DENSE)
            const unsigned cols_addr = use_list ? cols_base + ring_c : fused_base + 2u * (unsigned)cb.pos;
            const unsigned st_addr = stage_base + ring_s;
            if (BITS == 4) {
#pragma unroll
                for (int u = 0; u < SUBS; ++u) {
                    const int e = min(u * SLOTS + slot, vm1);
                    const unsigned kk = DENSE ? (unsigned)(cb.pos + e) : (pre ? pre[u] : col_at(cols_addr, e));
                    if (DENSE) cp_async_16(st_addr + lane * 16 + u * 512, b_codes + (size_t)kk * B);
                    else cp_async_16_l2_64(st_addr + lane * 16 + u * 512, b_codes + (size_t)kk * B);
                }
            } else {
                // 3-bit blocks (48 or 24 bytes): the chunk's bytes in copies of CB bytes, lane after lane
                constexpr int NC = CH * B / CB / 32;
#pragma unroll
                for (int q = 0; q < NC; ++q) {
                    const int off = (q * 32 + lane) * CB;    // byte offset inside the chunk's stage
                    const int e = min(off / B, vm1), part = off % B;
                    const unsigned kk = DENSE ? (unsigned)(cb.pos + e) : col_at(cols_addr, e);
                    const uint8_t* src = b_codes + (size_t)kk * B + part;
                    if (CB == 16) {
                        if (DENSE) cp_async_16(st_addr + off, src);
                        else cp_async_16_l2_64(st_addr + off, src);
                    } else {
                        cp_async_8(st_addr + off, src);
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < EPL; ++q) {
                // the aligned 4-byte word that holds each fp16 value (index rounded down to even)
                const int e = min(lane + 32 * q, vm1);
                const unsigned kk = DENSE ? (unsigned)(cb.pos + e) : ((pre && BITS == 4) ? pre[SUBS + q] : col_at(cols_addr, e));
                const unsigned mdst = st_addr + kMetaOff + 4u * (lane + 32 * q);
                const int mo = (int)kk - (int)((kk ^ b_par) & 1u);  // may be -1 only when r*n is odd: still inside the array
                if (!ODD_N || kk != (unsigned)(n - 1)) {
                    cp_async_4_ca(mdst, xb + (kk & ~1u));
                    cp_async_4(mdst + CH * 4, b_scales + mo);
                    cp_async_4(mdst + 2 * CH * 4, b_zeros + mo);
                } else {
                    // n odd: the word of the last column may reach past the end of an array; fetch directly
                    sts_u32(mdst, (unsigned)__ldg(xb + kk) << ((kk & 1u) * 16));
                    sts_u32(mdst + CH * 4, (unsigned)__ldg(b_scales + kk) << (((kk ^ b_par) & 1u) * 16));
                    sts_u32(mdst + 2 * CH * 4, (unsigned)__ldg(b_zeros + kk) << (((kk ^ b_par) & 1u) * 16));
                }
            }
            cb.advance(pc, warp);
        }
    };

    // The column numbers stage B will need at the end of this iteration, read before the arithmetic so
    // that the shared-memory latency hides under it (4-bit sparse path only).
    auto prep_b = [&](unsigned ring_c, unsigned* pre) {
        if (!DENSE && BITS == 4 && cb.valid(pc)) {
            const int vm1 = min(cb.p1 - cb.pos, CH) - 1;
            const unsigned cols_addr = use_list ? cols_base + ring_c : fused_base + 2u * (unsigned)cb.pos;
#pragma unroll
            for (int u = 0; u < SUBS; ++u) pre[u] = col_at(cols_addr, min(u * SLOTS + slot, vm1));
#pragma unroll
            for (int q = 0; q < EPL; ++q) pre[SUBS + q] = col_at(cols_addr, min(lane + 32 * q, vm1));
        }
    };

    // fill the pipeline: D chunks of columns, then D chunks of blocks (each needs its columns)
#pragma unroll 1
    for (int s = 0; s < D; ++s) {
        issue_a(s * kColsBytes);
        cp_async_commit();
    }
#pragma unroll 1
    for (int s = 0; s < D; ++s) {
        cp_async_wait<D - 1>();
        __syncwarp();
        issue_b(s * kStageBytes, s * kColsBytes, nullptr);
        issue_a((D + s) * kColsBytes);
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
        const unsigned c_par = ODD_N ? (unsigned)(((size_t)r * (size_t)n) & 1) : 0u;
        float zl = 0.0f;  // this lane's share of sum x_k * zero_rk
        for (int pos = p0 + warp * CH; pos < p1; pos += kWorkers * CH) {
            // ---- stage C of the oldest chunk: everything it needs is in commit groups that wait<D-1> covers
#ifdef SPQT_TRACE
            const long long tc0 = clock64();
#endif
            cp_async_wait<D - 1>();
            __syncwarp();
#ifdef SPQT_TRACE
            const long long tc1 = clock64();
#endif
            unsigned pre[SUBS + EPL];
            prep_b(rb_c, pre);
            const unsigned st_addr = stage_base + rc_s;
#ifdef SPQT_TRACE
            const long long tc2 = clock64();
#endif
            float a[EPL];  // x_k * scale_rk of the entries this lane holds (entry lane + 32 q)
#pragma unroll
            for (int q = 0; q < EPL; ++q) {
                const unsigned xw = lds_u32(st_addr + kMetaOff + 4u * (lane + 32 * q));
                const unsigned sw = lds_u32(st_addr + kMetaOff + 4u * (lane + 32 * q) + CH * 4);
                const unsigned zw = lds_u32(st_addr + kMetaOff + 4u * (lane + 32 * q) + 2 * CH * 4);
                const int e = min(lane + 32 * q, p1 - pos - 1);  // the entry whose metadata this lane holds
                unsigned kk;
                if (DENSE) kk = (unsigned)(pos + e);
                else kk = col_at(use_list ? cols_base + rc_c : fused_base + 2u * (unsigned)pos, e);
                const unsigned xs = (kk & 1u) * 16, ms = ((kk ^ c_par) & 1u) * 16;
                const float xf = __half2float(__ushort_as_half((unsigned short)(xw >> xs)));
                const float sf = __half2float(__ushort_as_half((unsigned short)(sw >> ms)));
                const float zf = __half2float(__ushort_as_half((unsigned short)(zw >> ms)));
                const float xin = (e == lane + 32 * q) ? xf : 0.0f;  // 0 past the end of the slice
                a[q] = xin * sf;                                      // exact
                zl = fmaf(xin, zf, zl);
            }
#pragma unroll
            for (int u = 0; u < SUBS; ++u) {
                const float au = __shfl_sync(0xffffffffu, a[(u * SLOTS) / 32], (u * SLOTS + slot) & 31);
                if (BITS == 4) {
                    const uint4 wv = lds_v4(st_addr + lane * 16 + u * 512);
                    fma_block16(acc, wv, au);
                } else {
                    // lane h of a block: words h and h+LPB of the 2-bit plane, word h of the 1-bit plane
                    const unsigned blk = st_addr + (u * SLOTS + slot) * B + 4u * h;
                    fma_block3(acc, lds_u32(blk), lds_u32(blk + 4u * LPB), lds_u32(blk + 8u * LPB), au);
                }
            }
            __syncwarp();  // every lane has read its part of the slots that B and A now refill
            issue_b(rc_s, rb_c, (!DENSE && BITS == 4) ? pre : nullptr);
            issue_a(rc_c);
            cp_async_commit();
            wrap(rc_s, kStageBytes, D * kStageBytes);
            wrap(rc_c, kColsBytes, 2 * D * kColsBytes);
            wrap(rb_c, kColsBytes, 2 * D * kColsBytes);
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

// ---------------------------------------------------------------- checked mode
// spqt_set_debug(1): before a sparse GEMV the index list is checked on the device (count in
// [0, n], every index in [0, n), no index twice for n up to kDebugBits).  A bad list sets the
// workspace's status word to 2 and the GEMV then runs with a count of 0 (y = 0) instead of reading
// wherever the indices point.  Two small extra launches per call; state is per device, not per stream.
constexpr int kDebugBits = 1 << 20;
static __device__ unsigned g_debug_bitmap[kDebugBits / 32];  // all zero between calls
static __device__ int g_debug_count;                         // the count the GEMV is given
static int g_debug = 0;

__global__ void debug_mark_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ count, int n,
                                  int* __restrict__ status)
{
    const int c = *count;
    bool bad = (c < 0 || c > n) && blockIdx.x == 0 && threadIdx.x == 0;
    const int lim = c < 0 ? 0 : (c > n ? n : c);  // idx holds n entries at most
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < lim; i += gridDim.x * blockDim.x) {
        const int k = idx[i];
        if (k < 0 || k >= n) {
            bad = true;
        } else if (n <= kDebugBits) {
            const unsigned bit = 1u << (k & 31);
            if (atomicOr(&g_debug_bitmap[k >> 5], bit) & bit) bad = true;  // seen before
        }
    }
    if (bad) atomicExch(status, 2);
}

__global__ void debug_clear_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ count, int n,
                                   const int* __restrict__ status)
{
    const int c = *count;
    const int lim = c < 0 ? 0 : (c > n ? n : c);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < lim; i += gridDim.x * blockDim.x) {
        const int k = idx[i];
        if (k >= 0 && k < n && n <= kDebugBits) g_debug_bitmap[k >> 5] = 0u;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) g_debug_count = (*status != 0) ? 0 : c;
}

// Launches the two kernels; returns the device address of the count the GEMV must use.
static spqt_status debug_check(const int32_t* idx, const int32_t* count, int n, int* status, cudaStream_t s,
                               const int32_t** checked_count)
{
    static int* count_addr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    if (count_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_debug_count) != cudaSuccess || p == nullptr) return SPQT_ERR_CUDA;
        count_addr[dev] = static_cast<int*>(p);
    }
    const int blocks = n < 256 * 64 ? (n + 255) / 256 : 64;
    debug_mark_kernel<<<blocks, 256, 0, s>>>(idx, count, n, status);
    debug_clear_kernel<<<blocks, 256, 0, s>>>(idx, count, n, status);
    if (cudaGetLastError() != cudaSuccess) return SPQT_ERR_CUDA;
    count_launch(2);
    *checked_count = count_addr[dev];
    return SPQT_OK;
}

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
    auto kernel = gemv_kernel<G, BITS, DENSE, ODD_N, FUSED, false>;
    auto kernel_c = gemv_kernel<G, BITS, DENSE, ODD_N, FUSED, true>;  // the thread-block-cluster variant
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPQT_ERR_CUDA;
    const int smem = (int)sizeof(GemvSmem<G, BITS>);
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
            cudaFuncSetAttribute(kernel_c, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
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
    unsigned long long* words = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + header_bytes(f.R));
    float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + header_bytes(f.R) + tagged_bytes(f));
    float* zpartials = partials + (size_t)f.R * slots * G;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(P);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int nattr = 0;
    if (!g_no_pdl) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    // A whole number (2..8) of CTAs per block-row: launch them as one thread-block cluster each, if the
    // device can hold all the clusters at once (asked once per kernel, cluster size and device).
    int cluster_k = 0;
    if (!g_no_cluster && f.R <= P && P % f.R == 0 && P / f.R >= 2 && P / f.R <= kMaxCluster) {
        const int k = P / f.R;
        static signed char fits[64][kMaxCluster + 1][149] = {};  // [device][k][clusters]: 0 unknown, 1 yes, -1 no
        const int nclusters = P / k;
        if (nclusters <= 148) {
            signed char& known = fits[dev][k][nclusters];
            attr[nattr].id = cudaLaunchAttributeClusterDimension;
            attr[nattr].val.clusterDim.x = k;
            attr[nattr].val.clusterDim.y = 1;
            attr[nattr].val.clusterDim.z = 1;
            if (known == 0) {
                cfg.attrs = attr;
                cfg.numAttrs = nattr + 1;
                int can = 0;
                if (cudaOccupancyMaxActiveClusters(&can, kernel_c, &cfg) == cudaSuccess && can >= nclusters) known = 1;
                else { known = -1; (void)cudaGetLastError(); }
            }
            if (known == 1) { cluster_k = k; ++nattr; }
        }
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    const cudaError_t err = cudaLaunchKernelEx(
        &cfg, cluster_k ? kernel_c : kernel, static_cast<const uint8_t*>(codes), static_cast<const __half*>(scales),
        static_cast<const __half*>(zeros), f.R, f.n, static_cast<const __half*>(x), idx, count,
        static_cast<__half*>(y), counters, status, words, partials, zpartials, slots,
        magic_of((unsigned)P), magic_of((unsigned)f.R), cluster_k, fa.t, fa.idx_out, fa.count_out);
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
    if (!DENSE && !FUSED && g_debug) {
        st = debug_check(idx, count, n, static_cast<int*>(workspace) + f.R, s, &count);
        if (st != SPQT_OK) return st;
    }
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
    // The scratch keeps whatever the previous call (or an interrupted one, or one of another shape)
    // left: the arrival counters, the status word and the tagged words must start at zero.
    if (cudaMemsetAsync(scratch_addr[dev], 0, header_bytes(f.R) + tagged_bytes(f), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return SPQT_ERR_CUDA;
    return gemv_entry<false>(codes, scales, zeros, m, n, bits, group, x, idx, count, y,
                             scratch_addr[dev], kStaticScratchBytes, stream);
}

spqt_status spqt_set_debug(int on)
{
    spqt::g_debug = on ? 1 : 0;
    return SPQT_OK;
}

spqt_status spqt_set_tuning(int gemv_ctas, int reserved)
{
    if (gemv_ctas < 0 || reserved < 0 || reserved > 3) return SPQT_ERR_INVALID_ARG;
    spqt::g_tune_ctas = gemv_ctas;
    spqt::g_no_pdl = reserved & 1;
    spqt::g_no_cluster = (reserved >> 1) & 1;
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
