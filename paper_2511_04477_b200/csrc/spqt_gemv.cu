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
// The list a CTA works from lives in shared memory as one 32-bit word per active
// entry: the column number in the low half, the fp16 bits of x_k in the high half.
// The prologue builds it: from idx and x (sparse call), by scanning x itself (the
// call that collects the indices in the same launch: every CTA scans x, counts the
// active entries of every 256-entry piece and expands only the pieces that overlap
// the list positions its own slices cover), or not at all (dense call).  When the
// part of the list a CTA needs exceeds the shared-memory window, the window is
// rebuilt between spans of the slice.
//
// Inside a CTA, every worker warp owns a contiguous part of each slice and runs its
// own copy pipeline over chunks of 32 list entries (64 with groups of 64 rows: 2 KB
// of 4-bit codes either way), kDepth chunks in flight; nothing is shared between
// the warps until the end of a segment.  Per chunk:
//   issue    lane e reads the word of entry e, copies the 4-byte (scale, zero) pair
//            of block (r, k_e) and keeps the entry word with the chunk; the code
//            blocks are copied 16 bytes per lane, the lanes of a block adjacent so
//            that every 32-byte sector crosses once, with 64-byte L2 granularity so
//            that an inactive neighbour block is not dragged in (cp.async).  The
//            dense call instead fetches the chunk's codes, pairs and x values with
//            three bulk copies issued by one lane (they are contiguous).
//   consume  lane e turns its pair into a = x_k*scale (exact in fp32) and
//            x_k*zero, writes the packed multiplier pair of its entry to
//            shared memory; then every lane does the dequantize-FMA work on its 16
//            codes of each block, reading the block's multiplier back.
// Entries past the end of a part are clamped to its last entry with weight 0, and
// the 512-byte steps of a chunk that hold no entry are skipped.  Two more warps,
// the writers (one per hand-over buffer), add the workers' sums at the end of a
// segment, publish the partial and, if this CTA is the last contributor of the
// block-row, produce y; they wait for the workers at a hardware barrier and for
// other CTAs with waits bounded in wall time (on expiry the workspace's status word
// is set and the kernel returns).
//
// Arithmetic:  y[j] = sum_k a_k * code_jk + sum_k x_k * zero_rk.  A 4-bit code
// becomes an fp32 operand with no conversion: a word whose bits above bit 22 are
// zero IS an fp32 subnormal, its integer value times 2^-149, and the multiplier
// a*2^93 is an exact power-of-two rescale, so each product is a*value*2^-56 up to
// the single rounding of the FMA.  Per 16-bit half-word the operands are its low
// 4, 8, 12 and 16 bits (u_j = q_0 + 16 q_1 + ... + 16^j q_j: three masks, the last
// needs none); the sums over the list are linear in them, so the per-code sums
// come back at the end of a segment as (U_j - U_{j-1}) / 16^j.  Under one logic op
// and one FMA per weight; two FMAs are issued as one packed fma.rn.f32x2.
#include <cstddef>

#include "spqt_common.cuh"

namespace spqt {

#ifndef SPQT_WORKERS
#define SPQT_WORKERS 16
#endif
#ifndef SPQT_DEPTH
#define SPQT_DEPTH 3
#endif
#ifndef SPQT_CAP
#define SPQT_CAP 12288
#endif
constexpr int kWorkers = SPQT_WORKERS;   // compute warps
constexpr int kWriters = 2;              // writer warps; segment sg goes to writer sg % kWriters
constexpr int kWriterWarp = kWorkers;    // the first of them
constexpr int kWarps = kWorkers + kWriters;
constexpr int kGemvThreads = kWarps * 32;
// list entries per chunk: 2 KB of 4-bit code blocks for either group size (32 blocks of 128 rows, 64 of 64)
__host__ __device__ constexpr int chunk_entries(int group) { return 32 * (128 / group); }
constexpr int kDepth = SPQT_DEPTH;       // chunks in flight per warp
constexpr unsigned long long kWaitNs = 1000000000ull;  // bound on every mbarrier wait: one second
constexpr int kMaxCluster = 8;           // largest thread-block cluster (CTAs of one block-row) used
constexpr int kCap = SPQT_CAP;              // list entries a CTA keeps in shared memory at a time
constexpr int kMaxListN = 65535;         // column numbers travel as 16 bits
constexpr int kMaxFusedN = 32768;        // longest x the in-kernel scan handles (128 pieces of 256 entries)
constexpr int kMaxPieces = kMaxFusedN / 256;

enum : int { kModeList = 0, kModeFused = 1, kModeDense = 2 };
enum : int { kFlagIdentity = 1, kFlagXs = 2, kFlagStatic = 4 };
constexpr int kMaxStaticSeg = 8;         // block-rows per CTA the static-partition ablation handles

static int g_tune_ctas = 0;  // 0 = one CTA per SM
int g_no_pdl = 0;            // 1 = plain stream-ordered launches (also read by the index-collection launch)
static int g_no_cluster = 0; // 1 = never launch thread-block clusters
static int g_static_partition = 0;  // 1 = ablation: static partition of the matrix columns instead of the list

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
        alignas(16) unsigned meta[CH];            // (scale, zero) pair of entry e
        alignas(16) unsigned xc[CH];              // list calls: the entry word; dense call: CH fp16 values of x
    };
    Stage stage[kWorkers][kDepth];                 // (the prologue borrows this area for its copy of x and its masks)
    alignas(16) float mult[kWorkers][CH][2];       // packed multiplier pair (a, a) * 2^93 of every entry of the chunk in work
    alignas(16) float red[2][kWorkers][G];         // per-warp partial sums of a finished segment
    float red_z[2][kWorkers];                      // and their offset terms
    alignas(8) uint64_t full[kWorkers][kDepth];    // dense call: completion of a stage's bulk copies
    uint64_t red_full[2], red_empty[2];
    // thread-block clusters only: partial sums the other CTAs of the cluster store here (CTA rank 0)
    alignas(16) float xred[kMaxCluster][G + 4];
    uint64_t xbar;                                 // counts their arrivals
    alignas(16) int tot[kMaxPieces];               // in-kernel scan: active entries of every 256 entries of x
    int static_table[kMaxStaticSeg][kWorkers + 1]; // ablation: list positions of a static column partition
    alignas(16) unsigned ent[kCap];                // the resident part of the list: x bits << 16 | column
};

struct GemvArgs {
    const uint8_t* codes;
    const unsigned* meta;       // (scale, zero) pairs
    int R, n;
    const __half* x;
    const int32_t* idx;
    const int32_t* count;
    __half* y;
    int* counters;
    int* status;
    unsigned long long* words;
    float* partials;
    float* zpartials;
    int max_slots;
    unsigned magic_p, magic_r;
    int cluster_k;
    float thr;
    int32_t* idx_out;
    int32_t* count_out;
    int flags;
};

template <int G, int BITS, int MODE, bool CLUSTER>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const GemvArgs a)
{
    constexpr int B = G * BITS / 8;
    constexpr int LPB = G / 32;       // copies: lanes per 4-bit block (16 bytes each)
    constexpr int CB = (B % 16 == 0) ? 16 : 8;   // bytes per copy: 3-bit blocks of 64 rows are only 8-byte aligned
    static_assert(BITS == 3 || BITS == 4, "3- or 4-bit codes");
    constexpr int SLOTS = 32 / LPB;   // copies: 4-bit blocks per 512-byte round
    constexpr int CH = chunk_entries(G);  // list entries per chunk
    constexpr int EPL = CH / 32;          // entries whose metadata a lane holds
    constexpr int SUBS = CH / SLOTS;      // copies: rounds per chunk
    // arithmetic: LM lanes share a block, each owns 16 of its rows (16 accumulators per lane: half the
    // registers of a 32-row share, which is what lets twice the warps stay resident)
    constexpr int LM = G / 16;
    constexpr int SLM = 32 / LM;          // blocks per step
    constexpr int MSUBS = CH / SLM;       // steps per chunk
    constexpr int KEEP = 16 / SLM;        // values per lane after the in-warp reduce-scatter
    constexpr int D = kDepth;
    constexpr bool DENSE = MODE == kModeDense;
    constexpr bool FUSED = MODE == kModeFused;
    using Smem = GemvSmem<G, BITS>;
    using Stage = typename Smem::Stage;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

    const int tid = threadIdx.x, lane = tid & 31;
    // the warp number through a shuffle: the compiler then knows it is the same in every lane and keeps
    // everything derived from it (the work map, the stage addresses) in uniform registers
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int P = gridDim.x, c = blockIdx.x;
    const int n = a.n, R = a.R;
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.red_full[b], kWorkers);
            mbar_init(&sm.red_empty[b], 1);
        }
        if (DENSE) {
            for (int w = 0; w < kWorkers; ++w)
                for (int s = 0; s < D; ++s) mbar_init(&sm.full[w][s], 1);
        }
        if (CLUSTER) mbar_init(&sm.xbar, a.cluster_k - 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Cluster launch (cluster_k CTAs work on one block-row and CTA rank 0 collects their sums): nobody
    // may touch another CTA's barrier before it is initialised.  Arrive now, wait much later.
    if (CLUSTER) cluster_arrive();

    Piece pc;
    pc.init_rows(R, P, c, a.magic_p, a.magic_r);

    // A hint only (no data is consumed before the wait below): pull x, and a given list, towards L2 while
    // the previous kernel of the stream drains.  A few CTAs do it for all.  (Measured: 1 to 2 % of a decode
    // layer's linears when x has left L2 since it was written.)
    if (!DENSE && (c & 7) == 0) {
        const char* xp = reinterpret_cast<const char*>(a.x);
        for (int off = tid * 128; off < 2 * n; off += kGemvThreads * 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(xp + off));
        if (!FUSED && a.idx != nullptr) {
            const char* ip = reinterpret_cast<const char*>(a.idx);
            for (int off = tid * 128; off < 4 * n; off += kGemvThreads * 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(ip + off));
        }
    }
    // Programmatic dependent launch: this grid may have been started while the previous kernel of
    // the stream was still draining.  Nothing above touches memory another kernel writes; everything
    // below waits for that kernel to complete, and lets the next kernel of the stream start early in turn.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ------------------------------------------------------------ prologue: the list in shared memory
    // Scratch borrowed from the stage area until the pipeline starts: a copy of x (16-bit words,
    // padded to whole 256-entry pieces) and, for the in-kernel scan, one activity byte per lane and piece.
    const int nv = (n + 255) >> 8;
    const unsigned xs_addr = smem_u32(&sm.stage[0][0]);
    unsigned char* const pm = reinterpret_cast<unsigned char*>(&sm.stage[0][0]) + (size_t)nv * 512;
    const unsigned short* const xg = reinterpret_cast<const unsigned short*>(a.x);
    const bool vec_ok = (reinterpret_cast<uintptr_t>(a.x) & 15) == 0;
    const bool has_xs = FUSED || (a.flags & kFlagXs) != 0;
    const unsigned ent_base = smem_u32(&sm.ent[0]);

    // piece li of x (entries 256 li + 8 lane .. + 7) from global memory, zero past the end
    auto load_piece = [&](int li) -> uint4 {
        const int k0 = li * 256 + lane * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (vec_ok && k0 + 8 <= n) {
            v = __ldg(reinterpret_cast<const uint4*>(a.x + k0));
        } else if (k0 < n) {
            unsigned short hv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) hv[e] = (k0 + e < n) ? __ldg(xg + k0 + e) : (unsigned short)0;
            v.x = hv[0] | ((unsigned)hv[1] << 16);
            v.y = hv[2] | ((unsigned)hv[3] << 16);
            v.z = hv[4] | ((unsigned)hv[5] << 16);
            v.w = hv[6] | ((unsigned)hv[7] << 16);
        }
        return v;
    };

    // Copy x to shared memory; the in-kernel scan also records which entries are active and how many
    // per piece.  Run by the warps gw = 0..NW-1 of a group; the caller synchronises the group afterwards.
    auto stage_x = [&](int gw, int NW) {
        constexpr int kPiecesPerRound = 4;   // loads of one round share a round trip
        // the largest fp16 value not above t (any negative value if t < 0: everything but NaN is
        // active; +inf if t is NaN or +inf: nothing is)
        const float thr = a.thr;
        const __half thr_h = (thr != thr) ? __ushort_as_half((unsigned short)0x7c00)
                                          : (thr < 0.0f ? __float2half_rn(-1.0f) : __float2half_rd(thr));
        const __half2 thr_h2 = __half2half2(thr_h);
        if (FUSED) {
            for (int i = nv + gw * 32 + lane; i < kMaxPieces; i += NW * 32) sm.tot[i] = 0;
        }
#pragma unroll 1
        for (int l0 = gw; l0 < nv; l0 += kPiecesPerRound * NW) {
            uint4 xv[kPiecesPerRound];
#pragma unroll
            for (int j = 0; j < kPiecesPerRound; ++j) {
                const int li = l0 + j * NW;
                xv[j] = make_uint4(0u, 0u, 0u, 0u);
                if (li < nv) xv[j] = load_piece(li);  // uniform across the warp
            }
#pragma unroll
            for (int j = 0; j < kPiecesPerRound; ++j) {
                const int li = l0 + j * NW, k0 = li * 256 + lane * 8;
                if (li < nv) {
                    sts_v4(xs_addr + (unsigned)li * 512u + (unsigned)lane * 16u, xv[j]);
                    if (FUSED) {
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
                        if (lane == 0) sm.tot[li] = (int)tot;
                    }
                }
            }
        }
    };

    // The window [lo, hi) of the list into sm.ent, by the threads gt = 0..NT-1 (warps gw = 0..NW-1) of
    // a group.  The in-kernel scan also writes the list positions [olo, ohi) of the index list the
    // call returns.  The caller synchronises the group before (x staged) and afterwards.
    auto build_window = [&](int lo, int hi, int olo, int ohi, int gw, int NW) {
        if (FUSED) {
            // lane l holds the totals of pieces 4l..4l+3; sums over the pieces below a given one come
            // from one warp reduction each
            int tot4[4];
            {
                const int4 t4 = *reinterpret_cast<const int4*>(&sm.tot[lane * 4]);
                tot4[0] = t4.x; tot4[1] = t4.y; tot4[2] = t4.z; tot4[3] = t4.w;
            }
            const unsigned len = (unsigned)max(hi - lo, 0), olen = (unsigned)max(ohi - olo, 0);
#pragma unroll 1
            for (int li = gw; li < nv; li += NW) {
                unsigned below = 0;  // active entries of this lane's pieces that come before piece li
#pragma unroll
                for (int q = 0; q < 4; ++q) below += (lane * 4 + q < li) ? (unsigned)tot4[q] : 0u;
                const int base = (int)__reduce_add_sync(0xffffffffu, below);
                const int q = li & 3;
                const int tsel = q == 0 ? tot4[0] : q == 1 ? tot4[1] : q == 2 ? tot4[2] : tot4[3];
                const int end = base + __shfl_sync(0xffffffffu, tsel, li >> 2);
                const bool in_win = end > lo && base < hi, in_out = end > olo && base < ohi;
                if (!in_win && !in_out) continue;  // uniform across the warp
                const unsigned m8 = pm[li * 32 + lane];
                const uint4 xv = lds_v4(xs_addr + (unsigned)li * 512u + (unsigned)lane * 16u);
                const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w};
                const int c8 = __popc(m8);
                int incl = c8;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += up;
                }
                int pos = base + incl - c8;
                const int col0 = li * 256 + lane * 8;
                // one predicated store per entry (a divergent branch per entry would cost far more)
                if (in_win) {
                    int p2 = pos;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const unsigned on = (m8 >> e) & 1u, d = (unsigned)(p2 - lo);
                        const unsigned xb = (e & 1) ? (xw[e >> 1] & 0xffff0000u) : (xw[e >> 1] << 16);
                        st_shared_u32_if(on & (d < len ? 1u : 0u), ent_base + 4u * d, xb | (unsigned)(col0 + e));
                        p2 += (int)on;
                    }
                }
                if (in_out) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const unsigned on = (m8 >> e) & 1u, d = (unsigned)(pos - olo);
                        st_global_if(on & (d < olen ? 1u : 0u), a.idx_out + pos, col0 + e);
                        pos += (int)on;
                    }
                }
            }
        } else if (!DENSE) {
            const bool identity = (a.flags & kFlagIdentity) != 0;
            const int NT = NW * 32, gt = gw * 32 + lane;
#pragma unroll 4
            for (int i = gt; i < hi - lo; i += NT) {
                const unsigned col = identity ? (unsigned)(lo + i) : (unsigned)__ldg(a.idx + lo + i);
                const unsigned xb = has_xs ? lds_u16(xs_addr + 2u * col) : (unsigned)__ldg(xg + col);
                sm.ent[i] = (xb << 16) | col;
            }
        }
    };

    int count = 0;
    bool resident = true;
    int win_lo = 0;  // list position of sm.ent[0]
    if (DENSE) {
        count = n;
        pc.set_count(n, 8);
    } else {
        if (!FUSED) count = (a.flags & kFlagIdentity) ? n : __ldg(a.count);  // in flight while x is staged
        // A given list that fits the window whole is copied whole, whatever the count turns out to be
        // (idx holds n entries): its first entries are then loaded beside x and the count, in the same
        // round trip, instead of after them.  Entries past the count are never used.
        constexpr int kEarly = 8;
        const bool whole_list = !FUSED && !(a.flags & kFlagIdentity) && has_xs && n <= kCap;
        int early[kEarly];
        if (whole_list) {
#pragma unroll
            for (int j = 0; j < kEarly; ++j) {
                const int i = tid + j * kGemvThreads;
                early[j] = i < n ? __ldg(a.idx + i) : 0;
            }
        }
        if (has_xs) stage_x(warp, kWarps);
        __syncthreads();
        if (whole_list) {
#pragma unroll
            for (int j = 0; j < kEarly; ++j) {
                const int i = tid + j * kGemvThreads;
                const unsigned col = min((unsigned)early[j], (unsigned)(n - 1));   // past the count: anything, but in range
                if (i < n) sm.ent[i] = (lds_u16(xs_addr + 2u * col) << 16) | col;
            }
            for (int i = tid + kEarly * kGemvThreads; i < n; i += kGemvThreads) {
                const unsigned col = min((unsigned)__ldg(a.idx + i), (unsigned)(n - 1));
                sm.ent[i] = (lds_u16(xs_addr + 2u * col) << 16) | col;
            }
        }
        if (FUSED) {
            const int4 t4 = *reinterpret_cast<const int4*>(&sm.tot[lane * 4]);
            count = (int)__reduce_add_sync(0xffffffffu, (unsigned)(t4.x + t4.y + t4.z + t4.w));
            if (c == 0 && tid == 0) *a.count_out = count;
        }
        pc.set_count(count);
        if (FUSED && (a.flags & kFlagStatic) && pc.r_last - pc.r_first < kMaxStaticSeg) {
            // Ablation, the paper's "sparse without load balancing": every CTA, and inside it every warp,
            // takes a fixed range of the matrix COLUMNS of its block-row and works on whatever active
            // entries fall into it.  Boundary j of the CTA's column range in a block-row becomes the list
            // position "active entries below that column", read off the scan: the totals of the pieces
            // below, plus the activity bits below the column inside its piece.
            const int nseg = pc.r_last - pc.r_first + 1;
            int tot4[4];
            {
                const int4 t4 = *reinterpret_cast<const int4*>(&sm.tot[lane * 4]);
                tot4[0] = t4.x; tot4[1] = t4.y; tot4[2] = t4.z; tot4[3] = t4.w;
            }
#pragma unroll 1
            for (int q = warp; q < nseg * (kWorkers + 1); q += kWarps) {
                const int sgi = q / (kWorkers + 1), j = q % (kWorkers + 1);
                unsigned u0, u1;
                pc.fraction(pc.r_first + sgi, &u0, &u1);
                const int k0 = (int)((u0 * (unsigned)n) / (unsigned)P), k1 = (int)((u1 * (unsigned)n) / (unsigned)P);
                const int kb = k0 + (int)(((long long)(k1 - k0) * j) / kWorkers);
                const int piece = kb >> 8, lane_of = (kb & 255) >> 3, bit = kb & 7;
                unsigned below = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) below += (lane * 4 + i < piece) ? (unsigned)tot4[i] : 0u;
                const unsigned m8 = piece < nv ? pm[piece * 32 + lane] : 0u;
                below += lane < lane_of ? (unsigned)__popc(m8) : (lane == lane_of ? (unsigned)__popc(m8 & ((1u << bit) - 1u)) : 0u);
                const int posk = (int)__reduce_add_sync(0xffffffffu, below);
                if (lane == 0) sm.static_table[sgi][j] = posk;
            }
            __syncthreads();
            pc.table = &sm.static_table[0][0];
        }
        // list positions this CTA will read: the union of its slices.  (A piece that spans several
        // block-rows ends the first one and begins the last one: its slices cover the whole list
        // between them.)
        int need_lo = 0, need_hi = count;
        if (pc.r_first == pc.r_last) pc.slice(pc.r_first, &need_lo, &need_hi);
        if (pc.table != nullptr && pc.r_first != pc.r_last) {
            // a static partition: the CTA's column ranges in its first and last block-row, and whole rows between
            int a0, b0, a1, b1;
            pc.slice(pc.r_first, &a0, &b0);
            pc.slice(pc.r_last, &a1, &b1);
            need_lo = pc.r_last - pc.r_first > 1 ? 0 : min(a0, a1);
            need_hi = pc.r_last - pc.r_first > 1 ? count : max(b0, b1);
        }
        resident = (need_hi - need_lo) <= kCap;
        if (!resident && pc.table != nullptr) {
            // (the ablation does not rebuild windows: long lists take the balanced partition)
            pc.table = nullptr;
            need_lo = 0;
            need_hi = count;
            if (pc.r_first == pc.r_last) pc.slice(pc.r_first, &need_lo, &need_hi);
        }
        int olo = 0, ohi = 0;  // the part of the returned index list this CTA writes: its slice of block-row 0
        if (FUSED && pc.r_first == 0) pc.slice(0, &olo, &ohi);
        if (whole_list) {
            win_lo = 0;          // the whole list is in place already
            resident = true;
        } else if (resident) {
            win_lo = need_lo;
            build_window(need_lo, need_hi, olo, ohi, warp, kWarps);
        } else {
            // the window of the first span; the workers rebuild it for every later span
            int p0, p1;
            pc.slice(pc.r_first, &p0, &p1);
            win_lo = p0;
            const int whi = min(p1, p0 + kCap);
            build_window(p0, whi, max(olo, p0), min(ohi, whi), warp, kWarps);
        }
        __syncthreads();  // the list is in place; the stage area is free for the pipeline
    }
    if (CLUSTER) cluster_wait();  // every CTA of the cluster has initialised its barriers by now

    if (warp >= kWriterWarp) {
        // ------------------------------------------------------------ writers
        // Two warps, one per hand-over buffer, so that the chains of dependent L2 round trips
        // (store, fence, counter, read back) of consecutive segments overlap.
        constexpr int RPL = G / 32;  // rows per lane
        constexpr int kStride = G + 2;  // words per contributing CTA: G sums, the offset term, one of padding
        const int wr = warp - kWriterWarp;
        __half* const y = a.y;
        int* const counters = a.counters;
        bool ok = true;
        for (int r = pc.r_first + wr, sg = wr; r <= pc.r_last; r += kWriters, sg += kWriters) {
            const int b = sg & 1;  // hand-over buffer of this segment
            int first, nslots;
            pc.contributors(r, &first, &nslots);
            const int mine = c - first;
            unsigned long long* const row_words = a.words + (size_t)r * kTagSlots * kStride;
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
                    if (it == 0) t0 = global_ns();
                    else if (global_ns() - t0 > kWaitNs) break;
                    __nanosleep(400);   // a look every fraction of a microsecond: the watching must not take issue slots from the workers
                }
                if (spec) {
#pragma unroll
                    for (int j = 0; j < kSpec; ++j) oz[j] = __shfl_sync(0xffffffffu, oz[j], 0);
                }
            }
            handover_wait(b, (kWorkers + 1) * 32);
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
                for (int s = 1; s < a.cluster_k; ++s) {
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
                const size_t pslot = (size_t)r * a.max_slots + mine;
#pragma unroll
                for (int i = 0; i < RPL; ++i) __stcg(a.partials + pslot * G + lane * RPL + i, v[i]);
                if (lane == 0) __stcg(a.zpartials + pslot, zpart);
                __threadfence();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(counters + r, 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev != nslots - 1) continue;
                __threadfence();
                const float* p = a.partials + (size_t)r * a.max_slots * G + lane * RPL;
                const float* zp = a.zpartials + (size_t)r * a.max_slots;
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
        if (!ok && lane == 0) atomicExch(a.status, 1);
        return;
    }

    // ---------------------------------------------------------------- workers
    // Everything the loop touches in shared memory is addressed with 32-bit shared addresses kept in
    // registers, and the control around a chunk is kept to a handful of instructions: the loop is
    // bound by instruction issue and by the half-rate integer pipe, so every instruction outside the
    // arithmetic counts.  Per chunk k of a warp: ISSUE(k) the copies; once they have landed PREP(k),
    // the multipliers of its entries; MATH(k); then ISSUE(k+D) into the stage MATH(k) has freed.
    constexpr unsigned kStageBytes = (unsigned)sizeof(Stage);
    constexpr unsigned kMetaOff = (unsigned)offsetof(Stage, meta);
    constexpr unsigned kXcOff = (unsigned)offsetof(Stage, xc);
    const int slot = lane / LPB, h = lane % LPB;   // copies
    const int mslot = lane / LM, mh = lane % LM;   // arithmetic
    const unsigned stage_base = smem_u32(&sm.stage[warp][0]);
    const unsigned mult_base = smem_u32(&sm.mult[warp][0][0]);
    const unsigned full_base = smem_u32(&sm.full[warp][0]);
    const unsigned lane0 = lane == 0 ? 1u : 0u;

    // block-row constants of the issue side, refreshed when it enters a new block-row
    const uint8_t* b_codes = nullptr;   // codes of the block-row (list calls: this lane's 16-byte part)
    const unsigned* b_meta = nullptr;   // (scale, zero) pairs of the block-row
    const uint8_t* d_codes = nullptr;   // dense call: where the issue side's next chunk starts in the three arrays
    const unsigned* d_meta = nullptr;
    const __half* d_x = nullptr;
    auto enter_row = [&](int r, int pos) {
        const size_t row_base = (size_t)r * (size_t)n;
        b_codes = a.codes + row_base * B + ((!DENSE && BITS == 4) ? 16 * h : 0);
        b_meta = a.meta + row_base;
        if (DENSE) {
            d_codes = b_codes + (size_t)pos * B;
            d_meta = b_meta + pos;
            d_x = a.x + pos;
        }
    };

    // the list words of the entries a lane handles in the chunk at list position pos (FULL: all CH
    // entries exist; else the entries past the end of the part read the part's last entry again)
    auto load_entries = [&](int pos, int valid, bool full, unsigned* ev) {
        const unsigned ent_addr = ent_base + 4u * (unsigned)(pos - win_lo);
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            const int e = lane + 32 * q;
            ev[q] = lds_u32(ent_addr + 4u * (unsigned)(full ? e : min(e, valid - 1)));
        }
    };

    // ISSUE: the copies of one chunk (entries pos .. pos+valid-1 of the current block-row's list) into a stage
    auto issue = [&](int pos, int valid, bool full, unsigned st_addr, unsigned bar_addr) {
        if (DENSE) {
            // the chunk's blocks, pairs and x values are contiguous: three bulk copies by one lane, from
            // three pointers that simply advance (computing the addresses afresh for every chunk took
            // five times the instructions)
            if (full) {
                mbar_expect_tx_if(lane0, bar_addr, (unsigned)CH * (B + 6));
                bulk_copy_if(lane0, st_addr, d_codes, (unsigned)CH * B, bar_addr);
                bulk_copy_if(lane0, st_addr + kMetaOff, d_meta, (unsigned)CH * 4, bar_addr);
                bulk_copy_if(lane0, st_addr + kXcOff, d_x, (unsigned)CH * 2, bar_addr);
            } else {
                mbar_expect_tx_if(lane0, bar_addr, (unsigned)valid * (B + 6));
                bulk_copy_if(lane0, st_addr, d_codes, (unsigned)valid * B, bar_addr);
                bulk_copy_if(lane0, st_addr + kMetaOff, d_meta, (unsigned)valid * 4, bar_addr);
                bulk_copy_if(lane0, st_addr + kXcOff, d_x, (unsigned)valid * 2, bar_addr);
            }
            d_codes += CH * B;
            d_meta += CH;
            d_x += CH;
            return;
        }
        unsigned col[EPL];
        load_entries(pos, valid, full, col);
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            col[q] &= 0xffffu;
            cp_async_4(st_addr + kMetaOff + 4u * (lane + 32 * q), b_meta + col[q]);
        }
        if (BITS == 4) {
            // (steps past the end of the part copy the part's last block again: an L2 hit, and no branch)
#pragma unroll
            for (int u = 0; u < SUBS; ++u) {
                const unsigned cu = __shfl_sync(0xffffffffu, col[(u * SLOTS) / 32], (u * SLOTS + slot) & 31);
                cp_async_16_l2_64(st_addr + lane * 16 + u * 512, b_codes + (size_t)cu * B);
            }
        } else {
            // 3-bit blocks (48 or 24 bytes): the chunk's bytes in copies of CB bytes, lane after lane
            constexpr int NC = CH * B / CB / 32;
#pragma unroll
            for (int q = 0; q < NC; ++q) {
                const int off = (q * 32 + lane) * CB;    // byte offset inside the chunk's stage
                const int e = off / B, part = off % B;
                const unsigned cu = __shfl_sync(0xffffffffu, col[(q * 32 * CB / B) / 32], e & 31);
                const uint8_t* src = b_codes + (size_t)cu * B + part;
                if (CB == 16) cp_async_16_l2_64(st_addr + off, src);
                else cp_async_8(st_addr + off, src);
            }
        }
    };

    unsigned long long acc[8];  // 16 fp32 sums, two per register
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0ull;
    float zl = 0.0f;     // this lane's share of sum x_k * zero_rk of the current segment

    // PREP: lane e turns the pair of its entry into a = x_k*scale (exact in fp32), written as the packed
    // multiplier pair (a, a) * 2^93, and adds x_k*zero to its share of the offset term
    auto prep = [&](unsigned st_addr, int pos, int valid, bool full) {
        unsigned ev[EPL];
        if (!DENSE) load_entries(pos, valid, full, ev);
#pragma unroll
        for (int q = 0; q < EPL; ++q) {
            const int e = lane + 32 * q;
            const unsigned mz = lds_u32(st_addr + kMetaOff + 4u * e);
            const unsigned xb = DENSE ? lds_u16(st_addr + kXcOff + 2u * e) : (ev[q] >> 16);
            const float xf = __half2float(__ushort_as_half((unsigned short)xb));
            const float sf = __half2float(__ushort_as_half((unsigned short)(mz & 0xffffu)));
            const float zf = __half2float(__ushort_as_half((unsigned short)(mz >> 16)));
            float am = xf * sf;   // exact
            float zt = xf * zf;   // exact
            if (!full) {          // an entry past the end of the part: weight 0
                am = e < valid ? am : 0.0f;
                zt = e < valid ? zt : 0.0f;
            }
            zl += zt;
            const unsigned long long aa = pack2(am, am);
            sts_u64(mult_base + 8u * e, fmul2(aa, pack2(0x1p93f, 0x1p93f)));
        }
    };

    // MATH: one step of a chunk: SLM blocks, each lane 16 codes of one of them
    auto step = [&](unsigned st_addr, int u) {
        const unsigned long long mm = lds_u64(mult_base + 8u * (u * SLM + mslot));
        if (BITS == 4) {
            const uint2 wv = lds_v2(st_addr + lane * 8 + u * 256);
            fma_block8_cum(acc, wv, mm);
        } else {
            // lane t of a block: word t of the 2-bit plane (G/16 words); its top bits are the even
            // (t < LM/2) or odd bits of word t mod LM/2 of the 1-bit plane
            const unsigned blk = st_addr + (u * SLM + mslot) * B;
            const unsigned w2 = lds_u32(blk + 4u * mh);
            const unsigned w1 = lds_u32(blk + (G / 4) + 4u * (mh % (LM / 2))) >> (mh / (LM / 2));
            fma_block3_cum(acc, w2, w1, mm);
        }
    };

    // Stage ring: chunk number k of this warp (in issue order = consume order) uses stage k mod D, so
    // ISSUE(k+D) refills the stage MATH(k) has just read.  wi: where the issue side stands in the
    // warp's sequence of chunks (it runs ahead of the arithmetic, across block-rows); wc: the arithmetic.
    unsigned rc = 0;   // byte offset of the arithmetic's stage
    unsigned bc = 0;   // dense call: byte offset of that stage's barrier, and its phase parity
    unsigned par = 0;
    Walker wi, wc;
    wc.first(pc, warp, resident);
    wi = wc;
    bool ok = true;
    // moves the issue side to its next non-empty part (within the current span only when the window is
    // rebuilt between spans); false when there is none
    auto seek_issue = [&]() -> bool {
        if (resident) {
            while (wi.valid(pc) && !wi.has_chunk()) wi.next_span(pc, warp, true);
        }
        const bool more = wi.valid(pc) && wi.has_chunk();
        if (more) enter_row(wi.r, wi.pos);
        return more;
    };
    bool more_i = seek_issue();
    // ISSUE of the warp's next chunk, if there is one, into the stage at byte offset rs; one commit
    // group per call either way
    auto issue_next = [&](unsigned rs, unsigned bs) {
        if (more_i) {
            const int left = wi.end - wi.pos;
            if (left >= CH) issue(wi.pos, CH, true, stage_base + rs, full_base + bs);
            else issue(wi.pos, left, false, stage_base + rs, full_base + bs);
            wi.pos += CH;
            if (wi.pos >= wi.end) more_i = seek_issue();
        }
        if (!DENSE) cp_async_commit();
    };
    // fills the pipeline, starting with the stage the arithmetic will read next
    auto prime = [&]() {
        unsigned rs = rc, bs = bc;
#pragma unroll 1
        for (int s = 0; s < D; ++s) {
            issue_next(rs, bs);
            rs = (rs + kStageBytes == D * kStageBytes) ? 0u : rs + kStageBytes;
            bs = (bs + 8u == D * 8u) ? 0u : bs + 8u;
        }
    };
    prime();

    int sg = 0;
    while (wc.valid(pc)) {
#pragma unroll 1
        for (int pos = wc.pos; pos < wc.end; pos += CH) {
            const int left = wc.end - pos;
            if (DENSE) {
                if (ok) ok = mbar_wait_addr(full_base + bc, par);
            } else {
                cp_async_wait<D - 1>();
                __syncwarp();
            }
            const unsigned st_addr = stage_base + rc;
            if (left >= CH) {
                prep(st_addr, pos, CH, true);
                __syncwarp();
                // a full chunk: straight-line code (branches between the steps made the compiler shuffle
                // the accumulators around them, half as many instructions again)
#pragma unroll
                for (int u = 0; u < MSUBS; ++u) step(st_addr, u);
            } else {
                prep(st_addr, pos, left, false);
                __syncwarp();
                // the last chunk of a part: only the steps that hold entries
                const int nsub = (left + SLM - 1) / SLM;
#pragma unroll 1
                for (int u = 0; u < nsub; ++u) step(st_addr, u);
            }
            __syncwarp();  // every lane is done with this chunk's stage and multipliers
            issue_next(rc, bc);
            if (rc + kStageBytes == D * kStageBytes) { rc = 0u; bc = 0u; par ^= 1u; } else { rc += kStageBytes; bc += 8u; }
        }
        if (wc.last_of_segment()) {
            // ---- end of the segment: in-warp reduce-scatter over the column slots, then hand the
            // per-warp sums to the writer warp
            const int b = sg & 1;
            if (sg >= 2 && ok) ok = mbar_wait(&sm.red_empty[b], ((sg >> 1) - 1) & 1);
            float accf[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                unpack2(acc[i], accf[2 * i], accf[2 * i + 1]);
                acc[i] = 0ull;
            }
            // lanes that differ in the bits above log2(LM) hold sums of the same rows
            float t8[8], t4[4], keep[4];
            halve<16>(accf, t8, lane, 16);
            halve<8>(t8, t4, lane, 8);
            uncumulate(t4);   // the four values are the cumulative sums of one half-word
            if (LM == 8) {
#pragma unroll
                for (int i = 0; i < 4; ++i) keep[i] = t4[i];
            } else {
                float t2[2];
                halve<4>(t4, t2, lane, 4);
                keep[0] = t2[0];
                keep[1] = t2[1];
            }
            const int a_base = mslot * KEEP;
#pragma unroll
            for (int i = 0; i < KEEP; ++i) {
                const int ai = a_base + i;  // accumulator index = word*8 + nibble
                const int cw = ai >> 3, e2 = ai & 7;
                const int row = (BITS == 4)
                                    ? 8 * mh + 4 * cw + (e2 >> 1) + (e2 & 1) * (G / 2)
                                    : 4 * mh + (e2 >> 1) + (G / 4) * (2 * (e2 & 1) + cw);
                sm.red[b][warp][row] = keep[i] * 0x1p56f;  // undo the 2^-56 of the subnormal trick
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) zl += __shfl_xor_sync(0xffffffffu, zl, o);
            if (lane == 0) sm.red_z[b][warp] = zl;
            zl = 0.0f;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.red_full[b]);   // what the watching writer tests
            handover_arrive(b, (kWorkers + 1) * 32);       // what it finally waits on
            ++sg;
        }
        wc.next_span(pc, warp, resident);
        if (!DENSE && !resident && wc.valid(pc)) {
            // The next span needs another part of the list: every worker has drained its pipeline (the
            // span's chunks are consumed), so the stage area and the window can be rebuilt.
            cp_async_wait<0>();
            worker_barrier(kWorkers * 32);
            if (has_xs) stage_x(warp, kWorkers);
            worker_barrier(kWorkers * 32);
            int olo = 0, ohi = 0;
            if (FUSED && wc.r == 0) { olo = wc.lo; ohi = wc.hi; }
            win_lo = wc.lo;
            build_window(wc.lo, wc.hi, olo, ohi, warp, kWorkers);
            worker_barrier(kWorkers * 32);
            wi = wc;
            more_i = seek_issue();
            prime();
        }
    }
    if (!DENSE) cp_async_wait<0>();
    if (!ok && lane == 0) atomicExch(a.status, 1);
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
static __device__ int g_debug_bad;                           // verdict of the call being checked
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
    if (bad) {
        atomicExch(status, 2);       // sticky, for the caller
        atomicExch(&g_debug_bad, 1); // this call's verdict
    }
}

__global__ void debug_clear_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ count, int n)
{
    const int c = *count;
    const int lim = c < 0 ? 0 : (c > n ? n : c);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < lim; i += gridDim.x * blockDim.x) {
        const int k = idx[i];
        if (k >= 0 && k < n && n <= kDebugBits) g_debug_bitmap[k >> 5] = 0u;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        g_debug_count = g_debug_bad ? 0 : c;
        g_debug_bad = 0;  // ready for the next checked call
    }
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
    debug_clear_kernel<<<1, 256, 0, s>>>(idx, count, n);
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

// Grid sizes found by spqt_autotune, per (shape, format, kind of call).  Process-wide, small, searched
// linearly; not thread-safe (like spqt_set_tuning).
struct TunedEntry {
    int m, n, bits, group, mode, ctas;
};
constexpr int kMaxTuned = 256;
static TunedEntry g_tuned[kMaxTuned];
static int g_tuned_count = 0;

static int tuned_ctas(const Format& f, int mode)
{
    for (int i = 0; i < g_tuned_count; ++i) {
        const TunedEntry& e = g_tuned[i];
        if (e.m == f.m && e.n == f.n && e.bits == f.bits && e.group == f.group && e.mode == mode) return e.ctas;
    }
    return 0;
}

static void store_tuned(const Format& f, int mode, int ctas)
{
    for (int i = 0; i < g_tuned_count; ++i) {
        TunedEntry& e = g_tuned[i];
        if (e.m == f.m && e.n == f.n && e.bits == f.bits && e.group == f.group && e.mode == mode) {
            e.ctas = ctas;
            return;
        }
    }
    if (g_tuned_count < kMaxTuned) g_tuned[g_tuned_count++] = TunedEntry{f.m, f.n, f.bits, f.group, mode, ctas};
}

// Bytes of the stage area the prologue may borrow, and what it needs for an x of n entries.
template <int G, int BITS>
constexpr size_t stage_area_bytes() { return sizeof(GemvSmem<G, BITS>::stage); }
inline size_t scratch_bytes(int n, bool fused) { return (size_t)((n + 255) / 256) * (fused ? 544 : 512); }

template <int G, int BITS>
static bool fused_fits(int n) { return n <= kMaxFusedN && scratch_bytes(n, true) <= stage_area_bytes<G, BITS>(); }

template <int G, int BITS, int MODE>
static spqt_status launch_gemv(const Format& f, const void* codes, const void* meta, const void* x,
                               const int32_t* idx, const int32_t* count, void* y, void* workspace,
                               cudaStream_t s, FusedArgs fa, int flags)
{
    auto kernel = gemv_kernel<G, BITS, MODE, false>;
    auto kernel_c = gemv_kernel<G, BITS, MODE, true>;  // the thread-block-cluster variant
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
    const int tuned = g_tune_ctas > 0 ? g_tune_ctas : tuned_ctas(f, MODE);
    int P = tuned > 0 ? tuned : sms;
    if (tuned == 0 && f.R <= P) {
        // With few block-rows, a whole number of CTAs per block-row (if that keeps >= 85 % of the SMs
        // busy; 70 % for light launches, below) gives every CTA a single segment: no CTA then carries two
        // aggregation chains.
        int k = P / f.R;
        // A small matrix gains nothing from more than four CTAs per block-row: the combination of many
        // partial sums then costs more than the extra CTAs save (measured: 1024 x 4096 takes 6.8 us on 144
        // CTAs, 4.9 us on 32).  "Small": under 256 KB of blocks per CTA at four CTAs per block-row.
        const size_t row_bytes = (size_t)f.n * (size_t)(f.B + 4);
        bool small = k > 4 && row_bytes / 4 < (size_t(256) << 10);
        if (small) k = 4;
        // A block-row of under 96 KB is not worth cutting at all once there are 32 of them (measured:
        // 4096 x 1024 takes 4.0 / 4.5 / 3.8 us -- given list, index collection inside, dense -- on 32 CTAs
        // against 4.5 / 5.5 / 3.8 on 128; 8192 x 1024 4.1 / 4.6 / 3.8 on 64 against 4.8 / 5.5 / 4.2 on 128).
        if (k > 1 && f.R >= 32 && row_bytes < (size_t(96) << 10)) {
            k = 1;
            small = true;
        }
        // While a CTA's share stays under half a megabyte the launch is latency-bound, and leaving up to 30 %
        // of the SMs idle costs less than partial sums that cross CTAs in a ragged pattern
        // (measured: 14336 x 4096 on 112 CTAs, one block-row each, 8.9 us against 9.7 us on 148; 13824 x 5120
        // on 108 CTAs 8.7 against 9.6 us).
        const size_t share = (size_t)f.R * row_bytes / (size_t)P;
        const bool light = share < (size_t(512) << 10);
        // The dense call streams every block: from about a third of a megabyte per CTA the idle SMs cost more than
        // the ragged pieces (measured, 64 block-rows: 8192 x 28672 takes 28.5 us on 148 CTAs against 31.1 us on
        // 128, 8192 x 16384 18.3 against 19.3 us, 8192 x 8192 11.7 against 11.2 us; the sparse calls, with half
        // the bytes, stay better off on 128).
        const bool heavy_dense = MODE == kModeDense && share >= (size_t(320) << 10);
        if (small || (!heavy_dense && k * f.R * 100 >= (light ? 70 : 85) * P)) P = k * f.R;
    }
    // no more CTAs than pieces of at least 64 columns of one block-row
    const long long pieces = (long long)f.R * ((f.n + 63) / 64);
    if (P > pieces) P = (int)pieces;
    if (P > kMaxCtas) P = kMaxCtas;
    if (P < 1) P = 1;
    const int slots = max_slots(f.R);
    GemvArgs ga;
    ga.codes = static_cast<const uint8_t*>(codes);
    ga.meta = static_cast<const unsigned*>(meta);
    ga.R = f.R;
    ga.n = f.n;
    ga.x = static_cast<const __half*>(x);
    ga.idx = idx;
    ga.count = count;
    ga.y = static_cast<__half*>(y);
    ga.counters = static_cast<int*>(workspace);
    ga.status = ga.counters + f.R;
    ga.words = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace) + header_bytes(f.R));
    ga.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + header_bytes(f.R) + tagged_bytes(f));
    ga.zpartials = ga.partials + (size_t)f.R * slots * G;
    ga.max_slots = slots;
    ga.magic_p = magic_of((unsigned)P);
    ga.magic_r = magic_of((unsigned)f.R);
    ga.thr = fa.t;
    ga.idx_out = fa.idx_out;
    ga.count_out = fa.count_out;
    ga.flags = flags;
    if (MODE == kModeList && scratch_bytes(f.n, false) <= stage_area_bytes<G, BITS>()) ga.flags |= kFlagXs;
    if (MODE == kModeFused && g_static_partition) ga.flags |= kFlagStatic;
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
    // Not for the call that collects the indices inside: alone, or behind launches of its own kind, it gains
    // 0.3-0.45 us from a cluster like the others, but in a stream that alternates it with launches that fill
    // every SM (the stacked gate|up matrix of a decoder layer) every such pair of launches was measured 1.4-1.8 us
    // slower than the sum of its parts (0.2-0.6 us for the other kinds of call): a layer's four launches take
    // 37.1 us without these clusters and 38.7 us with them.  The CTAs of a cluster can only start together.
    if (!g_no_cluster && MODE != kModeFused && f.R <= P && P % f.R == 0 && P / f.R >= 2 && P / f.R <= kMaxCluster) {
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
    ga.cluster_k = cluster_k;
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, cluster_k ? kernel_c : kernel, ga);
    count_launch();
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SPQT_OK : SPQT_ERR_CUDA;
}

// Everything that can be checked on the host, in the order the header documents; nothing is put on
// the stream before all of it has passed.
static spqt_status check_gemv_args(const void* codes, const void* meta, int m, int n, int bits, int group,
                                   const void* x, const int32_t* idx, const int32_t* count, bool dense, void* y,
                                   void* workspace, size_t ws_bytes, Format* f)
{
    if (!codes || !meta || !x || !y || !workspace) return SPQT_ERR_INVALID_ARG;
    if (!dense && (!idx || !count)) return SPQT_ERR_INVALID_ARG;
    spqt_status st = make_format(m, n, bits, group, f);
    if (st != SPQT_OK) return st;
    if (!aligned(codes, 16) || !aligned(meta, 16) || !aligned(x, 2) || !aligned(y, 2) || !aligned(workspace, 16) ||
        (!dense && (!aligned(idx, 4) || !aligned(count, 4))))
        return SPQT_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(*f)) return SPQT_ERR_WORKSPACE;
    if ((long long)f->R * kMaxCtas >= (1ll << 31)) return SPQT_ERR_UNSUPPORTED;  // the work map is 32-bit
    return SPQT_OK;
}

template <int MODE>
static spqt_status gemv_dispatch(const Format& f, const void* codes, const void* meta, const void* x,
                                 const int32_t* idx, const int32_t* count, void* y, void* workspace,
                                 cudaStream_t s, FusedArgs fa, int flags)
{
    if (f.bits == 4 && f.group == 128) return launch_gemv<128, 4, MODE>(f, codes, meta, x, idx, count, y, workspace, s, fa, flags);
    if (f.bits == 4 && f.group == 64) return launch_gemv<64, 4, MODE>(f, codes, meta, x, idx, count, y, workspace, s, fa, flags);
    if (f.bits == 3 && f.group == 128) return launch_gemv<128, 3, MODE>(f, codes, meta, x, idx, count, y, workspace, s, fa, flags);
    if (f.bits == 3 && f.group == 64) return launch_gemv<64, 3, MODE>(f, codes, meta, x, idx, count, y, workspace, s, fa, flags);
    return SPQT_ERR_UNSUPPORTED;
}

static bool fused_fits_format(const Format& f)
{
    if (f.bits == 4 && f.group == 128) return fused_fits<128, 4>(f.n);
    if (f.bits == 4 && f.group == 64) return fused_fits<64, 4>(f.n);
    if (f.bits == 3 && f.group == 128) return fused_fits<128, 3>(f.n);
    return fused_fits<64, 3>(f.n);
}

// The sparse call after its arguments have been checked.
static spqt_status sparse_checked(const Format& f, const void* codes, const void* meta, const void* x,
                                  const int32_t* idx, const int32_t* count, void* y, void* workspace, cudaStream_t s)
{
    if (f.n > kMaxListN) return SPQT_ERR_UNSUPPORTED;
    if (g_debug) {
        spqt_status st = debug_check(idx, count, f.n, static_cast<int*>(workspace) + f.R, s, &count);
        if (st != SPQT_OK) return st;
    }
    return gemv_dispatch<kModeList>(f, codes, meta, x, idx, count, y, workspace, s, FusedArgs{0.0f, nullptr, nullptr}, 0);
}

}  // namespace spqt

// Scratch of the entry point that allocates nothing: one block-row counter array, status word and
// partial-sum area, resident in every device that loads the library until the process exits.
constexpr size_t kStaticScratchBytes = size_t(1) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the scratch on the current device (looked up once per device); nullptr on error.
static void* static_scratch_address()
{
    // In host code the array's name is only a handle; the device address has to be asked for,
    // once per device, with that device current.
    static void* scratch_addr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return nullptr;
        scratch_addr[dev] = p;
    }
    return scratch_addr[dev];
}

extern "C" {

spqt_status spqt_sparse_gemv(const void* codes, const void* scale_zero,
                             int m, int n, int bits, int group,
                             const void* x, const int32_t* idx, const int32_t* count,
                             void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = check_gemv_args(codes, scale_zero, m, n, bits, group, x, idx, count, false, y, workspace,
                                     workspace_bytes, &f);
    if (st != SPQT_OK) return st;
    return sparse_checked(f, codes, scale_zero, x, idx, count, y, workspace, static_cast<cudaStream_t>(stream));
}

spqt_status spqt_sparsify_gemv(const void* codes, const void* scale_zero,
                               int m, int n, int bits, int group,
                               const void* x, float t, int32_t* idx, int32_t* count,
                               void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = check_gemv_args(codes, scale_zero, m, n, bits, group, x, idx, count, false, y, workspace,
                                     workspace_bytes, &f);
    if (st != SPQT_OK) return st;
    if (n > kMaxListN) return SPQT_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!fused_fits_format(f)) {
        // too long for the in-kernel scan: the same result from the two separate launches
        st = spqt_sparsify(x, n, t, idx, count, stream);
        if (st != SPQT_OK) return st;
        return gemv_dispatch<kModeList>(f, codes, scale_zero, x, idx, count, y, workspace, s,
                                        FusedArgs{0.0f, nullptr, nullptr}, 0);
    }
    return gemv_dispatch<kModeFused>(f, codes, scale_zero, x, nullptr, nullptr, y, workspace, s,
                                     FusedArgs{t, idx, count}, 0);
}

spqt_status spqt_dense_gemv(const void* codes, const void* scale_zero,
                            int m, int n, int bits, int group, const void* x,
                            void* y, void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = check_gemv_args(codes, scale_zero, m, n, bits, group, x, nullptr, nullptr, true, y, workspace,
                                     workspace_bytes, &f);
    if (st != SPQT_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const FusedArgs none{0.0f, nullptr, nullptr};
    // whole chunks of a block-row by bulk copies when every chunk starts on a 16-byte boundary
    if ((n & 7) == 0 && aligned(x, 16))
        return gemv_dispatch<kModeDense>(f, codes, scale_zero, x, nullptr, nullptr, y, workspace, s, none, 0);
    if (n > kMaxListN) return SPQT_ERR_UNSUPPORTED;
    // otherwise the list path over the identity list
    return gemv_dispatch<kModeList>(f, codes, scale_zero, x, nullptr, nullptr, y, workspace, s, none, kFlagIdentity);
}

spqt_status spqt_sparse_gemv_static(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x, const int32_t* idx, const int32_t* count,
                                    void* y, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (workspace_bytes(f) > kStaticScratchBytes) return SPQT_ERR_WORKSPACE;  // problem too large for the built-in scratch
    void* const scratch = static_scratch_address();
    if (scratch == nullptr) return SPQT_ERR_CUDA;
    st = check_gemv_args(codes, scale_zero, m, n, bits, group, x, idx, count, false, y, scratch, kStaticScratchBytes, &f);
    if (st != SPQT_OK) return st;
    if (n > kMaxListN) return SPQT_ERR_UNSUPPORTED;
    // The scratch keeps whatever the previous call (or an interrupted one, or one of another shape)
    // left: the arrival counters, the status word and the tagged words must start at zero.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(scratch, 0, header_bytes(f.R) + tagged_bytes(f), s) != cudaSuccess) return SPQT_ERR_CUDA;
    return sparse_checked(f, codes, scale_zero, x, idx, count, y, scratch, s);
}

// Reads a status word (device) into *status_host, waits, and maps it to a return value.
static spqt_status read_status_word(const int* word, int* status_host, cudaStream_t s)
{
    if (cudaMemcpyAsync(status_host, word, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return SPQT_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SPQT_ERR_CUDA;
    return *status_host == 0 ? SPQT_OK : (*status_host == 1 ? SPQT_ERR_TIMEOUT : SPQT_ERR_INVALID_ARG);
}

spqt_status spqt_static_status(int m, int group, int* status_host, void* stream)
{
    if (!status_host || m <= 0 || (group != 64 && group != 128) || m % group) return SPQT_ERR_INVALID_ARG;
    void* const scratch = static_scratch_address();
    if (scratch == nullptr) return SPQT_ERR_CUDA;
    return read_status_word(static_cast<const int*>(scratch) + m / group, status_host, static_cast<cudaStream_t>(stream));
}

spqt_status spqt_autotune(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                          const void* x, float t, int32_t* idx, int32_t* count, void* y,
                          void* workspace, size_t workspace_bytes, void* flush, size_t flush_bytes,
                          int* ctas_sparse, int* ctas_dense, void* stream)
{
    using namespace spqt;
    Format f;
    spqt_status st = check_gemv_args(codes, scale_zero, m, n, bits, group, x, idx, count, false, y, workspace,
                                     workspace_bytes, &f);
    if (st != SPQT_OK) return st;
    if (n > kMaxListN) return SPQT_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int sms = sm_count();
    if (sms <= 0) return SPQT_ERR_CUDA;
    // candidates: one CTA per SM, and every whole number (1..8) of CTAs per block-row that fits
    int cand[10], ncand = 0;
    cand[ncand++] = sms;
    for (int k = 1; k <= kMaxCluster; ++k)
        if ((long long)k * f.R <= sms && k * f.R != sms) cand[ncand++] = k * f.R;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SPQT_ERR_CUDA;
    const int saved = g_tune_ctas;
    const bool fused_ok = fused_fits_format(f);
    int best[2] = {0, 0};
    st = SPQT_OK;
    for (int kind = 0; kind < 2 && st == SPQT_OK; ++kind) {   // 0: index collection + sparse product, 1: dense product
        float best_ms = 0.0f;
        for (int ci = 0; ci < ncand && st == SPQT_OK; ++ci) {
            g_tune_ctas = cand[ci];
            float ms_min = 0.0f;
            for (int rep = 0; rep < 6 && st == SPQT_OK; ++rep) {   // the first repetition warms up
                if (flush && flush_bytes && cudaMemsetAsync(flush, rep, flush_bytes, s) != cudaSuccess) st = SPQT_ERR_CUDA;
                if (cudaEventRecord(e0, s) != cudaSuccess) st = SPQT_ERR_CUDA;
                if (st == SPQT_OK) {
                    if (kind == 0) st = spqt_sparsify_gemv(codes, scale_zero, m, n, bits, group, x, t, idx, count, y, workspace, workspace_bytes, stream);
                    else st = spqt_dense_gemv(codes, scale_zero, m, n, bits, group, x, y, workspace, workspace_bytes, stream);
                }
                if (cudaEventRecord(e1, s) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) st = SPQT_ERR_CUDA;
                float ms = 0.0f;
                if (st == SPQT_OK && cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) st = SPQT_ERR_CUDA;
                if (rep > 0 && (ms_min == 0.0f || ms < ms_min)) ms_min = ms;
            }
            if (st == SPQT_OK && (best[kind] == 0 || ms_min < best_ms)) {
                best[kind] = cand[ci];
                best_ms = ms_min;
            }
        }
    }
    g_tune_ctas = saved;
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (st != SPQT_OK) return st;
    store_tuned(f, fused_ok ? kModeFused : kModeList, best[0]);
    if (fused_ok) store_tuned(f, kModeList, best[0]);
    store_tuned(f, (n & 7) == 0 && aligned(x, 16) ? kModeDense : kModeList, best[1]);
    if (ctas_sparse) *ctas_sparse = best[0];
    if (ctas_dense) *ctas_dense = best[1];
    return SPQT_OK;
}

spqt_status spqt_set_debug(int on)
{
    spqt::g_debug = on ? 1 : 0;
    return SPQT_OK;
}

spqt_status spqt_set_tuning(int gemv_ctas, int reserved)
{
    if (gemv_ctas < 0 || reserved < 0 || reserved > 7) return SPQT_ERR_INVALID_ARG;
    spqt::g_tune_ctas = gemv_ctas;
    spqt::g_no_pdl = reserved & 1;
    spqt::g_no_cluster = (reserved >> 1) & 1;
    spqt::g_static_partition = (reserved >> 2) & 1;
    return SPQT_OK;
}

spqt_status spqt_workspace_status(const void* workspace, int m, int group, int* status_host, void* stream)
{
    if (!workspace || !status_host || m <= 0 || (group != 64 && group != 128) || m % group) return SPQT_ERR_INVALID_ARG;
    return read_status_word(static_cast<const int*>(workspace) + m / group, status_host, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
