// The work map of the GEMV kernel: which block-rows, and which slices of the active index list,
// belong to which CTA and warp (32-bit arithmetic, divisions by multiply-high).  Included by
// spqt_gemv.cu only, after its compile-time constants (kWorkers, kCap).
#pragma once

namespace spqt {

// floor(v / d) for any 32-bit v from the multiplier m = floor((2^32 - 1) / d): the high product is
// the quotient or one less (the multiplier falls short of 2^32 / d by at most 1), one compare fixes it.
__host__ __device__ __forceinline__ unsigned magic_of(unsigned d) { return 0xffffffffu / d; }
__device__ __forceinline__ unsigned magic_div(unsigned v, unsigned d, unsigned m)
{
    const unsigned q = __umulhi(v, m);
    return q + ((v - q * d >= d) ? 1u : 0u);
}

// The piece of CTA c: block-rows r_first..r_last, and of each the slice of the active list that
// belongs to this CTA.  The R block-rows are laid end to end and cut into P equal pieces; the
// fraction [u0,u1) of a block-row is the slice [u0*count/P, u1*count/P) of the list.  Uniform across
// the CTA.  `unit` scales the slices: the dense path counts in groups of 8 columns so that every
// slice starts on a 16-byte boundary of x.
struct Piece {
    int R, P, c, count, unit, r_first, r_last;
    unsigned mP, mR;  // multipliers of magic_div for P and R, computed by the host
    unsigned qc, rc;  // count = qc * P + rc: keeps the slice arithmetic in 32 bits (the host checks R * P < 2^31)
    // Ablation (no load balancing): list positions of the boundaries of a static partition of the matrix
    // COLUMNS, [segment][kWorkers + 1] in shared memory; nullptr = the balanced partition of the list.
    const int* table;

    // the block-rows of the piece do not depend on the count: computed while the count is being fetched
    __device__ __forceinline__ void init_rows(int R_, int P_, int c_, unsigned mP_, unsigned mR_)
    {
        R = R_; P = P_; c = c_;
        mP = mP_;
        mR = mR_;
        unit = 1;
        table = nullptr;
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R;
        r_first = (int)magic_div(lo, (unsigned)P, mP);
        r_last = (int)magic_div(hi - 1u, (unsigned)P, mP);
    }
    // count_ list entries, in units of unit_ entries (count_ a multiple of unit_)
    __device__ __forceinline__ void set_count(int count_, int unit_ = 1)
    {
        unit = unit_;
        count = count_ / unit_;
        qc = magic_div((unsigned)count, (unsigned)P, mP);
        rc = (unsigned)count - qc * (unsigned)P;
    }
    // floor(u * count / P) for 0 <= u <= P
    __device__ __forceinline__ int scaled(unsigned u) const { return (int)(u * qc + magic_div(u * rc, (unsigned)P, mP)); }
    // the fraction [u0, u1) / P of block-row `row` that belongs to this CTA
    __device__ __forceinline__ void fraction(int row, unsigned* u0, unsigned* u1) const
    {
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R, base = (unsigned)row * (unsigned)P;
        *u0 = (lo > base ? lo : base) - base;
        *u1 = (hi < base + (unsigned)P ? hi : base + (unsigned)P) - base;
    }
    __device__ __forceinline__ void slice(int row, int* a, int* b) const
    {
        if (table != nullptr) {
            const int* t = table + (row - r_first) * (kWorkers + 1);
            *a = t[0];
            *b = t[kWorkers];
            return;
        }
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R, base = (unsigned)row * (unsigned)P;
        const unsigned u0 = (lo > base ? lo : base) - base;
        const unsigned u1 = (hi < base + (unsigned)P ? hi : base + (unsigned)P) - base;
        *a = scaled(u0) * unit;
        *b = scaled(u1) * unit;
    }
    // contributors to block-row `row`: CTAs first .. first+n-1
    __device__ __forceinline__ void contributors(int row, int* first, int* n) const
    {
        const unsigned f = magic_div((unsigned)row * (unsigned)P, (unsigned)R, mR);
        const unsigned l = magic_div(((unsigned)row + 1u) * (unsigned)P - 1u, (unsigned)R, mR);
        *first = (int)f;
        *n = (int)(l - f + 1u);
    }
};

// The part [a,b) of the span [lo,hi) that worker warp `warp` processes: the span is cut into
// kWorkers contiguous parts whose boundaries are multiples of 8 entries from lo.
__device__ __forceinline__ void warp_part(const Piece& pc, int r, int lo, int hi, int warp, int* a, int* b)
{
    if (pc.table != nullptr) {  // static column partition: the warp's column range, as list positions
        const int* t = pc.table + (r - pc.r_first) * (kWorkers + 1);
        *a = t[warp];
        *b = t[warp + 1];
        return;
    }
    const int q = (hi - lo + 7) >> 3;
    const int ua = (warp * q) / kWorkers, ub = ((warp + 1) * q) / kWorkers;
    *a = lo + 8 * ua;
    *b = min(lo + 8 * ub, hi);
}

// A warp's walk over its work.  The CTA's slice of a block-row (a segment) is processed as one span
// when the list entries the CTA needs are all resident in shared memory, else as consecutive spans
// of at most kCap entries (the shared-memory window is rebuilt between them).  Within a span the
// warp owns the part [pos, end).
struct Walker {
    int r, lo, hi, seg_hi;
    int pos, end;
    __device__ __forceinline__ bool valid(const Piece& pc) const { return r <= pc.r_last; }
    __device__ __forceinline__ void open_segment(const Piece& pc, int warp, bool resident)
    {
        if (r <= pc.r_last) {
            int p0, p1;
            pc.slice(r, &p0, &p1);
            seg_hi = p1;
            lo = p0;
            hi = resident ? p1 : min(p1, p0 + kCap);
            warp_part(pc, r, lo, hi, warp, &pos, &end);
        }
    }
    __device__ __forceinline__ void first(const Piece& pc, int warp, bool resident)
    {
        r = pc.r_first;
        open_segment(pc, warp, resident);
    }
    __device__ __forceinline__ bool last_of_segment() const { return hi >= seg_hi; }
    __device__ __forceinline__ void next_span(const Piece& pc, int warp, bool resident)
    {
        if (hi < seg_hi) {
            lo = hi;
            hi = min(seg_hi, lo + kCap);
            warp_part(pc, r, lo, hi, warp, &pos, &end);
        } else {
            ++r;
            open_segment(pc, warp, resident);
        }
    }
    __device__ __forceinline__ bool has_chunk() const { return pos < end; }
};

}  // namespace spqt
