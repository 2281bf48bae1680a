// The work map of the GEMV kernel: which block-rows, and which slices of the active index list,
// belong to which CTA and warp (32-bit arithmetic, divisions by multiply-high).  Included by
// spqt_gemv.cu only, after its compile-time constants (kWorkers).
#pragma once

namespace spqt {

// ---------------------------------------------------------------- work map

// The piece of CTA c: block-rows r_first..r_last, and of each the slice of the
// active list that belongs to this CTA.  Uniform across the CTA.

// floor(v / d) for any 32-bit v from the multiplier m = floor((2^32 - 1) / d): the high product is
// the quotient or one less (the multiplier falls short of 2^32 / d by at most 1), one compare fixes it.
__host__ __device__ __forceinline__ unsigned magic_of(unsigned d) { return 0xffffffffu / d; }
__device__ __forceinline__ unsigned magic_div(unsigned v, unsigned d, unsigned m)
{
    const unsigned q = __umulhi(v, m);
    return q + ((v - q * d >= d) ? 1u : 0u);
}

struct Piece {
    int R, P, c, count, r_first, r_last;
    unsigned mP, mR;  // multipliers of magic_div for P and R, computed by the host
    unsigned qc, rc;  // count = qc * P + rc: keeps the slice arithmetic in 32 bits (the host checks R * P < 2^31)

    // the block-rows of the piece do not depend on the count: computed while the count is being fetched
    __device__ __forceinline__ void init_rows(int R_, int P_, int c_, unsigned mP_, unsigned mR_)
    {
        R = R_; P = P_; c = c_;
        mP = mP_;
        mR = mR_;
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R;
        r_first = (int)magic_div(lo, (unsigned)P, mP);
        r_last = (int)magic_div(hi - 1u, (unsigned)P, mP);
    }
    __device__ __forceinline__ void set_count(int count_)
    {
        count = count_;
        qc = magic_div((unsigned)count, (unsigned)P, mP);
        rc = (unsigned)count - qc * (unsigned)P;
    }
    // floor(u * count / P) for 0 <= u <= P
    __device__ __forceinline__ int scaled(unsigned u) const { return (int)(u * qc + magic_div(u * rc, (unsigned)P, mP)); }
    __device__ __forceinline__ void slice_compute(int row, int* a, int* b) const
    {
        const unsigned lo = (unsigned)c * (unsigned)R, hi = lo + (unsigned)R, base = (unsigned)row * (unsigned)P;
        const unsigned u0 = (lo > base ? lo : base) - base;
        const unsigned u1 = (hi < base + (unsigned)P ? hi : base + (unsigned)P) - base;
        *a = scaled(u0);
        *b = scaled(u1);
    }
    __device__ __forceinline__ void slice(int row, int* a, int* b) const { slice_compute(row, a, b); }
    // contributors to block-row `row`: CTAs first .. first+n-1
    __device__ __forceinline__ void contributors(int row, int* first, int* n) const
    {
        const unsigned f = magic_div((unsigned)row * (unsigned)P, (unsigned)R, mR);
        const unsigned l = magic_div(((unsigned)row + 1u) * (unsigned)P - 1u, (unsigned)R, mR);
        *first = (int)f;
        *n = (int)(l - f + 1u);
    }
};

// A warp's position in its sequence of chunks: list position `pos` of the
// chunk's first entry inside block-row r (whose slice ends at p1).
struct Cursor {
    int r, pos, p1;
    int chunk;  // list entries per chunk (32 or 64, by format)
    __device__ __forceinline__ void settle(const Piece& pc, int warp)
    {
        while (r <= pc.r_last && pos >= p1) {
            ++r;
            if (r <= pc.r_last) {
                int p0;
                pc.slice(r, &p0, &p1);
                pos = p0 + warp * chunk;
            }
        }
    }
    __device__ __forceinline__ void init(const Piece& pc, int warp, int chunk_)
    {
        chunk = chunk_;
        r = pc.r_first;
        int p0;
        pc.slice(r, &p0, &p1);
        pos = p0 + warp * chunk;
        settle(pc, warp);
    }
    __device__ __forceinline__ bool valid(const Piece& pc) const { return r <= pc.r_last; }
    __device__ __forceinline__ void advance(const Piece& pc, int warp)
    {
        pos += kWorkers * chunk;
        if (pos >= p1) settle(pc, warp);
    }
};

}  // namespace spqt
