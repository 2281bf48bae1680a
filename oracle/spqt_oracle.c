/*
 * SpQt CPU oracle  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct statement of what the activation-sparse,
 * group-quantized GEMV computes.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it.  It shares no code,
 * header, table or constant with the CUDA library and is never a fallback.
 *
 * Notation (the paper's): W is m x n (m outputs, n inputs), y = W x
 * (Sec. 4.2.1, "(m,n) x (n,1)").  A quantization group ("superblock") is G
 * consecutive ROWS of ONE column; superblocks are stored row-major over
 * (block-row r, column k) -- the zigzag layout of Sec. 4.1.2, items (1),(2).
 * An input entry whose magnitude does not exceed the threshold is treated as
 * zero and its whole column of W is skipped (Sec. 2, "Dynamic Sparsity").
 * The index list idx[0:n_ns] of the surviving entries is what the sparse
 * GEMV consumes (Sec. 4.2.3).
 *
 * Every function below is the definition written out: no blocking, fusion or
 * reordering.  Floating point is fp64 except in the quantizer, whose steps
 * are single correctly-rounded IEEE fp32 operations (so that any conforming
 * implementation produces the same bytes); build with -ffp-contract=off.
 *
 * Parity status: every exported function is pinned by tests that do not go
 * through this file's own arithmetic (hand-worked example with exactly
 * representable values, closed forms, brute force, quantizer invariants,
 * numpy's float16 for the two conversions).  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- fp16 <-> fp32
 * IEEE binary16 bit patterns travel as uint16_t.  Widening is exact; narrowing
 * rounds to nearest, ties to even.  Both are pinned against numpy.float16.   */

static float half_to_float(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    float v;
    if (e == 0)
        v = ldexpf((float)f, -24);              /* zero / subnormal: f * 2^-24 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexpf((float)(1024 + f), e - 25);  /* (1 + f/1024) * 2^(e-15)     */
    return sign ? -v : v;
}

static uint16_t float_to_half(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t a = u & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);   /* NaN            */
    if (a >= 0x477ff000u) return (uint16_t)(sign | 0x7c00u);  /* >= 65520 -> Inf */
    if (a < 0x38800000u) {
        /* below 2^-14: the result is a multiple of 2^-24 (possibly 1024 of
         * them, which is exactly the smallest normal, encoded 0x0400).       */
        double d = (double)fabsf(x) * 16777216.0;             /* exact          */
        return (uint16_t)(sign | (uint16_t)nearbyint(d));     /* ties to even   */
    }
    uint32_t mant = a & 0x7fffffu;
    uint32_t e = (a >> 23) - 127 + 15;                        /* 1..30          */
    uint32_t h = (e << 10) | (mant >> 13);
    uint32_t rem = mant & 0x1fffu;
    if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) h++;   /* carry is fine  */
    return (uint16_t)(sign | h);
}

void spqt_oracle_half_to_float(const uint16_t* h, float* f, size_t count)
{
    for (size_t i = 0; i < count; ++i) f[i] = half_to_float(h[i]);
}

void spqt_oracle_float_to_half(const float* f, uint16_t* h, size_t count)
{
    for (size_t i = 0; i < count; ++i) h[i] = float_to_half(f[i]);
}

/* ---------------------------------------------------------------- geometry    */

static int bad_format(int m, int n, int bits, int group)
{
    if (m <= 0 || n <= 0) return 1;
    if (bits != 3 && bits != 4) return 1;
    if (group <= 0 || group % 2) return 1;
    if (bits == 3 && group % 8) return 1;
    if (m % group) return 1;
    return 0;
}

/* bytes of codes per superblock */
static size_t block_bytes(int bits, int group) { return (size_t)group * (size_t)bits / 8; }

size_t spqt_oracle_block_bytes(int bits, int group) { return block_bytes(bits, group); }

/* ---------------------------------------------------------------- quantizer
 * Asymmetric min/max round-to-nearest per superblock (group-wise scheme with a
 * scale and an additive offset per block, Sec. 2 / Sec. 4.1.1; any group-based
 * scheme and bit-width is admissible, Sec. 4.1.3).
 *   z  = min_i w_i                       (an fp16 value, kept exactly; a minimum or maximum
 *                                         that is zero is taken as +0.0 whatever the signs of
 *                                         the zeros in the group: the values are the same and
 *                                         the stored bytes do not depend on the order of the rows)
 *   s  = fp16( (max_i w_i - z) / qmax )  (fp32 subtract, fp32 divide, RN-even)
 *   q_i = clamp( rint( (w_i - z) / s ), 0, qmax ),  all zero when s == 0
 * W: fp16 bits, row-major, leading dimension ldw.
 * q: natural-order codes, one byte each, q[j*n + k].
 * scales, zeros: fp16 bits, index r*n + k.                                    */
int spqt_oracle_quantize(const uint16_t* W, int m, int n, int ldw, int bits, int group,
                         uint8_t* q, uint16_t* scales, uint16_t* zeros)
{
    if (bad_format(m, n, bits, group) || ldw < n) return 1;
    const int qmax = (1 << bits) - 1;
    const int R = m / group;
    for (int r = 0; r < R; ++r) {
        for (int k = 0; k < n; ++k) {
            float lo = INFINITY, hi = -INFINITY;
            for (int i = 0; i < group; ++i) {
                float w = half_to_float(W[(size_t)(r * group + i) * ldw + k]);
                if (w < lo) lo = w;
                if (w > hi) hi = w;
            }
            if (lo == 0.0f) lo = 0.0f;                   /* a zero extreme of either sign is +0.0 */
            if (hi == 0.0f) hi = 0.0f;
            volatile float range = hi - lo;              /* one fp32 subtract */
            volatile float s32 = range / (float)qmax;    /* one fp32 divide   */
            uint16_t sh = float_to_half(s32);
            float sf = half_to_float(sh);
            scales[(size_t)r * n + k] = sh;
            zeros[(size_t)r * n + k] = float_to_half(lo);   /* exact: lo is an fp16 value */
            for (int i = 0; i < group; ++i) {
                int code = 0;
                if (sf != 0.0f) {
                    float w = half_to_float(W[(size_t)(r * group + i) * ldw + k]);
                    volatile float d = w - lo;           /* one fp32 subtract */
                    volatile float t = d / sf;           /* one fp32 divide   */
                    float c = rintf(t);                  /* ties to even      */
                    if (c < 0.0f) c = 0.0f;
                    if (c > (float)qmax) c = (float)qmax;
                    code = (int)c;
                }
                q[(size_t)(r * group + i) * n + k] = (uint8_t)code;
            }
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- zigzag layout
 * Superblock (r,k) occupies bytes [(r*n+k)*B, (r*n+k+1)*B) of `codes`
 * (row-major over (block-row, column), Sec. 4.1.2 item (2)).
 * Inside a 4-bit block, byte i (i < G/2) holds code i in its low nibble and
 * code i+G/2 in its high nibble.
 * A 3-bit block is a 2-bit plane followed by a 1-bit plane:
 *   byte j (j < G/4)        = sum_{u<4} (code[j + u*G/4] & 3) << 2u
 *   byte G/4 + j (j < G/8)  = sum_{u<8} (code[j + u*G/8] >> 2) << u             */

static void put_block(uint8_t* blk, const uint8_t* c /* G codes */, int bits, int G)
{
    memset(blk, 0, block_bytes(bits, G));
    if (bits == 4) {
        for (int i = 0; i < G / 2; ++i)
            blk[i] = (uint8_t)((c[i] & 15) | ((c[i + G / 2] & 15) << 4));
    } else {
        for (int j = 0; j < G / 4; ++j)
            for (int u = 0; u < 4; ++u)
                blk[j] |= (uint8_t)((c[j + u * (G / 4)] & 3) << (2 * u));
        for (int j = 0; j < G / 8; ++j)
            for (int u = 0; u < 8; ++u)
                blk[G / 4 + j] |= (uint8_t)(((c[j + u * (G / 8)] >> 2) & 1) << u);
    }
}

/* code of row i (0 <= i < G) inside one block */
static int get_code(const uint8_t* blk, int i, int bits, int G)
{
    if (bits == 4) {
        int half = G / 2;
        return (i < half) ? (blk[i] & 15) : (blk[i - half] >> 4);
    } else {
        int q4 = G / 4, q8 = G / 8;
        int low2 = (blk[i % q4] >> (2 * (i / q4))) & 3;
        int top1 = (blk[q4 + i % q8] >> (i / q8)) & 1;
        return low2 | (top1 << 2);
    }
}

int spqt_oracle_pack_codes(const uint8_t* q, int m, int n, int bits, int group, uint8_t* codes)
{
    if (bad_format(m, n, bits, group) || group > 1024) return 1;
    const size_t B = block_bytes(bits, group);
    const int R = m / group;
    uint8_t col[1024];
    for (int r = 0; r < R; ++r)
        for (int k = 0; k < n; ++k) {
            for (int i = 0; i < group; ++i) col[i] = q[(size_t)(r * group + i) * n + k];
            put_block(codes + ((size_t)r * n + k) * B, col, bits, group);
        }
    return 0;
}

int spqt_oracle_unpack_codes(const uint8_t* codes, int m, int n, int bits, int group, uint8_t* q)
{
    if (bad_format(m, n, bits, group)) return 1;
    const size_t B = block_bytes(bits, group);
    const int R = m / group;
    for (int r = 0; r < R; ++r)
        for (int k = 0; k < n; ++k)
            for (int i = 0; i < group; ++i)
                q[(size_t)(r * group + i) * n + k] =
                    (uint8_t)get_code(codes + ((size_t)r * n + k) * B, i, bits, group);
    return 0;
}

/* quantize + lay out: what the offline conversion step produces (Sec. 3.2) */
int spqt_oracle_pack(const uint16_t* W, int m, int n, int ldw, int bits, int group,
                     uint8_t* q_scratch /* m*n bytes */, uint8_t* codes,
                     uint16_t* scales, uint16_t* zeros)
{
    int rc = spqt_oracle_quantize(W, m, n, ldw, bits, group, q_scratch, scales, zeros);
    if (rc) return rc;
    return spqt_oracle_pack_codes(q_scratch, m, n, bits, group, codes);
}

/* ---------------------------------------------------------------- dequantized weight
 * What[j][k] = s_rk * q_jk + z_rk in fp64 (exact: 11-bit x 4-bit + 11-bit).    */
static double weight_at(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                        int n, int bits, int G, int j, int k)
{
    int r = j / G, i = j % G;
    size_t b = (size_t)r * n + k;
    int code = get_code(codes + b * block_bytes(bits, G), i, bits, G);
    return (double)half_to_float(scales[b]) * (double)code + (double)half_to_float(zeros[b]);
}

int spqt_oracle_dequantize(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                           int m, int n, int bits, int group, double* What /* m*n */)
{
    if (bad_format(m, n, bits, group)) return 1;
    for (int j = 0; j < m; ++j)
        for (int k = 0; k < n; ++k)
            What[(size_t)j * n + k] = weight_at(codes, scales, zeros, n, bits, group, j, k);
    return 0;
}

/* ---------------------------------------------------------------- sparse index collection
 * idx = all k with |x_k| > t, ascending; *count = how many (Sec. 4.2.3: a
 * contiguous list of the indices of the entries above the threshold).  The
 * comparison is strict and is made after exact widening; NaN is never active. */
int spqt_oracle_sparsify(const uint16_t* x, int n, float t, int32_t* idx, int32_t* count)
{
    if (n < 0) return 1;
    int32_t c = 0;
    for (int k = 0; k < n; ++k)
        if (fabs((double)half_to_float(x[k])) > (double)t) idx[c++] = k;
    *count = c;
    return 0;
}

/* ---------------------------------------------------------------- sparse GEMV
 * y[j] = sum_{i<count} What[j][idx[i]] * x[idx[i]], fp64, in list order, for
 * the rows listed in `rows` (all m rows when rows == NULL).  bound[j] is the
 * same sum over absolute values (the tolerance is stated relative to it).
 * Rows are independent; the OpenMP pragma only spreads them over cores.        */
int spqt_oracle_sparse_gemv(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                            int m, int n, int bits, int group,
                            const uint16_t* x, const int32_t* idx, int32_t count,
                            const int32_t* rows, int n_rows,
                            double* y, double* bound)
{
    if (bad_format(m, n, bits, group) || count < 0 || count > n) return 1;
    const int nr = rows ? n_rows : m;
    for (int i = 0; i < count; ++i)
        if (idx[i] < 0 || idx[i] >= n) return 2;
    for (int a = 0; a < nr; ++a)
        if (rows && (rows[a] < 0 || rows[a] >= m)) return 3;
#pragma omp parallel for schedule(static)
    for (int a = 0; a < nr; ++a) {
        int j = rows ? rows[a] : a;
        double acc = 0.0, bnd = 0.0;
        for (int i = 0; i < count; ++i) {
            int k = idx[i];
            double w = weight_at(codes, scales, zeros, n, bits, group, j, k);
            double xv = (double)half_to_float(x[k]);
            acc += w * xv;
            bnd += fabs(w) * fabs(xv);
        }
        y[a] = acc;
        if (bound) bound[a] = bnd;
    }
    return 0;
}

/* dense GEMV over the same packed buffer: every column, no index list */
int spqt_oracle_dense_gemv(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros,
                           int m, int n, int bits, int group, const uint16_t* x,
                           const int32_t* rows, int n_rows, double* y, double* bound)
{
    if (bad_format(m, n, bits, group)) return 1;
    const int nr = rows ? n_rows : m;
    for (int a = 0; a < nr; ++a)
        if (rows && (rows[a] < 0 || rows[a] >= m)) return 3;
#pragma omp parallel for schedule(static)
    for (int a = 0; a < nr; ++a) {
        int j = rows ? rows[a] : a;
        double acc = 0.0, bnd = 0.0;
        for (int k = 0; k < n; ++k) {
            double w = weight_at(codes, scales, zeros, n, bits, group, j, k);
            double xv = (double)half_to_float(x[k]);
            acc += w * xv;
            bnd += fabs(w) * fabs(xv);
        }
        y[a] = acc;
        if (bound) bound[a] = bnd;
    }
    return 0;
}

/* ---------------------------------------------------------------- load-balanced partition
 * Worker w of S takes idx[floor(w*count/S) : floor((w+1)*count/S)) -- the even
 * split of the ACTIVE list over the workers of a block-row (Sec. 4.2.3; the
 * paper's example: 9 active entries over 3 workers -> 3 each).                 */
int spqt_oracle_partition(int32_t count, int S, int32_t* begin /* S+1 */)
{
    if (count < 0 || S <= 0) return 1;
    for (int w = 0; w <= S; ++w) begin[w] = (int32_t)(((int64_t)w * count) / S);
    return 0;
}

int spqt_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void spqt_oracle_set_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}
