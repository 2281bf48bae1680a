/*
 * spqt.h -- C ABI of the SpQt hot path for NVIDIA B200 (sm_100a).
 *
 * SpQt ("Enabling Dynamic Sparsity in Quantized LLM Inference") runs every
 * decode-time linear layer y = W x as: (1) collect the indices of the hidden
 * state entries whose magnitude exceeds a calibrated threshold, (2) multiply
 * only the matching columns of the group-quantized W, which is stored in the
 * "zigzag" layout so that a skipped column is a run of whole quantization
 * blocks.  This library is that path and nothing else.
 *
 * Conventions
 *   W is m x n: m output features (rows), n input features (columns), y = W x
 *   (paper Sec. 4.2.1).  G = group size, b = bits per code, R = m / G
 *   block-rows, B = G*b/8 bytes of codes per block.
 *   Every pointer is a DEVICE pointer unless its name ends in _host.
 *   `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *   stream).  All calls are asynchronous on that stream and never synchronise
 *   the device, except the *_host entry point and spqt_workspace_status, which
 *   say so.
 *   The caller owns every buffer; the library allocates nothing, frees nothing
 *   and keeps no pointer after a call returns.
 *
 * Data layout (paper Sec. 4.1.2: column-aligned grouping, row-major block storage)
 *   A block (r,k) is the G codes of rows r*G .. r*G+G-1 of column k.
 *   codes : R*n blocks of B bytes; block (r,k) starts at byte (r*n + k)*B.
 *           4-bit block: byte i (i < G/2) = code[i] | code[i + G/2] << 4.
 *           3-bit block: G/4 bytes of a 2-bit plane, byte j = sum_{u<4}
 *           (code[j + u*G/4] & 3) << 2u, then G/8 bytes of a 1-bit plane,
 *           byte j = sum_{u<8} (code[j + u*G/8] >> 2) << u.
 *   scale_zero : R*n pairs of fp16 in the same block order: the pair of block
 *           (r,k) is at fp16 index 2*(r*n + k): first the scale, then the zero.
 *           A weight is What[r*G+i][k] = scale[r,k] * code_i + zero[r,k]
 *           ("zero" is the additive offset of the block, its minimum).
 *
 * Errors
 *   Every entry point returns a spqt_status.  Arguments that can be checked on
 *   the host are checked before anything is put on the stream; a failed check
 *   launches nothing.  The contents of idx/count are trusted (indices in [0,n),
 *   no duplicates, count <= n) unless checked mode is on.
 */
#ifndef SPQT_H
#define SPQT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPQT_OK = 0,
    SPQT_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, ldw < n; a bad index list (checked mode) */
    SPQT_ERR_UNSUPPORTED = 2, /* bits not in {3,4}, group not in {64,128}, m % group != 0, n too large     */
    SPQT_ERR_ALIGNMENT = 3,   /* a pointer is not aligned as documented                                    */
    SPQT_ERR_WORKSPACE = 4,   /* workspace smaller than spqt_packed_sizes reports                          */
    SPQT_ERR_CUDA = 5,        /* the CUDA runtime reported an error (launch, copy, query)                  */
    SPQT_ERR_TIMEOUT = 6      /* a bounded wait inside a kernel expired (seen through spqt_workspace_status) */
} spqt_status;

/* Human-readable name of a status code; never NULL. */
const char* spqt_status_string(int status);

/* Library version, major*1000 + minor. */
int spqt_version(void);

/*
 * Sizes in bytes of the buffers a problem needs (layout of paper Sec. 4.1.2: R*n
 * blocks; one scale and one offset per block, Sec. 4.1.1).  Any out-pointer may
 * be NULL.  Needs no GPU.  gemv_workspace_bytes covers every GEMV entry point.
 */
spqt_status spqt_packed_sizes(int m, int n, int bits, int group,
                              size_t* codes_bytes, size_t* scale_zero_bytes,
                              size_t* gemv_workspace_bytes);

/*
 * Offline conversion: quantize W group by group and write it in zigzag order
 * (paper Sec. 3.2, Sec. 4.1.2; run once per model, Sec. 5).
 * Per block: zero = min of the G weights; scale = fp16((max - zero) / (2^b - 1)),
 * the subtraction and division each one IEEE fp32 operation; code_i =
 * clamp(rint((w_i - zero) / scale), 0, 2^b - 1) with ties to even, all zero when
 * scale == 0.  A minimum or maximum that is zero counts as +0.0 whatever the
 * signs of the zeros in the group.  Results are bit-reproducible.
 *   W          : fp16, row-major [m][ldw], ldw >= n, 2-byte aligned.
 *   codes      : R*n*B bytes, 16-byte aligned.
 *   scale_zero : 2*R*n fp16, 16-byte aligned.
 */
spqt_status spqt_pack(const void* W, int m, int n, int ldw, int bits, int group,
                      void* codes, void* scale_zero, void* stream);

/*
 * Inverse of the layout step of spqt_pack (a checking aid for the layout of
 * paper Sec. 4.1.2): natural-order codes, one byte each, q_u8[j*n + k] = code
 * of row j, column k.
 */
spqt_status spqt_unpack(const void* codes, int m, int n, int bits, int group,
                        void* q_u8, void* stream);

/*
 * Sparse index collection (paper Sec. 4.2.3, the index-collecting kernel):
 * idx[0:*count] = every k with |x_k| > t, in ascending order; *count = how many.
 * The comparison is strict and exact (fp16 widened); NaN entries are never
 * active.  idx must hold n entries.  x: fp16[n], 2-byte aligned.  idx, count:
 * int32, 4-byte aligned.  n == 0 is allowed and writes *count = 0.
 */
spqt_status spqt_sparsify(const void* x, int n, float t,
                          int32_t* idx, int32_t* count, void* stream);

/*
 * Load-balanced sparse GEMV over the zigzag layout (paper Sec. 4.2.2 and 4.2.3):
 *   y[j] = sum_{i < *count} What[j][idx[i]] * x[idx[i]],  j in [0,m), y fp16.
 * For every block-row the index list -- not the matrix columns -- is split
 * evenly over the workers of that block-row; partial sums are accumulated in
 * fp32 and combined in a fixed order, so a call is bit-reproducible.  idx may be
 * in any order.  *count == 0 gives y = 0.
 *   codes, scale_zero : as written by spqt_pack, 16-byte aligned.
 *   x : fp16[n], 2-byte aligned.  idx : int32[>= *count].  count : int32 on the device.
 *   y : fp16[m], 2-byte aligned.
 *   workspace : gemv_workspace_bytes of device memory, 16-byte aligned, zeroed
 *       ONCE by the caller before its first use; every call leaves it ready for
 *       the next.  Two calls that may overlap on the GPU need two workspaces.
 * Supported: bits 4 or 3 with group 64 or 128; n <= 65535 (column numbers travel as 16 bits).
 */
spqt_status spqt_sparse_gemv(const void* codes, const void* scale_zero,
                             int m, int n, int bits, int group,
                             const void* x, const int32_t* idx, const int32_t* count,
                             void* y, void* workspace, size_t workspace_bytes, void* stream);

/*
 * spqt_sparsify followed by spqt_sparse_gemv in ONE launch (the paper runs the index collection as
 * a kernel of its own before every GEMV, Sec. 4.2.3; on this GPU a separate launch plus the
 * count -> idx -> blocks chain of dependent reads costs more than a small GEMV itself).  Results
 * are identical to the two calls: idx[0:*count] ascending, *count, and the same y bits.  idx (n
 * entries) and count are written; the other arguments are those of spqt_sparse_gemv.  When x is too
 * long for the in-kernel scan (n above about 30000) the two kernels are launched one after the
 * other instead.
 */
spqt_status spqt_sparsify_gemv(const void* codes, const void* scale_zero,
                               int m, int n, int bits, int group,
                               const void* x, float t, int32_t* idx, int32_t* count,
                               void* y, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same kernel over all n columns with no index list: the dense GEMV on the
 * zigzag layout (paper Sec. 4.2.2), the sparsity-free comparison.  Any n when n is a multiple of 8
 * and x is 16-byte aligned (whole chunks of a block-row are then fetched by bulk copies); otherwise
 * n <= 65535.
 */
spqt_status spqt_dense_gemv(const void* codes, const void* scale_zero,
                            int m, int n, int bits, int group, const void* x,
                            void* y, void* workspace, size_t workspace_bytes, void* stream);

/*
 * spqt_sparse_gemv for callers that cannot give it a workspace.  (The paper has no counterpart:
 * this is a packaging of the call above, same arithmetic, same result bits.)
 *
 * Some hosts of this library may not obtain device memory themselves: a custom operator running
 * inside a framework whose allocator owns the whole device, or a serving loop that has frozen its
 * memory map after start-up and will not tolerate the device-wide stall of a cudaMalloc.  For them
 * the workspace is a 1 MiB array compiled into the library (static __device__ storage: every GPU
 * that loads the library carries it until the process exits).  The call allocates nothing and
 * frees nothing; inputs and outputs are still the caller's.
 *
 *   - Problems whose workspace (spqt_packed_sizes: gemv_workspace_bytes) exceeds 1 MiB are refused
 *     with SPQT_ERR_WORKSPACE; every Llama-shaped layer used in this repository fits.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and keeps it; make that first call before any stream capture begins, and
 *     from one host thread (the look-up is not guarded against two threads making it at once).
 *   - All calls on a device share the one array, which still holds the previous call's contents; the
 *     part that must start at zero (arrival counters, status word, the tagged words that carry partial
 *     sums between thread blocks: up to about 0.9 MiB) is cleared on `stream` before the kernel, after
 *     every argument check has passed.  Two calls that may overlap on the GPU (different streams, no
 *     ordering) race on it: order them, or use spqt_sparse_gemv with separate workspaces.
 *   - Because the status word is cleared per call, it describes the last call only: read it with
 *     spqt_static_status after that call.
 * Other arguments, alignment rules and error codes are those of spqt_sparse_gemv.
 */
spqt_status spqt_sparse_gemv_static(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x, const int32_t* idx, const int32_t* count,
                                    void* y, void* stream);

/*
 * Status word of the built-in scratch after the last spqt_sparse_gemv_static call on this device
 * and stream (same meaning and return value as spqt_workspace_status; waits for the stream).
 * m and group are those of that call.
 */
spqt_status spqt_static_status(int m, int group, int* status_host, void* stream);

/*
 * One decode-time linear layer from HOST activations (paper Sec. 3.2: hidden
 * state -> index collection with the layer's threshold -> sparse GEMV):
 * copies x_host (fp16[n]) to x_dev, runs spqt_sparsify_gemv (same results as
 * spqt_sparsify followed by spqt_sparse_gemv), copies y (fp16[m]) to y_host and
 * waits for the stream.  x_host / y_host
 * should be pinned (then a one-CTA kernel fetches x over the bus instead of the copy
 * engine, whose start-up latency is several times the transfer of a few KB, and the
 * GEMV kernel writes y straight into y_host: no copy back); x_dev (fp16[n]), idx_dev
 * (int32[n]), count_dev (int32[1]) and y_dev (fp16[m]) are caller-provided
 * device staging buffers.  This entry point synchronises.
 */
spqt_status spqt_sparse_linear_host(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x_host, float t, void* y_host,
                                    void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same without the wait at the end: everything is enqueued on `stream` and the call returns; y_host
 * is valid once the caller has synchronised the stream (several linears of a token step can be enqueued
 * one after the other, each with its own staging buffers and workspace, and waited for once).  x_host
 * must stay unchanged until then; pageable x_host / y_host make the copies synchronous, not wrong.
 */
spqt_status spqt_sparse_linear_host_async(const void* codes, const void* scale_zero,
                                          int m, int n, int bits, int group,
                                          const void* x_host, float t, void* y_host,
                                          void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * A token step recorded once and replayed: the host-buffer linears of a step (each described like the
 * arguments of spqt_sparse_linear_host_async: same meaning and alignment of every field) are captured,
 * in order, into one CUDA graph -- the transfer of every x from its x_host (all of them at the head of the
 * step), per linear the launch that collects the indices and multiplies, and the way y reaches y_host -- so
 * that a step costs the host one launch call.
 *   spqt_host_step_create  : builds the graph (allocates host-side CUDA objects; not a hot-path call;
 *                            nothing runs on the device).  The pointers, shapes and thresholds are fixed
 *                            from here on; the CONTENTS of the x_host buffers are read at every launch.
 *                            The linears must not share staging buffers or workspaces; x_host and y_host
 *                            must be pinned memory (a copy from pageable memory cannot be recorded:
 *                            SPQT_ERR_CUDA).  Returns a handle
 *                            in *step; SPQT_ERR_CUDA if the capture fails, the failing linear's status if
 *                            one of them is refused.
 *   spqt_host_step_launch  : enqueues one replay on `stream`; asynchronous; the y_host buffers are valid
 *                            once the caller has synchronised the stream.  One replay at a time per handle.
 *   spqt_host_step_destroy : frees the handle (after its last replay has finished).
 * Not thread-safe per handle.  No counterpart in the paper (its linears live inside llama.cpp's graph).
 */
typedef struct {
    const void* codes;
    const void* scale_zero;
    int m, n, bits, group;
    const void* x_host;
    float t;
    void* y_host;
    void* x_dev;
    int32_t* idx_dev;
    int32_t* count_dev;
    void* y_dev;
    void* workspace;
    size_t workspace_bytes;
} spqt_host_linear;

spqt_status spqt_host_step_create(const spqt_host_linear* linears, int count, void** step);
spqt_status spqt_host_step_launch(void* step, void* stream);
spqt_status spqt_host_step_destroy(void* step);

/*
 * Tuning aid: number of CTAs of the GEMV grid (0 restores the built-in rule, one
 * persistent CTA per SM; values above 512 are clamped).  `no_overlap` is a set of bits, 0 by
 * default: bit 0 launches the GEMV kernels strictly stream-ordered instead of letting a GEMV start
 * (and wait inside the kernel) while the previous kernel of the stream drains; bit 1 never launches
 * thread-block clusters (otherwise, in spqt_sparse_gemv and spqt_dense_gemv, the 2..8 CTAs that share a
 * block-row combine their sums through shared memory when the device can hold all the clusters at once); bit 2 is an ablation, the paper's
 * "sparse without load balancing" (Sec. 6): spqt_sparsify_gemv then gives every CTA, and inside it every
 * warp, a fixed range of the matrix columns of its block-row instead of an even share of the active
 * list (same results up to the order of partial sums; lists longer than the shared-memory window and
 * CTAs with more than 8 block-rows keep the balanced partition).
 * Any value gives the same results up to the order of partial sums.
 * Process-wide, not thread-safe.
 */
spqt_status spqt_set_tuning(int gemv_ctas, int no_overlap);

/*
 * Small batch: B = 1..8 decode rows at once (paper Sec. 3.3 and Sec. 4.1.3 expect beam search with
 * small beams on the same layout; Sec. 5: with more than one token the system dispatches dense kernels).
 * The sparse call multiplies every row over the UNION of the rows' active sets:
 *   idx[0:*count] = every k with |X[b][k]| > t for at least one row b, ascending;
 *   Y[b][j] = sum_{i < *count} What[j][idx[i]] * X[b][idx[i]]   for every row b
 * (a row's entries at or below the threshold in columns of the union are used with their values: the
 * block is read for the batch anyway, so this is never less accurate than thresholding row by row).
 * Every active block is fetched once for the whole batch.  The dense call is the same over all n
 * columns.  Dispatch rule: with one row use spqt_sparsify_gemv; with 2..8 rows the sparse call here
 * as long as the union keeps some sparsity (the union of B sets that are each 50 % sparse is
 * 1 - 2^-B dense), the dense call otherwise and for prompts; rows beyond 8 in further calls.
 *   X : fp16 [batch][ldx], ldx >= n, 2-byte aligned.   Y : fp16 [batch][ldy], ldy >= m.
 *   idx : int32[n], count : int32, both on the device, written by the sparse call.
 *   workspace : spqt_gemm_small_workspace bytes, 16-byte aligned, zeroed ONCE by the caller; every call
 *       leaves it ready for the next.  Sums are added in a fixed order: calls are bit-reproducible.
 * Batches of 5..8 rows run as two passes of four rows over the same list.  Two launches (three for
 * more than four rows) per sparse call; asynchronous on `stream`.  The sparse call needs n <= 65535
 * (SPQT_ERR_UNSUPPORTED beyond).
 */
spqt_status spqt_gemm_small_workspace(int m, int n, int bits, int group, size_t* workspace_bytes);
spqt_status spqt_sparse_gemm_small(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                   const void* X, int ldx, int batch, float t, int32_t* idx, int32_t* count,
                                   void* Y, int ldy, void* workspace, size_t workspace_bytes, void* stream);
spqt_status spqt_dense_gemm_small(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                                  const void* X, int ldx, int batch, void* Y, int ldy,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Comparison baseline, not part of the method: the conventional ROW-WISE grouping the paper contrasts
 * its layout with (paper Sec. 2 and Sec. 4.1.1: groups of consecutive weights of one row suit a
 * row-parallel GEMV but conflict with column sparsity; Sec. 6 compares the dense kernel over the zigzag
 * layout with the stock row-wise one on 15 shapes).  Same quantizer as spqt_pack, 4-bit only:
 *   block (j, g) = the codes of columns g*group .. g*group+group-1 of row j, at byte
 *                  (j*(n/group) + g) * group/2; byte i of a block = code i | code (i + group/2) << 4;
 *   scale_zero   = fp16 pairs (scale, zero) in the same block order.
 * n must be a multiple of group (SPQT_ERR_UNSUPPORTED otherwise; any m >= 1); bits must be 4.
 *   spqt_rowwise_packed_sizes : bytes of codes (m*n/2) and of scale_zero (4*m*n/group); host only.
 *   spqt_rowwise_pack         : W fp16 row-major [m][ldw >= n] (2-byte aligned) -> codes, scale_zero
 *                               (both 16-byte aligned, caller-allocated).
 *   spqt_rowwise_dense_gemv   : y[j] = sum_k What[j][k] * x[k] over all n columns; x fp16[n], y fp16[m]
 *                               (2-byte aligned); n <= 16384 (SPQT_ERR_UNSUPPORTED beyond: a row must fit
 *                               the 16 warps of a CTA).  Needs no workspace: every row is summed inside one
 *                               CTA, in a fixed order (bit-reproducible).
 * All device pointers; asynchronous on `stream`; nothing is allocated or retained.
 */
spqt_status spqt_rowwise_packed_sizes(int m, int n, int bits, int group,
                                      size_t* codes_bytes, size_t* scale_zero_bytes);
spqt_status spqt_rowwise_pack(const void* W, int m, int n, int ldw, int bits, int group,
                              void* codes, void* scale_zero, void* stream);
spqt_status spqt_rowwise_dense_gemv(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x, void* y, void* stream);
/*
 * The same product with the entries at or below the threshold treated as zero (|x[k]| > t is active, as in
 * spqt_sparsify; NaN is never active): what activation sparsity can do on the row-wise layout, where a
 * sparse column is scattered over a group of every row (paper Sec. 2, Sec. 4.1.1) -- no block can be
 * skipped, every byte is still read, only the contributions vanish.  Same arguments and limits.
 */
spqt_status spqt_rowwise_thresholded_gemv(const void* codes, const void* scale_zero,
                                          int m, int n, int bits, int group,
                                          const void* x, float t, void* y, void* stream);

/*
 * The two-level format the paper's implementation builds on (paper Sec. 2: superblocks of 256 weights
 * split into eight blocks of 32, 4-bit codes, a 6-bit scale and a 6-bit minimum per block, a 16-bit scale
 * and minimum per superblock), in the zigzag arrangement of Sec. 4.1.2: a superblock is 256 consecutive
 * ROWS of one column; superblock (r, k) is record r*n + k.  A record is 144 bytes:
 *   bytes 0..127   codes, byte i = q_i | q_{i+128} << 4            (rows r*256 + i and r*256 + 128 + i)
 *   bytes 128..139 the sixteen 6-bit fields sc_0..sc_7, m_0..m_7 as a little-endian bit string
 *                  (field f at bits 6f..6f+5)
 *   bytes 140..143 d, dmin: fp16, little-endian
 * and row j of block i (rows 32i..32i+31 of the superblock) dequantizes to  d*sc_i*q_j - dmin*m_i.
 * The paper states neither the rounding rule nor the bit arrangement; the rule implemented (every step
 * one IEEE fp32 operation, rint = round to nearest even, zeros of either sign count as +0.0):
 *   lo_i = min(min_j w_j, 0), step_i = (max_j w_j - lo_i)/15, neg_i = 0 - lo_i;
 *   d = fp16(max_i step_i/63), dmin = fp16(max_i neg_i/63);
 *   sc_i = min(rint(step_i/d), 63), m_i = min(rint(neg_i/dmin), 63)   (0 when the divisor is 0);
 *   q_j = clamp(rint((w_j + dmin*m_i)/(d*sc_i)), 0, 15)                 (0 when d*sc_i is 0).
 * m must be a multiple of 256 (SPQT_ERR_UNSUPPORTED otherwise); any n >= 1.
 *   spqt_kq_packed_sizes : bytes of the records (144*n*m/256) and of the GEMV workspace; host only.
 *   spqt_kq_pack         : W fp16 row-major [m][ldw >= n] (2-byte aligned) -> records (16-byte aligned).
 *   spqt_kq_sparse_gemv  : y[j] = sum_{i < *count} What[j][idx[i]] * x[idx[i]]; idx, count as written by
 *                          spqt_sparsify (any order of distinct in-range columns; trusted); x fp16[n],
 *                          y fp16[m] (2-byte aligned).
 *   spqt_kq_dense_gemv   : the same over all n columns.
 *   workspace : workspace_bytes of device memory, 16-byte aligned, zeroed ONCE by the caller; every call
 *               leaves it ready for the next (SPQT_ERR_WORKSPACE if too small).  Sums are added in a fixed
 *               order: calls are bit-reproducible.
 * All device pointers; asynchronous on `stream`; nothing is allocated or retained.
 */
spqt_status spqt_kq_packed_sizes(int m, int n, size_t* records_bytes, size_t* workspace_bytes);
spqt_status spqt_kq_pack(const void* W, int m, int n, int ldw, void* records, void* stream);
spqt_status spqt_kq_sparse_gemv(const void* records, int m, int n, const void* x,
                                const int32_t* idx, const int32_t* count, void* y,
                                void* workspace, size_t workspace_bytes, void* stream);
spqt_status spqt_kq_dense_gemv(const void* records, int m, int n, const void* x, void* y,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same format with other code widths (paper Sec. 4.1.3: the grouping works for any code width from
 * 2 to 8 bits).  bits = 2, 4, 5, 6 or 8 (SPQT_ERR_UNSUPPORTED otherwise); bits = 4 is exactly the format
 * above.  2^bits - 1 takes the place of 15 in the rule, and only the code bytes of a record change:
 *   bits = 8 : bytes 0..255, byte i = q_i; record of 272 bytes (fields at 256, d and dmin at 268)
 *   bits = 2 : bytes 0..63,  byte i = q_i | q_{i+64} << 2 | q_{i+128} << 4 | q_{i+192} << 6;
 *              record of 80 bytes (fields at 64, d and dmin at 76)
 *   bits = 5 : bytes 0..127 the low four bits, byte i = (q_i & 15) | (q_{i+128} & 15) << 4; bytes 128..159
 *              the fifth bit of every row, bit j%8 of byte 128 + j/8; record of 176 bytes
 *   bits = 6 : bytes 0..127 as for 5; bytes 128..191 the high two bits h = q >> 4, byte 128 + i =
 *              h_i | h_{i+64} << 2 | h_{i+128} << 4 | h_{i+192} << 6; record of 208 bytes
 * (the fields follow the code bytes, then d and dmin).
 * Arguments, workspace, alignment and error behaviour as for the spqt_kq_* calls; the workspace does not
 * depend on the width.
 */
spqt_status spqt_kqw_packed_sizes(int m, int n, int bits, size_t* records_bytes, size_t* workspace_bytes);
spqt_status spqt_kqw_pack(const void* W, int m, int n, int ldw, int bits, void* records, void* stream);
spqt_status spqt_kqw_sparse_gemv(const void* records, int m, int n, int bits, const void* x,
                                 const int32_t* idx, const int32_t* count, void* y,
                                 void* workspace, size_t workspace_bytes, void* stream);
spqt_status spqt_kqw_dense_gemv(const void* records, int m, int n, int bits, const void* x, void* y,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Threshold calibration (paper Sec. 5, the calibration threshold tool; Sec. 3.2: thresholds are
 * computed once per sparsity level from calibration activations).  *threshold (a device float) =
 * the nearest-rank order statistic of |x| over the pool x[0:count] of fp16 calibration activations:
 * the ceil(sparsity * N)-th smallest magnitude (1-based; N = the entries that are not NaN), so that at
 * least that fraction of the pool is inactive under "active <=> |x| > threshold".  sparsity <= 0, or an
 * empty pool, gives -1 (nothing dropped).  Exact: a histogram over the 2^15 fp16 magnitudes.
 *   x : fp16[count], 2-byte aligned; the activations of one site (or of all the matrices that share an
 *       input), over as many calibration tokens as wanted, concatenated.
 *   workspace : 131072 bytes, 4-byte aligned, zeroed ONCE by the caller; every call leaves it zeroed.
 * The two modes of the paper's tool sit on top of this call in paper_2511_04477_b200/calibrate.py:
 * one global sparsity for every site, or per-matrix sparsities averaged over the matrices that share an
 * input ({q,k,v}, {gate,up}) so that they share one threshold and one index collection.
 */
spqt_status spqt_calibrate_threshold(const void* x, size_t count, double sparsity, float* threshold,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Per-shape profiling (paper Sec. 3.2: GEMV shapes are profiled per platform to pick the kernel's
 * hyper-parameters; Sec. 6, hyper-parameter study).  Times the call that collects the indices and
 * multiplies (spqt_sparsify_gemv with threshold t on x) and the dense call on this problem for a set
 * of grid sizes -- one CTA per SM, and every whole number 1..8 of CTAs per block-row that fits the
 * device -- and remembers the fastest of each for this (m, n, bits, group): later calls of
 * spqt_sparsify_gemv / spqt_sparse_gemv and of spqt_dense_gemv with the same shape use them
 * (spqt_set_tuning with a non-zero grid size still overrides).  Results of those calls do not change
 * beyond the order of partial sums.  Arguments are those of spqt_sparsify_gemv; idx, count and y are
 * overwritten.  If `flush` is not NULL its flush_bytes bytes are rewritten before every timed launch, so
 * that a buffer larger than L2 makes the weights come from HBM as in steady-state decoding.
 * ctas_sparse / ctas_dense (host, may be NULL) receive the choices.  Synchronises the stream many
 * times; call it once per shape at start-up, outside any stream capture.  The table holds 256 shapes,
 * is process-wide and not thread-safe.
 */
spqt_status spqt_autotune(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                          const void* x, float t, int32_t* idx, int32_t* count, void* y,
                          void* workspace, size_t workspace_bytes, void* flush, size_t flush_bytes,
                          int* ctas_sparse, int* ctas_dense, void* stream);

/*
 * Checked mode (off by default; paper Sec. 4.2.3 assumes a well-formed index list and so does the
 * normal path).  With on != 0, spqt_sparse_gemv and spqt_sparse_gemv_static first check the list on
 * the device: *count in [0, n], every index in [0, n), and, for n <= 1048576, no index twice.  A bad
 * list sets the workspace's status word to 2 and the product is computed with a count of 0 (y = 0)
 * instead of reading wherever the indices point.  The verdict is per call: a later call with a good
 * list on the same workspace computes its product normally, although the status word stays set until
 * the caller zeroes the workspace.  Costs two small extra launches per call; the check keeps its
 * state per device, so checked calls on one device must not overlap.  Process-wide, not thread-safe.
 */
spqt_status spqt_set_debug(int on);

/*
 * Reads the workspace's status word into *status_host (a host int) and waits for
 * the stream: 0 = every GEMV that used this workspace ran to completion;
 * 1 = a bounded wait expired inside a GEMV kernel (which then returned early,
 * leaving y unspecified); 2 = checked mode found a bad index list.  The word is
 * sticky until the caller zeroes the workspace again.  Returns SPQT_OK for 0,
 * SPQT_ERR_TIMEOUT for 1 and SPQT_ERR_INVALID_ARG for 2 (after writing *status_host).
 */
spqt_status spqt_workspace_status(const void* workspace, int m, int group, int* status_host, void* stream);

/*
 * Measurement aid, not part of the method (the paper has no counterpart): reads `bytes` of device
 * memory at `buf` (128-byte aligned) into shared memory in 64-byte blocks with the copy instruction
 * the GEMV uses, and adds the number of bytes it fetched to *moved (a device counter the caller
 * zeroes).  pattern 0: every block (the achievable read rate); pattern 1: one randomly chosen half
 * of every 128-byte line (the gather a sparse GEMV performs at 50 % block density).  Time it with
 * events on `stream`; the buffer should be much larger than L2.
 */
spqt_status spqt_probe_read(const void* buf, size_t bytes, int pattern,
                            unsigned long long* moved, void* stream);

/*
 * Measurement aid, not part of the method: the dequantize-FMA arithmetic of the GEMV loop alone.  One
 * CTA of 16 warps per SM; every warp runs `chunks_per_warp` (>= 1) full 2 KB chunks of 4-bit codes with
 * groups of 128 rows (eight 512-byte steps each) on operands that already sit in shared memory: no
 * copies, no list handling, no reduction.  `sink` (device, sink_floats >= 512 per SM or
 * SPQT_ERR_INVALID_ARG; written so that the arithmetic is kept) receives meaningless sums; *chunks_total (host) receives the number of chunks
 * the launch processes.  Time it with events on `stream`: chunks per second times the bytes a chunk
 * stands for (2176 with its metadata) is the bandwidth at which instruction issue alone saturates.
 */
spqt_status spqt_probe_arith(int chunks_per_warp, float* sink, size_t sink_floats,
                             unsigned long long* chunks_total, void* stream);

/* Number of kernels the library has launched in this process (a counter for
 * benchmarks; not synchronised with the device). */
unsigned long long spqt_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPQT_H */
