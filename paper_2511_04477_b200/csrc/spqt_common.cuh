// Shared host-side helpers of the SpQt CUDA library (argument checks, geometry,
// device properties).  No kernel code lives here.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/spqt.h"

namespace spqt {

struct Format {
    int m, n, bits, group;
    int R;          // block-rows
    int B;          // bytes of codes per block
    size_t blocks;  // R * n
};

// Validates the format and fills the derived sizes.
inline spqt_status make_format(int m, int n, int bits, int group, Format* f)
{
    if (m <= 0 || n <= 0) return SPQT_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4) return SPQT_ERR_UNSUPPORTED;
    if (group != 64 && group != 128) return SPQT_ERR_UNSUPPORTED;
    if (m % group != 0) return SPQT_ERR_UNSUPPORTED;
    f->m = m; f->n = n; f->bits = bits; f->group = group;
    f->R = m / group;
    f->B = group * bits / 8;
    f->blocks = (size_t)f->R * (size_t)n;
    return SPQT_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Largest grid any tuning may use for a GEMV; the workspace is sized for it
// (independent of the device, so sizes can be computed without a GPU).
constexpr int kMaxCtas = 512;

// Upper bound on the number of CTAs that contribute partial sums to one block-row.
inline int max_slots(int R) { return (kMaxCtas + R - 1) / R + 1; }

// Block-rows with at most kTagSlots contributing CTAs exchange their partial sums as tagged 64-bit
// words, the others as plain fp32 values behind a fence.
constexpr int kTagSlots = 4;

// Workspace layout: [R] int32 arrival counters (kept zero between calls), one
// int32 status word (non-zero after a bounded wait expired), padded to 256 B;
// then 64-bit words [R][kTagSlots][G + 2]: per contributing CTA the G partial sums
// of the block-row, its offset-term partial and a word of padding, each an fp32
// value with a tag in the high half (all zero between calls); then, only when a
// block-row can have more than kTagSlots contributors, fp32 partials
// [R][slots][G] and offset-term partials [R][slots] (contents irrelevant between calls).
inline size_t header_bytes(int R) { return (((size_t)(R + 1) * 4 + 255) / 256) * 256; }

inline size_t tagged_bytes(const Format& f)
{
    return (size_t)f.R * kTagSlots * (size_t)(f.group + 2) * sizeof(unsigned long long);
}

inline size_t workspace_bytes(const Format& f)
{
    const int slots = max_slots(f.R);
    const size_t plain = slots > kTagSlots ? (size_t)f.R * (size_t)slots * (size_t)(f.group + 1) * sizeof(float) : 0;
    return header_bytes(f.R) + tagged_bytes(f) + plain;
}

extern int g_no_pdl;          // 1 = launch strictly stream-ordered (spqt_set_tuning)
int sm_count();               // SMs of the current device (cached per device); <= 0 on error
void count_launch(int k = 1); // bump the process-wide launch counter

// Index collection over `batch` rows of X (columns active in at least one row, ascending; n < 2^16), one launch.
spqt_status launch_sparsify_rows(const __half* X, int ldx, int batch, int n, float t, int32_t* idx, int32_t* count,
                                 cudaStream_t stream);

}  // namespace spqt
