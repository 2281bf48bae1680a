// Device-side building blocks of the GEMV kernel: PTX wrappers (mbarriers with bounded waits,
// cp.async, bulk copies, tagged 64-bit words, shared-memory accesses by 32-bit address,
// thread-block-cluster primitives, predicated stores) and the packed-FMA dequantization arithmetic.
// Included by spqt_gemv.cu only, after its compile-time constants.
#pragma once

namespace spqt {

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

// One non-blocking look at the phase with the given parity.
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

// Bounded wait for the phase with the given parity; false when the bound
// (wall time, so that a logic error can never hold the GPU) expires.  One try_wait
// blocks for up to about 4 us on this GPU (with or without the time hint), re-testing
// the barrier about every 60 ns while it does, a dozen instructions each time: far
// fewer than a software spin on test_wait, but not nothing -- which is why the long
// wait of the writer warps is a hardware barrier instead (handover_wait below).
constexpr unsigned kSuspendNs = 100000u;  // the time hint of one try_wait
__device__ __forceinline__ bool mbar_wait_addr(unsigned addr, unsigned parity)
{
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kSuspendNs)
            : "memory");
        if (done) return true;
        if (it == 0) t0 = global_ns();
        else if (global_ns() - t0 > kWaitNs) return false;
    }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) { return mbar_wait_addr(smem_u32(bar), parity); }

// Bulk copies (the dense path: whole chunks of a block-row are contiguous).  The copy completes on
// the mbarrier by the number of bytes it moved; one thread first announces the total with expect_tx.
// Source, destination and size are multiples of 16 bytes.  This GPU's own memory only, no multicast.
__device__ __forceinline__ void mbar_expect_tx(unsigned bar_addr, unsigned bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar_addr), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_copy(unsigned smem_dst, const void* gmem_src, unsigned bytes, unsigned bar_addr)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
                 "l"(gmem_src), "r"(bytes), "r"(bar_addr)
                 : "memory");
}
// the same under a predicate (no branch: one lane of a warp issues for all)
__device__ __forceinline__ void mbar_expect_tx_if(unsigned cond, unsigned bar_addr, unsigned bytes)
{
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 st;\n\tsetp.ne.u32 p, %0, 0;\n\t"
                 "@p mbarrier.arrive.expect_tx.shared::cta.b64 st, [%1], %2;\n\t}" ::"r"(cond), "r"(bar_addr), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_copy_if(unsigned cond, unsigned smem_dst, const void* gmem_src, unsigned bytes,
                                             unsigned bar_addr)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t"
                 "@p cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%1], [%2], %3, [%4];\n\t}" ::"r"(cond),
                 "r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar_addr)
                 : "memory");
}
// barrier among the worker warps only (id 1); every worker warp must reach it
__device__ __forceinline__ void worker_barrier(int threads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
}

// Hand-over of a finished segment from the worker warps to its writer warp (hardware barriers 2 and
// 3, one per hand-over buffer): the workers arrive without waiting, the writer waits.  A warp waiting
// at a hardware barrier issues nothing, whereas a warp in mbarrier.try_wait re-tests the barrier
// about every 60 ns (a dozen instructions each time, measured from the instruction mix) on the
// scheduler it shares with four worker warps.  Like __syncthreads it cannot time out: every worker warp
// passes every segment end, whatever its bounded waits returned.
// (threads = all worker threads plus the writer's 32)
__device__ __forceinline__ void handover_arrive(int b, int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(2 + b), "r"(threads) : "memory");
}
__device__ __forceinline__ void handover_wait(int b, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(2 + b), "r"(threads) : "memory");
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
// A partial sum travels between CTAs as one 64-bit word: the fp32 value in the low half, a non-zero
// tag in the high half.  One aligned 64-bit access is indivisible, so a reader that sees the tag has
// the value: no fence is needed between the two.
constexpr unsigned long long kTagBit = 1ull << 32;
__device__ __forceinline__ unsigned long long ld_word(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_word(unsigned long long* p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.b64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// shared-memory accesses by 32-bit shared address
__device__ __forceinline__ unsigned lds_u32(unsigned addr)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds_u16(unsigned addr)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds_v4(unsigned addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint2 lds_v2(unsigned addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u32(unsigned addr, unsigned v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts_v4(unsigned addr, const uint4& v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// two packed multiplier pairs (four fp32 values) of one list entry
__device__ __forceinline__ void lds_pairs(unsigned addr, unsigned long long& a, unsigned long long& b)
{
    asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr) : "memory");
}
__device__ __forceinline__ void sts_pairs(unsigned addr, unsigned long long a, unsigned long long b)
{
    asm volatile("st.shared.v2.u64 [%0], {%1, %2};" ::"r"(addr), "l"(a), "l"(b) : "memory");
}
__device__ __forceinline__ void st_shared_u32_if(unsigned cond, unsigned smem_dst, unsigned v)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p st.shared.u32 [%1], %2;\n\t}" ::"r"(cond), "r"(smem_dst), "r"(v) : "memory");
}

// ---- thread-block clusters: the CTAs of one block-row hand their sums to CTA rank 0 through its
// shared memory
__device__ __forceinline__ void cluster_arrive()
{
    // relaxed: the only thing the other CTAs must see, the barrier initialisation, has its own fence
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait()
{
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in the CTA of the given rank
__device__ __forceinline__ unsigned cluster_map(unsigned smem_addr, unsigned rank)
{
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(unsigned addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(unsigned remote_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
// Bounded wait with cluster-scope acquire (the data were written by other CTAs of the cluster).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, unsigned parity)
{
    const unsigned addr = smem_u32(bar);
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(kSuspendNs)
            : "memory");
        if (done) return true;
        if (it == 0) t0 = global_ns();
        else if (global_ns() - t0 > kWaitNs) return false;
    }
}

// stores under a predicate (never a branch)
__device__ __forceinline__ void st_shared_u16_if(unsigned cond, unsigned smem_dst, int v)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p st.shared.u16 [%1], %2;\n\t}" ::"r"(cond), "r"(smem_dst), "h"((unsigned short)v) : "memory");
}
__device__ __forceinline__ void st_global_if(unsigned cond, int* dst, int v)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p st.global.u32 [%1], %2;\n\t}" ::"r"(cond), "l"(dst), "r"(v) : "memory");
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
// times a*2^-56.  Codes 0..3 are masked in place, codes 4..7 after a shift by 16, so that both
// halves use the same two multiplier pairs m01 = a*(2^93, 2^89) and m23 = a*(2^85, 2^81).
__device__ __forceinline__ void fma_word(unsigned long long* acc, unsigned w, unsigned long long m01,
                                         unsigned long long m23)
{
    const unsigned v = w >> 16;
    ffma2(acc[0], pack2(__uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000f0u)), m01);
    ffma2(acc[1], pack2(__uint_as_float(w & 0x00000f00u), __uint_as_float(w & 0x0000f000u)), m23);
    ffma2(acc[2], pack2(__uint_as_float(v & 0x0000000fu), __uint_as_float(v & 0x000000f0u)), m01);
    ffma2(acc[3], pack2(__uint_as_float(v & 0x00000f00u), __uint_as_float(v & 0x0000f000u)), m23);
}

// d = a * b on both lanes
__device__ __forceinline__ unsigned long long fmul2(unsigned long long a, unsigned long long b)
{
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// acc (16 fp32 sums in 8 registers) += the 16 codes of a lane's 8 bytes, each times a (scaled by
// 2^-56), given the multiplier pairs m01 = a*(2^93, 2^89) and m23 = a*(2^85, 2^81).
__device__ __forceinline__ void fma_block8(unsigned long long* acc, const uint2& w, unsigned long long m01,
                                           unsigned long long m23)
{
    fma_word(acc + 0, w.x, m01, m23);
    fma_word(acc + 4, w.y, m01, m23);
}

// 3-bit codes: w2 is a word of the 2-bit plane (byte i, field v = bits 2v..2v+1), w1 the matching word
// of the 1-bit plane, already shifted so that bit 2v of byte i is the top bit of the code in field v.
// The fields are first widened to two words of eight 4-bit codes (fields v = {0,2}, then {1,3}; low
// nibble first), then treated like 4-bit codes.
__device__ __forceinline__ void fma_block3(unsigned long long* acc, unsigned w2, unsigned w1, unsigned long long m01,
                                           unsigned long long m23)
{
    const unsigned c0 = (w2 & 0x33333333u) | ((w1 << 2) & 0x44444444u);
    const unsigned c1 = ((w2 >> 2) & 0x33333333u) | (w1 & 0x44444444u);
    fma_block8(acc, make_uint2(c0, c1), m01, m23);
}

// The cumulative form of the same arithmetic, for blocks whose codes all share one multiplier a
// (mm = (a, a) * 2^93).  Instead of the four codes q0..q3 of a 16-bit half-word, the four sums
// u_j = q0 + 16 q1 + ... + 16^j q_j (the half-word masked to its low 4(j+1) bits, a subnormal like the
// single codes) are accumulated: the top one needs no mask, so a word costs seven masks and a shift
// instead of eight and a shift, and one multiplier pair instead of two.  The sums are linear in the
// codes, so the sum over the list of a*q_j is recovered once per segment as (U_j - U_{j-1}) / 16^j;
// every U_j is dominated by its own top code, which keeps the rounding error of that difference at
// the level of a direct sum (a factor 1 + 1/16 + ... above it at most).
__device__ __forceinline__ void fma_word_cum(unsigned long long* acc, unsigned w, unsigned long long mm)
{
    const unsigned v = w >> 16;
    ffma2(acc[0], pack2(__uint_as_float(w & 0x0000000fu), __uint_as_float(w & 0x000000ffu)), mm);
    ffma2(acc[1], pack2(__uint_as_float(w & 0x00000fffu), __uint_as_float(w & 0x0000ffffu)), mm);
    ffma2(acc[2], pack2(__uint_as_float(v & 0x0000000fu), __uint_as_float(v & 0x000000ffu)), mm);
    ffma2(acc[3], pack2(__uint_as_float(v & 0x00000fffu), __uint_as_float(v)), mm);
}
__device__ __forceinline__ void fma_block8_cum(unsigned long long* acc, const uint2& w, unsigned long long mm)
{
    fma_word_cum(acc + 0, w.x, mm);
    fma_word_cum(acc + 4, w.y, mm);
}
__device__ __forceinline__ void fma_block3_cum(unsigned long long* acc, unsigned w2, unsigned w1, unsigned long long mm)
{
    const unsigned c0 = (w2 & 0x33333333u) | ((w1 << 2) & 0x44444444u);
    const unsigned c1 = ((w2 >> 2) & 0x33333333u) | (w1 & 0x44444444u);
    fma_block8_cum(acc, make_uint2(c0, c1), mm);
}
// u[0..3] = the four cumulative sums of one half-word -> the four code sums, each still times 2^-56
__device__ __forceinline__ void uncumulate(float* u)
{
    const float s1 = (u[1] - u[0]) * 0x1p-4f, s2 = (u[2] - u[1]) * 0x1p-8f, s3 = (u[3] - u[2]) * 0x1p-12f;
    u[1] = s1;
    u[2] = s2;
    u[3] = s3;
}
__device__ __forceinline__ unsigned long long lds_u64(unsigned addr)
{
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u64(unsigned addr, unsigned long long v)
{
    asm volatile("st.shared.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
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

}  // namespace spqt
