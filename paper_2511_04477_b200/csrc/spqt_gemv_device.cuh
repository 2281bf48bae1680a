// Device-side building blocks of the GEMV kernel: PTX wrappers (mbarriers with bounded waits,
// cp.async, tagged 64-bit words, shared-memory accesses by 32-bit address, thread-block-cluster
// primitives, predicated stores) and the packed-FMA dequantization arithmetic.  Included by
// spqt_gemv.cu only, after its compile-time constants.
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
__device__ __forceinline__ void sts_u32(unsigned addr, unsigned v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
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
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
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

// acc (32 fp32 sums in 16 registers) += the 32 codes of a lane's 16 bytes, each times a (scaled by 2^-56).
__device__ __forceinline__ void fma_block16(unsigned long long* acc, const uint4& w, float a)
{
    const unsigned long long aa = pack2(a, a);
    const unsigned long long m01 = fmul2(aa, pack2(0x1p93f, 0x1p89f)), m23 = fmul2(aa, pack2(0x1p85f, 0x1p81f));
    fma_word(acc + 0, w.x, m01, m23);
    fma_word(acc + 4, w.y, m01, m23);
    fma_word(acc + 8, w.z, m01, m23);
    fma_word(acc + 12, w.w, m01, m23);
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

}  // namespace spqt
