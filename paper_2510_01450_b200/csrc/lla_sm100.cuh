// sm_100a building blocks shared by the tensor-core kernels: mbarrier, TMA, tcgen05 / TMEM wrappers.
#pragma once

#include <cuda.h>

#include "lla_common.cuh"

namespace lla {
namespace sm100 {

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-suspending probe: a dedicated issuing warp that has nothing else to do wakes faster by
// spinning on this than by letting try_wait put it to sleep.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
constexpr long long kWaitClocks = 1ll << 31;   // default cap of a bounded wait (about a second)
// Bounded wait: gives up after `cap` clock ticks or as soon as another thread flagged an abort.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long cap = kWaitClocks) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > cap) {
            *abort_flag = 1;
            return false;
        }
    }
}
// Bounded wait of the exit path: for work this thread issued itself (copies, MMAs) to finish before the
// block's shared memory and TMEM go away.  Ignores the abort flag, which is already set there.
__device__ __forceinline__ bool mbar_wait_landed(uint32_t bar, uint32_t parity, long long cap = kWaitClocks) {
    const long long t0 = clock64();
    while (!mbar_try(bar, parity))
        if (clock64() - t0 > cap) return false;
    return true;
}
// OR of a predicate over the threads of named barrier `id` (every thread gets the result)
__device__ __forceinline__ bool bar_or(int id, int threads, bool v) {
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
                 "barrier.cta.red.or.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"((uint32_t)v), "r"(id), "r"(threads) : "memory");
    return r != 0;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void named_sync_compute() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z, int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

__device__ __forceinline__ uint32_t elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P1;\n\telect.sync _|P1, 0xffffffff;\n\tselp.u32 %0, 1, 0, P1;\n\t}" : "=r"(pred));
    return pred;
}
__device__ __forceinline__ void tc_commit_el(uint32_t el, uint32_t bar) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %0, 0;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%1];\n\t}"
                 ::"r"(el), "r"(bar) : "memory");
}

// 32 consecutive TMEM columns of this thread's lane -> registers (and back)
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr) : "memory");
}
// 16 consecutive TMEM columns of this thread's lane -> registers
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(addr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t addr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// two fp32 lanes in one 64-bit register (sm_100 packed fp32 arithmetic)
__device__ __forceinline__ uint64_t pk2(float lo, float hi) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) { uint64_t r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) { uint64_t r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) { uint64_t r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) { uint64_t r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
// Split two fp32 values into bf16 hi + lo pairs without touching the conversion unit (which shares
// the transcendental pipe with exp2): hi is the value truncated to its top 16 bits, lo the
// truncated exact remainder, so hi + lo keeps 16 mantissa bits.  Returns the packed hi pair and
// writes the packed lo pair; element `a` goes to the low half-word.
__device__ __forceinline__ uint32_t split_bf16x2(float a, float b, uint32_t& lo) {
    const uint32_t ua = __float_as_uint(a), ub = __float_as_uint(b);
    const uint32_t hi = __byte_perm(ua, ub, 0x7632);
    const float ra = a - __uint_as_float(ua & 0xFFFF0000u), rb = b - __uint_as_float(ub & 0xFFFF0000u);
    lo = __byte_perm(__float_as_uint(ra), __float_as_uint(rb), 0x7632);
    return hi;
}
// 16 consecutive TMEM columns of this thread's lane <- registers
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
// {lo16: fp16(a), hi16: fp16(b)}, round to nearest, values beyond the fp16 range saturate to the largest finite one
__device__ __forceinline__ uint32_t pack_f16(float a, float b) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}
// {hi16: bf16(a), lo16: bf16(b)}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(a), "f"(b));
    return r;
}

// kind::f16 instruction descriptor: fp32 accumulator, both operands bf16 (f16 = 0) or both fp16 (f16 = 1).
// The two format fields are set alike: an MMA with an fp16 A operand and a bf16 B operand raised "illegal
// instruction" on B200.
constexpr uint32_t make_idesc(int M, int N, int a_mn, int b_mn, int f16 = 0) {
    return (1u << 4) | (f16 ? 0u : (1u << 7) | (1u << 10)) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// tcgen05.mma issue and shared-memory matrix descriptors
// ------------------------------------------------------------------------------------------------
// MMA issue.  The whole MMA warp runs these convergently and the instructions are predicated on the
// elected lane (el != 0): issuing from a divergent single-thread branch instead costs ~100 clocks
// per instruction (operands have to be moved into uniform registers one by one), three times the
// execution time of a 128x64x16 MMA.
// D[tmem] (+)= A[smem] * B[smem] over 64 elements of K (4 instructions, both operands K-major:
// +32 bytes = 2 descriptor units per step).  acc0 = 0 overwrites D with the first product.
__device__ __forceinline__ void mma_ss_k64(uint32_t el, uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u64 a1, %2, 2; add.u64 a2, %2, 4; add.u64 a3, %2, 6;\n\t"
        "add.u64 b1, %3, 2; add.u64 b2, %3, 4; add.u64 b3, %3, 6;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], %2, %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a1, b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a2, b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a3, b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// D[tmem] (+)= (U_hi + U_lo)[tmem] * B[smem] over 64 keys: per 16-key step the hi operand sits at
// a + 16*step and the lo operand 8 columns further; B is MN-major (+2048 bytes = 128 units per step).
__device__ __forceinline__ void mma_ts_hilo_k64(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a0l, a1, a1l, a2, a2l, a3, a3l;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u32 a0l, %2, 8; add.u32 a1, %2, 16; add.u32 a1l, %2, 24; add.u32 a2, %2, 32;\n\t"
        "add.u32 a2l, %2, 40; add.u32 a3, %2, 48; add.u32 a3l, %2, 56;\n\t"
        "add.u64 b1, %3, 128; add.u64 b2, %3, 256; add.u64 b3, %3, 384;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a0l], %3, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1l], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2l], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3], b3, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3l], b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// D[tmem] (+)= U[tmem] * B[smem] over 64 keys with U a single 16-bit operand: the compute threads leave the
// 16-key steps 0, 1 at columns a, a + 8 and the steps 2, 3 at a + 32, a + 40 (each 32-key pass writes into
// the columns it read its scores from).
__device__ __forceinline__ void mma_ts_k64(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u32 a1, %2, 8; add.u32 a2, %2, 32; add.u32 a3, %2, 40;\n\t"
        "add.u64 b1, %3, 128; add.u64 b2, %3, 256; add.u64 b3, %3, 384;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3], b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// The same with the four 16-element steps of the TMEM operand in consecutive groups of 8 columns.
__device__ __forceinline__ void mma_ts_k64c(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u32 a1, %2, 8; add.u32 a2, %2, 16; add.u32 a3, %2, 24;\n\t"
        "add.u64 b1, %3, 128; add.u64 b2, %3, 256; add.u64 b3, %3, 384;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3], b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// D[tmem] (+)= U_hi[tmem] * B[smem] over 64 keys: only the hi halves of the operand pairs laid out as for
// mma_ts_hilo_k64 (16 columns per 16-key step), B MN-major.
__device__ __forceinline__ void mma_ts_hi_k64(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u32 a1, %2, 16; add.u32 a2, %2, 32; add.u32 a3, %2, 48;\n\t"
        "add.u64 b1, %3, 128; add.u64 b2, %3, 256; add.u64 b3, %3, 384;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3], b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem] over 64 elements of K with B K-major (a 64-row tile as TMA leaves it): the
// operand in TMEM holds its four 16-element steps in consecutive groups of 8 columns, B advances 32 bytes a step.
__device__ __forceinline__ void mma_ts_kmajor_k64(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 b1, b2, b3;\n\t.reg .b32 a1, a2, a3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u32 a1, %2, 8; add.u32 a2, %2, 16; add.u32 a3, %2, 24;\n\t"
        "add.u64 b1, %3, 2; add.u64 b2, %3, 4; add.u64 b3, %3, 6;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a1], b1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a2], b2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [a3], b3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc0) : "memory");
}
// Shared-memory matrix descriptors (128-byte swizzle, tile base 1024-byte aligned).
//   K-major:  rows of 128 bytes, 8-row groups 1024 bytes apart; a 16-element K step is +32 bytes.
//   MN-major: rows (one per K index) of 128 bytes holding 64 contiguous MN elements; 8-row groups
//             1024 bytes apart; a 16-element K step is +2048 bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo_bytes = 16) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);         // start address
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;    // leading byte offset: distance between the 64-wide
                                                         // column groups of an MN-major operand wider than 64
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset
    d |= (uint64_t)1 << 46;                              // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;                              // SWIZZLE_128B
    return d;
}

// byte offset of the 16-byte chunk `chunk` (8 bf16) of row `row` in a swizzled 128 x 64 bf16 tile
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// ------------------------------------------------------------------------------------------------
// Host: tensor-map encoding through the driver entry point (no link-time dependency on libcuda)
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}


// [outer, rows, 64] bf16 tensor viewed as 3-D, box = 64 columns x box_rows rows x 1, 128-byte swizzle
inline bool make_map_bf16_64(CUtensorMap* map, const void* base, int outer, int rows, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)outer};
    const cuuint64_t strides[2] = {128, (cuuint64_t)rows * 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 [outer][rows][cols] (cols a multiple of 64), box = 64 columns x box_rows rows, 128B swizzle:
// one copy per 64-column sub-tile, x coordinate 64 * sub.
inline bool make_map_bf16(CUtensorMap* map, const void* base, int outer, int rows, int cols, int box_rows,
                          CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)outer};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)rows * cols * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, dtype, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 16-bit [batches][heads][rows][cols] tensor with element strides (sb, sh, sr, 1), all multiples of 8 elements:
// 4-D map, box = 64 columns x box_rows rows x 1 x 1, 128B swizzle.  Coordinates (column, row, head, batch).
inline bool make_map_16bit_4d(CUtensorMap* map, const void* base, int batches, int heads, long long rows, int cols,
                              long long sb, long long sh, long long sr, int box_rows, CUtensorMapDataType dtype) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batches};
    // a dimension of extent 1 still needs a stride that is a multiple of 16 bytes and below 2^40
    const cuuint64_t strides[3] = {(cuuint64_t)sr * 2, (cuuint64_t)(heads > 1 ? sh : sr) * 2, (cuuint64_t)(batches > 1 ? sb : sr) * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, dtype, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 [outer][rows][cols] records (cols * 4 a multiple of 16 bytes), box = all columns x box_rows rows, no swizzle:
// rows past the end of an `outer` unit arrive as zeros.
inline bool make_map_f32_rows(CUtensorMap* map, const void* base, int outer, int rows, int cols, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)outer};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)rows * cols * 4};
    const cuuint32_t box[3] = {(cuuint32_t)cols, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace sm100
}  // namespace lla
