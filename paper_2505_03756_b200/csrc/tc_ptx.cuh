// tcgen05 / TMEM / TMA / mbarrier wrappers (inline PTX for sm_100a) shared by the tensor-core kernels.
#pragma once
#include <cuda.h>
#include <stdint.h>
#include "mma_utils.cuh"

namespace tc {

constexpr uint32_t WAIT_LIMIT = 1u << 22;   // polls of one bounded mbarrier wait

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
// Bounded wait: false when the CTA is aborting or the limit ran out (which raises the abort flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// AND of a predicate over the `count` threads that meet at named barrier `id` (all of them get the result).
__device__ __forceinline__ bool group_and(bool mine, int id, int count) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "barrier.cta.red.and.pred q, %2, %3, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r) : "r"(mine ? 1u : 0u), "r"(id), "r"(count) : "memory");
  return r != 0;
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

#define TM_REGS(r, o) \
  "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define TM_IN(r, o) \
  "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])

// 32 consecutive TMEM columns of this thread's lane -> 32 registers (the warp reads its 32 lanes).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : TM_REGS(r, 0), TM_REGS(r, 8), TM_REGS(r, 16), TM_REGS(r, 24)
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), TM_IN(r, 0), TM_IN(r, 8), TM_IN(r, 16), TM_IN(r, 24) : "memory");
}
// 16 consecutive TMEM columns of this thread's lane -> 16 registers.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : TM_REGS(r, 0), TM_REGS(r, 8)
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D(tmem) (+)= A(tmem, bf16 pairs packed in 32-bit columns, row = lane) * B(smem descriptor).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 registers -> 16 consecutive TMEM columns of this thread's lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), TM_IN(r, 0), TM_IN(r, 8) : "memory");
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout code 2), descriptor version 1.
// K-major operands: lbo unused (1), sbo = 1024 (8 rows of 128 bytes).  MN-major: lbo = distance
// between 64-element groups along MN, sbo = 1024 (8 rows along K).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// The same descriptor as two 32-bit halves: the high half is fixed per layout and the low half is the start address / 16
// (plus the leading-offset field), so stepping through a tile is one 32-bit add.
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) { return (sbo_bytes >> 4) | (1u << 14) | (2u << 29); }

// Variants for a converged warp: every lane executes the call, one elected lane issues the instruction.  The
// operands then depend on nothing lane-specific.
__device__ __forceinline__ void umma_ss_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_ts_elect(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit_elect(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}
// One 128 x 128 x 128 score tile as a single block: an elected lane of the converged warp issues the eight k-steps and the
// commit.  Low descriptor words step by constants: Q is [half][128 rows][128 B] (k-steps 32 B apart, the halves 16 KiB),
// K is eight pages of [8-key group][half][8 keys][128 B] (k-steps 32 B apart, the halves 1 KiB).
__device__ __forceinline__ void umma_s_tile_elect(uint32_t d_tmem, uint32_t q_lo, uint32_t k_lo, uint32_t q_hi, uint32_t k_hi,
                                                  uint32_t idesc, uint32_t commit_bar) {
  asm volatile(
      "{\n\t.reg .pred e, pt, pf;\n\t.reg .b64 da, db;\n\t.reg .b32 a, b;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.eq.u32 pt, 0, 0;\n\tsetp.ne.u32 pf, 0, 0;\n\t"
      "add.u32 a, %1, 0;\n\tadd.u32 b, %2, 0;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pf;\n\t"
      "add.u32 a, %1, 2;\n\tadd.u32 b, %2, 2;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 4;\n\tadd.u32 b, %2, 4;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 6;\n\tadd.u32 b, %2, 6;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 1024;\n\tadd.u32 b, %2, 64;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 1026;\n\tadd.u32 b, %2, 66;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 1028;\n\tadd.u32 b, %2, 68;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "add.u32 a, %1, 1030;\n\tadd.u32 b, %2, 70;\n\tmov.b64 da, {a, %3};\n\tmov.b64 db, {b, %4};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, pt;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%6];\n\t}"
      ::"r"(d_tmem), "r"(q_lo), "r"(k_lo), "r"(q_hi), "r"(k_hi), "r"(idesc), "r"(commit_bar) : "memory");
}
// O (+)= P V for one 128-key tile: P as bf16 pairs in TMEM (8 columns per k-step), V as eight 4 KiB pages, one per k-step.
__device__ __forceinline__ void umma_pv_tile_elect(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_lo, uint32_t v_hi, uint32_t idesc,
                                                   uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred e, pt, p0;\n\t.reg .b64 db;\n\t.reg .b32 a, b;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.eq.u32 pt, 0, 0;\n\tsetp.ne.u32 p0, %5, 0;\n\t"
      "add.u32 a, %1, 0;\n\tadd.u32 b, %2, 0;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, p0;\n\t"
      "add.u32 a, %1, 8;\n\tadd.u32 b, %2, 256;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 16;\n\tadd.u32 b, %2, 512;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 24;\n\tadd.u32 b, %2, 768;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 32;\n\tadd.u32 b, %2, 1024;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 40;\n\tadd.u32 b, %2, 1280;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 48;\n\tadd.u32 b, %2, 1536;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "add.u32 a, %1, 56;\n\tadd.u32 b, %2, 1792;\n\tmov.b64 db, {b, %3};\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], db, %4, pt;\n\t"
      "}"
      ::"r"(o_tmem), "r"(p_tmem), "r"(v_lo), "r"(v_hi), "r"(idesc), "r"(accumulate_first) : "memory");
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n; b_mn = B operand is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

}  // namespace tc
