// 5th-generation tensor-core primitives (tcgen05 + tensor memory), sm_100a only: TMEM allocation,
// shared-memory matrix descriptors for the 128-byte-swizzled canonical layouts, instruction
// descriptors for bf16 x bf16 -> fp32, MMA issue with A from shared or tensor memory, commit to an
// mbarrier, and 32-lane x 32-column loads / stores between registers and tensor memory.
#pragma once
#include <stdint.h>

#include "gf_device.cuh"

namespace gf {

// ---- tensor memory ----------------------------------------------------------------------------
// Allocation is warp-collective; the base address (lane 0, first column) is written to shared
// memory.  ncols is a power of two in [32, 512].  The allocating warp must also deallocate.
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// Makes generic-proxy shared-memory writes visible to the async proxy (tensor-core operand reads).
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// ---- descriptors ------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle.  Canonical layouts (T = 8 bf16 = 16 bytes):
//   K-major  operand [rows][64 elements]: a row is 128 bytes, 8 rows form a 1024-byte atom, the
//            next 8 rows are sbo bytes further; lbo is unused.  One MMA consumes 16 elements
//            (32 bytes) of every row: advance the start address by 32 bytes per K step.
//   MN-major operand [k][64 elements of M/N]: a k-row is 128 bytes, 8 k-rows form an atom, the
//            next 8 k-rows are sbo bytes further, the next 64 M/N elements lbo bytes further.
//            One MMA consumes 16 k-rows: advance the start address by 2 * sbo per K step.
__host__ __device__ constexpr uint64_t tc_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46) /* descriptor version */ |
         ((uint64_t)2 << 61) /* 128-byte swizzle */;
}
// Instruction descriptor: D fp32, A and B bf16, A K-major, B K-major or MN-major, M x N tile.
__host__ __device__ constexpr uint32_t tc_idesc_bf16(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

// ---- MMA (one thread issues for the CTA); K = 16 per instruction --------------------------------
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// A (M x 16, bf16 pairs packed in 8 columns) from tensor memory.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// ---- whole K loops in one asm block ------------------------------------------------------------
// The issuing thread is alone on its scheduler, so every instruction between two MMAs costs issue
// latency.  These blocks keep the two predicates and the descriptor halves in registers and spend
// one 32-bit add per operand and MMA (the start address is the low field of a descriptor; adding
// to the low word cannot carry out of it for shared-memory addresses).
#define GF_MMA_SS_STEP(OFF, PRED)                                              \
  "add.u32 ta, alo, " #OFF ";\n\tmov.b64 da, {ta, ahi};\n\t"                  \
  "add.u32 tb, blo, " #OFF ";\n\tmov.b64 db, {tb, bhi};\n\t"                  \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, " #PRED ";\n\t"
// S = A B^T over K = 64 * CB elements: both operands K-major, 128-row column blocks 16384 bytes
// apart, 32 bytes per K step inside a column block.  The first MMA overwrites the accumulator.
template <int CB>
__device__ __forceinline__ void umma_ss_kloop(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  if constexpr (CB == 2) {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b32 alo, ahi, blo, bhi, ta, tb;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 pf, 0, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "mov.b64 {alo, ahi}, %1;\n\tmov.b64 {blo, bhi}, %2;\n\t"
        GF_MMA_SS_STEP(0, pf) GF_MMA_SS_STEP(2, pt) GF_MMA_SS_STEP(4, pt) GF_MMA_SS_STEP(6, pt)
        GF_MMA_SS_STEP(1024, pt) GF_MMA_SS_STEP(1026, pt) GF_MMA_SS_STEP(1028, pt) GF_MMA_SS_STEP(1030, pt)
        "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred pf, pt;\n\t.reg .b32 alo, ahi, blo, bhi, ta, tb;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 pf, 0, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
        "mov.b64 {alo, ahi}, %1;\n\tmov.b64 {blo, bhi}, %2;\n\t"
        GF_MMA_SS_STEP(0, pf) GF_MMA_SS_STEP(2, pt) GF_MMA_SS_STEP(4, pt) GF_MMA_SS_STEP(6, pt)
        "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
  }
}
#undef GF_MMA_SS_STEP

#define GF_MMA_TS_STEP(AOFF, BOFF, PRED)                                       \
  "add.u32 ta, %1, " #AOFF ";\n\t"                                             \
  "add.u32 tb, blo, " #BOFF ";\n\tmov.b64 db, {tb, bhi};\n\t"                  \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, " #PRED ";\n\t"
// O (+)= P V over 128 tokens: P as bf16 pairs in tensor memory (tokens 0..63 at columns 0..31, tokens
// 64..127 at columns 64..95 of a_tmem), V MN-major with 16 token rows = 2048 bytes per K step.
__device__ __forceinline__ void umma_ts_kloop8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred pf, pt;\n\t.reg .b32 blo, bhi, ta, tb;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 pf, %4, 0;\n\tsetp.eq.b32 pt, 0, 0;\n\t"
      "mov.b64 {blo, bhi}, %2;\n\t"
      GF_MMA_TS_STEP(0, 0, pf) GF_MMA_TS_STEP(8, 128, pt) GF_MMA_TS_STEP(16, 256, pt) GF_MMA_TS_STEP(24, 384, pt)
      GF_MMA_TS_STEP(64, 512, pt) GF_MMA_TS_STEP(72, 640, pt) GF_MMA_TS_STEP(80, 768, pt) GF_MMA_TS_STEP(88, 896, pt)
      "}" ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate_first)
      : "memory");
}
#undef GF_MMA_TS_STEP

// ---- registers <-> tensor memory: thread i of the warp owns lane (lane base + i) ---------------
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,"
      "%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
      "%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// ---- packed fp32 pairs and three-input max (halve the instruction count of the softmax) --------
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

}  // namespace gf
