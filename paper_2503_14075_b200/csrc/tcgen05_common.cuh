// PTX wrappers shared by the tcgen05 tree-attention kernels: shared-memory and instruction
// descriptors, tcgen05.mma / commit / ld / st, TMA box loads, bounded mbarrier waits.
#pragma once

#include "tree_attn.cuh"

namespace twig {

constexpr int kSpinLimit = 1 << 22;

// ---- descriptors -------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
// lbo_bytes is the distance between 64-element groups along the leading (MN) dimension
// and is only meaningful for MN-major operands.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffff) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;      // descriptor version of this architecture
  d |= (uint64_t)2 << 61;      // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = m (64 or 128), A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with the A operand in tensor memory (M rows in the lanes, two consecutive-K bf16 per
// 32-bit column): only B comes through shared memory.
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One box of the 5-D cache tensor map -> shared memory; completion is counted on `bar`.
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int pos,
                                            int head, int batch, int layer) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(pos), "r"(head), "r"(batch), "r"(layer)
      : "memory");
}
// One box of a 4-D tensor map (x, position, head, batch) -> shared memory; completion is counted on `bar`.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int pos,
                                            int head, int batch) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(pos), "r"(head), "r"(batch)
      : "memory");
}
// Bounded wait on an mbarrier phase; false when the limit ran out or another role has failed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *fail) {
  for (int i = 0; i < kSpinLimit; ++i) {
    if ((i & 1023) == 1023 && *fail) return false;
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}

#define TWIG_R8(a, o) "=r"(a[o]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]), "=r"(a[o + 7])
// 32 consecutive fp32 columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : TWIG_R8(v, 0), TWIG_R8(v, 8), TWIG_R8(v, 16), TWIG_R8(v, 24)
      : "r"(taddr));
}
// 64 consecutive fp32 columns of 16 lanes (the 16 lanes from the address's lane on), spread over
// the warp like an mma.sync accumulator: for every 8-column group g, lane t holds columns
// 8g + 2(t % 4) + {0, 1} of row t / 4 in v[4g], v[4g+1] and of row t / 4 + 8 in v[4g+2], v[4g+3].
__device__ __forceinline__ void tmem_ld_16rows_64cols(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : TWIG_R8(v, 0), TWIG_R8(v, 8), TWIG_R8(v, 16), TWIG_R8(v, 24)
      : "r"(taddr));
}
#undef TWIG_R8
#define TWIG_S8(a, o) "r"(a[o]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7])
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), TWIG_S8(v, 0), TWIG_S8(v, 8), TWIG_S8(v, 16), TWIG_S8(v, 24)
      : "memory");
}
// 16 consecutive columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), TWIG_S8(v, 0), TWIG_S8(v, 8)
      : "memory");
}
#undef TWIG_S8
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 2^x by range reduction and a cubic on the FMA pipe (relative error < 1e-3, far below the
// bf16 rounding of P); used for half of the elements so that the special-function unit and
// the FMA pipe share the exponentials.  Arguments below -126 give 2^-126 (in effect 0).
__device__ __forceinline__ float poly_exp2(float x) {
  x = fmaxf(x, -126.f);
  const float t = x + 12582912.f;                 // 1.5 * 2^23: rounds x to the nearest integer
  const float f = x - (t - 12582912.f);           // in [-0.5, 0.5]
  float r = fmaf(f, 0.0555041f, 0.2402265f);
  r = fmaf(r, f, 0.6931472f);
  r = fmaf(r, f, 1.f);
  return __int_as_float(__float_as_int(r) + (__float_as_int(t) << 23));   // * 2^n (the magic's bits shift out)
}

}  // namespace twig
