// Declarations shared by the two tree-attention kernels (the mma.sync path and
// the tcgen05 path): launch parameters and small PTX wrappers.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include "twig_common.cuh"

namespace twig {

struct AttnParams {
  const __nv_bfloat16 *q, *tree_k, *tree_v, *cache_k, *cache_v;   // cache_* point at the layer
  long long c_sb, c_sh, c_sp;
  const int *kv_len, *n_nodes, *parent;
  __nv_bfloat16 *out;
  float *lse;
  int *dev_status;
  int t_max, n_q_heads, n_kv_heads, group, max_len, row_blocks;
  // whole cache (all layers), for the tensor maps of the tcgen05 path
  const __nv_bfloat16 *cache_k0, *cache_v0;
  long long c_sl;
  int layer, n_layers, batch;
  int early_prefix;   // TWIG_ATTN_EARLY_PREFIX of the call
  int early_query;    // TWIG_ATTN_EARLY_QUERY as well (mma.sync kernel)
  float scale_log2;   // softmax_scale * log2(e)
  // host side only: launch with programmatic stream serialization, forced key splits (0: automatic),
  // the caller's scratch (persistent kernel)
  int overlap, forced_splits;
  int stream_policy;   // persistent kernel: 0 chosen on the device, 1 equal shares, 2 whole items
  unsigned char *ws;
  size_t ws_bytes;
};

// ---- small PTX wrappers ----------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float2 unpack_f16(uint32_t w) {
  return __half22float2(*reinterpret_cast<__half2 *>(&w));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// ---- mbarrier + asynchronous stores into a cluster peer's shared memory ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence_cluster() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA's window) in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// stores into a cluster CTA's shared memory (this CTA's own included); that CTA's mbarrier
// counts the bytes once they have landed
__device__ __forceinline__ void st_async_b32x2(uint32_t dst, uint32_t a, uint32_t b, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];"
               ::"r"(dst), "r"(a), "r"(b), "r"(bar) : "memory");
}
__device__ __forceinline__ void st_async_b32x4(uint32_t dst, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(dst), "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar) : "memory");
}
__device__ __forceinline__ void st_async_f32x2(uint32_t dst, float a, float b, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
               ::"r"(dst), "f"(a), "f"(b), "r"(bar) : "memory");
}

__device__ __forceinline__ void st_async_f32x4(uint32_t dst, float a, float b, float c, float d, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(dst), "f"(a), "f"(b), "f"(c), "f"(d), "r"(bar) : "memory");
}

// Partial rows cross between CTAs as fp16 of O / l (bounded by the largest |V| among the row's keys)
// times a power of two that brings the row's largest entry into [1, 2): fp16 then keeps 11 bits of
// every entry down to 2^-15 of that maximum, whatever the magnitude of V.  `amax` is that largest
// |O / l|; `down` scales the row before the conversion, `up` = 1 / down travels with the row's (m, l).
// Zero, infinite and NaN maxima are left unscaled.
__device__ __forceinline__ void row_scale(float amax, float &down, float &up) {
  const int ebits = (int)((__float_as_uint(amax) >> 23) & 0xffu);
  const bool scalable = ebits > 0 && ebits < 255;
  down = scalable ? __uint_as_float((uint32_t)(254 - ebits) << 23) : 1.f;
  up = scalable ? __uint_as_float((uint32_t)ebits << 23) : 1.f;
}

// exp2 on the special-function unit; fast_exp2(-inf) = +0
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Tensor maps (TMA) over the whole K and the whole V cache, dims (d, pos, head, batch, layer), boxes of
// 64 columns x box_rows rows with the 128-byte swizzle; kept in a small host table per cache layout.
struct CacheMaps {
  alignas(64) CUtensorMap kmap;
  alignas(64) CUtensorMap vmap;
};
bool cache_maps(const AttnParams &p, int box_rows, CacheMaps *out);

// tcgen05 path (tree_attn_umma.cu): head_dim 128, rows = t_max * group.
twig_status launch_tree_attn_umma(AttnParams &p, int batch, int rows, cudaStream_t st);
// persistent tcgen05 path (tree_attn_stream.cu): the same shapes, needs the caller's scratch
twig_status launch_tree_attn_stream(AttnParams &p, int batch, int rows, cudaStream_t st);
size_t tree_attn_stream_workspace_bytes(int batch, int n_q_heads, int max_nodes);
int pick_splits(int items, int max_tiles, int ctas_per_sm, int forced);

}  // namespace twig
