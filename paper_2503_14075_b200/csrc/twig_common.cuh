// Shared device/host helpers for the twig kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "twig.h"

namespace twig {

// Host-side view of a twig_kv with everything the kernels need by value.
struct KvView {
  const __nv_bfloat16 *k, *v;
  long long stride_layer, stride_batch, stride_head, stride_pos;
  int n_layers, batch, n_kv_heads, head_dim, max_len;
};

struct KvViewMut {
  __nv_bfloat16 *k, *v;
  long long stride_layer, stride_batch, stride_head, stride_pos;
  int n_layers, batch, n_kv_heads, head_dim, max_len;
};

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks a twig_kv: pointers, head_dim, and that every row starts on 16 bytes.
inline twig_status check_kv(const twig_kv *kv) {
  if (!kv || !kv->k || !kv->v) return TWIG_ERR_NULL;
  if (kv->head_dim != 64 && kv->head_dim != 128) return TWIG_ERR_UNSUPPORTED;
  if (kv->n_layers <= 0 || kv->batch <= 0 || kv->n_kv_heads <= 0 || kv->max_len <= 0)
    return TWIG_ERR_SHAPE;
  if (kv->batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (kv->stride_pos < kv->head_dim) return TWIG_ERR_SHAPE;
  if (!aligned16(kv->k) || !aligned16(kv->v)) return TWIG_ERR_ALIGN;
  if ((kv->stride_layer | kv->stride_batch | kv->stride_head | kv->stride_pos) & 7)
    return TWIG_ERR_ALIGN;
  return TWIG_OK;
}

inline KvView view_of(const twig_kv *kv) {
  KvView w;
  w.k = static_cast<const __nv_bfloat16 *>(kv->k);
  w.v = static_cast<const __nv_bfloat16 *>(kv->v);
  w.stride_layer = kv->stride_layer;
  w.stride_batch = kv->stride_batch;
  w.stride_head = kv->stride_head;
  w.stride_pos = kv->stride_pos;
  w.n_layers = kv->n_layers;
  w.batch = kv->batch;
  w.n_kv_heads = kv->n_kv_heads;
  w.head_dim = kv->head_dim;
  w.max_len = kv->max_len;
  return w;
}

inline KvViewMut view_of_mut(const twig_kv *kv) {
  KvViewMut w;
  w.k = static_cast<__nv_bfloat16 *>(kv->k);
  w.v = static_cast<__nv_bfloat16 *>(kv->v);
  w.stride_layer = kv->stride_layer;
  w.stride_batch = kv->stride_batch;
  w.stride_head = kv->stride_head;
  w.stride_pos = kv->stride_pos;
  w.n_layers = kv->n_layers;
  w.batch = kv->batch;
  w.n_kv_heads = kv->n_kv_heads;
  w.head_dim = kv->head_dim;
  w.max_len = kv->max_len;
  return w;
}

// Whether kernels are launched with programmatic stream serialization (the next kernel of the
// stream may be scheduled while this one drains; it waits on the device before reading anything).
bool launch_overlap_enabled();

// Launch configuration with programmatic stream serialization: the kernel may be scheduled while its
// predecessor in the stream drains; it waits on the device before it reads that kernel's output.
struct PdlLaunch {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  PdlLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t st) {
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = launch_overlap_enabled() ? 1 : 0;
  }
};

inline twig_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}

#ifdef __CUDACC__
// First statement of every kernel that may be launched with programmatic stream serialization:
// wait until the preceding kernel of the stream has completed and its writes are visible, then
// allow the following kernel to be scheduled.  A no-op for ordinary launches.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ void flag_status(int *dev_status, int b, int code) {
  if (dev_status) atomicMax(dev_status + b, code);
}

__device__ __forceinline__ uint4 ld_nc_16(const void *p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ void st_16(void *p, const uint4 &r) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z),
               "r"(r.w)
               : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
#endif

}  // namespace twig
