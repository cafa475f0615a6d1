// Tree acceptance of tree-based self-speculative decoding (Sec. 5.4,
// Appendix A, Algorithm 2): the target walks the draft tree from the root,
// accepting at each level a child whose token equals its own prediction, and
// adds one bonus token; the accepted nodes' K/V rows of every layer are then
// appended to the KV cache (the rejected nodes' rows are simply never copied).
#include "twig_common.cuh"

namespace twig {

constexpr int kAcceptThreads = 256;
constexpr int kAcceptSlicesPerCta = 4;   // (layer, kv head) slices copied by one CTA

// completion ticket per batch slot: the last CTA of a request to finish its
// copies publishes the new kv_len; the ticket returns to 0 for the next call.
__device__ unsigned int g_accept_ticket[TWIG_MAX_BATCH];

template <int D>
__global__ void __launch_bounds__(kAcceptThreads)
tree_accept_compact_kernel(const int *__restrict__ parent, const int *__restrict__ draft_tok,
                           const int *__restrict__ base_argmax, const int *__restrict__ n_nodes,
                           int t_max, int d_max, const __nv_bfloat16 *__restrict__ tree_k,
                           const __nv_bfloat16 *__restrict__ tree_v, KvViewMut cache, int *kv_len,
                           int *__restrict__ accept_len, int *__restrict__ path_out,
                           int *__restrict__ bonus_tok, int *dev_status) {
  constexpr int LPR = D / 8;
  __shared__ int s_parent[TWIG_MAX_NODES], s_tok[TWIG_MAX_NODES], s_tgt[TWIG_MAX_NODES];
  __shared__ int s_path[TWIG_MAX_NODES];
  __shared__ int s_bad, s_best, s_len;

  grid_dependency_sync();
  const int b = blockIdx.y, tid = threadIdx.x;
  const int n = n_nodes[b];
  if (n == 0) return;                                   // idle request
  const bool first = blockIdx.x == 0 && tid == 0;
  if (n < 0 || n > t_max) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
    return;
  }
  if (tid == 0) {
    s_bad = 0;
    s_best = -1;
  }
  __syncthreads();
  if (tid < n) {
    const int p = parent[(long long)b * t_max + tid];
    s_parent[tid] = p;
    s_tok[tid] = draft_tok[(long long)b * t_max + tid];
    s_tgt[tid] = base_argmax[(long long)b * t_max + tid];
    if ((tid == 0) ? (p != -1) : (p < 0 || p >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
    return;
  }
  // node i is accepted iff every edge on its root path matches; key orders by
  // depth first, then by lower index
  if (tid < n) {
    int x = tid, depth = 0;
    bool ok = true;
    while (x > 0) {                    // parent[x] < x, so this ends within n steps
      const int p = s_parent[x];
      ok = ok && (s_tok[x] == s_tgt[p]);
      x = p;
      ++depth;
    }
    if (ok) atomicMax(&s_best, depth * TWIG_MAX_NODES + (TWIG_MAX_NODES - 1 - tid));
  }
  __syncthreads();
  const int alen = s_best / TWIG_MAX_NODES;
  const int winner = TWIG_MAX_NODES - 1 - (s_best % TWIG_MAX_NODES);
  const int base = kv_len[b];
  if (alen + 1 > d_max || base < 0 || base + alen + 1 > cache.max_len) {
    if (first) flag_status(dev_status, b, alen + 1 > d_max ? TWIG_DEV_BAD_TREE : TWIG_DEV_OVERFLOW);
    return;
  }
  if (tid == 0) {
    int x = winner;
    for (int j = alen; j >= 0; --j) {
      s_path[j] = x;
      x = s_parent[x];
    }
    s_len = alen;
  }
  __syncthreads();
  if (blockIdx.x == 0) {
    if (tid < d_max) path_out[(long long)b * d_max + tid] = (tid <= alen) ? s_path[tid] : -1;
    if (tid == 0) {
      accept_len[b] = alen;
      bonus_tok[b] = s_tgt[winner];
    }
  }

  // copy rows path[0..alen] of the slices this CTA owns, K and V
  const int n_slices = cache.n_layers * cache.n_kv_heads;
  const int slice0 = blockIdx.x * kAcceptSlicesPerCta;
  const int rows = alen + 1;
  const int items = kAcceptSlicesPerCta * rows * 2 * LPR;
  for (int it = tid; it < items; it += kAcceptThreads) {
    const int sub = it % LPR;
    int r = it / LPR;
    const int which = r & 1;
    r >>= 1;
    const int j = r % rows, slice = slice0 + r / rows;
    if (slice >= n_slices) continue;
    const int layer = slice / cache.n_kv_heads, h = slice % cache.n_kv_heads;
    const long long toff = ((((long long)layer * cache.batch + b) * cache.n_kv_heads + h) * t_max + s_path[j]) * D + sub * 8;
    const long long coff = layer * cache.stride_layer + b * cache.stride_batch + h * cache.stride_head +
                           (long long)(base + j) * cache.stride_pos + sub * 8;
    const uint4 val = ld_nc_16((which ? tree_v : tree_k) + toff);
    st_16((which ? cache.v : cache.k) + coff, val);
  }

  // every CTA has read kv_len[b] above; the last one to arrive updates it
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(&g_accept_ticket[b], 1u);
    if (t == gridDim.x - 1) {
      g_accept_ticket[b] = 0;
      kv_len[b] = base + alen + 1;
      __threadfence();
    }
  }
}

// ---------------------------------------------------------------------------
// Greedy target token per tree node: argmax over the vocabulary, lowest index on ties.
// One CTA per (request, node) row; 16-byte loads, 8 in flight per thread.
// ---------------------------------------------------------------------------
constexpr int kArgmaxThreads = 256;

__device__ __forceinline__ void argmax_take(float v, int i, float &best, int &bi) {
  if (v > best || (v == best && i < bi)) {
    best = v;
    bi = i;
  }
}

template <bool FP32>
__global__ void __launch_bounds__(kArgmaxThreads)
base_argmax_kernel(const void *__restrict__ logits, long long row_stride, int vocab,
                   const int *__restrict__ n_nodes, int t_max, int *__restrict__ out, int *dev_status) {
  constexpr int EPC = FP32 ? 4 : 8;                 // elements per 16-byte chunk
  __shared__ float s_v[kArgmaxThreads / 32];
  __shared__ int s_i[kArgmaxThreads / 32];
  grid_dependency_sync();
  const int b = blockIdx.y, node = blockIdx.x, tid = threadIdx.x;
  const int n = n_nodes[b];
  if (n < 0 || n > t_max) {
    if (node == 0 && tid == 0) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
    return;
  }
  if (node >= n) return;
  const unsigned char *row = static_cast<const unsigned char *>(logits) +
                             ((long long)b * t_max + node) * row_stride * (FP32 ? 4 : 2);
  float best = -INFINITY;
  int bi = 0x7fffffff;
  const int chunks = vocab / EPC;
  auto take_chunk = [&](const uint4 &w, int c) {
    const int base = c * EPC;
    if (FP32) {
      argmax_take(__uint_as_float(w.x), base, best, bi);
      argmax_take(__uint_as_float(w.y), base + 1, best, bi);
      argmax_take(__uint_as_float(w.z), base + 2, best, bi);
      argmax_take(__uint_as_float(w.w), base + 3, best, bi);
    } else {
      argmax_take(bf16_lo(w.x), base, best, bi);
      argmax_take(bf16_hi(w.x), base + 1, best, bi);
      argmax_take(bf16_lo(w.y), base + 2, best, bi);
      argmax_take(bf16_hi(w.y), base + 3, best, bi);
      argmax_take(bf16_lo(w.z), base + 4, best, bi);
      argmax_take(bf16_hi(w.z), base + 5, best, bi);
      argmax_take(bf16_lo(w.w), base + 6, best, bi);
      argmax_take(bf16_hi(w.w), base + 7, best, bi);
    }
  };
  constexpr int kDeep = 8;                          // 16-byte loads in flight per thread
  // (every batch is predicated, so that a row that is no multiple of the batch never falls back to one
  // load per round trip)
  for (int c0 = tid; c0 < chunks; c0 += kDeep * kArgmaxThreads) {
    uint4 w[kDeep];
#pragma unroll
    for (int u = 0; u < kDeep; ++u) {
      const int c = c0 + u * kArgmaxThreads;
      if (c < chunks) w[u] = ld_nc_16(row + (long long)c * 16);
    }
#pragma unroll
    for (int u = 0; u < kDeep; ++u) {
      const int c = c0 + u * kArgmaxThreads;
      if (c < chunks) take_chunk(w[u], c);
    }
  }
  for (int i = chunks * EPC + tid; i < vocab; i += kArgmaxThreads) {     // tail that is no whole chunk
    const float v = FP32 ? reinterpret_cast<const float *>(row)[i]
                         : __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(row)[i]);
    argmax_take(v, i, best, bi);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    argmax_take(ov, oi, best, bi);
  }
  if ((tid & 31) == 0) {
    s_v[tid >> 5] = best;
    s_i[tid >> 5] = bi;
  }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kArgmaxThreads / 32; ++w) argmax_take(s_v[w], s_i[w], best, bi);
    out[(long long)b * t_max + node] = bi;
  }
}

}  // namespace twig

using namespace twig;

extern "C" twig_status tree_base_argmax(const void *logits, int32_t logits_fp32, int64_t row_stride,
                                        int32_t vocab, const int32_t *n_nodes, int32_t batch,
                                        int32_t t_max, int32_t *base_argmax, int32_t *dev_status,
                                        void *stream) {
  if (!logits || !n_nodes || !base_argmax) return TWIG_ERR_NULL;
  if (vocab <= 0 || batch <= 0 || t_max <= 0 || row_stride < vocab) return TWIG_ERR_SHAPE;
  if (t_max > TWIG_MAX_NODES || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  const int esz = logits_fp32 ? 4 : 2;
  if (!aligned16(logits) || (row_stride * esz) % 16) return TWIG_ERR_ALIGN;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(t_max, batch);
  cfg.blockDim = dim3(kArgmaxThreads);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = launch_overlap_enabled() ? 1 : 0;
  const long long rs = row_stride;
  const cudaError_t err =
      logits_fp32 ? cudaLaunchKernelEx(&cfg, base_argmax_kernel<true>, logits, rs, vocab, n_nodes, t_max, base_argmax, dev_status)
                  : cudaLaunchKernelEx(&cfg, base_argmax_kernel<false>, logits, rs, vocab, n_nodes, t_max, base_argmax, dev_status);
  return err == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}


extern "C" twig_status tree_accept_compact(const int32_t *parent, const int32_t *draft_tok,
                                           const int32_t *base_argmax, const int32_t *n_nodes,
                                           int32_t t_max, int32_t d_max, const void *tree_k_all,
                                           const void *tree_v_all, const twig_kv *cache,
                                           int32_t *kv_len, int32_t *accept_len, int32_t *path,
                                           int32_t *bonus_tok, int32_t *dev_status, void *stream) {
  if (!parent || !draft_tok || !base_argmax || !n_nodes || !tree_k_all || !tree_v_all || !kv_len ||
      !accept_len || !path || !bonus_tok)
    return TWIG_ERR_NULL;
  twig_status s = check_kv(cache);
  if (s != TWIG_OK) return s;
  if (t_max <= 0 || d_max <= 0) return TWIG_ERR_SHAPE;
  if (t_max > TWIG_MAX_NODES || d_max > TWIG_MAX_NODES) return TWIG_ERR_UNSUPPORTED;
  if (!aligned16(tree_k_all) || !aligned16(tree_v_all)) return TWIG_ERR_ALIGN;
  const int n_slices = cache->n_layers * cache->n_kv_heads;
  dim3 grid((n_slices + kAcceptSlicesPerCta - 1) / kAcceptSlicesPerCta, cache->batch);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto tk = static_cast<const __nv_bfloat16 *>(tree_k_all);
  auto tv = static_cast<const __nv_bfloat16 *>(tree_v_all);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kAcceptThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = launch_overlap_enabled() ? 1 : 0;
  const KvViewMut cv = view_of_mut(cache);
  const cudaError_t err =
      cache->head_dim == 128
          ? cudaLaunchKernelEx(&cfg, tree_accept_compact_kernel<128>, parent, draft_tok, base_argmax, n_nodes, t_max,
                               d_max, tk, tv, cv, kv_len, accept_len, path, bonus_tok, dev_status)
          : cudaLaunchKernelEx(&cfg, tree_accept_compact_kernel<64>, parent, draft_tok, base_argmax, n_nodes, t_max,
                               d_max, tk, tv, cv, kv_len, accept_len, path, bonus_tok, dev_status);
  if (err != cudaSuccess) return TWIG_ERR_CUDA;
  return launch_status();
}
