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

}  // namespace twig

using namespace twig;

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
