// Chain drafting of sequence self-speculative decoding with its early exit (Appendix A,
// "Self-speculative decoding"; Algorithm 1's draft loop): the draft model predicts up to
// delta tokens one after another and stops early once the probability of the token it has
// just predicted falls below theta; that token still belongs to the draft.  The draft model
// runs between the calls (its logits are inputs); one call takes one draft distribution per
// request, picks the greedy token (lowest id among equal logits), computes its probability,
// appends it to the request's chain (node n's parent is node n - 1, the layout tree attention
// and acceptance take: a chain is a tree) and decides whether the request goes on drafting.
// Requests that have stopped ignore further calls, so a batch can be driven through delta
// calls without reading anything back.
#include "twig_common.cuh"

namespace twig {

constexpr int kChainThreads = 512;

// running (maximum, its first index, sum of exp(x - maximum))
struct MaxSum {
  float m, s;
  int i;
};
__device__ __forceinline__ void ms_take(MaxSum &a, float x, int i) {
  if (x > a.m) {
    a.s = a.s * __expf(a.m - x) + 1.f;      // (exp(-inf) = 0 for the first element)
    a.m = x;
    a.i = i;
  } else if (x > -INFINITY) {                // (a logit of -inf adds nothing, also before any finite one)
    a.s += __expf(x - a.m);
  }
}
__device__ __forceinline__ void ms_merge(MaxSum &a, const MaxSum &b) {
  if (b.m > a.m || (b.m == a.m && b.i < a.i)) {
    a.s = b.s + a.s * __expf(a.m - b.m);
    a.m = b.m;
    a.i = b.i;
  } else if (b.m > -INFINITY) {
    a.s += b.s * __expf(b.m - a.m);
  }
}

template <bool FP32>
__global__ void __launch_bounds__(kChainThreads)
chain_draft_step_kernel(const void *__restrict__ logits, long long row_stride, int vocab, int max_draft,
                        float threshold, int *__restrict__ parent, int *__restrict__ draft_tok,
                        float *__restrict__ tok_prob, int *__restrict__ n_nodes, int *__restrict__ active,
                        int t_max, int *dev_status) {
  constexpr int EPC = FP32 ? 4 : 8;                 // elements per 16-byte chunk
  __shared__ MaxSum s_part[kChainThreads / 32];
  grid_dependency_sync();
  const int b = blockIdx.x, tid = threadIdx.x;
  if (active[b] == 0) return;
  const int n = n_nodes[b];
  if (n < 1 || n >= t_max) {                        // no root yet, or no room for another node
    if (tid == 0) {
      flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
      active[b] = 0;
    }
    return;
  }
  const unsigned char *row = static_cast<const unsigned char *>(logits) + (long long)b * row_stride * (FP32 ? 4 : 2);
  MaxSum acc{-INFINITY, 0.f, 0x7fffffff};
  const int chunks = vocab / EPC;
  auto take_chunk = [&](const uint4 &w, int c) {
    const int base = c * EPC;
    if (FP32) {
      ms_take(acc, __uint_as_float(w.x), base);
      ms_take(acc, __uint_as_float(w.y), base + 1);
      ms_take(acc, __uint_as_float(w.z), base + 2);
      ms_take(acc, __uint_as_float(w.w), base + 3);
    } else {
      ms_take(acc, bf16_lo(w.x), base);
      ms_take(acc, bf16_hi(w.x), base + 1);
      ms_take(acc, bf16_lo(w.y), base + 2);
      ms_take(acc, bf16_hi(w.y), base + 3);
      ms_take(acc, bf16_lo(w.z), base + 4);
      ms_take(acc, bf16_hi(w.z), base + 5);
      ms_take(acc, bf16_lo(w.w), base + 6);
      ms_take(acc, bf16_hi(w.w), base + 7);
    }
  };
  int c = tid;
  constexpr int kDeep = 4;                          // 16-byte loads in flight per thread
  for (; c + (kDeep - 1) * kChainThreads < chunks; c += kDeep * kChainThreads) {
    uint4 w[kDeep];
#pragma unroll
    for (int u = 0; u < kDeep; ++u) w[u] = ld_nc_16(row + (long long)(c + u * kChainThreads) * 16);
#pragma unroll
    for (int u = 0; u < kDeep; ++u) take_chunk(w[u], c + u * kChainThreads);
  }
  for (; c < chunks; c += kChainThreads) take_chunk(ld_nc_16(row + (long long)c * 16), c);
  for (int i = chunks * EPC + tid; i < vocab; i += kChainThreads) {     // tail that is no whole chunk
    const float v = FP32 ? reinterpret_cast<const float *>(row)[i]
                         : __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(row)[i]);
    ms_take(acc, v, i);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum other;
    other.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
    other.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
    other.i = __shfl_xor_sync(0xffffffffu, acc.i, o);
    ms_merge(acc, other);
  }
  if ((tid & 31) == 0) s_part[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kChainThreads / 32; ++w) ms_merge(acc, s_part[w]);
    const float prob = 1.f / acc.s;                 // softmax(row)[token]: the token's logit is the maximum
    const long long at = (long long)b * t_max + n;
    parent[at] = n - 1;
    draft_tok[at] = acc.i;
    if (tok_prob) tok_prob[at] = prob;
    n_nodes[b] = n + 1;
    // n draft tokens now (the root is node 0): stop at delta of them or below the confidence threshold
    if (n >= max_draft || prob < threshold) active[b] = 0;
  }
}

__global__ void chain_draft_reset_kernel(int *parent, int *draft_tok, float *tok_prob, int *n_nodes, int *active,
                                         int t_max, int batch) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < batch * t_max) {
    parent[idx] = -1;
    draft_tok[idx] = idx % t_max == 0 ? -1 : 0;
    if (tok_prob) tok_prob[idx] = idx % t_max == 0 ? 1.f : 0.f;
  }
  if (idx < batch) {
    n_nodes[idx] = 1;        // the root: the last accepted token
    active[idx] = 1;
  }
}

}  // namespace twig

using namespace twig;

extern "C" twig_status chain_draft_reset(int32_t *parent, int32_t *draft_tok, float *tok_prob, int32_t *n_nodes,
                                         int32_t *active, int32_t t_max, int32_t batch, void *stream) {
  if (!parent || !draft_tok || !n_nodes || !active) return TWIG_ERR_NULL;
  if (t_max <= 0 || batch <= 0) return TWIG_ERR_SHAPE;
  if (t_max > TWIG_MAX_NODES || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  const int total = batch * t_max;
  chain_draft_reset_kernel<<<(total + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      parent, draft_tok, tok_prob, n_nodes, active, t_max, batch);
  return launch_status();
}

extern "C" twig_status chain_draft_step(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                                        int32_t max_draft, float threshold, int32_t *parent, int32_t *draft_tok,
                                        float *tok_prob, int32_t *n_nodes, int32_t *active, int32_t t_max,
                                        int32_t batch, int32_t *dev_status, void *stream) {
  if (!logits || !parent || !draft_tok || !n_nodes || !active) return TWIG_ERR_NULL;
  if (vocab <= 0 || batch <= 0 || t_max <= 0 || row_stride < vocab || max_draft <= 0) return TWIG_ERR_SHAPE;
  if (max_draft + 1 > t_max) return TWIG_ERR_SHAPE;            // the root and delta draft tokens must fit
  if (t_max > TWIG_MAX_NODES || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (!(threshold >= 0.f)) return TWIG_ERR_SHAPE;               // (also refuses NaN)
  const int esz = logits_fp32 ? 4 : 2;
  if (!aligned16(logits) || (row_stride * esz) % 16) return TWIG_ERR_ALIGN;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(batch);
  cfg.blockDim = dim3(kChainThreads);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = launch_overlap_enabled() ? 1 : 0;
  const long long rs = row_stride;
  const cudaError_t err =
      logits_fp32 ? cudaLaunchKernelEx(&cfg, chain_draft_step_kernel<true>, logits, rs, vocab, max_draft, threshold, parent,
                                       draft_tok, tok_prob, n_nodes, active, t_max, dev_status)
                  : cudaLaunchKernelEx(&cfg, chain_draft_step_kernel<false>, logits, rs, vocab, max_draft, threshold, parent,
                                       draft_tok, tok_prob, n_nodes, active, t_max, dev_status);
  return err == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}
