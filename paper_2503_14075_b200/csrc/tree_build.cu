// Draft-side token tree of tree-based self-speculative decoding (Sec. 4.3; Appendix, "Tree-based
// self-speculative decoding"): level by level, every node selected for expansion gets its E most
// probable next tokens as children; the K best nodes of a level are expanded at the next; at the end
// the tree is cut to N_max nodes.  A node's score is the log of the joint probability of its path.
// The draft model itself runs between these calls: its logits are inputs.
//
// Tree state per request (capacity `cap` nodes, node 0 = root): token, parent, score, all in
// creation order (a parent always precedes its children).
#include "twig_common.cuh"

namespace twig {

namespace {

constexpr int kTopThreads = 512;
constexpr int kMaxE = 16;            // children per expanded node
constexpr int kMaxCand = 1024;       // entries at or above the threshold that the short list holds
constexpr int kSelThreads = 256;

// (value, index) order of the top lists: larger value first, equal values: lower index first
__device__ __forceinline__ bool comes_first(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

// One CTA per (expansion slot, request): log-sum-exp of the row and its E largest logits.
// The row is read from global memory once and kept in shared memory (when it fits).  The E-th
// largest of the half-warp groups' maxima is a lower bound of the E-th largest logit, so one more pass
// over the staged row collects the few entries at or above it into a short list; the E selection
// rounds run over that list (over the whole row if the list overflows, e.g. a row of equal logits).
// Round e finds the best entry that comes strictly after round e-1's winner in the (value, index)
// order, so nothing has to be marked as taken and no lane takes a long branch.
template <bool FP32>
__global__ void __launch_bounds__(kTopThreads)
tree_expand_kernel(const void *__restrict__ logits, long long row_stride, int vocab, int rows,
                   const int *__restrict__ src_node, int E, int level_base, int cap, int staged,
                   int *__restrict__ node_tok, int *__restrict__ node_parent, float *__restrict__ node_score,
                   int *dev_status) {
  constexpr int EPC = FP32 ? 4 : 8;
  extern __shared__ __align__(16) unsigned char row_s[];
  __shared__ float s_v[kTopThreads / 32];
  __shared__ int s_i[kTopThreads / 32];
  __shared__ float s_m[kTopThreads / 32], s_s[kTopThreads / 32];
  __shared__ float s_top_v[kMaxE];
  __shared__ int s_top_i[kMaxE];
  __shared__ float s_tmax[kTopThreads / 16];       // maxima of the half-warp groups
  __shared__ float s_cand_v[kMaxCand];
  __shared__ int s_cand_i[kMaxCand];
  __shared__ int s_n_cand;
  const int r = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = src_node[(long long)b * rows + r];
  if (u < 0) return;                                       // unused slot
  const int first = level_base + r * E;
  if (u >= level_base || first + E > cap) {
    if (tid == 0) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
    return;
  }
  const unsigned char *row = static_cast<const unsigned char *>(logits) +
                             ((long long)b * rows + r) * row_stride * (FP32 ? 4 : 2);
  auto element = [&](const unsigned char *base, int i) {
    return FP32 ? reinterpret_cast<const float *>(base)[i]
                : __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(base)[i]);
  };
  auto unpack = [&](const uint4 &w, float (&v)[8]) {
    if (FP32) {
      v[0] = __uint_as_float(w.x); v[1] = __uint_as_float(w.y); v[2] = __uint_as_float(w.z); v[3] = __uint_as_float(w.w);
    } else {
      v[0] = bf16_lo(w.x); v[1] = bf16_hi(w.x); v[2] = bf16_lo(w.y); v[3] = bf16_hi(w.y);
      v[4] = bf16_lo(w.z); v[5] = bf16_hi(w.z); v[6] = bf16_lo(w.w); v[7] = bf16_hi(w.w);
    }
  };
  const int chunks = vocab / EPC;

  // ---- pass over global memory: stage the row, running (max, sum of exp) per thread ----
  float m = -INFINITY, s = 0.f;
  float t_max = -INFINITY;                       // (equals m; kept apart for clarity)
  auto soft = [&](float v) {
    t_max = fmaxf(t_max, v);
    const float nm = fmaxf(m, v);
    s = s * __expf(m - nm) + __expf(v - nm);      // (m = -inf: s is 0 and exp(-inf) = 0)
    m = nm;
  };
  for (int c = tid; c < chunks; c += kTopThreads) {
    const uint4 w = ld_nc_16(row + (long long)c * 16);
    if (staged) *reinterpret_cast<uint4 *>(row_s + (size_t)c * 16) = w;
    float v[8];
    unpack(w, v);
    float cm = v[0];
#pragma unroll
    for (int k = 1; k < EPC; ++k) cm = fmaxf(cm, v[k]);
    t_max = fmaxf(t_max, cm);
    const float nm = fmaxf(m, cm);
    float acc = s * __expf(m - nm);
#pragma unroll
    for (int k = 0; k < EPC; ++k) acc += __expf(v[k] - nm);
    s = acc;
    m = nm;
  }
  for (int i = chunks * EPC + tid; i < vocab; i += kTopThreads) {
    const float v = element(row, i);
    if (staged) {
      if (FP32) reinterpret_cast<float *>(row_s)[i] = v;
      else reinterpret_cast<__nv_bfloat16 *>(row_s)[i] = reinterpret_cast<const __nv_bfloat16 *>(row)[i];
    }
    soft(v);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, s, o);
    const float nm = fmaxf(m, om);
    s = (m == -INFINITY ? 0.f : s * __expf(m - nm)) + (om == -INFINITY ? 0.f : os * __expf(om - nm));
    m = nm;
  }
  if (lane == 0) {
    s_m[warp] = m;
    s_s[warp] = s;
  }
  __syncthreads();                         // (also: the staged row is complete)
  float M = -INFINITY;
  for (int w = 0; w < kTopThreads / 32; ++w) M = fmaxf(M, s_m[w]);
  float S = 0.f;
  for (int w = 0; w < kTopThreads / 32; ++w) S += s_m[w] == -INFINITY ? 0.f : s_s[w] * __expf(s_m[w] - M);
  const float lse = M + logf(S);

  // ---- threshold: the E-th largest of the maxima of the 32 half-warp groups (E <= 16 distinct
  // entries are at or above it, so it is a lower bound of the E-th largest logit) ----
  const unsigned char *src = staged ? row_s : row;
  float g_max = t_max;
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) g_max = fmaxf(g_max, __shfl_xor_sync(0xffffffffu, g_max, o));
  constexpr int kGroups = kTopThreads / 16;
  if ((lane & 15) == 0) s_tmax[tid >> 4] = g_max;
  if (tid == 0) s_n_cand = 0;
  __syncthreads();
  if (tid < kGroups) {
    const float mine = s_tmax[tid];
    int above = 0;                                   // group maxima ranked before mine (ties: lower group first)
    for (int j = 0; j < kGroups; ++j) above += (s_tmax[j] > mine || (s_tmax[j] == mine && j < tid)) ? 1 : 0;
    if (above == E - 1) s_v[0] = mine;               // exactly one group has this rank
  }
  __syncthreads();
  const float thr = s_v[0];
  __syncthreads();
  for (int c = tid; c < chunks; c += kTopThreads) {
    const uint4 w = *reinterpret_cast<const uint4 *>(src + (size_t)c * 16);
    float v[8];
    unpack(w, v);
#pragma unroll
    for (int k = 0; k < EPC; ++k)
      if (v[k] >= thr) {
        const int at = atomicAdd(&s_n_cand, 1);
        if (at < kMaxCand) {
          s_cand_v[at] = v[k];
          s_cand_i[at] = c * EPC + k;
        }
      }
  }
  for (int i = chunks * EPC + tid; i < vocab; i += kTopThreads) {
    const float v = element(src, i);
    if (v >= thr) {
      const int at = atomicAdd(&s_n_cand, 1);
      if (at < kMaxCand) {
        s_cand_v[at] = v;
        s_cand_i[at] = i;
      }
    }
  }
  __syncthreads();
  const int n_cand = s_n_cand;
  const bool short_list = n_cand <= kMaxCand;       // (n_cand >= E always: the E maxima are in it)

  // ---- E rounds over the short list (or the whole row) ----
  float pv = INFINITY;                     // previous winner; every finite logit comes after (+inf, -1)
  int pi = -1;
  for (int e = 0; e < E; ++e) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    auto offer = [&](float v, int i) {
      const bool after_prev = pv > v || (pv == v && pi < i);
      if (after_prev && comes_first(v, i, bv, bi)) {
        bv = v;
        bi = i;
      }
    };
    if (short_list)
      for (int j = tid; j < n_cand; j += kTopThreads) offer(s_cand_v[j], s_cand_i[j]);
    for (int c = tid; c < (short_list ? 0 : chunks); c += kTopThreads) {
      const uint4 w = *reinterpret_cast<const uint4 *>(src + (size_t)c * 16);
      float v[8];
      int ix[8];
      unpack(w, v);
      // entries at or before the previous winner drop out; then a tournament inside the chunk (equal
      // values: the left, lower-index entry stays), and one comparison with the running best
#pragma unroll
      for (int k = 0; k < EPC; ++k) {
        ix[k] = c * EPC + k;
        const bool after_prev = pv > v[k] || (pv == v[k] && pi < ix[k]);
        v[k] = after_prev ? v[k] : -INFINITY;
      }
#pragma unroll
      for (int span = 1; span < EPC; span <<= 1)
#pragma unroll
        for (int k = 0; k + span < EPC; k += 2 * span)
          if (v[k + span] > v[k]) {
            v[k] = v[k + span];
            ix[k] = ix[k + span];
          }
      if (v[0] > -INFINITY && comes_first(v[0], ix[0], bv, bi)) {
        bv = v[0];
        bi = ix[0];
      }
    }
    if (!short_list)
      for (int i = chunks * EPC + tid; i < vocab; i += kTopThreads) offer(element(src, i), i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (comes_first(ov, oi, bv, bi)) {
        bv = ov;
        bi = oi;
      }
    }
    if (lane == 0) {
      s_v[warp] = bv;
      s_i[warp] = bi;
    }
    __syncthreads();
    pv = s_v[0];
    pi = s_i[0];
#pragma unroll
    for (int w = 1; w < kTopThreads / 32; ++w)
      if (comes_first(s_v[w], s_i[w], pv, pi)) {
        pv = s_v[w];
        pi = s_i[w];
      }
    if (tid == 0) {
      s_top_v[e] = pv;
      s_top_i[e] = pi;
    }
    __syncthreads();                       // s_v / s_i are free for the next round
  }
  if (tid < E) {
    const long long at = (long long)b * cap + first + tid;
    node_tok[at] = s_top_i[tid];
    node_parent[at] = u;
    node_score[at] = node_score[(long long)b * cap + u] + (s_top_v[tid] - lse);
  }
}

// One CTA per request.  Ranks the nodes lo..hi-1 by (score desc, id asc) and takes the first `take`:
//  * expansion mode (parent_out == nullptr): their ids, ascending, to sel_out[b, 0..take) (-1 padded);
//  * final mode: the root and the selected nodes are renumbered in creation order and written as
//    parent_out / tok_out [b, t_max] with n_nodes_out[b]; kept_out[b, i] = the old id of new node i.
__global__ void __launch_bounds__(kSelThreads)
tree_select_kernel(const float *__restrict__ node_score, const int *__restrict__ node_tok,
                   const int *__restrict__ node_parent, int cap, int lo, int hi, int take,
                   int *__restrict__ sel_out, int sel_stride, int *__restrict__ parent_out,
                   int *__restrict__ tok_out, int *__restrict__ n_nodes_out, int *__restrict__ kept_out,
                   int t_max, int *dev_status) {
  extern __shared__ unsigned char sel_smem[];
  float *sc = reinterpret_cast<float *>(sel_smem);                 // [hi]
  int *new_id = reinterpret_cast<int *>(sel_smem) + cap;           // [hi]: position among the kept, or -1
  const int b = blockIdx.x, tid = threadIdx.x;
  const float *score = node_score + (long long)b * cap;
  for (int i = tid; i < hi; i += kSelThreads) {
    sc[i] = score[i];
    new_id[i] = -1;
  }
  __syncthreads();
  const bool final_mode = parent_out != nullptr;
  for (int i = lo + tid; i < hi; i += kSelThreads) {
    int rank = 0;
    const float v = sc[i];
    for (int j = lo; j < hi; ++j) rank += comes_first(sc[j], j, v, i) ? 1 : 0;
    if (rank < take) new_id[i] = 0;                                // selected (position follows)
  }
  if (final_mode && tid == 0) new_id[0] = 0;                       // the root is always kept
  __syncthreads();
  const int from = final_mode ? 0 : lo;
  for (int i = from + tid; i < hi; i += kSelThreads) {
    if (new_id[i] < 0) continue;
    int pos = 0;
    for (int j = from; j < i; ++j) pos += new_id[j] >= 0 ? 1 : 0;
    // (positions are written after every thread has counted)
    sc[i] = __int_as_float(pos);
  }
  __syncthreads();
  for (int i = from + tid; i < hi; i += kSelThreads)
    if (new_id[i] >= 0) new_id[i] = __float_as_int(sc[i]);
  __syncthreads();
  if (!final_mode) {
    for (int k = tid; k < sel_stride; k += kSelThreads) sel_out[(long long)b * sel_stride + k] = -1;
    __syncthreads();
    for (int i = lo + tid; i < hi; i += kSelThreads)
      if (new_id[i] >= 0 && new_id[i] < sel_stride) sel_out[(long long)b * sel_stride + new_id[i]] = i;
    return;
  }
  int total = 0;
  for (int j = 0; j < hi; ++j) total += new_id[j] >= 0 ? 1 : 0;    // (hi <= a few hundred)
  if (tid == 0) n_nodes_out[b] = total;
  for (int k = total + tid; k < t_max; k += kSelThreads) {
    parent_out[(long long)b * t_max + k] = -1;
    tok_out[(long long)b * t_max + k] = 0;
    if (kept_out) kept_out[(long long)b * t_max + k] = -1;
  }
  for (int i = tid; i < hi; i += kSelThreads) {
    const int ni = new_id[i];
    if (ni < 0) continue;
    int np = -1;
    if (i > 0) {
      np = new_id[node_parent[(long long)b * cap + i]];
      if (np < 0) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);   // kept set not closed under parents
    }
    parent_out[(long long)b * t_max + ni] = np;
    tok_out[(long long)b * t_max + ni] = i > 0 ? node_tok[(long long)b * cap + i] : -1;
    if (kept_out) kept_out[(long long)b * t_max + ni] = i;
  }
}

}  // namespace

}  // namespace twig

using namespace twig;

extern "C" twig_status tree_reset(int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                                  int32_t batch, void *stream) {
  if (!node_tok || !node_parent || !node_score) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0) return TWIG_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // node 0 of every request: token -1, parent -1, score 0 (the other entries are written before they are read)
  if (cudaMemset2DAsync(node_tok, (size_t)cap * 4, 0xff, 4, batch, st) != cudaSuccess) return TWIG_ERR_CUDA;
  if (cudaMemset2DAsync(node_parent, (size_t)cap * 4, 0xff, 4, batch, st) != cudaSuccess) return TWIG_ERR_CUDA;
  if (cudaMemset2DAsync(node_score, (size_t)cap * 4, 0, 4, batch, st) != cudaSuccess) return TWIG_ERR_CUDA;
  return TWIG_OK;
}

extern "C" twig_status tree_expand_level(const void *logits, int32_t logits_fp32, int64_t row_stride,
                                         int32_t vocab, int32_t rows, const int32_t *src_node, int32_t n_children,
                                         int32_t level_base, int32_t *node_tok, int32_t *node_parent,
                                         float *node_score, int32_t cap, int32_t batch, int32_t *dev_status,
                                         void *stream) {
  if (!logits || !src_node || !node_tok || !node_parent || !node_score) return TWIG_ERR_NULL;
  if (vocab <= 0 || rows <= 0 || batch <= 0 || cap <= 0 || level_base <= 0 || row_stride < vocab) return TWIG_ERR_SHAPE;
  if (n_children <= 0 || n_children > kMaxE || n_children > vocab) return TWIG_ERR_UNSUPPORTED;
  if (batch > TWIG_MAX_BATCH || rows > 65535) return TWIG_ERR_UNSUPPORTED;
  if (level_base + (long long)rows * n_children > cap) return TWIG_ERR_SHAPE;
  const int esz = logits_fp32 ? 4 : 2;
  if (!aligned16(logits) || (row_stride * esz) % 16) return TWIG_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dim3 grid(rows, batch);
  // the row is staged in shared memory when it fits (else the selection rounds re-read it through L2)
  const size_t row_bytes = ((size_t)vocab * esz + 15) & ~(size_t)15;
  const int staged = row_bytes <= 200 * 1024;
  const size_t smem = staged ? row_bytes : 0;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_expand_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(tree_expand_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  if (logits_fp32)
    tree_expand_kernel<true><<<grid, kTopThreads, smem, st>>>(logits, row_stride, vocab, rows, src_node, n_children,
        level_base, cap, staged, node_tok, node_parent, node_score, dev_status);
  else
    tree_expand_kernel<false><<<grid, kTopThreads, smem, st>>>(logits, row_stride, vocab, rows, src_node, n_children,
        level_base, cap, staged, node_tok, node_parent, node_score, dev_status);
  return launch_status();
}

static twig_status launch_select(const float *node_score, const int32_t *node_tok, const int32_t *node_parent,
                                 int cap, int lo, int hi, int take, int *sel_out, int sel_stride, int *parent_out,
                                 int *tok_out, int *n_nodes_out, int *kept_out, int t_max, int batch,
                                 int *dev_status, cudaStream_t st) {
  const size_t smem = (size_t)cap * 8;
  if (smem > 48 * 1024) return TWIG_ERR_UNSUPPORTED;
  tree_select_kernel<<<batch, kSelThreads, smem, st>>>(node_score, node_tok, node_parent, cap, lo, hi, take, sel_out,
                                                       sel_stride, parent_out, tok_out, n_nodes_out, kept_out, t_max,
                                                       dev_status);
  return launch_status();
}

extern "C" twig_status tree_select_expansion(const float *node_score, int32_t cap, int32_t level_lo, int32_t level_hi,
                                             int32_t n_select, int32_t *expand_node, int32_t batch,
                                             int32_t *dev_status, void *stream) {
  if (!node_score || !expand_node) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0 || n_select <= 0 || level_lo < 0 || level_hi <= level_lo || level_hi > cap)
    return TWIG_ERR_SHAPE;
  if (batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (n_select > level_hi - level_lo) return TWIG_ERR_SHAPE;     // every expansion row gets a node
  return launch_select(node_score, nullptr, nullptr, cap, level_lo, level_hi, n_select, expand_node, n_select, nullptr,
                       nullptr, nullptr, nullptr, 0, batch, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" twig_status tree_finalize(const int32_t *node_tok, const int32_t *node_parent, const float *node_score,
                                     int32_t cap, int32_t n_built, int32_t n_max, int32_t *parent, int32_t *draft_tok,
                                     int32_t *n_nodes, int32_t *kept_node, int32_t t_max, int32_t batch,
                                     int32_t *dev_status, void *stream) {
  if (!node_tok || !node_parent || !node_score || !parent || !draft_tok || !n_nodes) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0 || n_built <= 0 || n_built > cap || n_max <= 0 || t_max <= 0) return TWIG_ERR_SHAPE;
  if (n_max > t_max || t_max > TWIG_MAX_NODES || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  return launch_select(node_score, node_tok, node_parent, cap, 1, n_built, n_max - 1, nullptr, 0, parent, draft_tok,
                       n_nodes, kept_node, t_max, batch, dev_status, static_cast<cudaStream_t>(stream));
}
