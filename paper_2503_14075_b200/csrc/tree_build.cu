// Draft-side token tree of tree-based self-speculative decoding (Sec. 4.3; Appendix, "Tree-based
// self-speculative decoding"): level by level, every node selected for expansion gets its E most
// probable next tokens as children; the K best nodes of a level are expanded at the next; at the end
// the tree is cut to N_max nodes.  A node's score is the log of the joint probability of its path.
// The draft model itself runs between these calls: its logits are inputs.
//
// Tree state per request (capacity `cap` nodes, node 0 = root): token, parent, score, all in
// creation order (a parent always precedes its children).
//
// A level costs one launch: the expansion kernel's CTAs of a request take a ticket when their
// children are written, and the last of them runs the step that consumes the level (the choice of the
// next level's expansion nodes, or the final pruning).  The two steps also exist as launches of
// their own.
#include "twig_common.cuh"

namespace twig {

namespace {

constexpr int kTopThreads = 512;
constexpr int kMaxE = 16;            // children per expanded node
constexpr int kMaxCand = 1024;       // entries at or above the threshold that the short list holds
constexpr int kSelThreads = 256;
constexpr int kBatchLoads = 8;       // 16-byte loads a thread has in flight while the row streams in

// (value, index) order of the top lists: larger value first, equal values: lower index first
__device__ __forceinline__ bool comes_first(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

// What follows a level: the ranking of nodes lo..hi-1 by (score desc, id asc), of which the first
// `take` are kept.
//  * expansion mode (parent_out == nullptr): their ids, ascending, to sel_out[b, 0..take) (-1 padded);
//  * final mode: the root and the selected nodes are renumbered in creation order and written as
//    parent_out / tok_out [b, t_max] with n_nodes_out[b]; kept_out[b, i] = the old id of new node i.
struct SelectArgs {
  int lo, hi, take;
  int *sel_out;
  int sel_stride;
  int *parent_out, *tok_out, *n_nodes_out, *kept_out;
  int t_max;
};

// Runs in one CTA (all of its threads) for request b.  `work` holds 2*cap words of shared memory.
// The tree state is read through L2: inside the expansion kernel the nodes of the new level were
// written by other CTAs a moment ago, and a line of this SM's L1 may predate them.
__device__ void select_nodes(const SelectArgs &a, int b, int cap, const float *node_score, const int *node_tok,
                             const int *node_parent, unsigned char *work, int *dev_status) {
  __shared__ int s_warp_kept[32];
  float *sc = reinterpret_cast<float *>(work);                     // [hi]
  int *new_id = reinterpret_cast<int *>(work) + cap;               // [hi]: position among the kept, or -1
  const int tid = threadIdx.x, nt = blockDim.x;
  const int lo = a.lo, hi = a.hi;
  const float *score = node_score + (long long)b * cap;
  for (int i = tid; i < hi; i += nt) {
    sc[i] = __ldcg(score + i);
    new_id[i] = -1;
  }
  __syncthreads();
  const bool final_mode = a.parent_out != nullptr;
  for (int i = lo + tid; i < hi; i += nt) {
    // rank in the (score desc, id asc) order: older nodes with a score at least as high, younger
    // nodes with a higher one
    int rank = 0;
    const float v = sc[i];
#pragma unroll 4
    for (int j = lo; j < i; ++j) rank += sc[j] >= v ? 1 : 0;
#pragma unroll 4
    for (int j = i + 1; j < hi; ++j) rank += sc[j] > v ? 1 : 0;
    if (rank < a.take) new_id[i] = 0;                              // selected (position follows)
  }
  if (final_mode && tid == 0) new_id[0] = 0;                       // the root is always kept
  __syncthreads();
  // positions among the kept, in id order: ballots inside a warp, warp totals across the CTA
  const int from = final_mode ? 0 : lo;
  const int lane = tid & 31, warp = tid >> 5, n_warps = (nt + 31) >> 5;
  int total = 0;                                                   // (the same in every thread)
  for (int i0 = from; i0 < hi; i0 += nt) {
    const int i = i0 + tid;
    const bool kept = i < hi && new_id[i] >= 0;
    const unsigned votes = __ballot_sync(0xffffffffu, kept);
    if (lane == 0) s_warp_kept[warp] = __popc(votes);
    __syncthreads();
    int before = 0, all = 0;
    for (int w = 0; w < n_warps; ++w) {
      const int c = s_warp_kept[w];
      before += w < warp ? c : 0;
      all += c;
    }
    if (kept) new_id[i] = total + before + __popc(votes & ((1u << lane) - 1u));
    total += all;
    __syncthreads();
  }
  if (!final_mode) {
    for (int k = tid; k < a.sel_stride; k += nt) a.sel_out[(long long)b * a.sel_stride + k] = -1;
    __syncthreads();
    for (int i = lo + tid; i < hi; i += nt)
      if (new_id[i] >= 0 && new_id[i] < a.sel_stride) a.sel_out[(long long)b * a.sel_stride + new_id[i]] = i;
    return;
  }
  if (tid == 0) a.n_nodes_out[b] = total;
  const int t_max = a.t_max;
  for (int k = total + tid; k < t_max; k += nt) {
    a.parent_out[(long long)b * t_max + k] = -1;
    a.tok_out[(long long)b * t_max + k] = 0;
    if (a.kept_out) a.kept_out[(long long)b * t_max + k] = -1;
  }
  for (int i = tid; i < hi; i += nt) {
    const int ni = new_id[i];
    if (ni < 0) continue;
    int np = -1;
    if (i > 0) {
      const int par = __ldcg(node_parent + (long long)b * cap + i);
      np = par >= 0 && par < i ? new_id[par] : -1;
      if (np < 0) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);   // not a tree, or the kept set is not closed under parents
    }
    a.parent_out[(long long)b * t_max + ni] = np;
    a.tok_out[(long long)b * t_max + ni] = i > 0 ? __ldcg(node_tok + (long long)b * cap + i) : -1;
    if (a.kept_out) a.kept_out[(long long)b * t_max + ni] = i;
  }
}

// The selection as a launch of its own: one CTA per request.
__global__ void __launch_bounds__(kSelThreads)
tree_select_kernel(const float *node_score, const int *node_tok, const int *node_parent, int cap, SelectArgs a,
                   int *dev_status) {
  extern __shared__ __align__(16) unsigned char sel_smem[];
  grid_dependency_sync();
  select_nodes(a, blockIdx.x, cap, node_score, node_tok, node_parent, sel_smem, dev_status);
}

// One CTA per (expansion slot, request): log-sum-exp of the row and its E largest logits.
// The row is read from global memory once, eight 16-byte loads per thread in flight, and kept in
// shared memory (when it fits).  The E-th largest of the half-warp groups' maxima is a lower bound of
// the E-th largest logit, so one more pass over the staged row collects the few entries at or above
// it into a short list, which is ranked by counting (every candidate counts the candidates that come
// before it in the (value, index) order).  If the list overflows (e.g. a row of equal logits), E
// selection rounds run over the whole row instead: round e finds the best entry that comes strictly
// after round e-1's winner, so nothing has to be marked as taken.
// Writes the children's tokens, parents and scores; `row_s` is free again on return.  The row's
// address does not depend on the source node u, so u is looked at only once the row's loads are in
// flight; a row whose u turns out to be unusable is read for nothing.
template <bool FP32>
__device__ __forceinline__ void expand_row(const unsigned char *__restrict__ row, int vocab, int E, int staged,
                                           unsigned char *row_s, int u, int level_base, long long base, int first,
                                           int *node_tok, int *node_parent, float *node_score) {
  constexpr int EPC = FP32 ? 4 : 8;
  __shared__ float s_v[kTopThreads / 32];
  __shared__ int s_i[kTopThreads / 32];
  __shared__ float s_m[kTopThreads / 32], s_s[kTopThreads / 32];
  __shared__ float s_top_v[kMaxE];
  __shared__ int s_top_i[kMaxE];
  __shared__ float s_tmax[kTopThreads / 16];       // maxima of the half-warp groups
  __shared__ float s_cand_v[kMaxCand];
  __shared__ int s_cand_i[kMaxCand];
  __shared__ int s_n_cand;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    const float ref = nm == -INFINITY ? 0.f : nm;   // (only -inf so far: every term is exp(-inf) = 0)
    s = s * __expf(m - ref) + __expf(v - ref);      // (m = -inf: s is 0 and exp(-inf) = 0)
    m = nm;
  };
  for (int c0 = tid; c0 < chunks; c0 += kTopThreads * kBatchLoads) {
    uint4 w[kBatchLoads];
#pragma unroll
    for (int q = 0; q < kBatchLoads; ++q) {
      const int c = c0 + q * kTopThreads;
      if (c < chunks) w[q] = ld_nc_16(row + (long long)c * 16);
    }
#pragma unroll
    for (int q = 0; q < kBatchLoads; ++q) {
      const int c = c0 + q * kTopThreads;
      if (c >= chunks) break;
      if (staged) *reinterpret_cast<uint4 *>(row_s + (size_t)c * 16) = w[q];
      float v[8];
      unpack(w[q], v);
      float cm = v[0];
#pragma unroll
      for (int k = 1; k < EPC; ++k) cm = fmaxf(cm, v[k]);
      t_max = fmaxf(t_max, cm);
      const float nm = fmaxf(m, cm);
      const float ref = nm == -INFINITY ? 0.f : nm;
      float acc = s * __expf(m - ref);
#pragma unroll
      for (int k = 0; k < EPC; ++k) acc += __expf(v[k] - ref);
      s = acc;
      m = nm;
    }
  }
  for (int i = chunks * EPC + tid; i < vocab; i += kTopThreads) {
    const float v = element(row, i);
    if (staged) {
      if (FP32) reinterpret_cast<float *>(row_s)[i] = v;
      else reinterpret_cast<__nv_bfloat16 *>(row_s)[i] = reinterpret_cast<const __nv_bfloat16 *>(row)[i];
    }
    soft(v);
  }
  // (the root's score is 0 by definition; its entry may be written by another CTA of this launch)
  const bool usable = u >= 0 && u < level_base;
  const float parent_score = usable && u > 0 ? __ldcg(node_score + base + u) : 0.f;
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

  // ---- the short list ranked by counting (indices are distinct, so ranks are) ----
  if (short_list) {
    for (int j = tid; j < n_cand; j += kTopThreads) {
      const float v = s_cand_v[j];
      const int i = s_cand_i[j];
      int rank = 0;
      for (int q = 0; q < n_cand; ++q) rank += comes_first(s_cand_v[q], s_cand_i[q], v, i) ? 1 : 0;
      if (rank < E) {
        s_top_v[rank] = v;
        s_top_i[rank] = i;
      }
    }
    __syncthreads();
  }
  // ---- or E rounds over the whole row ----
  float pv = INFINITY;                     // previous winner; every finite logit comes after (+inf, -1)
  int pi = -1;
  for (int e = 0; e < (short_list ? 0 : E); ++e) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    auto offer = [&](float v, int i) {
      const bool after_prev = pv > v || (pv == v && pi < i);
      if (after_prev && comes_first(v, i, bv, bi)) {
        bv = v;
        bi = i;
      }
    };
    for (int c = tid; c < chunks; c += kTopThreads) {
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
  if (tid < E && (usable || u < 0)) {        // an unused slot's children: nobody selects them
    const long long at = base + first + tid;
    node_tok[at] = usable ? s_top_i[tid] : 0;
    node_parent[at] = usable ? u : -1;
    node_score[at] = usable ? parent_score + (s_top_v[tid] - lse) : -INFINITY;
  }
  __syncthreads();                         // (the caller may reuse row_s)
}

// Grid (rows, batch).  `ticket` (one counter per request, zero before the launch and zero again after
// it) selects the one-launch form: the request's last CTA to finish runs `tail`.
template <bool FP32>
__global__ void __launch_bounds__(kTopThreads, 2)
tree_expand_kernel(const void *__restrict__ logits, long long row_stride, int vocab, int rows,
                   const int *__restrict__ src_node, int E, int level_base, int cap, int staged, int *node_tok,
                   int *node_parent, float *node_score, int *ticket, SelectArgs tail, int *dev_status) {
  extern __shared__ __align__(16) unsigned char row_s[];
  __shared__ int s_last;
  grid_dependency_sync();
  const int r = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int u = src_node[(long long)b * rows + r];
  const int first = level_base + r * E;
  const long long base = (long long)b * cap;
  if (level_base == 1 && r == 0 && tid == 0) {             // the first level also writes the root
    node_tok[base] = -1;
    node_parent[base] = -1;
    node_score[base] = 0.f;
  }
  if (first + E <= cap) {
    const unsigned char *row = static_cast<const unsigned char *>(logits) +
                               ((long long)b * rows + r) * row_stride * (FP32 ? 4 : 2);
    expand_row<FP32>(row, vocab, E, staged, row_s, u, level_base, base, first, node_tok, node_parent, node_score);
  }
  if ((first + E > cap || u >= level_base) && tid == 0) flag_status(dev_status, b, TWIG_DEV_BAD_TREE);
  if (!ticket) return;
  // ---- the last CTA of the request to get here has every node of the level in view (a request
  // with one row has one CTA; expand_row ended with a CTA-wide barrier) ----
  if (rows > 1) {
    if (tid == 0) {
      __threadfence();
      const int last = atomicAdd(ticket + b, 1) == rows - 1 ? 1 : 0;
      if (last) {
        __threadfence();
        ticket[b] = 0;
      }
      s_last = last;
    }
    __syncthreads();
    if (!s_last) return;
  }
  select_nodes(tail, b, cap, node_score, node_tok, node_parent, row_s, dev_status);
}

// Node 0 of every request: token -1, parent -1, score 0.
__global__ void tree_reset_kernel(int *node_tok, int *node_parent, float *node_score, int cap, int batch) {
  grid_dependency_sync();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  node_tok[(long long)b * cap] = -1;
  node_parent[(long long)b * cap] = -1;
  node_score[(long long)b * cap] = 0.f;
}

}  // namespace

}  // namespace twig

using namespace twig;


extern "C" twig_status tree_reset(int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                                  int32_t batch, void *stream) {
  if (!node_tok || !node_parent || !node_score) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0) return TWIG_ERR_SHAPE;
  PdlLaunch L(dim3((batch + 127) / 128), dim3(128), 0, static_cast<cudaStream_t>(stream));
  if (cudaLaunchKernelEx(&L.cfg, tree_reset_kernel, node_tok, node_parent, node_score, cap, batch) != cudaSuccess)
    return TWIG_ERR_CUDA;
  return launch_status();
}

namespace {

constexpr size_t kMaxStagedRow = 200 * 1024;     // a staged row and the static arrays fit one SM's shared memory
constexpr size_t kMaxSelectSmem = 48 * 1024;     // two words per node

twig_status check_expand(const void *logits, int logits_fp32, long long row_stride, int vocab, int rows,
                         const int *src_node, int n_children, int level_base, const int *node_tok,
                         const int *node_parent, const float *node_score, int cap, int batch) {
  if (!logits || !src_node || !node_tok || !node_parent || !node_score) return TWIG_ERR_NULL;
  if (vocab <= 0 || rows <= 0 || batch <= 0 || cap <= 0 || level_base <= 0 || row_stride < vocab) return TWIG_ERR_SHAPE;
  if (n_children <= 0 || n_children > kMaxE || n_children > vocab) return TWIG_ERR_UNSUPPORTED;
  if (batch > TWIG_MAX_BATCH || rows > 65535) return TWIG_ERR_UNSUPPORTED;
  if (level_base + (long long)rows * n_children > cap) return TWIG_ERR_SHAPE;
  const int esz = logits_fp32 ? 4 : 2;
  if (!aligned16(logits) || (row_stride * esz) % 16) return TWIG_ERR_ALIGN;
  return TWIG_OK;
}

// `ticket` == nullptr: the expansion alone.
twig_status launch_expand(const void *logits, int logits_fp32, long long row_stride, int vocab, int rows,
                          const int *src_node, int E, int level_base, int *node_tok, int *node_parent,
                          float *node_score, int cap, int batch, int *ticket, const SelectArgs &tail,
                          int *dev_status, cudaStream_t st) {
  const int esz = logits_fp32 ? 4 : 2;
  // the row is staged in shared memory when it fits (else the later passes re-read it through L2)
  const size_t row_bytes = ((size_t)vocab * esz + 15) & ~(size_t)15;
  const int staged = row_bytes <= kMaxStagedRow;
  size_t smem = staged ? row_bytes : 0;
  if (ticket && smem < (size_t)cap * 8) smem = (size_t)cap * 8;      // the tail's two words per node
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_expand_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxStagedRow) != cudaSuccess ||
        cudaFuncSetAttribute(tree_expand_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxStagedRow) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  PdlLaunch L(dim3(rows, batch), dim3(kTopThreads), smem, st);
  const cudaError_t err =
      logits_fp32 ? cudaLaunchKernelEx(&L.cfg, tree_expand_kernel<true>, logits, row_stride, vocab, rows, src_node, E,
                                       level_base, cap, staged, node_tok, node_parent, node_score, ticket, tail, dev_status)
                  : cudaLaunchKernelEx(&L.cfg, tree_expand_kernel<false>, logits, row_stride, vocab, rows, src_node, E,
                                       level_base, cap, staged, node_tok, node_parent, node_score, ticket, tail, dev_status);
  if (err != cudaSuccess) return TWIG_ERR_CUDA;
  return launch_status();
}

twig_status launch_select(const float *node_score, const int32_t *node_tok, const int32_t *node_parent, int cap,
                          const SelectArgs &a, int batch, int *dev_status, cudaStream_t st) {
  const size_t smem = (size_t)cap * 8;
  if (smem > kMaxSelectSmem) return TWIG_ERR_UNSUPPORTED;
  PdlLaunch L(dim3(batch), dim3(kSelThreads), smem, st);
  if (cudaLaunchKernelEx(&L.cfg, tree_select_kernel, node_score, node_tok, node_parent, cap, a, dev_status) != cudaSuccess)
    return TWIG_ERR_CUDA;
  return launch_status();
}

twig_status expansion_args(int cap, int level_lo, int level_hi, int n_select, int *expand_node, int batch, SelectArgs *a) {
  if (!expand_node) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0 || n_select <= 0 || level_lo < 0 || level_hi <= level_lo || level_hi > cap)
    return TWIG_ERR_SHAPE;
  if (batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (n_select > level_hi - level_lo) return TWIG_ERR_SHAPE;     // every expansion row gets a node
  *a = SelectArgs{level_lo, level_hi, n_select, expand_node, n_select, nullptr, nullptr, nullptr, nullptr, 0};
  return TWIG_OK;
}

twig_status final_args(int cap, int n_built, int n_max, int *parent, int *draft_tok, int *n_nodes, int *kept_node,
                       int t_max, int batch, SelectArgs *a) {
  if (!parent || !draft_tok || !n_nodes) return TWIG_ERR_NULL;
  if (cap <= 0 || batch <= 0 || n_built <= 0 || n_built > cap || n_max <= 0 || t_max <= 0) return TWIG_ERR_SHAPE;
  if (n_max > t_max || t_max > TWIG_MAX_NODES || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  *a = SelectArgs{1, n_built, n_max - 1, nullptr, 0, parent, draft_tok, n_nodes, kept_node, t_max};
  return TWIG_OK;
}

}  // namespace

extern "C" twig_status tree_expand_level(const void *logits, int32_t logits_fp32, int64_t row_stride,
                                         int32_t vocab, int32_t rows, const int32_t *src_node, int32_t n_children,
                                         int32_t level_base, int32_t *node_tok, int32_t *node_parent,
                                         float *node_score, int32_t cap, int32_t batch, int32_t *dev_status,
                                         void *stream) {
  const twig_status ok = check_expand(logits, logits_fp32, row_stride, vocab, rows, src_node, n_children, level_base,
                                      node_tok, node_parent, node_score, cap, batch);
  if (ok != TWIG_OK) return ok;
  return launch_expand(logits, logits_fp32, row_stride, vocab, rows, src_node, n_children, level_base, node_tok,
                       node_parent, node_score, cap, batch, nullptr, SelectArgs{}, dev_status,
                       static_cast<cudaStream_t>(stream));
}

extern "C" twig_status tree_select_expansion(const float *node_score, int32_t cap, int32_t level_lo, int32_t level_hi,
                                             int32_t n_select, int32_t *expand_node, int32_t batch,
                                             int32_t *dev_status, void *stream) {
  if (!node_score) return TWIG_ERR_NULL;
  SelectArgs a;
  const twig_status ok = expansion_args(cap, level_lo, level_hi, n_select, expand_node, batch, &a);
  if (ok != TWIG_OK) return ok;
  return launch_select(node_score, nullptr, nullptr, cap, a, batch, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" twig_status tree_finalize(const int32_t *node_tok, const int32_t *node_parent, const float *node_score,
                                     int32_t cap, int32_t n_built, int32_t n_max, int32_t *parent, int32_t *draft_tok,
                                     int32_t *n_nodes, int32_t *kept_node, int32_t t_max, int32_t batch,
                                     int32_t *dev_status, void *stream) {
  if (!node_tok || !node_parent || !node_score) return TWIG_ERR_NULL;
  SelectArgs a;
  const twig_status ok = final_args(cap, n_built, n_max, parent, draft_tok, n_nodes, kept_node, t_max, batch, &a);
  if (ok != TWIG_OK) return ok;
  return launch_select(node_score, node_tok, node_parent, cap, a, batch, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" twig_status tree_grow_level(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                                       int32_t rows, const int32_t *src_node, int32_t n_children, int32_t level_base,
                                       int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                                       int32_t batch, int32_t n_select, int32_t *expand_node, int32_t n_max,
                                       int32_t *parent, int32_t *draft_tok, int32_t *n_nodes, int32_t *kept_node,
                                       int32_t t_max, int32_t *ticket, int32_t *dev_status, void *stream) {
  twig_status ok = check_expand(logits, logits_fp32, row_stride, vocab, rows, src_node, n_children, level_base,
                                node_tok, node_parent, node_score, cap, batch);
  if (ok != TWIG_OK) return ok;
  if (!ticket) return TWIG_ERR_NULL;
  if ((size_t)cap * 8 > kMaxSelectSmem) return TWIG_ERR_UNSUPPORTED;
  const int level_hi = level_base + rows * n_children;
  SelectArgs a;
  ok = n_select > 0 ? expansion_args(cap, level_base, level_hi, n_select, expand_node, batch, &a)
                    : final_args(cap, level_hi, n_max, parent, draft_tok, n_nodes, kept_node, t_max, batch, &a);
  if (ok != TWIG_OK) return ok;
  return launch_expand(logits, logits_fp32, row_stride, vocab, rows, src_node, n_children, level_base, node_tok,
                       node_parent, node_score, cap, batch, ticket, a, dev_status, static_cast<cudaStream_t>(stream));
}
