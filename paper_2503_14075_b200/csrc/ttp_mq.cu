// Multi-query pruning guide of Eq. 3: the attention that the textual tokens after the image pay to
// every visual token, summed over those tokens and averaged over heads,
//   a[m] = (1/H) sum_h sum_i softmax_{j <= t_i}(q_i . k_j / sqrt(d))[vis_start + m],
// t_i = vis_start + n_vis + i the prompt position of text token i.  Unlike the single-query score
// this is an N x L attention-map reduction: S = Q_text K^T runs on tensor cores (bf16
// mma.sync.m16n8k16, fp32 accumulation).  A thread-block cluster owns 64 query rows of one head and
// walks the keys twice, its CTAs sharing the key tiles: once for the rows' softmax statistics
// (max, sum; exchanged through distributed shared memory), once more over the visual span for
// the normalised probabilities, whose column sums go to the block's own slice of the scratch;
// a second kernel adds the slices in a fixed order, so the result does not depend on scheduling.
#include <cooperative_groups.h>

#include "tree_attn.cuh"

namespace cg = cooperative_groups;

namespace twig {

namespace {

constexpr int kMqRows = 64;       // query rows per CTA (4 warps x 16)
constexpr int kMqKeys = 64;       // keys per tile
constexpr int kMqThreads = 128;

// [rows x D] bf16 tile as D/64 panels of 128-byte rows; 16-byte chunks XORed with the row
__device__ __forceinline__ uint32_t mq_off(int r, int c) {
  return (uint32_t)((c >> 3) * 64 * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kMqThreads)
ttp_mq_partial_kernel(const __nv_bfloat16 *__restrict__ q_text, int n_text_max,
                      const __nv_bfloat16 *__restrict__ k, long long ksb, long long ksh, long long ksp,
                      int k_max_len, const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                      const int *__restrict__ n_vis, int n_q_heads, int group, float scale_log2,
                      float *__restrict__ partial, int m_max, int *dev_status) {
  constexpr int CPR = D / 8, KS = D / 16, NT = kMqKeys / 8;
  constexpr int TILE_BYTES = 64 * D * 2;
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ float s_col[4][kMqKeys];
  __shared__ float2 s_ml[8][kMqRows];            // (max, sum) of every row from every CTA of the cluster

  cg::cluster_group cluster = cg::this_cluster();
  const int n_splits = cluster.num_blocks(), split = cluster.block_rank();
  const int qb = blockIdx.x / n_splits, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b];
  const int n_text = lp - vs - nv;
  if (lp < 0 || lp > k_max_len || vs < 0 || nv < 0 || nv > m_max || n_text < 0 || n_text > n_text_max) {
    if (tid == 0 && qb == 0 && h == 0) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
    return;
  }
  const int row0 = qb * kMqRows;
  if (row0 >= n_text || nv == 0) return;          // (the reduction reads only the blocks that exist)
  const int rows = min(kMqRows, n_text - row0);
  const int t_first = vs + nv + row0;             // prompt position of this block's first query

  const uint32_t q_s = smem_u32(smem), k_s = q_s + TILE_BYTES;
  const __nv_bfloat16 *qsrc = q_text + (((long long)b * n_q_heads + h) * n_text_max + row0) * D;
  const __nv_bfloat16 *ksrc = k + b * ksb + (h / group) * ksh;

  for (int cid = tid; cid < kMqRows * CPR; cid += kMqThreads) {       // Q tile; rows past the last are zero
    const int r = cid / CPR, c = cid % CPR;
    cp_async_16(q_s + mq_off(r, c), qsrc + (long long)(r < rows ? r : 0) * D + c * 8, r < rows);
  }
  auto load_keys = [&](int t, int stage) {                            // keys 64 t .. 64 t + 63, zero past the prompt
    for (int cid = tid; cid < kMqKeys * CPR; cid += kMqThreads) {
      const int r = cid / CPR, c = cid % CPR;
      const int j = t * kMqKeys + r;
      cp_async_16(k_s + stage * TILE_BYTES + mq_off(r, c), ksrc + (long long)(j < lp ? j : 0) * ksp + c * 8, j < lp);
    }
  };

  const int gq = lane >> 2, tq = lane & 3;
  const int r_lo = warp * 16 + gq, r_hi = r_lo + 8;
  // last key each of this thread's two rows may see (its own position); -1 for rows past the last
  const int see_lo = r_lo < rows ? t_first + r_lo : -1, see_hi = r_hi < rows ? t_first + r_hi : -1;
  const uint32_t q_frag = q_s + (warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * 128;
  const int sw = lane & 7;
  uint32_t qf[KS][4];                  // this warp's Q fragments: the same for every key tile

  // S = Q K^T of this warp's 16 rows against the 64 keys of a stage, scaled into the exp2 domain
  // and masked (causal; keys past the prompt)
  auto scores_of = [&](int t, int stage, float (&s)[NT][4]) {
    const uint32_t kst = k_s + stage * TILE_BYTES;
#pragma unroll
    for (int i = 0; i < NT; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t kb[4];
        const int key = np * 16 + (lane & 7) + (lane >> 4) * 8;
        ldsm_x4(kst + mq_off(key, ks * 2 + ((lane >> 3) & 1)), kb);
        mma_bf16(s[2 * np], qf[ks], kb[0], kb[1]);
        mma_bf16(s[2 * np + 1], qf[ks], kb[2], kb[3]);
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = t * kMqKeys + nt * 8 + tq * 2 + (e & 1);
        s[nt][e] = j <= ((e & 2) ? see_hi : see_lo) ? s[nt][e] * scale_log2 : -INFINITY;
      }
  };

  // ---- pass 1: running maximum and sum of every row over its causal span ----
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const int n_t1 = (t_first + rows - 1) / kMqKeys + 1;        // tiles up to the last query's own position
  const int per1 = (n_t1 + n_splits - 1) / n_splits;
  const int t_begin1 = split * per1, t_end1 = min(n_t1, t_begin1 + per1);     // this CTA's share
  if (t_begin1 < t_end1) load_keys(t_begin1, 0);
  cp_async_commit();                                          // (this group also carries Q)
  cp_async_wait<0>();
  __syncthreads();
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const int c = ks * 2 + (lane >> 4);
    ldsm_x4(q_frag + (c >> 3) * 64 * 128 + (((c & 7) ^ sw) << 4), qf[ks]);
  }
  for (int t = t_begin1; t < t_end1; ++t) {
    const int it = t - t_begin1;
    if (t + 1 < t_end1) load_keys(t + 1, (it + 1) & 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    float s[NT][4];
    scores_of(t, it & 1, s);
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float use_lo = mn_lo == -INFINITY ? 0.f : mn_lo, use_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      sum_lo += fast_exp2(s[nt][0] - use_lo) + fast_exp2(s[nt][1] - use_lo);
      sum_hi += fast_exp2(s[nt][2] - use_hi) + fast_exp2(s[nt][3] - use_hi);
    }
    l_lo = l_lo * fast_exp2(m_lo - use_lo) + sum_lo;
    l_hi = l_hi * fast_exp2(m_hi - use_hi) + sum_hi;
    m_lo = mn_lo;
    m_hi = mn_hi;
    __syncthreads();                    // every warp is done with this stage before it is refilled
  }
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  // every CTA of the cluster tells every other its rows' (max, sum); then all hold the same totals
  if (n_splits > 1) {
    if (tq == 0) {
      for (int c = 0; c < n_splits; ++c) {
        float2 *dst = cluster.map_shared_rank(&s_ml[split][0], c);
        dst[r_lo] = make_float2(m_lo, l_lo);
        dst[r_hi] = make_float2(m_hi, l_hi);
      }
    }
    cluster.sync();
    float M_lo = -INFINITY, M_hi = -INFINITY;
    for (int c = 0; c < n_splits; ++c) {
      M_lo = fmaxf(M_lo, s_ml[c][r_lo].x);
      M_hi = fmaxf(M_hi, s_ml[c][r_hi].x);
    }
    const float U_lo = M_lo == -INFINITY ? 0.f : M_lo, U_hi = M_hi == -INFINITY ? 0.f : M_hi;
    float L_lo = 0.f, L_hi = 0.f;
    for (int c = 0; c < n_splits; ++c) {          // index order: the same sum in every CTA
      L_lo += s_ml[c][r_lo].y * fast_exp2(s_ml[c][r_lo].x - U_lo);
      L_hi += s_ml[c][r_hi].y * fast_exp2(s_ml[c][r_hi].x - U_hi);
    }
    m_lo = M_lo;
    m_hi = M_hi;
    l_lo = L_lo;
    l_hi = L_hi;
  }
  const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
  const float use_lo = m_lo == -INFINITY ? 0.f : m_lo, use_hi = m_hi == -INFINITY ? 0.f : m_hi;

  // ---- pass 2: normalised probabilities over the visual span, summed down the 64 rows ----
  float *out = partial + (((long long)b * n_q_heads + h) * (gridDim.x / n_splits) + qb) * m_max;
  const int t_vis0 = vs / kMqKeys, n_t2 = (vs + nv - 1) / kMqKeys + 1 - t_vis0;
  const int per2 = (n_t2 + n_splits - 1) / n_splits;
  const int t_begin2 = t_vis0 + split * per2, t_end2 = min(t_vis0 + n_t2, t_begin2 + per2);
  if (t_begin2 < t_end2) load_keys(t_begin2, 0);
  cp_async_commit();
  for (int t = t_begin2; t < t_end2; ++t) {
    const int it = t - t_begin2;
    if (t + 1 < t_end2) load_keys(t + 1, (it + 1) & 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    float s[NT][4];
    scores_of(t, it & 1, s);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float c0 = fast_exp2(s[nt][0] - use_lo) * inv_lo + fast_exp2(s[nt][2] - use_hi) * inv_hi;
      float c1 = fast_exp2(s[nt][1] - use_lo) * inv_lo + fast_exp2(s[nt][3] - use_hi) * inv_hi;
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {          // down the warp's 16 rows (lanes that share tq)
        c0 += __shfl_xor_sync(0xffffffffu, c0, o);
        c1 += __shfl_xor_sync(0xffffffffu, c1, o);
      }
      if (gq == 0) {
        s_col[warp][nt * 8 + tq * 2] = c0;
        s_col[warp][nt * 8 + tq * 2 + 1] = c1;
      }
    }
    __syncthreads();
    if (tid < kMqKeys) {
      const int m = t * kMqKeys + tid - vs;
      if (m >= 0 && m < nv) out[m] = (s_col[0][tid] + s_col[1][tid]) + (s_col[2][tid] + s_col[3][tid]);
    }
    __syncthreads();                    // s_col and this stage are free again
  }
  cp_async_wait<0>();
}

// scores[b, m] = (1/H) sum over heads and query blocks, in index order; 0 past n_vis
__global__ void ttp_mq_reduce_kernel(const float *__restrict__ partial, int n_blocks_max, int n_q_heads,
                                     int n_text_max, const int *__restrict__ prefix_len,
                                     const int *__restrict__ vis_start, const int *__restrict__ n_vis,
                                     int k_max_len, float *__restrict__ scores, int m_max) {
  const int b = blockIdx.y, m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= m_max) return;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b];
  const int n_text = lp - vs - nv;
  float acc = 0.f;
  if (lp >= 0 && lp <= k_max_len && vs >= 0 && nv >= 0 && nv <= m_max && n_text > 0 && n_text <= n_text_max && m < nv) {
    const int nqb = (n_text + kMqRows - 1) / kMqRows;
    for (int h = 0; h < n_q_heads; ++h)
      for (int qb = 0; qb < nqb; ++qb)
        acc += partial[(((long long)b * n_q_heads + h) * n_blocks_max + qb) * m_max + m];
    acc /= (float)n_q_heads;
  }
  scores[(long long)b * m_max + m] = acc;
}

}  // namespace

}  // namespace twig

using namespace twig;

extern "C" size_t ttp_multiquery_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t n_text_max, int32_t m_max) {
  if (batch <= 0 || n_q_heads <= 0 || n_text_max <= 0 || m_max <= 0) return 0;
  return (size_t)batch * n_q_heads * ((n_text_max + kMqRows - 1) / kMqRows) * m_max * sizeof(float);
}

extern "C" twig_status ttp_score_multiquery(const void *q_text, int32_t n_text_max, const void *twig_k,
                                            int64_t k_stride_batch, int64_t k_stride_head, int64_t k_stride_pos,
                                            int32_t k_max_len, const int32_t *prefix_len, const int32_t *vis_start,
                                            const int32_t *n_vis, int32_t batch, int32_t n_q_heads,
                                            int32_t n_kv_heads, int32_t head_dim, float softmax_scale,
                                            float *scores, int32_t m_max, int32_t *dev_status, void *ws,
                                            size_t ws_bytes, void *stream) {
  if (!q_text || !twig_k || !prefix_len || !vis_start || !n_vis || !scores || !ws) return TWIG_ERR_NULL;
  if (batch <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || k_max_len <= 0 || m_max <= 0 || n_text_max <= 0)
    return TWIG_ERR_SHAPE;
  if (n_q_heads % n_kv_heads || k_stride_pos < head_dim) return TWIG_ERR_SHAPE;
  if (head_dim != 64 && head_dim != 128) return TWIG_ERR_UNSUPPORTED;
  if (m_max > TWIG_MAX_VISUAL || batch > TWIG_MAX_BATCH || n_q_heads > 65535) return TWIG_ERR_UNSUPPORTED;
  if (!aligned16(q_text) || !aligned16(twig_k) || !aligned16(ws) ||
      ((k_stride_batch | k_stride_head | k_stride_pos) & 7))
    return TWIG_ERR_ALIGN;
  if (ws_bytes < ttp_multiquery_workspace_bytes(batch, n_q_heads, n_text_max, m_max)) return TWIG_ERR_WORKSPACE;
  const int n_blocks = (n_text_max + kMqRows - 1) / kMqRows;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.f / sqrtf((float)head_dim);
  const float scale_log2 = scale * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto q = static_cast<const __nv_bfloat16 *>(q_text);
  auto k = static_cast<const __nv_bfloat16 *>(twig_k);
  float *partial = static_cast<float *>(ws);
  const int group = n_q_heads / n_kv_heads;
  // key tiles are shared by the CTAs of a cluster: as many as still fit one wave (4 CTAs per SM)
  int n_splits = 8;
  while (n_splits > 1 && (long long)n_blocks * n_q_heads * batch * n_splits > 4 * 148) n_splits >>= 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_blocks * n_splits, n_q_heads, batch);
  cfg.blockDim = dim3(kMqThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t err;
  if (head_dim == 128) {
    constexpr int smem = 3 * 64 * 128 * 2;
    static bool attr_set = false;
    if (!attr_set) {
      if (cudaFuncSetAttribute(ttp_mq_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return TWIG_ERR_CUDA;
      attr_set = true;
    }
    cfg.dynamicSmemBytes = smem;
    err = cudaLaunchKernelEx(&cfg, ttp_mq_partial_kernel<128>, q, n_text_max, k, (long long)k_stride_batch,
                             (long long)k_stride_head, (long long)k_stride_pos, k_max_len, prefix_len, vis_start, n_vis,
                             n_q_heads, group, scale_log2, partial, m_max, dev_status);
  } else {
    cfg.dynamicSmemBytes = 3 * 64 * 64 * 2;
    err = cudaLaunchKernelEx(&cfg, ttp_mq_partial_kernel<64>, q, n_text_max, k, (long long)k_stride_batch,
                             (long long)k_stride_head, (long long)k_stride_pos, k_max_len, prefix_len, vis_start, n_vis,
                             n_q_heads, group, scale_log2, partial, m_max, dev_status);
  }
  if (err != cudaSuccess) return TWIG_ERR_CUDA;
  if (cudaGetLastError() != cudaSuccess) return TWIG_ERR_CUDA;
  ttp_mq_reduce_kernel<<<dim3((m_max + 255) / 256, batch), 256, 0, st>>>(partial, n_blocks, n_q_heads, n_text_max,
      prefix_len, vis_start, n_vis, k_max_len, scores, m_max);
  return launch_status();
}
