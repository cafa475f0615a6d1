// Multi-query pruning guide of Eq. 3: the attention that the textual tokens after the image pay to
// every visual token, summed over those tokens and averaged over heads,
//   a[m] = (1/H) sum_h sum_i softmax_{j <= t_i}(q_i . k_j / sqrt(d))[vis_start + m],
// t_i = vis_start + n_vis + i the prompt position of text token i.  Unlike the single-query score
// this is an N x L attention-map reduction.  Three kernels, each launched so that it may be
// scheduled while its predecessor drains:
//   1. probabilities: a CTA takes 64 query rows of one head and one chunk of kChunk keys.  Q and the
//      chunk go to shared memory in the 128-byte-swizzled layout of the matrix descriptors, one
//      thread issues S = Q K^T (tcgen05.mma, M = 64, N = kChunk, fp32 in tensor memory), the four
//      warps read their 16 rows back, mask (causal), and write the chunk's row maxima and sums of
//      exponentials plus the exponentials themselves, relative to the chunk's row maximum, as fp16.
//      Every key is read once and every product and exponential is computed once.
//   2. column sums: a CTA merges the chunks' statistics of its 64 rows into the rows' softmax
//      denominators and adds up, down the rows, the stored exponentials of a few visual chunks, each
//      row weighted by exp2(chunk max - row max) / row sum.
//   3. the sum over heads and row blocks in index order, so that the result does not depend on
//      scheduling.
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>

#include "tcgen05_common.cuh"

namespace twig {

namespace {

constexpr int kMqRows = 64;        // query rows per CTA (one M = 64 accumulator; 16 rows per lane quadrant)
constexpr int kMqThreads = 256;     // two warps per lane quadrant of the accumulator: half of a chunk's columns each
constexpr int kChunk = 128;        // keys per CTA of the first kernel = fp32 columns of tensor memory
constexpr int kSumThreads = 256;
constexpr int kSumChunks = 4;      // visual chunks per CTA of the second kernel

// [rows x D] bf16 tile as D/64 panels of `panel_rows` 128-byte rows; 16-byte chunks XORed with the row
__device__ __forceinline__ uint32_t mq_off(int r, int c, int panel_rows) {
  return (uint32_t)((c >> 3) * panel_rows * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

struct MqLayout {
  int lp, vs, nv, n_text;
  bool ok;
};
__device__ __forceinline__ MqLayout mq_layout(const int *prefix_len, const int *vis_start, const int *n_vis, int b,
                                              int k_max_len, int m_max, int n_text_max) {
  MqLayout y;
  y.lp = prefix_len[b];
  y.vs = vis_start[b];
  y.nv = n_vis[b];
  y.n_text = y.lp - y.vs - y.nv;
  y.ok = y.lp >= 0 && y.lp <= k_max_len && y.vs >= 0 && y.nv >= 0 && y.nv <= m_max && y.n_text >= 0 &&
         y.n_text <= n_text_max;
  return y;
}

// Scratch: probabilities [item][chunk][64 rows][kChunk] fp16, statistics [item][chunk][64 rows]
// (max, sum), partial column sums [item][m_max]; item = (request, head, row block).
struct MqScratch {
  __half *probs;
  float2 *stats;
  float *partial;
};
inline size_t mq_probs_bytes(size_t items, int n_chunks) { return items * n_chunks * kMqRows * kChunk * sizeof(__half); }
inline size_t mq_stats_bytes(size_t items, int n_chunks) { return items * n_chunks * kMqRows * sizeof(float2); }
inline size_t mq_partial_bytes(size_t items, int m_max) { return ((items * m_max * sizeof(float)) + 15) & ~(size_t)15; }

// ---- 1. probabilities and per-chunk statistics ----
// grid (n_groups * n_row_blocks, heads, batch); blockIdx.x = row block * n_groups + group.  A CTA walks
// `chunks_per_cta` consecutive chunks of its item with Q loaded once and the key tiles double
// buffered: the loads of the next chunk are in flight while this chunk's product is read back.
template <int D, int NBUF>
__global__ void __launch_bounds__(kMqThreads)
ttp_mq_probs_kernel(const __nv_bfloat16 *__restrict__ q_text, int n_text_max,
                    const __nv_bfloat16 *__restrict__ k, long long ksb, long long ksh, long long ksp,
                    int k_max_len, const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                    const int *__restrict__ n_vis, int n_q_heads, int group, float scale_log2, int n_chunks,
                    int n_row_blocks, int n_groups, int chunks_per_cta, MqScratch ws, int m_max, int *dev_status) {
  constexpr int CPR = D / 8;                         // 16-byte pieces per row
  constexpr int Q_BYTES = kMqRows * D * 2;
  constexpr int K_BYTES = kChunk * D * 2;
  constexpr int P_PITCH = kChunk * 2 + 16;           // staged fp16 row (+16: rows start in different banks)
  extern __shared__ __align__(1024) unsigned char smem[];   // Q | NBUF key tiles | staged probabilities
  __shared__ __align__(8) unsigned long long s_bar[2];   // product into accumulator 0 / 1 complete
  __shared__ uint32_t s_tmem;
  __shared__ volatile int s_fail;
  __shared__ float s_xm[2][kMqRows], s_xl[kMqRows];      // what the two column halves tell each other

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = blockIdx.x % n_groups, qb = blockIdx.x / n_groups, h = blockIdx.y, b = blockIdx.z;
  grid_dependency_sync();
  const MqLayout y = mq_layout(prefix_len, vis_start, n_vis, b, k_max_len, m_max, n_text_max);
  if (!y.ok) {
    if (tid == 0 && blockIdx.x == 0 && h == 0) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
    return;
  }
  const int row0 = qb * kMqRows;
  if (row0 >= y.n_text || y.nv == 0) return;          // (the later stages read only what exists)
  const int rows = min(kMqRows, y.n_text - row0);
  const int t_first = y.vs + y.nv + row0;             // prompt position of this block's first query
  const int n_c = (t_first + rows - 1) / kChunk + 1;  // chunks that hold a key some row sees
  const int c_begin = grp * chunks_per_cta, c_end = min(n_c, c_begin + chunks_per_cta);
  if (c_begin >= c_end) return;

  if (tid == 0) {
    s_fail = 0;
    mbar_init(smem_u32(&s_bar[0]), 1);                // one tcgen05.commit per use
    mbar_init(smem_u32(&s_bar[1]), 1);
    mbar_init_fence_cluster();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(2 * kChunk) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  const uint32_t q_s = smem_u32(smem), k_s = q_s + Q_BYTES;
  const __nv_bfloat16 *qsrc = q_text + (((long long)b * n_q_heads + h) * n_text_max + row0) * D;
  const __nv_bfloat16 *ksrc = k + b * ksb + (h / group) * ksh;
  // a thread copies the same 16-byte piece of every RS-th row: RS is a multiple of 8, so the swizzle
  // term of its shared-memory offset is the same for all of them
  constexpr int RS = kMqThreads / CPR, SWEEPS = kChunk / RS;
  static_assert(RS % 8 == 0 && kChunk % RS == 0, "row sweeps");
  const int lr = tid / CPR, lc = tid % CPR;
  const uint32_t k_off0 = mq_off(lr, lc, kChunk);
  const __nv_bfloat16 *kpiece = ksrc + lc * 8;
  auto load_keys = [&](int c, int buf) {              // keys of chunk c, zero past the prompt
    const uint32_t dst = k_s + buf * K_BYTES + k_off0;
    const int jbase = c * kChunk + lr;
#pragma unroll
    for (int i = 0; i < SWEEPS; ++i) {
      const int j = jbase + i * RS;
      const bool in = j < y.lp;
      cp_async_16(dst + i * RS * 128, kpiece + (long long)(in ? j : 0) * ksp, in);
    }
  };
  load_keys(c_begin, 0);
  for (int cid = tid; cid < kMqRows * CPR; cid += kMqThreads) {      // Q rows, zero past the last
    const int r = cid / CPR, cc = cid % CPR;
    cp_async_16(q_s + mq_off(r, cc, kMqRows), qsrc + (long long)(r < rows ? r : 0) * D + cc * 8, r < rows);
  }
  cp_async_commit();
#pragma unroll
  for (int i = 1; i < NBUF; ++i) {
    if (c_begin + i < c_end) load_keys(c_begin + i, i);
    cp_async_commit();                                // (one group per chunk, empty or not)
  }

  // accumulator row r sits in lane 32 (r / 16) + r % 16 of tensor memory; warps w and w + 4 read rows
  // 16 w .. 16 w + 15 (lane quadrant w), the first 64 columns of a chunk and the last 64; for every
  // 8-column group g a thread holds columns 8 g + 2 (lane % 4) + {0, 1} of rows lane / 4 and lane / 4 + 8
  const int quad = warp & 3, half = warp >> 2;
  const int gq = lane >> 2, tq = lane & 3;
  const int r_lo = quad * 16 + gq, r_hi = r_lo + 8;
  // last key each of this thread's two rows may see (its own position); -1 for rows past the last
  const int see_lo = r_lo < rows ? t_first + r_lo : -1, see_hi = r_hi < rows ? t_first + r_hi : -1;
  const long long item = ((long long)b * n_q_heads + h) * n_row_blocks + qb;
  unsigned char *stage = smem + Q_BYTES + NBUF * K_BYTES;
  const int n_it = c_end - c_begin;
  auto issue_product = [&](int it) {                  // S(it) = Q K(it)^T into accumulator it & 1 (one thread)
    constexpr uint32_t kIdesc = instr_desc(kMqRows, kChunk, false);
    const uint32_t acc = s_tmem + (it & 1) * kChunk;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint32_t qa = q_s + (ks >> 2) * kMqRows * 128 + (ks & 3) * 32;
      const uint32_t ka = k_s + (it % NBUF) * K_BYTES + (ks >> 2) * kChunk * 128 + (ks & 3) * 32;
      umma(acc, smem_desc(qa, 16), smem_desc(ka, 16), kIdesc, ks > 0);
    }
    umma_commit(smem_u32(&s_bar[it & 1]));
  };
  // what the cp.async of every thread wrote is handed to the tensor core
  auto publish_tiles = [&]() {
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  };
  cp_async_wait<NBUF - 1>();                          // chunk 0 and Q have landed
  publish_tiles();
  if (tid == 0) issue_product(0);
  bool ok = true;
  for (int it = 0; it < n_it; ++it) {
    const int c = c_begin + it, acc = it & 1, j0 = c * kChunk;
    if (it + 1 < n_it) {
      // the next chunk's product is issued before this chunk is read back.  The barrier also says that
      // every warp is done with the accumulator and the stage of chunk it - 1.
      cp_async_wait<NBUF - 2>();                      // chunk it + 1 has landed
      publish_tiles();
      if (tid == 0) issue_product(it + 1);
    }
    ok = __syncthreads_and(mbar_wait(smem_u32(&s_bar[acc]), (it >> 1) & 1, &s_fail) ? 1 : 0) != 0;      // (the same in every thread)
    tc_fence_after();
    if (!ok) break;
    if (it + NBUF < n_it) load_keys(c + NBUF, it % NBUF);   // this chunk's tile has been consumed
    cp_async_commit();

    const uint32_t t_acc = s_tmem + acc * kChunk + ((uint32_t)(quad * 32) << 16) + half * 64;
    uint32_t v[32];
    tmem_ld_16rows_64cols(t_acc, v);
    tmem_ld_wait();
    float m_lo, m_hi, l_lo, l_hi;
    // MASKED: the chunk holds keys that some row does not see (its own successors, or keys past the
    // prompt).  Otherwise every row, the zero rows past the last included (their entries are finite
    // and the next stage gives them weight 0), takes every key.
    auto soft = [&](auto masked_tag) {
      constexpr bool MASKED = decltype(masked_tag)::value;
      m_lo = -INFINITY;
      m_hi = -INFINITY;
#pragma unroll
      for (int g = 0; g < 8; ++g)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int j = j0 + half * 64 + g * 8 + tq * 2 + e;
          if (!MASKED || j <= see_lo) m_lo = fmaxf(m_lo, __uint_as_float(v[4 * g + e]));
          if (!MASKED || j <= see_hi) m_hi = fmaxf(m_hi, __uint_as_float(v[4 * g + 2 + e]));
        }
      m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1));
      m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
      m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1));
      m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
      if (tq == 0) {
        s_xm[half][r_lo] = m_lo;
        s_xm[half][r_hi] = m_hi;
      }
      __syncthreads();
      // (the scale is positive: the maximum of the scaled scores is the scaled maximum)
      m_lo = fmaxf(m_lo, s_xm[half ^ 1][r_lo]) * scale_log2;
      m_hi = fmaxf(m_hi, s_xm[half ^ 1][r_hi]) * scale_log2;
      const float use_lo = m_lo == -INFINITY ? 0.f : m_lo, use_hi = m_hi == -INFINITY ? 0.f : m_hi;
      l_lo = 0.f;
      l_hi = 0.f;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        float p[4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int j = j0 + half * 64 + g * 8 + tq * 2 + e;
          p[e] = fast_exp2(fmaf(__uint_as_float(v[4 * g + e]), scale_log2, -use_lo));
          p[2 + e] = fast_exp2(fmaf(__uint_as_float(v[4 * g + 2 + e]), scale_log2, -use_hi));
          if (MASKED) {
            p[e] = j <= see_lo ? p[e] : 0.f;
            p[2 + e] = j <= see_hi ? p[2 + e] : 0.f;
          }
        }
        l_lo += p[0] + p[1];
        l_hi += p[2] + p[3];
        const int col = half * 64 + g * 8 + tq * 2;
        *reinterpret_cast<__half2 *>(stage + r_lo * P_PITCH + col * 2) = __floats2half2_rn(p[0], p[1]);
        *reinterpret_cast<__half2 *>(stage + r_hi * P_PITCH + col * 2) = __floats2half2_rn(p[2], p[3]);
      }
    };
    if (j0 + kChunk - 1 <= t_first) soft(std::false_type{});     // (the same branch in every thread)
    else soft(std::true_type{});
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    if (tq == 0 && half == 1) {
      s_xl[r_lo] = l_lo;
      s_xl[r_hi] = l_hi;
    }
    tc_fence_before();                                // (a later product overwrites the accumulator these threads read)
    __syncthreads();
    if (tq == 0 && half == 0) {
      float2 *st = ws.stats + (item * n_chunks + c) * kMqRows;
      st[r_lo] = make_float2(m_lo, l_lo + s_xl[r_lo]);
      st[r_hi] = make_float2(m_hi, l_hi + s_xl[r_hi]);
    }
    // the chunk's probabilities, 16 bytes per thread and row piece; only chunks that hold visual tokens
    if (j0 < y.vs + y.nv && j0 + kChunk > y.vs) {
      __half *dst = ws.probs + (item * n_chunks + c) * (long long)(kMqRows * kChunk);
      constexpr int PIECES = kChunk * 2 / 16, ROWS_PER_SWEEP = kMqThreads / PIECES;
      const int orow = tid / PIECES, opiece = tid % PIECES;
#pragma unroll
      for (int i = 0; i < kMqRows / ROWS_PER_SWEEP; ++i) {
        const int r = orow + i * ROWS_PER_SWEEP;
        st_16(dst + r * kChunk + opiece * 8, *reinterpret_cast<const uint4 *>(stage + r * P_PITCH + opiece * 16));
      }
    }
    // (the stage, s_xm and s_xl are next written after the barrier at the top of the next iteration;
    // the last iteration writes nothing after it)
  }
  cp_async_wait<0>();
  if (!ok && tid == 0) flag_status(dev_status, b, TWIG_DEV_INTERNAL);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem), "r"(2 * kChunk) : "memory");
}

// (max, sum) of two disjoint key sets -> of their union
__device__ __forceinline__ float2 merge_stats(float2 a, float2 b) {
  const float m = fmaxf(a.x, b.x);
  const float use = m == -INFINITY ? 0.f : m;
  return make_float2(m, a.y * fast_exp2(a.x - use) + b.y * fast_exp2(b.x - use));
}

// ---- 2. column sums of the normalised probabilities of one item over a few visual chunks ----
// grid (groups of kSumChunks visual chunks, heads * n_row_blocks, batch).  Three round trips to
// memory: the statistics, then every probability this CTA needs at once, then the stores.
__global__ void __launch_bounds__(kSumThreads)
ttp_mq_colsum_kernel(int n_text_max, int k_max_len, const int *__restrict__ prefix_len,
                     const int *__restrict__ vis_start, const int *__restrict__ n_vis, int n_q_heads, int n_chunks,
                     int n_row_blocks, MqScratch ws, int m_max) {
  constexpr int PAIRS = kChunk / 2;                  // column pairs of a chunk
  constexpr int RG = kSumThreads / PAIRS;            // row groups: thread (pair, rg) adds rows rg, rg + RG, ...
  constexpr int RPT = kMqRows / RG;                  // rows per thread and chunk
  constexpr int kMergeRegs = 8;                      // chunks per thread of the merge held in registers
  static_assert(kSumChunks * kMqRows == kSumThreads, "one thread per (chunk, row) weight");
  __shared__ float s_max[kMqRows], s_inv[kMqRows], s_f[kSumChunks][kMqRows];
  __shared__ float s_acc[kSumChunks][RG][kChunk];
  const int tid = threadIdx.x;
  const int h = blockIdx.y / n_row_blocks, qb = blockIdx.y % n_row_blocks, b = blockIdx.z;
  grid_dependency_sync();
  const MqLayout y = mq_layout(prefix_len, vis_start, n_vis, b, k_max_len, m_max, n_text_max);
  if (!y.ok) return;                                  // (flagged by the first kernel)
  const int row0 = qb * kMqRows;
  if (row0 >= y.n_text || y.nv == 0) return;
  const int rows = min(kMqRows, y.n_text - row0);
  const int c_first = y.vs / kChunk, c_last = (y.vs + y.nv - 1) / kChunk;
  const int c_begin = c_first + blockIdx.x * kSumChunks, c_end = min(c_last + 1, c_begin + kSumChunks);
  if (c_begin >= c_end) return;
  const long long item = ((long long)b * n_q_heads + h) * n_row_blocks + qb;
  const float2 *st = ws.stats + item * n_chunks * kMqRows;

  // the rows' softmax statistics over every chunk they see: four threads per row, then the four merged;
  // and, by the same token, the chunk maximum of every (chunk, row) this CTA weights
  const int n_c = (y.vs + y.nv + row0 + rows - 1) / kChunk + 1;
  const int wc = c_begin + tid / kMqRows, wr = tid % kMqRows;
  const float chunk_max = wc < c_end ? st[wc * kMqRows + wr].x : -INFINITY;
  {
    const int r = tid >> 2, q = tid & 3;
    float2 part[kMergeRegs];
#pragma unroll
    for (int i = 0; i < kMergeRegs; ++i) {
      const int c = q + 4 * i;
      part[i] = c < n_c ? st[c * kMqRows + r] : make_float2(-INFINITY, 0.f);
    }
    float2 acc = part[0];
#pragma unroll
    for (int i = 1; i < kMergeRegs; ++i) acc = merge_stats(acc, part[i]);
    for (int c = q + 4 * kMergeRegs; c < n_c; c += 4) acc = merge_stats(acc, st[c * kMqRows + r]);
#pragma unroll
    for (int o = 1; o < 4; o <<= 1) {
      float2 other;
      other.x = __shfl_xor_sync(0xffffffffu, acc.x, o);
      other.y = __shfl_xor_sync(0xffffffffu, acc.y, o);
      // (both partners must end up with the same bits: the lower lane's value goes first)
      acc = (q & o) ? merge_stats(other, acc) : merge_stats(acc, other);
    }
    if (q == 0) {
      s_max[r] = acc.x == -INFINITY ? 0.f : acc.x;
      s_inv[r] = r < rows && acc.y > 0.f ? 1.f / acc.y : 0.f;
    }
  }
  __syncthreads();
  s_f[tid / kMqRows][wr] = fast_exp2(chunk_max - s_max[wr]) * s_inv[wr];
  __syncthreads();

  const int pair = tid % PAIRS, rg = tid / PAIRS;
  const __half2 *src = reinterpret_cast<const __half2 *>(ws.probs + (item * n_chunks + c_begin) * (long long)(kMqRows * kChunk)) + pair;
  __half2 v[kSumChunks][RPT];
#pragma unroll
  for (int ci = 0; ci < kSumChunks; ++ci)
#pragma unroll
    for (int i = 0; i < RPT; ++i)
      v[ci][i] = c_begin + ci < c_end ? src[(long long)ci * (kMqRows * PAIRS) + (rg + i * RG) * PAIRS] : __half2();
#pragma unroll
  for (int ci = 0; ci < kSumChunks; ++ci) {
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const float2 f = __half22float2(v[ci][i]);
      a0 = fmaf(f.x, s_f[ci][rg + i * RG], a0);
      a1 = fmaf(f.y, s_f[ci][rg + i * RG], a1);
    }
    s_acc[ci][rg][2 * pair] = a0;
    s_acc[ci][rg][2 * pair + 1] = a1;
  }
  __syncthreads();
  float *out = ws.partial + item * m_max;
  for (int i = tid; i < kSumChunks * kChunk; i += kSumThreads) {
    const int ci = i / kChunk, col = i % kChunk;
    const int m = (c_begin + ci) * kChunk + col - y.vs;
    if (c_begin + ci < c_end && m >= 0 && m < y.nv) {
      float sum = 0.f;
#pragma unroll
      for (int g = 0; g < RG; ++g) sum += s_acc[ci][g][col];
      out[m] = sum;
    }
  }
}

// ---- 3. scores[b, m] = (1/H) sum over heads and row blocks, in index order; 0 past n_vis ----
__global__ void ttp_mq_reduce_kernel(const float *__restrict__ partial, int n_blocks_max, int n_q_heads,
                                     int n_text_max, const int *__restrict__ prefix_len,
                                     const int *__restrict__ vis_start, const int *__restrict__ n_vis,
                                     int k_max_len, float *__restrict__ scores, int m_max) {
  grid_dependency_sync();
  const int b = blockIdx.y, m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= m_max) return;
  const MqLayout y = mq_layout(prefix_len, vis_start, n_vis, b, k_max_len, m_max, n_text_max);
  float acc = 0.f;
  if (y.ok && y.n_text > 0 && m < y.nv) {
    const int nqb = (y.n_text + kMqRows - 1) / kMqRows;
    const int n_terms = n_q_heads * nqb;             // term t = (head t / nqb, row block t % nqb)
    constexpr int kBatch = 16;                       // loads in flight; the additions keep the index order
    for (int t0 = 0; t0 < n_terms; t0 += kBatch) {
      float v[kBatch];
#pragma unroll
      for (int i = 0; i < kBatch; ++i) {
        const int t = t0 + i;
        v[i] = t < n_terms ? partial[(((long long)b * n_q_heads + t / nqb) * n_blocks_max + t % nqb) * m_max + m] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < kBatch; ++i) acc += v[i];
    }
    acc /= (float)n_q_heads;
  }
  scores[(long long)b * m_max + m] = acc;
}

}  // namespace

}  // namespace twig

using namespace twig;

// `k_max_len`: the key tensor's length as passed to ttp_score_multiquery
extern "C" size_t ttp_multiquery_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t n_text_max, int32_t m_max,
                                                 int32_t k_max_len) {
  if (batch <= 0 || n_q_heads <= 0 || n_text_max <= 0 || m_max <= 0 || k_max_len <= 0) return 0;
  const size_t items = (size_t)batch * n_q_heads * ((n_text_max + kMqRows - 1) / kMqRows);
  const int n_chunks = (k_max_len + kChunk - 1) / kChunk;
  return mq_probs_bytes(items, n_chunks) + mq_stats_bytes(items, n_chunks) + mq_partial_bytes(items, m_max);
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
  if (ws_bytes < ttp_multiquery_workspace_bytes(batch, n_q_heads, n_text_max, m_max, k_max_len)) return TWIG_ERR_WORKSPACE;
  const int n_blocks = (n_text_max + kMqRows - 1) / kMqRows;
  const int n_chunks = (k_max_len + kChunk - 1) / kChunk;
  if ((long long)n_blocks * n_q_heads > 65535) return TWIG_ERR_UNSUPPORTED;
  const size_t items = (size_t)batch * n_q_heads * n_blocks;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.f / sqrtf((float)head_dim);
  if (!(scale > 0.f)) return TWIG_ERR_UNSUPPORTED;          // (the kernel scales row maxima: a positive scale keeps them maxima)
  const float scale_log2 = scale * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto q = static_cast<const __nv_bfloat16 *>(q_text);
  auto k = static_cast<const __nv_bfloat16 *>(twig_k);
  MqScratch sc;
  unsigned char *base = static_cast<unsigned char *>(ws);
  sc.probs = reinterpret_cast<__half *>(base);
  sc.stats = reinterpret_cast<float2 *>(base + mq_probs_bytes(items, n_chunks));
  sc.partial = reinterpret_cast<float *>(base + mq_probs_bytes(items, n_chunks) + mq_stats_bytes(items, n_chunks));
  const int group = n_q_heads / n_kv_heads;

  // Q, two key tiles, the staged probabilities; at least 78 KB so that no more than two CTAs share an SM
  // (each holds half of its tensor memory)
  constexpr int kBufs = 2;
  const size_t smem = std::max<size_t>((size_t)(kMqRows + kBufs * kChunk) * head_dim * 2 + kMqRows * (kChunk * 2 + 16), 78 * 1024);
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(ttp_mq_probs_kernel<128, kBufs>, cudaFuncAttributeMaxDynamicSharedMemorySize, 164 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(ttp_mq_probs_kernel<64, kBufs>, cudaFuncAttributeMaxDynamicSharedMemorySize, 164 * 1024) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  // chunks per CTA: walks long enough to pay for a CTA's start (Q, tensor memory), about two waves of CTAs
  // at two CTAs per SM (measured on 4 x 32 heads x 24 chunks: 1: 70 us, 3: 59, 6: 55, 12: 56, 24: 68 per call)
  const int chunks_per_cta = (int)std::min<long long>(8, std::max<long long>(1, (long long)items * n_chunks / (2 * 2 * 148)));
  const int n_groups = (n_chunks + chunks_per_cta - 1) / chunks_per_cta;
  {
    PdlLaunch L(dim3(n_groups * n_blocks, n_q_heads, batch), dim3(kMqThreads), smem, st);
    const cudaError_t err =
        head_dim == 128
            ? cudaLaunchKernelEx(&L.cfg, ttp_mq_probs_kernel<128, kBufs>, q, n_text_max, k, (long long)k_stride_batch,
                                 (long long)k_stride_head, (long long)k_stride_pos, k_max_len, prefix_len, vis_start,
                                 n_vis, n_q_heads, group, scale_log2, n_chunks, n_blocks, n_groups, chunks_per_cta, sc, m_max, dev_status)
            : cudaLaunchKernelEx(&L.cfg, ttp_mq_probs_kernel<64, kBufs>, q, n_text_max, k, (long long)k_stride_batch,
                                 (long long)k_stride_head, (long long)k_stride_pos, k_max_len, prefix_len, vis_start,
                                 n_vis, n_q_heads, group, scale_log2, n_chunks, n_blocks, n_groups, chunks_per_cta, sc, m_max, dev_status);
    if (err != cudaSuccess) return TWIG_ERR_CUDA;
  }
  {
    const int vis_chunks = (m_max + kChunk - 1) / kChunk + 1;       // a span of m_max keys touches at most this many chunks
    PdlLaunch L(dim3((vis_chunks + kSumChunks - 1) / kSumChunks, n_q_heads * n_blocks, batch), dim3(kSumThreads), 0, st);
    if (cudaLaunchKernelEx(&L.cfg, ttp_mq_colsum_kernel, n_text_max, k_max_len, prefix_len, vis_start, n_vis, n_q_heads,
                           n_chunks, n_blocks, sc, m_max) != cudaSuccess)
      return TWIG_ERR_CUDA;
  }
  {
    PdlLaunch L(dim3((m_max + 255) / 256, batch), dim3(256), 0, st);
    if (cudaLaunchKernelEx(&L.cfg, ttp_mq_reduce_kernel, (const float *)sc.partial, n_blocks, n_q_heads, n_text_max,
                           prefix_len, vis_start, n_vis, k_max_len, scores, m_max) != cudaSuccess)
      return TWIG_ERR_CUDA;
  }
  return launch_status();
}
