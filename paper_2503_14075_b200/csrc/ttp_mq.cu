// Multi-query pruning guide of Eq. 3: the attention that the textual tokens after the image pay to
// every visual token, summed over those tokens and averaged over heads,
//   a[m] = (1/H) sum_h sum_i softmax_{j <= t_i}(q_i . k_j / sqrt(d))[vis_start + m],
// t_i = vis_start + n_vis + i the prompt position of text token i.  Unlike the single-query score
// this is an N x L attention-map reduction.  Three kernels, each launched so that it may be
// scheduled while its predecessor drains:
//   1. probabilities: a CTA takes 64 query rows of one head and a run of kChunk-key chunks.  Q (cp.async)
//      and the key tiles (TMA) go to shared memory in the 128-byte-swizzled layout of the matrix
//      descriptors, one thread issues S = Q K^T per chunk (tcgen05.mma, M = 64, N = kChunk, fp32 in
//      tensor memory), eight warps read the accumulator back, mask (causal), and write, per half-chunk
//      of 64 keys, the rows' maxima and sums of exponentials plus the exponentials themselves,
//      relative to the half-chunk's row maximum, as fp16.  Every key is read once and every product
//      and exponential is computed once.
//   2. column sums: a CTA merges the half-chunks' statistics of its 64 rows into the rows' softmax
//      denominators and adds up, down the rows, the stored exponentials of a few visual chunks, each
//      row weighted by exp2(half-chunk max - row max) / row sum.
//   3. the sum over heads and row blocks in index order, so that the result does not depend on
//      scheduling.
#include <cuda_fp16.h>

#include <algorithm>
#include <mutex>
#include <type_traits>

#include "tcgen05_common.cuh"

namespace twig {

namespace {

constexpr int kMqRows = 64;        // query rows per CTA (one M = 64 accumulator; 16 rows per lane quadrant)
constexpr int kMqSoftWarps = 8;    // two warps per lane quadrant of the accumulator: half of a chunk's columns each
constexpr int kMqThreads = 32 * (kMqSoftWarps + 1);   // and the warp that moves tiles and issues products
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

// Scratch: probabilities [item][chunk][64 rows][kChunk] fp16, statistics [item][half-chunk][64 rows]
// (max, sum: one pair per 64 keys), partial column sums [item][m_max]; item = (request, head, row block).
struct MqScratch {
  __half *probs;
  float2 *stats;
  float *partial;
};
inline size_t mq_probs_bytes(size_t items, int n_chunks) { return items * n_chunks * kMqRows * kChunk * sizeof(__half); }
inline size_t mq_stats_bytes(size_t items, int n_chunks) { return items * 2 * n_chunks * kMqRows * sizeof(float2); }
inline size_t mq_partial_bytes(size_t items, int m_max) { return ((items * m_max * sizeof(float)) + 15) & ~(size_t)15; }

// ---- 1. probabilities and per-chunk statistics ----
// grid (n_groups * n_row_blocks, heads, batch); blockIdx.x = row block * n_groups + group.  A CTA walks
// `chunks_per_cta` consecutive chunks of its item.  Nine warps in two roles that meet only at mbarriers:
//   warp 8, one thread: brings the key tiles (TMA boxes of the 4-D map over K: 64 columns x 128 rows,
//     128-byte swizzle, completion counted on the buffer's barrier) into NBUF buffers, a buffer being
//     refilled as soon as the product that read it has completed, and issues S(t) = Q K(t)^T into one of
//     two accumulators in tensor memory as soon as the tile is there and the accumulator has been read;
//   warps 0-7: warps w and w + 4 own the rows of lane quadrant w (16 rows), the first and the last 64
//     columns of a chunk (a half-chunk with statistics of its own): tcgen05.ld, release the accumulator,
//     mask, row max, exponentials, row sums, staged per warp and stored 16 bytes per lane.
// Keys past the prompt are read as they are (past the tensor: as zeros): no query sees them.
template <int D, int NBUF>
__global__ void __launch_bounds__(kMqThreads)
ttp_mq_probs_kernel(const __nv_bfloat16 *__restrict__ q_text, int n_text_max, const __grid_constant__ CUtensorMap kmap,
                    int k_max_len, const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                    const int *__restrict__ n_vis, int n_q_heads, int group, float scale_log2, int n_chunks,
                    int n_row_blocks, int n_groups, int chunks_per_cta, MqScratch ws, int m_max, int *dev_status) {
  constexpr int CPR = D / 8;                         // 16-byte pieces per row
  constexpr int Q_BYTES = kMqRows * D * 2;
  constexpr int K_BYTES = kChunk * D * 2;
  constexpr int P_PITCH = 64 * 2 + 16;               // a warp's staged fp16 row of 64 columns (+16: bank spread)
  constexpr int WARP_STAGE = 16 * P_PITCH;
  extern __shared__ __align__(1024) unsigned char smem[];   // Q | NBUF key tiles | eight warps' stages
  // barriers: tile landed [NBUF], product complete [2], accumulator read [2]
  __shared__ __align__(8) unsigned long long s_bar[NBUF + 4];
  __shared__ uint32_t s_tmem;
  __shared__ volatile int s_fail;

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
  const int n_it = c_end - c_begin;

  const uint32_t bars = smem_u32(s_bar);
  auto bar_full = [&](int buf) { return bars + 8 * buf; };
  auto bar_ready = [&](int acc) { return bars + 8 * (NBUF + acc); };
  auto bar_read = [&](int acc) { return bars + 8 * (NBUF + 2 + acc); };
  const uint32_t q_s = smem_u32(smem), k_s = q_s + Q_BYTES;
  auto load_tile = [&](int it) {                      // (one thread) key tile of chunk c_begin + it into buffer it % NBUF
    const int buf = it % NBUF;
    mbar_arrive_expect_tx(bar_full(buf), K_BYTES);
#pragma unroll
    for (int pnl = 0; pnl < D / 64; ++pnl)
      tma_load_4d(k_s + buf * K_BYTES + pnl * kChunk * 128, &kmap, bar_full(buf), pnl * 64, (c_begin + it) * kChunk,
                  h / group, b);
  };
  if (tid == kMqSoftWarps * 32) {
    // the thread that moves the tiles sets up their barriers and has the first tiles on their way
    // before anything else of the CTA is ready
    for (int i = 0; i < NBUF; ++i) mbar_init(bar_full(i), 1);      // one arrival that announces the bytes
    mbar_init_fence_cluster();
    fence_async_smem();
    for (int it = 0; it < NBUF && it < n_it; ++it) load_tile(it);
  }
  if (tid == 0) {
    s_fail = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_ready(i), 1);                                  // one tcgen05.commit
      mbar_init(bar_read(i), kMqSoftWarps);                        // every softmax warp once
    }
    mbar_init_fence_cluster();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(2 * kChunk) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }

  // Q rows (zero past the last) by the softmax warps; one barrier of the whole CTA hands them, the
  // barriers and the tensor-memory address to everybody
  if (warp < kMqSoftWarps) {
    const __nv_bfloat16 *qsrc = q_text + (((long long)b * n_q_heads + h) * n_text_max + row0) * D;
    for (int cid = tid; cid < kMqRows * CPR; cid += kMqSoftWarps * 32) {
      const int r = cid / CPR, cc = cid % CPR;
      cp_async_16(q_s + mq_off(r, cc, kMqRows), qsrc + (long long)(r < rows ? r : 0) * D + cc * 8, r < rows);
    }
    cp_async_commit();
    cp_async_wait<0>();
    fence_async_smem();                               // the tensor core reads what these threads wrote
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int *fail = &s_fail;

  if (warp == kMqSoftWarps) {
    // ================= tiles and products (one thread) =================
    if (lane == 0) {
      constexpr uint32_t kIdesc = instr_desc(kMqRows, kChunk, false);
      bool ok = true;
      for (int it = 0; it < n_it; ++it) {
        const int buf = it % NBUF, acc = it & 1;
        ok = mbar_wait(bar_full(buf), (it / NBUF) & 1, fail);
        if (ok && it >= 2) ok = mbar_wait(bar_read(acc), ((it - 2) >> 1) & 1, fail);     // S(it - 2) has been read
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t qa = q_s + (ks >> 2) * kMqRows * 128 + (ks & 3) * 32;
          const uint32_t ka = k_s + buf * K_BYTES + (ks >> 2) * kChunk * 128 + (ks & 3) * 32;
          umma(tmem + acc * kChunk, smem_desc(qa, 16), smem_desc(ka, 16), kIdesc, ks > 0);
        }
        umma_commit(bar_ready(acc));
        if (it + NBUF < n_it) {                       // the buffer is refilled once this product has read it
          ok = mbar_wait(bar_ready(acc), (it >> 1) & 1, fail);
          if (!ok) break;
          load_tile(it + NBUF);
        }
      }
      if (!ok) s_fail = 1;
    }
  } else {
    // ================= read-back: statistics and exponentials (warps 0-7) =================
    // accumulator row r sits in lane 32 (r / 16) + r % 16 of tensor memory; warps w and w + 4 read rows
    // 16 w .. 16 w + 15 (lane quadrant w), the first 64 columns of a chunk and the last 64: two
    // half-chunks with statistics of their own, so the warps never wait for one another.  For every
    // 8-column group g a thread holds columns 8 g + 2 (lane % 4) + {0, 1} of rows lane / 4 and lane / 4 + 8.
    const int quad = warp & 3, half = warp >> 2;
    const int gq = lane >> 2, tq = lane & 3;
    const int r_lo = quad * 16 + gq, r_hi = r_lo + 8;
    // last key each of this thread's two rows may see (its own position); -1 for rows past the last
    const int see_lo = r_lo < rows ? t_first + r_lo : -1, see_hi = r_hi < rows ? t_first + r_hi : -1;
    const long long item = ((long long)b * n_q_heads + h) * n_row_blocks + qb;
    unsigned char *stage = smem + Q_BYTES + NBUF * K_BYTES + warp * WARP_STAGE;
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
      const int c = c_begin + it, acc = it & 1, j0 = c * kChunk + half * 64;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_ready(acc), (it >> 1) & 1, fail));
      if (!ok) break;
      tc_fence_after();
      uint32_t v[32];
      tmem_ld_16rows_64cols(tmem + acc * kChunk + ((uint32_t)(quad * 32) << 16) + half * 64, v);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_read(acc));      // the product after next may overwrite the accumulator
      float m_lo, m_hi, l_lo, l_hi;
      // MASKED: the half-chunk holds keys that some row does not see (its own successors, or keys past the
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
            const int j = j0 + g * 8 + tq * 2 + e;
            if (!MASKED || j <= see_lo) m_lo = fmaxf(m_lo, __uint_as_float(v[4 * g + e]));
            if (!MASKED || j <= see_hi) m_hi = fmaxf(m_hi, __uint_as_float(v[4 * g + 2 + e]));
          }
        m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1));
        m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
        m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1));
        m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
        // (the scale is positive: the maximum of the scaled scores is the scaled maximum)
        m_lo *= scale_log2;
        m_hi *= scale_log2;
        const float use_lo = m_lo == -INFINITY ? 0.f : m_lo, use_hi = m_hi == -INFINITY ? 0.f : m_hi;
        l_lo = 0.f;
        l_hi = 0.f;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          float p[4];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int j = j0 + g * 8 + tq * 2 + e;
            p[e] = fast_exp2(fmaf(__uint_as_float(v[4 * g + e]), scale_log2, -use_lo));
            p[2 + e] = fast_exp2(fmaf(__uint_as_float(v[4 * g + 2 + e]), scale_log2, -use_hi));
            if (MASKED) {
              p[e] = j <= see_lo ? p[e] : 0.f;
              p[2 + e] = j <= see_hi ? p[2 + e] : 0.f;
            }
          }
          l_lo += p[0] + p[1];
          l_hi += p[2] + p[3];
          const int col = g * 8 + tq * 2;
          *reinterpret_cast<__half2 *>(stage + gq * P_PITCH + col * 2) = __floats2half2_rn(p[0], p[1]);
          *reinterpret_cast<__half2 *>(stage + (gq + 8) * P_PITCH + col * 2) = __floats2half2_rn(p[2], p[3]);
        }
      };
      if (j0 + 63 <= t_first) soft(std::false_type{});     // (the same branch in every thread of the warp)
      else soft(std::true_type{});
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
      l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
      l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
      if (tq == 0) {
        float2 *st = ws.stats + (item * (2 * n_chunks) + 2 * c + half) * kMqRows;
        st[r_lo] = make_float2(m_lo, l_lo);
        st[r_hi] = make_float2(m_hi, l_hi);
      }
      __syncwarp();
      // the warp's 16 rows x 64 columns, 16 bytes per lane; only chunks that hold visual tokens
      if (c * kChunk < y.vs + y.nv && (c + 1) * kChunk > y.vs) {
        __half *dst = ws.probs + (item * n_chunks + c) * (long long)(kMqRows * kChunk) + (quad * 16) * kChunk + half * 64;
        const int orow = lane >> 3, opiece = lane & 7;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = orow + 4 * i;
          st_16(dst + r * kChunk + opiece * 8, *reinterpret_cast<const uint4 *>(stage + r * P_PITCH + opiece * 16));
        }
      }
      __syncwarp();                                   // the stage is read before the next chunk is staged
    }
    if (!ok) s_fail = 1;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (s_fail && tid == 0) flag_status(dev_status, b, TWIG_DEV_INTERNAL);
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kChunk) : "memory");
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
  constexpr int kMergeRegs = 12;                     // half-chunks per thread of the merge held in registers
  static_assert(2 * kSumChunks * kMqRows == 2 * kSumThreads, "two (half-chunk, row) weights per thread");
  __shared__ float s_max[kMqRows], s_inv[kMqRows], s_f[2 * kSumChunks][kMqRows];
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
  const float2 *st = ws.stats + item * (2 * n_chunks) * kMqRows;       // [half-chunk][row]

  // the rows' softmax statistics over every half-chunk they see: four threads per row, then the four
  // merged; and, by the same token, the maxima of the (half-chunk, row) pairs this CTA weights
  const int n_c = 2 * ((y.vs + y.nv + row0 + rows - 1) / kChunk + 1);
  const int wr = tid % kMqRows;
  float half_max[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int wh = 2 * c_begin + tid / kMqRows + i * (kSumThreads / kMqRows);
    half_max[i] = wh < 2 * c_end ? st[wh * kMqRows + wr].x : -INFINITY;
  }
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
#pragma unroll
  for (int i = 0; i < 2; ++i)
    s_f[tid / kMqRows + i * (kSumThreads / kMqRows)][wr] = fast_exp2(half_max[i] - s_max[wr]) * s_inv[wr];
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
      const float w = s_f[2 * ci + pair / (PAIRS / 2)][rg + i * RG];      // (the pair's half of the chunk)
      a0 = fmaf(f.x, w, a0);
      a1 = fmaf(f.y, w, a1);
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

// 4-D tensor map over the key tensor: (head_dim, position, kv head, request), boxes of 64 columns x
// kChunk rows with the 128-byte swizzle (one panel of a key tile).  Rows past k_max_len read as zeros.
typedef CUresult (*MqEncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool mq_key_map(CUtensorMap *out, const void *k, long long ksb, long long ksh, long long ksp, int k_max_len, int n_kv_heads,
                int batch, int head_dim) {
  static std::mutex mu;
  static MqEncodeTiledFn fn = nullptr;
  static bool tried = false;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!tried) {
      tried = true;
      void *ptr = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
          qres == cudaDriverEntryPointSuccess)
        fn = reinterpret_cast<MqEncodeTiledFn>(ptr);
    }
  }
  if (!fn || ksp <= 0) return false;
  // (a stride of an extent-1 dimension is never used, but must be a valid one)
  if (n_kv_heads == 1 || ksh <= 0) ksh = ksp;
  if (batch == 1 || ksb <= 0) ksb = ksp;
  const cuuint64_t dims[4] = {(cuuint64_t)head_dim, (cuuint64_t)k_max_len, (cuuint64_t)n_kv_heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)ksp * 2, (cuuint64_t)ksh * 2, (cuuint64_t)ksb * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)kChunk, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(k), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
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
  MqScratch sc;
  unsigned char *base = static_cast<unsigned char *>(ws);
  sc.probs = reinterpret_cast<__half *>(base);
  sc.stats = reinterpret_cast<float2 *>(base + mq_probs_bytes(items, n_chunks));
  sc.partial = reinterpret_cast<float *>(base + mq_probs_bytes(items, n_chunks) + mq_stats_bytes(items, n_chunks));
  const int group = n_q_heads / n_kv_heads;
  alignas(64) CUtensorMap kmap;
  if (!mq_key_map(&kmap, twig_k, k_stride_batch, k_stride_head, k_stride_pos, k_max_len, n_kv_heads, batch, head_dim))
    return TWIG_ERR_UNSUPPORTED;                      // (no tensor map: there is no other path)

  // Q, two key tiles, the warps' stages; at least 78 KB so that no more than two CTAs share an SM
  // (each holds half of its tensor memory)
  constexpr int kBufs = 2;
  const size_t smem = std::max<size_t>((size_t)(kMqRows + kBufs * kChunk) * head_dim * 2 + kMqSoftWarps * 16 * (64 * 2 + 16), 78 * 1024);
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(ttp_mq_probs_kernel<128, kBufs>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(ttp_mq_probs_kernel<64, kBufs>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  // chunks per CTA: walks long enough to pay for a CTA's start (Q, tensor memory, the first tiles' latency),
  // about 3.5 CTAs per SM in all (measured on 4 x 32 heads x 24 chunks, per call: 2 chunks 61 us, 4: 53, 6: 51,
  // 8: 52, 12: 50, 24: 56)
  const long long total_chunks = (long long)items * n_chunks;
  const int chunks_per_cta = (int)std::min<long long>(12, std::max<long long>(1, (total_chunks + 517) / 518));
  const int n_groups = (n_chunks + chunks_per_cta - 1) / chunks_per_cta;
  {
    PdlLaunch L(dim3(n_groups * n_blocks, n_q_heads, batch), dim3(kMqThreads), smem, st);
    const cudaError_t err =
        head_dim == 128
            ? cudaLaunchKernelEx(&L.cfg, ttp_mq_probs_kernel<128, kBufs>, q, n_text_max, kmap, k_max_len, prefix_len, vis_start,
                                 n_vis, n_q_heads, group, scale_log2, n_chunks, n_blocks, n_groups, chunks_per_cta, sc, m_max, dev_status)
            : cudaLaunchKernelEx(&L.cfg, ttp_mq_probs_kernel<64, kBufs>, q, n_text_max, kmap, k_max_len, prefix_len, vis_start,
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
