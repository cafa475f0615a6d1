// Tree attention of the verification pass (Sec. 5.4, Appendix A, Algorithm 2;
// Eq. 2 with the causal mask replaced by the tree's ancestor mask).
//
// Every draft-tree node attends to the whole cached prefix, to its ancestors
// and to itself.  The T*G query rows that share one kv head (T nodes, G query
// heads per kv head) form the M side of two dense contractions, S = Q K^T and
// O = P V, run on bf16 tensor-core MMA with fp32 accumulation.  The key axis
// (prefix rows followed by the tree's own rows) is cut into tiles; a thread
// block cluster splits the tiles between its CTAs, every CTA keeps a
// flash-style running (max, sum, O) per row, and the partial results are
// merged through distributed shared memory (each CTA pushes its per-row partial
// to the CTA that owns the row), so nothing but Q, K, V and the final output
// touches HBM.
#include <cooperative_groups.h>

#include "tree_attn.cuh"

namespace cg = cooperative_groups;

namespace twig {

// Byte offset of 16-byte chunk `c` of row `r` in a [rows x D] bf16 tile.  The
// tile is stored as D/64 panels of 128-byte rows; within a panel the chunk
// index is XORed with (row & 7), which makes ldmatrix conflict-free.
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return (uint32_t)((c >> 3) * ROWS * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D_, int WM_, int WN_, int KC_, int STAGES_, int MIN_CTAS_>
struct AttnCfg {
  static constexpr int D = D_, WM = WM_, WN = WN_, KC = KC_, STAGES = STAGES_, MIN_CTAS = MIN_CTAS_;
  static constexpr int ROWS = 16 * WM;          // query rows per CTA
  static constexpr int KT = KC * WN;            // keys per tile
  static constexpr int DW = D / WN;             // output columns per warp
  static constexpr int THREADS = 32 * WM * WN;
  static constexpr int CPR = D / 8;             // 16-byte chunks per row
  static constexpr int Q_BYTES = ROWS * D * 2;
  static constexpr int P_BYTES = WN > 1 ? ROWS * KT * 2 : 0;   // bf16 probabilities of one tile
  static constexpr int TILE_BYTES = KT * D * 2;
  static constexpr int STAGE_BYTES = 2 * STAGES * TILE_BYTES;
  static constexpr int RECV_BYTES = ROWS * D * 2;              // the per-split partials a CTA owns (fp16)
  static_assert(KT == 64, "a row of P is one 128-byte swizzled line");
  static_assert(DW % 16 == 0 && KC % 16 == 0, "warp slices are whole ldmatrix.x4 steps");
  // The small, latency-bound variants (one CTA per SM is enough for them) keep the split-merge
  // buffer outside the stage ring: peers may then push as soon as they are done, and one
  // cluster barrier of the epilogue goes away.  The others reuse the ring after the key loop.
  static constexpr bool RECV_OWN = ROWS <= 32;
  // The same variants spend far less time computing a tile than waiting for it, so they keep the
  // whole ring in flight (a stage is refilled after its tile has been used) instead of one stage
  // less (refilled before): STAGES rather than STAGES - 1 tiles are requested up front.
  static constexpr bool FULL_RING = ROWS <= 32;
  static constexpr int PRE = FULL_RING ? STAGES : STAGES - 1;
  static_assert(RECV_OWN || RECV_BYTES <= STAGE_BYTES, "the receive buffer must fit in the stage ring");
  static constexpr int P_OFFSET = Q_BYTES;
  static constexpr int K_OFFSET = Q_BYTES + P_BYTES;
  static constexpr int RECV_OFFSET = RECV_OWN ? K_OFFSET + STAGE_BYTES : K_OFFSET;
  static constexpr int SMEM_BYTES = K_OFFSET + STAGE_BYTES + (RECV_OWN ? RECV_BYTES : 0);
};

// The WM x WN warps of a CTA: warp (wm, wn) owns query rows [16 wm, 16 wm + 16).  For S = Q K^T it
// takes the KC keys [wn KC, wn KC + KC) of the tile; the WN warps of a row group agree on the row
// maxima through shared memory and leave their bf16 probabilities there; for O += P V every warp
// reads all KT probabilities of its rows and accumulates the DW output columns [wn DW, wn DW + DW).
// No warp ever holds another's partial O, so nothing but maxima, probabilities and row sums is
// exchanged inside the CTA.
template <class C>
__global__ void __launch_bounds__(C::THREADS, C::MIN_CTAS)
tree_attn_kernel(const AttnParams p) {
  constexpr int D = C::D, ROWS = C::ROWS, KT = C::KT, KC = C::KC, WN = C::WN, STAGES = C::STAGES;
  constexpr int NT = KC / 8;       // key n-tiles of S per warp per tile
  constexpr int OT = C::DW / 8;    // head-dim n-tiles of O per warp
  constexpr int KS = D / 16;       // k-steps of Q K^T
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long s_mask[TWIG_MAX_NODES];
  __shared__ int s_par[TWIG_MAX_NODES];
  __shared__ float s_stat[WN][ROWS];                            // row maxima of a tile, later row sums
  __shared__ float s_amax[WN][ROWS];                            // largest |O| of a row over a warp's columns
  __shared__ float4 r_ml[ROWS];                                 // received (m, l, row scale): [sender][owned row]
  __shared__ int s_bad;
  __shared__ __align__(8) unsigned long long s_recv_bar;       // counts the bytes peers have pushed to this CTA

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp / WN, wn = warp % WN;
  const int split = blockIdx.x, n_splits = gridDim.x;
  const int hk = blockIdx.y / p.row_blocks, rb = blockIdx.y % p.row_blocks;
  const int b = blockIdx.z;
  // barrier of the WN warps that share a row group (ids 1..WM; 0 is __syncthreads)
  auto group_sync = [&]() {
    if (WN > 1) asm volatile("bar.sync %0, %1;" ::"r"(1 + wm), "n"(32 * WN) : "memory");
  };

  // Normally nothing is read before the preceding kernel of the stream has completed.  With
  // `early_prefix` the caller has promised that the preceding kernel writes neither the lengths,
  // the parent array nor cache rows below kv_len: those are then read (and the prefix tiles
  // prefetched) while that kernel is still draining, and only Q and the tree's rows wait.
  if (!p.early_prefix) grid_dependency_sync();
  // ---- per-request metadata; every exit below is uniform over the cluster ----
  const int n = p.n_nodes[b], L = p.kv_len[b];
  const int my_parent = tid < p.t_max ? p.parent[(long long)b * p.t_max + tid] : -1;   // (in flight with n, L)
  // A CTA that leaves early still waits for the preceding kernel first: the kernel after this one
  // only waits for this one, so every CTA has to carry the dependency on.
  const bool first = split == 0 && blockIdx.y == 0 && tid == 0;
  const int rows_total = n * p.group, row0 = rb * ROWS;
  if (n <= 0 || n > p.t_max || L < 0 || L > p.max_len || row0 >= rows_total) {
    if (p.early_prefix) grid_dependency_sync();       // (also with early_query: nothing was launched early yet)
    if (first && (n < 0 || n > p.t_max)) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    else if (first && n > 0 && (L < 0 || L > p.max_len)) flag_status(p.dev_status, b, TWIG_DEV_OVERFLOW);
    return;
  }
  // Split merge: every CTA owns ROWS / n_splits rows and receives n_splits partials (m, l, O row)
  // for each of them; its barrier completes when all of those bytes have landed.
  const int rows_per = ROWS / n_splits;
  const uint32_t recv_bar = smem_u32(&s_recv_bar);
  if (n_splits > 1) {
    if (tid == 0) {
      // one arrival that announces the peers' bytes, one per warp for this CTA's own share
      mbar_init(recv_bar, 1 + C::THREADS / 32);
      mbar_arrive_expect_tx(recv_bar, (uint32_t)((n_splits - 1) * rows_per * (D * 2 + 16)));
      mbar_init_fence_cluster();
    }
    __syncthreads();
    // with its own receive buffer a CTA only has to be running before peers may write to it
    if (C::RECV_OWN) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  }

  const uint32_t q_s = smem_u32(smem);
  const uint32_t p_s = q_s + C::P_OFFSET;
  const uint32_t k_s = q_s + C::K_OFFSET;
  const uint32_t v_s = k_s + STAGES * C::TILE_BYTES;

  // ---- key tiles of this CTA --------------------------------------------------
  const int NK = L + n;
  const int n_tiles = (NK + KT - 1) / KT;
  const int per = (n_tiles + n_splits - 1) / n_splits;
  const int t_begin = split * per;
  const int t_end = min(n_tiles, t_begin + per);

  const __nv_bfloat16 *ck = p.cache_k + b * p.c_sb + hk * p.c_sh;
  const __nv_bfloat16 *cv = p.cache_v + b * p.c_sb + hk * p.c_sh;
  const __nv_bfloat16 *tk = p.tree_k + ((long long)b * p.n_kv_heads + hk) * p.t_max * D;
  const __nv_bfloat16 *tv = p.tree_v + ((long long)b * p.n_kv_heads + hk) * p.t_max * D;

  auto load_tile = [&](int t, int stage) {
    constexpr int CHUNKS = KT * C::CPR;
#pragma unroll
    for (int i = 0; i < (CHUNKS + C::THREADS - 1) / C::THREADS; ++i) {
      const int cid = i * C::THREADS + tid;
      if (CHUNKS % C::THREADS != 0 && cid >= CHUNKS) break;
      const int r = cid / C::CPR, c = cid % C::CPR;
      const int vj = t * KT + r;
      const __nv_bfloat16 *sk = ck, *sv = cv;
      bool valid = false;
      if (vj < L) {
        sk = ck + (long long)vj * p.c_sp + c * 8;
        sv = cv + (long long)vj * p.c_sp + c * 8;
        valid = true;
      } else if (vj < NK) {
        sk = tk + (vj - L) * D + c * 8;
        sv = tv + (vj - L) * D + c * 8;
        valid = true;
      }
      const uint32_t off = stage * C::TILE_BYTES + tile_off<KT>(r, c);
      cp_async_16(k_s + off, sk, valid);
      cp_async_16(v_s + off, sv, valid);
    }
  };

  // ---- start the copies first: Q tile (zero rows past the last row) and the first key tiles ----
  constexpr int PRE = C::PRE;
  bool prefetched[PRE > 0 ? PRE : 1];
  if (p.early_prefix) {
#pragma unroll
    for (int s = 0; s < PRE; ++s) {
      const int t = t_begin + s;
      prefetched[s] = t < t_end && t * KT + KT <= L;      // wholly inside the cached prefix
      if (prefetched[s]) load_tile(t, s);
      cp_async_commit();
    }
  }
  auto load_q = [&]() {
    constexpr int CHUNKS = ROWS * C::CPR;
#pragma unroll
    for (int i = 0; i < (CHUNKS + C::THREADS - 1) / C::THREADS; ++i) {
      const int cid = i * C::THREADS + tid;
      if (CHUNKS % C::THREADS != 0 && cid >= CHUNKS) break;
      const int r = cid / C::CPR, c = cid % C::CPR;
      const int gr = row0 + r;
      const bool valid = gr < rows_total;
      const int node = valid ? gr / p.group : 0, g = valid ? gr % p.group : 0;
      const __nv_bfloat16 *src =
          p.q + (((long long)b * p.t_max + node) * p.n_q_heads + hk * p.group + g) * D + c * 8;
      cp_async_16(q_s + tile_off<ROWS>(r, c), src, valid);
    }
  };
  if (!p.early_prefix) {
    load_q();
#pragma unroll
    for (int s = 0; s < PRE; ++s) {
      if (t_begin + s < t_end) load_tile(t_begin + s, s);
      cp_async_commit();        // the first group also carries Q
    }
  }

  // ---- while they fly: parent array -> shared memory, validation, ancestor masks ----
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (tid < n) {
    const int pr = my_parent;
    s_par[tid] = pr;
    if ((tid == 0) ? (pr != -1) : (pr < 0 || pr >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (p.early_prefix) grid_dependency_sync();
    if (first) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    cp_async_wait<0>();       // nothing may still be writing this CTA's shared memory
    return;
  }
  if (tid < n) {          // ancestor-or-self bitmask; parent[x] < x bounds the walk
    unsigned long long m = 0;
    int x = tid;
    while (x >= 0) {
      m |= 1ull << x;
      x = s_par[x];
    }
    s_mask[tid] = m;
  }
  __syncthreads();

  // ---- per-thread state --------------------------------------------------------
  const int gq = lane >> 2, tq = lane & 3;
  const int r_lo = wm * 16 + gq, r_hi = r_lo + 8;         // CTA-local rows of this thread
  // ancestor masks of this thread's two rows (0 for rows past the last one)
  unsigned long long mask_lo = 0ull, mask_hi = 0ull;
  {
    const int g_lo = row0 + r_lo, g_hi = row0 + r_hi;
    if (g_lo < rows_total) mask_lo = s_mask[p.group == 1 ? g_lo : g_lo / p.group];
    if (g_hi < rows_total) mask_hi = s_mask[p.group == 1 ? g_hi : g_hi / p.group];
  }

  if (p.early_prefix) {     // now wait for the preceding kernel; then Q and the tiles that hold tree rows
    // (with the second promise, that Q and the tree's rows are final as well, nothing is waited for
    // here: the wait moves down to just before this kernel's first store)
    if (!p.early_query) grid_dependency_sync();
    else asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    load_q();
#pragma unroll
    for (int s = 0; s < PRE; ++s)
      if (t_begin + s < t_end && !prefetched[s]) load_tile(t_begin + s, s);
    cp_async_commit();
    cp_async_wait<0>();
  }

  float o[OT][4];
#pragma unroll
  for (int i = 0; i < OT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;     // l: this warp's keys only
  const int sw = lane & 7;                                               // (row & 7) of this lane's ldmatrix row
  const uint32_t a_row = (wm * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * 128;   // A-operand row of this lane
  const uint32_t q_frag = q_s + a_row, p_frag = p_s + a_row;             // chunk added per k-step

  for (int t = t_begin; t < t_end; ++t) {
    const int it = t - t_begin;
    cp_async_wait<PRE - 1>();
    __syncthreads();
    if (!C::FULL_RING) {   // refill the stage that was consumed one iteration ago
      const int tn = t + STAGES - 1;
      if (tn < t_end) load_tile(tn, (it + STAGES - 1) % STAGES);
      cp_async_commit();
    }
    const int stage = it % STAGES;
    const uint32_t kst = k_s + stage * C::TILE_BYTES, vst = v_s + stage * C::TILE_BYTES;
    const int kbase = wn * KC;

    // S = Q K^T for this warp's KC keys
    float s[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t qf[4];
      {
        const int c = ks * 2 + (lane >> 4);
        ldsm_x4(q_frag + (c >> 3) * ROWS * 128 + (((c & 7) ^ sw) << 4), qf);
      }
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t kb[4];
        const int key = kbase + np * 16 + (lane & 7) + (lane >> 4) * 8;
        ldsm_x4(kst + tile_off<KT>(key, ks * 2 + ((lane >> 3) & 1)), kb);
        mma_bf16(s[2 * np], qf, kb[0], kb[1]);
        mma_bf16(s[2 * np + 1], qf, kb[2], kb[3]);
      }
    }

    // scale into the exp2 domain; mask the tile that holds the prefix end / the tree
    const int key0 = t * KT + kbase;
    if (key0 + KC > L) {
      // bit j of vis_*: key key0 + j is visible to the row (every prefix key; tree keys by the
      // ancestor mask, whose bits at and above n are clear, so keys past the last one are hidden)
      const int rel0 = key0 - L;                       // > -KC
      unsigned long long vis_lo, vis_hi;
      if (rel0 >= 0) {
        vis_lo = rel0 < 64 ? mask_lo >> rel0 : 0ull;
        vis_hi = rel0 < 64 ? mask_hi >> rel0 : 0ull;
      } else {
        const unsigned long long pre = (1ull << -rel0) - 1ull;
        vis_lo = (mask_lo << -rel0) | pre;
        vis_hi = (mask_hi << -rel0) | pre;
      }
      vis_lo >>= tq * 2;
      vis_hi >>= tq * 2;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned long long v = (e & 2) ? vis_hi : vis_lo;
          s[nt][e] = ((v >> (nt * 8 + (e & 1))) & 1ull) ? s[nt][e] * p.scale_log2 : -INFINITY;
        }
      }
    } else {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[nt][e] *= p.scale_log2;
      }
    }

    // online softmax: row maxima over this warp's keys, then over the WN warps of the row group
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
    if (WN > 1) {
      if (tq == 0) {
        s_stat[wn][r_lo] = mx_lo;
        s_stat[wn][r_hi] = mx_hi;
      }
      group_sync();
#pragma unroll
      for (int w = 0; w < WN; ++w) {
        mx_lo = fmaxf(mx_lo, s_stat[w][r_lo]);
        mx_hi = fmaxf(mx_hi, s_stat[w][r_hi]);
      }
    }
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float use_lo = mn_lo == -INFINITY ? 0.f : mn_lo, use_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
    const float a_lo = fast_exp2(m_lo - use_lo), a_hi = fast_exp2(m_hi - use_hi);
    m_lo = mn_lo;
    m_hi = mn_hi;
    float sum_lo = 0.f, sum_hi = 0.f;
    uint32_t pf[NT / 2][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float p0 = fast_exp2(s[nt][0] - use_lo), p1 = fast_exp2(s[nt][1] - use_lo);
      const float p2 = fast_exp2(s[nt][2] - use_hi), p3 = fast_exp2(s[nt][3] - use_hi);
      sum_lo += p0 + p1;
      sum_hi += p2 + p3;
      pf[nt / 2][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[nt / 2][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    l_lo = l_lo * a_lo + sum_lo;
    l_hi = l_hi * a_hi + sum_hi;
#pragma unroll
    for (int i = 0; i < OT; ++i) {
      o[i][0] *= a_lo;
      o[i][1] *= a_lo;
      o[i][2] *= a_hi;
      o[i][3] *= a_hi;
    }

    if (WN > 1) {
      // probabilities -> shared memory (rows of 128 bytes, 16-byte chunks XORed with the row)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int c = wn * NT + nt;
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(p_s + r_lo * 128 + ((c ^ (r_lo & 7)) << 4) + tq * 4),
                     "r"(pf[nt / 2][(nt & 1) * 2 + 0]) : "memory");
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(p_s + r_hi * 128 + ((c ^ (r_hi & 7)) << 4) + tq * 4),
                     "r"(pf[nt / 2][(nt & 1) * 2 + 1]) : "memory");
      }
      group_sync();
      // O[:, this warp's columns] += P[all keys of the tile] V
#pragma unroll
      for (int kk = 0; kk < KT / 16; ++kk) {
        uint32_t pa[4];
        ldsm_x4(p_frag + (((kk * 2 + (lane >> 4)) ^ sw) << 4), pa);
#pragma unroll
        for (int dp = 0; dp < OT / 2; ++dp) {
          uint32_t vb[4];
          const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          ldsm_x4_t(vst + tile_off<KT>(key, wn * OT + dp * 2 + (lane >> 4)), vb);
          mma_bf16(o[2 * dp], pa, vb[0], vb[1]);
          mma_bf16(o[2 * dp + 1], pa, vb[2], vb[3]);
        }
      }
    } else {
      // one warp per row group: the probabilities stay in registers
#pragma unroll
      for (int kk = 0; kk < NT / 2; ++kk) {
#pragma unroll
        for (int dp = 0; dp < OT / 2; ++dp) {
          uint32_t vb[4];
          const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          ldsm_x4_t(vst + tile_off<KT>(key, dp * 2 + (lane >> 4)), vb);
          mma_bf16(o[2 * dp], pf[kk], vb[0], vb[1]);
          mma_bf16(o[2 * dp + 1], pf[kk], vb[2], vb[3]);
        }
      }
    }
    if (C::FULL_RING) {    // refill this tile's own stage once every warp has finished with it
      const int tn = t + STAGES;
      if (tn < t_end) {
        __syncthreads();
        load_tile(tn, stage);
      }
      cp_async_commit();
    }
  }
  cp_async_wait<0>();

  // ---- row sums: add up the WN warps' shares; the rows' largest |O| -----
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  float amax_lo = 0.f, amax_hi = 0.f;
  {     // (rows pass through the fp16 buffer of the merge even when there is a single split)
#pragma unroll
    for (int i = 0; i < OT; ++i) {
      amax_lo = fmaxf(amax_lo, fmaxf(fabsf(o[i][0]), fabsf(o[i][1])));
      amax_hi = fmaxf(amax_hi, fmaxf(fabsf(o[i][2]), fabsf(o[i][3])));
    }
    amax_lo = fmaxf(amax_lo, __shfl_xor_sync(0xffffffffu, amax_lo, 1));
    amax_lo = fmaxf(amax_lo, __shfl_xor_sync(0xffffffffu, amax_lo, 2));
    amax_hi = fmaxf(amax_hi, __shfl_xor_sync(0xffffffffu, amax_hi, 1));
    amax_hi = fmaxf(amax_hi, __shfl_xor_sync(0xffffffffu, amax_hi, 2));
  }
  if (WN > 1) {
    // (every warp of the group has read the last tile's maxima: that was before the tile's second barrier)
    if (tq == 0) {
      s_stat[wn][r_lo] = l_lo;
      s_stat[wn][r_hi] = l_hi;
      s_amax[wn][r_lo] = amax_lo;
      s_amax[wn][r_hi] = amax_hi;
    }
    group_sync();
    l_lo = l_hi = 0.f;
#pragma unroll
    for (int w = 0; w < WN; ++w) {
      l_lo += s_stat[w][r_lo];
      l_hi += s_stat[w][r_hi];
      amax_lo = fmaxf(amax_lo, s_amax[w][r_lo]);
      amax_hi = fmaxf(amax_hi, s_amax[w][r_hi]);
    }
  }

  // ---- merge the key splits of the cluster ------------------------------------------
  // Each CTA writes its per-row partial (m, l, O / l as scaled fp16, see row_scale: finer than the
  // bf16 output whatever the magnitude of V) into the owner's shared memory (once the owner's
  // buffer is free: at once if it is a buffer of its own, else after every CTA of the cluster has
  // left its key loop) with asynchronous stores that report to the owner's barrier; the owner
  // waits for its bytes, combines its n_splits partials and stores.
  unsigned char *recv = smem + C::RECV_OFFSET;                 // [slot][D] fp16
  if (n_splits > 1) {
    if (C::RECV_OWN) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // every peer is running
    else cluster.sync();                        // every peer has left its key loop: the rings are free
  } else if (!C::RECV_OWN) {
    __syncthreads();                            // all warps are done with the stage ring
  }
  {
    // The two lanes of a quad pair swap halves so that each holds four consecutive floats of one
    // row: even lanes of the pair keep the low row, odd lanes the high row; 16-byte stores.
    const bool odd = tq & 1;
    const int r = odd ? r_hi : r_lo;
    const int owner = r / rows_per, lr = r % rows_per;
    const int slot = split * rows_per + lr;
    unsigned char *ro = recv + (size_t)slot * D * 2;
    const float my_l = odd ? l_hi : l_lo;
    // (a row that saw no key in this split carries m = -inf and counts for nothing)
    const bool seen = (odd ? m_hi : m_lo) > -INFINITY && my_l > 0.f;
    const float inv_l = seen ? 1.f / my_l : 0.f;
    float down, up;
    row_scale((odd ? amax_hi : amax_lo) * inv_l, down, up);
    const bool remote = owner != split;           // (n_splits == 1: never)
    const uint32_t ro_c = remote ? map_to_cta(smem_u32(ro), owner) : 0u;
    const uint32_t bar_c = remote ? map_to_cta(recv_bar, owner) : 0u;
#pragma unroll
    for (int i = 0; i < OT; ++i) {
      const float s0 = odd ? o[i][0] : o[i][2], s1 = odd ? o[i][1] : o[i][3];
      const float g0 = __shfl_xor_sync(0xffffffffu, s0, 1), g1 = __shfl_xor_sync(0xffffffffu, s1, 1);
      const float4 v = odd ? make_float4(g0, g1, o[i][2], o[i][3]) : make_float4(o[i][0], o[i][1], g0, g1);
      const uint32_t h0 = pack_f16(v.x * inv_l * down, v.y * inv_l * down), h1 = pack_f16(v.z * inv_l * down, v.w * inv_l * down);
      // 8-column groups of a row are XOR-swizzled by the row to spread banks
      const int off = ((((wn * OT + i) ^ (lr & 7)) << 3) + (tq >> 1) * 4) * 2;
      if (remote) st_async_b32x2(ro_c + off, h0, h1, bar_c);
      else *reinterpret_cast<uint2 *>(ro + off) = make_uint2(h0, h1);
    }
    if (wn == 0 && tq < 2) {
      const float mm = seen ? (odd ? m_hi : m_lo) : -INFINITY, ll = seen ? my_l : 0.f;
      if (remote) st_async_f32x4(map_to_cta(smem_u32(r_ml + slot), owner), mm, ll, up, 0.f, bar_c);
      else r_ml[slot] = make_float4(mm, ll, up, 0.f);
    }
  }
  if (n_splits > 1) {
    __syncwarp();                     // the lanes' own-share stores come before lane 0's arrival
    if (lane == 0) mbar_arrive(recv_bar);
    // bounded: a peer that never delivers is reported, not waited for
    bool landed = mbar_try_wait(recv_bar, 0);
    if (!landed) {
      unsigned long long t0, t1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
      do {                                                    // at most 0.2 s
        landed = mbar_try_wait(recv_bar, 0);
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
      } while (!landed && t1 - t0 < 200000000ull);
    }
    if (!landed) {
      if (tid == 0) flag_status(p.dev_status, b, TWIG_DEV_INTERNAL);
      return;
    }
  } else {
    __syncthreads();
  }

  if (p.early_query) asm volatile("griddepcontrol.wait;" ::: "memory");     // stores are ordered after the predecessor
  {
    constexpr int TPR = D / 4;                        // threads per row, 4 floats each
    constexpr int RPP = C::THREADS / TPR;             // rows per pass
    const int c4 = (tid % TPR) * 4;
    for (int lr = tid / TPR; lr < rows_per; lr += RPP) {
      const int gr = row0 + split * rows_per + lr;
      if (gr >= rows_total) continue;
      float mv[8];
      float mstar = -INFINITY;
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        mv[sd] = sd < n_splits ? r_ml[sd * rows_per + lr].x : -INFINITY;
        mstar = fmaxf(mstar, mv[sd]);
      }
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float lsum = 0.f;
      const int col = (((c4 >> 3) ^ (lr & 7)) << 3) + (c4 & 7);
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        if (sd < n_splits) {
          const float4 ml = r_ml[sd * rows_per + lr];
          const float wl = fast_exp2(mv[sd] - mstar) * ml.y;
          lsum += wl;
          const float wgt = wl * ml.z;
          const uint2 raw = *reinterpret_cast<const uint2 *>(recv + ((size_t)(sd * rows_per + lr) * D + col) * 2);
          const float2 v01 = unpack_f16(raw.x), v23 = unpack_f16(raw.y);
          acc.x = fmaf(wgt, v01.x, acc.x);
          acc.y = fmaf(wgt, v01.y, acc.y);
          acc.z = fmaf(wgt, v23.x, acc.z);
          acc.w = fmaf(wgt, v23.y, acc.w);
        }
      }
      const float inv = 1.f / lsum;
      const int node = gr / p.group, g = gr % p.group;
      const int h = hk * p.group + g;
      uint2 packed;
      packed.x = pack_bf16(acc.x * inv, acc.y * inv);
      packed.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2 *>(p.out + (((long long)b * p.t_max + node) * p.n_q_heads + h) * D + c4) = packed;
      if (p.lse && c4 == 0)
        p.lse[((long long)b * p.n_q_heads + h) * p.t_max + node] = (mstar + log2f(lsum)) * 0.6931471805599453f;
    }
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
template <class C>
static twig_status launch_attn(const AttnParams &p, int batch, int n_splits, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_attn_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, p.n_kv_heads * p.row_blocks, batch);
  cfg.blockDim = dim3(C::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap ? 2 : 1;
  if (cudaLaunchKernelEx(&cfg, tree_attn_kernel<C>, p) != cudaSuccess) return TWIG_ERR_CUDA;
  return TWIG_OK;
}

int pick_splits(int items, int max_tiles, int ctas_per_sm, int forced) {
  if (forced > 0) return forced;
  int s = 1;
  // double the key splits while all CTAs still fit in one wave
  while (s < 8 && items * s * 2 <= ctas_per_sm * 148 && s * 2 <= max_tiles) s *= 2;
  return s;
}

// warps that share the 64 keys of a tile in the 16- and 32-row variants
#ifndef TWIG_SMALL_WN
#define TWIG_SMALL_WN 4
#endif

template <int D>
static twig_status dispatch_attn(AttnParams &p, int batch, int rows, cudaStream_t st) {
  using C16 = AttnCfg<D, 1, TWIG_SMALL_WN, 64 / TWIG_SMALL_WN, 2, 2>;
  using C32 = AttnCfg<D, 2, TWIG_SMALL_WN, 64 / TWIG_SMALL_WN, 2, 2>;
  using C64 = AttnCfg<D, 4, 2, 32, 2, 2>;
  using C128 = AttnCfg<D, 8, 1, 64, 2, 1>;
  const int rows_per_cta = rows <= 16 ? 16 : rows <= 32 ? 32 : rows <= 64 ? 64 : 128;
  p.row_blocks = (rows + rows_per_cta - 1) / rows_per_cta;
  if ((long long)p.n_kv_heads * p.row_blocks > 65535) return TWIG_ERR_UNSUPPORTED;
  const int max_tiles = (p.max_len + p.t_max + 63) / 64;
  const int n_splits = pick_splits(batch * p.n_kv_heads * p.row_blocks, max_tiles, 2, p.forced_splits);
  switch (rows_per_cta) {
    case 16: return launch_attn<C16>(p, batch, n_splits, st);
    case 32: return launch_attn<C32>(p, batch, n_splits, st);
    case 64: return launch_attn<C64>(p, batch, n_splits, st);
    default: return launch_attn<C128>(p, batch, n_splits, st);
  }
}

}  // namespace twig

using namespace twig;

extern "C" twig_status tree_verify_attention_ex(const void *q, const void *tree_k, const void *tree_v,
                                                const twig_kv *cache, int32_t layer,
                                                const int32_t *kv_len, const int32_t *n_nodes,
                                                const int32_t *parent, int32_t t_max,
                                                int32_t n_q_heads, float softmax_scale, void *out,
                                                float *lse, int32_t *dev_status, void *ws,
                                                size_t ws_bytes, void *stream, uint32_t flags) {
  if (!q || !tree_k || !tree_v || !kv_len || !n_nodes || !parent || !out) return TWIG_ERR_NULL;
  twig_status s = check_kv(cache);
  if (s != TWIG_OK) return s;
  if (t_max <= 0 || n_q_heads <= 0 || layer < 0 || layer >= cache->n_layers) return TWIG_ERR_SHAPE;
  if (n_q_heads % cache->n_kv_heads) return TWIG_ERR_SHAPE;
  if (t_max > TWIG_MAX_NODES) return TWIG_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(tree_k) || !aligned16(tree_v) || !aligned16(out)) return TWIG_ERR_ALIGN;
  const int kernel = (int)((flags >> 1) & 3u);
  const int splits = (int)((flags >> 8) & 15u);
  if (splits != 0 && splits != 1 && splits != 2 && splits != 4 && splits != 8) return TWIG_ERR_UNSUPPORTED;
  if (ws_bytes > 0 && (!ws || !aligned16(ws))) return ws ? TWIG_ERR_ALIGN : TWIG_ERR_NULL;

  AttnParams p;
  p.q = static_cast<const __nv_bfloat16 *>(q);
  p.tree_k = static_cast<const __nv_bfloat16 *>(tree_k);
  p.tree_v = static_cast<const __nv_bfloat16 *>(tree_v);
  p.cache_k = static_cast<const __nv_bfloat16 *>(cache->k) + layer * cache->stride_layer;
  p.cache_v = static_cast<const __nv_bfloat16 *>(cache->v) + layer * cache->stride_layer;
  p.cache_k0 = static_cast<const __nv_bfloat16 *>(cache->k);
  p.cache_v0 = static_cast<const __nv_bfloat16 *>(cache->v);
  p.c_sl = cache->stride_layer;
  p.layer = layer;
  p.n_layers = cache->n_layers;
  p.batch = cache->batch;
  p.c_sb = cache->stride_batch;
  p.c_sh = cache->stride_head;
  p.c_sp = cache->stride_pos;
  p.kv_len = kv_len;
  p.n_nodes = n_nodes;
  p.parent = parent;
  p.out = static_cast<__nv_bfloat16 *>(out);
  p.lse = lse;
  p.dev_status = dev_status;
  p.t_max = t_max;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = cache->n_kv_heads;
  p.group = n_q_heads / cache->n_kv_heads;
  p.max_len = cache->max_len;
  p.row_blocks = 1;
  p.overlap = (launch_overlap_enabled() && !(flags & TWIG_ATTN_PLAIN_LAUNCH)) ? 1 : 0;
  p.early_prefix = ((flags & TWIG_ATTN_EARLY_PREFIX) && p.overlap) ? 1 : 0;
  p.early_query = (p.early_prefix && (flags & TWIG_ATTN_EARLY_QUERY)) ? 1 : 0;
  p.forced_splits = splits;
  p.stream_policy = (int)((flags >> 12) & 3u);
  if (p.stream_policy == 3) return TWIG_ERR_UNSUPPORTED;
  p.ws = static_cast<unsigned char *>(ws);
  p.ws_bytes = ws_bytes;
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.f / sqrtf((float)cache->head_dim);
  p.scale_log2 = scale * 1.4426950408889634f;
  const int rows = t_max * p.group;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool umma_ok = cache->head_dim == 128 && softmax_scale >= 0.f;
  // A kernel named in the flags is the kernel that runs: what it cannot do is an error, never a
  // quiet change of kernel.
  if (kernel == TWIG_ATTN_KERNEL_TCGEN05 || kernel == TWIG_ATTN_KERNEL_STREAM) {
    if (!umma_ok) return TWIG_ERR_UNSUPPORTED;
    return kernel == TWIG_ATTN_KERNEL_STREAM ? launch_tree_attn_stream(p, cache->batch, rows, st)
                                             : launch_tree_attn_umma(p, cache->batch, rows, st);
  }
  if (kernel == TWIG_ATTN_KERNEL_AUTO && umma_ok) {
    // automatic choice: the tcgen05 kernel with cluster splits once there are more than 32 query rows
    // per kv head or enough (request, kv head) pairs to fill the GPU, the mma.sync kernel for small,
    // latency-bound calls.  (The persistent kernel measured slower than the cluster kernel on every
    // shape tried, so it only runs when it is named.)
    const bool big = rows > 32 || (long long)cache->batch * cache->n_kv_heads >= 148;
    if (big) {
      const twig_status us = launch_tree_attn_umma(p, cache->batch, rows, st);
      if (us != TWIG_ERR_UNSUPPORTED) return us;     // no tensor map for this layout: the mma.sync kernel
    }
  }
  return cache->head_dim == 128 ? dispatch_attn<128>(p, cache->batch, rows, st)
                                : dispatch_attn<64>(p, cache->batch, rows, st);
}

extern "C" twig_status tree_verify_attention(const void *q, const void *tree_k, const void *tree_v,
                                             const twig_kv *cache, int32_t layer,
                                             const int32_t *kv_len, const int32_t *n_nodes,
                                             const int32_t *parent, int32_t t_max,
                                             int32_t n_q_heads, float softmax_scale, void *out,
                                             float *lse, int32_t *dev_status, void *ws,
                                             size_t ws_bytes, void *stream) {
  return tree_verify_attention_ex(q, tree_k, tree_v, cache, layer, kv_len, n_nodes, parent, t_max, n_q_heads,
                                  softmax_scale, out, lse, dev_status, ws, ws_bytes, stream, 0u);
}
