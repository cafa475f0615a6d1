// Tree attention of the verification pass on the 5th-generation tensor cores
// (Sec. 5.4, Appendix A, Algorithm 2; Eq. 2 with the tree's ancestor mask).
//
// One CTA owns up to ROWS query rows (tree node x query head of one kv head) and a
// share of the key tiles (64 or 128 keys each).  Its warps (six, or ten with 128-row accumulators)
// have three roles that only meet at mbarriers:
//   warp 4 (loader)   brings K and V tiles (units K0 V0 K1 V1 ...) into a ring of five to eight
//                     slots (UmmaCfg::SLOTS) in the 128-byte-swizzled layout the matrix descriptors
//                     name: tiles that lie wholly in the cached prefix by TMA (two 64-column boxes of
//                     a 5-D tensor map over the cache, completion counted on the slot's mbarrier),
//                     the tile that holds the prefix end and the tree's own rows by 16-byte
//                     cp.async with zero fill; a slot is refilled when the MMA that read it
//                     has completed;
//   warp 5 (issuer)   one thread issues S(t) = Q K(t)^T (tcgen05.mma, M = 64 or 128, N = keys of a
//                     tile, K = 8 x 16) two tiles ahead into a double-buffered S in tensor memory, and
//                     O += P(t) V(t) (N = 128, V read MN-major, accumulating in tensor memory) as
//                     soon as the softmax warps have published P(t);
//   warps 0-3 (softmax; with 128-row accumulators also warps 6-9, which take the second half of
//                     every tile's keys): tcgen05.ld of S, running max / sum, P (bf16).  With up
//                     to 64 rows the products use M = 64, whose accumulator rows sit in lanes 0-15
//                     of each of the four 32-lane quadrants of tensor memory (row r in lane
//                     32 (r / 16) + r % 16), so every warp works on 16 rows and P goes to shared
//                     memory; with 128 rows M = 128 and row r is lane r.
// Blocks of 128 rows keep both A operands in tensor memory instead (Q, written once by the softmax
// warps, and P, written over the first half of the S tile it came from): see UmmaCfg.
// The running maximum is only raised when a tile exceeds it by more than 2^8; then (rarely)
// the O accumulator is rescaled in tensor memory (ld, multiply, st).  P stays below 2^8,
// which bf16 and the fp32 sums hold without loss of accuracy.
// The instruction multiplies 64 or 128 rows; rows past ROWS read whatever follows in
// shared memory and land in lanes nobody reads.  Key splits of a cluster are merged
// through distributed shared memory as in the mma.sync kernel (each CTA pushes its
// per-row partial to the row's owner); without splits every thread stores its own row.
// Every wait is bounded: if one runs out the request is flagged TWIG_DEV_INTERNAL.
#include <cooperative_groups.h>
#include <cuda.h>

#include <mutex>

#include "tcgen05_common.cuh"

namespace cg = cooperative_groups;

namespace twig {

namespace {

constexpr int kD = 128;          // head_dim
// warps 0-3 softmax, warp 4 loader, warp 5 MMA issuer; with 128-row accumulators warps 6-9 are a
// second softmax group (UmmaCfg::THREADS)
constexpr int kMaxSlots = 8;                      // ring of K / V tiles (K0 V0 K1 V1 K2 ...)
constexpr float kLazyMax = 8.f;                   // raise the running max only beyond this (log2 units)

// KT = keys per tile: 64 (two CTAs per SM, 256 tensor-memory columns each) or 128 (one CTA per SM
// with all 512 columns: half as many, twice as large MMA instructions per key).
template <int ROWS, int KT>
struct UmmaCfg {
  static constexpr int TILE_BYTES = KT * kD * 2;         // one K (or V) tile: 16 or 32 KB
  static constexpr int PANEL_BYTES = KT * 128;           // 64-column panel of a K/V tile
  // 128-row blocks keep the A operands of both products in tensor memory: Q (loaded once) and P
  // (written by the softmax warps over the first half of the S tile it came from).  Both products
  // then read only their B operand (K or V) through shared memory, whose port is what limits a
  // CTA that streams 8 KB per MMA instruction; and the 96 KB that Q and two P buffers took go to
  // the ring of K / V tiles.
  static constexpr bool TMEM_AB = ROWS == 128;
  static constexpr int Q_BYTES = TMEM_AB ? 0 : ROWS * kD * 2;     // two 64-column panels of ROWS x 128 B
  static constexpr int P_ONE = TMEM_AB ? 0 : ROWS * KT * 2;       // ROWS x KT keys bf16, KT/64 panels of ROWS x 128 B
  // two P buffers where shared memory allows: the softmax of tile t+1 then never waits for P(t) V(t)
  // (64-key tiles with two CTAs per SM: one more ring slot measured better than the second P buffer)
  static constexpr int P_BUFS = (ROWS <= 64 && KT == 64) ? 1 : 2;
  static constexpr int P_BYTES = P_BUFS * P_ONE;
  static constexpr int SLOTS = TMEM_AB ? (KT == 128 ? 6 : 8) : (ROWS == 32 && KT == 64) ? 6 : 5;
  static constexpr int RING_BYTES = SLOTS * TILE_BYTES;
  // S: [0,KT) and [KT,2KT); O: [2KT, 2KT+128); Q (TMEM_AB): [2KT+128, 2KT+192), 64 columns of bf16 pairs
  static constexpr uint32_t TMEM_COLS = (KT == 64 && !TMEM_AB) ? 256 : 512;
  static constexpr uint32_t O_COL = 2 * KT;
  static constexpr uint32_t Q_COL = 2 * KT + 128;
  static constexpr int MIN_CTAS = (KT == 64 && ROWS <= 64) ? 2 : 1;     // (128 rows: shared memory allows one CTA per SM)
  static constexpr int RECV_BYTES = ROWS * kD * 4;
  static_assert(RECV_BYTES <= RING_BYTES, "split-merge buffer must fit in the stage ring");
  static_assert(Q_BYTES % 1024 == 0 && P_BYTES % 1024 == 0, "swizzled tiles start on 1024 bytes");
  static_assert(SLOTS <= kMaxSlots, "ring barriers");
  static constexpr int SMEM_BYTES = Q_BYTES + P_BYTES + RING_BYTES;
  static constexpr int MMA_M = ROWS <= 64 ? 64 : 128;
  static constexpr int ROWS_PER_WARP = MMA_M == 64 ? 16 : 32;    // rows a softmax warp owns
  // 128-row accumulators: two warps share the rows of a lane quadrant, half of a tile's keys each
  static constexpr int SOFT_GROUPS = MMA_M == 128 ? 2 : 1;
  static constexpr int THREADS = 32 * (6 + 4 * (SOFT_GROUPS - 1));
};

template <int ROWS, int KT>
__global__ void __launch_bounds__(UmmaCfg<ROWS, KT>::THREADS, UmmaCfg<ROWS, KT>::MIN_CTAS)
tree_attn_umma_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap,
                      const __grid_constant__ CUtensorMap vmap) {
  using C = UmmaCfg<ROWS, KT>;
  constexpr int kTileBytes = C::TILE_BYTES, kPanelBytes = C::PANEL_BYTES, kSlots = C::SLOTS;
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long s_mask[TWIG_MAX_NODES];
  // one scratch area, used in turn for: the parent array (set-up), the values the two softmax
  // groups exchange (key loop; [tile parity][key half][row]), the received (m, l) pairs of the
  // split merge ([sender][owned row])
  __shared__ __align__(16) float s_scratch[2 * 2 * 128];
  int *s_par = reinterpret_cast<int *>(s_scratch);
  float (*s_pair)[2][128] = reinterpret_cast<float (*)[2][128]>(s_scratch);
  float4 *r_ml = reinterpret_cast<float4 *>(s_scratch);
  __shared__ __align__(8) unsigned long long s_recv_bar;      // counts what peers push to this CTA (split merge)
  // barriers: full[5], empty[5] (ring slots), s_ready[2], p_ready[2], o_done[2], q_ready
  __shared__ __align__(8) unsigned long long s_bar[2 * kMaxSlots + 7];
  __shared__ uint32_t s_tmem;
  __shared__ int s_bad, s_fail;
  __shared__ volatile int s_never;                   // stays 0

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, n_splits = gridDim.x;
  const int hk = blockIdx.y / p.row_blocks, rb = blockIdx.y % p.row_blocks;
  const int b = blockIdx.z;

  const uint32_t q_s = smem_u32(smem);
  const uint32_t p_s = q_s + C::Q_BYTES;
  const uint32_t ring_s = p_s + C::P_BYTES;
  const uint32_t bars = smem_u32(s_bar);
  auto bar_full = [&](int slot) { return bars + 8 * slot; };
  auto bar_empty = [&](int slot) { return bars + 8 * (kMaxSlots + slot); };
  auto bar_s = [&](int buf) { return bars + 8 * (2 * kMaxSlots + buf); };
  auto bar_p = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 2 + buf); };
  auto bar_o = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 4 + buf); };
  const uint32_t bar_q = bars + 8 * (2 * kMaxSlots + 6);
  constexpr int PB = C::P_BUFS;

  // ---- what needs nothing from global memory comes first, while the preceding kernel of the
  // stream may still be draining: barriers (all but the one whose count depends on the request)
  // and tensor memory ----
  if (tid == 0) {
    s_bad = 0;
    s_fail = 0;
    s_never = 0;
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(bar_full(i), 32);       // every loader lane arrives once per unit
      mbar_init(bar_empty(i), 1);       // one tcgen05.commit
    }
    mbar_init(bar_s(0), 1);
    mbar_init(bar_s(1), 1);
    mbar_init(bar_o(0), 1);
    mbar_init(bar_o(1), 1);
    if (!C::TMEM_AB) mbar_init(bar_q, 32);     // (with Q in tensor memory: one arrival per softmax warp, set below)
    if (n_splits > 1) {
      // split merge: one arrival that announces the peers' bytes (every peer sends each of this
      // CTA's ROWS / n_splits rows as 128 fp16 and (m, l, row scale, -)), one per softmax warp for this
      // CTA's own share
      mbar_init(smem_u32(&s_recv_bar), 1 + 4);
      mbar_arrive_expect_tx(smem_u32(&s_recv_bar), (uint32_t)((n_splits - 1) * (ROWS / n_splits) * (kD * 2 + 16)));
    }
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {         // the two tensor maps (kernel parameters) into the descriptor cache
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&kmap)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&vmap)) : "memory");
  }
  // every exit before the key loop hands the tensor memory back
  auto leave = [&]() {
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 5) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem), "r"(C::TMEM_COLS) : "memory");
  };

  grid_dependency_sync();
  // ---- per-request metadata; every exit below is uniform over the cluster ----
  const int n = p.n_nodes[b], L = p.kv_len[b];
  const int my_parent = tid < p.t_max ? p.parent[(long long)b * p.t_max + tid] : -1;
  const bool first = split == 0 && blockIdx.y == 0 && tid == 0;
  const int rows_total = n * p.group, row0 = rb * ROWS;
  if (n <= 0 || n > p.t_max || L < 0 || L > p.max_len || row0 >= rows_total) {
    if (first && (n < 0 || n > p.t_max)) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    else if (first && n > 0 && (L < 0 || L > p.max_len)) flag_status(p.dev_status, b, TWIG_DEV_OVERFLOW);
    leave();
    return;
  }

  const int NK = L + n;
  const int n_tiles = (NK + KT - 1) / KT;
  const int per = (n_tiles + n_splits - 1) / n_splits;
  const int t_begin = split * per;
  const int t_end = min(n_tiles, t_begin + per);
  const int n_my = max(0, t_end - t_begin);
  // softmax warps that own rows of this request (a prefix of warps 0-3)
  constexpr int RPW = C::ROWS_PER_WARP;
  const int n_soft = min((ROWS + RPW - 1) / RPW, (rows_total - row0 + RPW - 1) / RPW);

  // ---- parents, validation, ancestor masks ---------------
  __syncthreads();
  if (tid < n) {
    s_par[tid] = my_parent;
    if ((tid == 0) ? (my_parent != -1) : (my_parent < 0 || my_parent >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (first) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    leave();
    return;
  }
  if (tid < n) {
    unsigned long long m = 0;
    int x = tid;
    while (x >= 0) {
      m |= 1ull << x;
      x = s_par[x];
    }
    s_mask[tid] = m;
  }
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) mbar_init(bar_p(i), n_soft * C::SOFT_GROUPS);      // one arrival per softmax warp
    if (C::TMEM_AB) mbar_init(bar_q, n_soft * C::SOFT_GROUPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t tmem_o = tmem + C::O_COL;
  volatile int *fail = &s_fail;

  // per-row state of the softmax threads (also used by the epilogue)
  const int row_local = C::MMA_M == 64 ? 16 * warp + lane : tid;
  const bool row_active = warp < 4 && lane < RPW && row_local < ROWS;
  const int gr = row0 + row_local;
  const bool row_valid = row_active && gr < rows_total;
  float m_run = -INFINITY, l_run = 0.f;     // m_run is in the exp2 domain (scaled logits)
  const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);     // this warp's 32 lanes

  if (warp == 4) {
    // ================= loader =================
    const __nv_bfloat16 *ck = p.cache_k + b * p.c_sb + hk * p.c_sh;
    const __nv_bfloat16 *cv = p.cache_v + b * p.c_sb + hk * p.c_sh;
    const __nv_bfloat16 *tk = p.tree_k + ((long long)b * p.n_kv_heads + hk) * p.t_max * kD;
    const __nv_bfloat16 *tv = p.tree_v + ((long long)b * p.n_kv_heads + hk) * p.t_max * kD;
    const int c = lane & 15, rbase = lane >> 4;      // chunk c of rows rbase, rbase + 2, ...
    const uint32_t panel = (uint32_t)((c >> 3) * kPanelBytes);
    // Q tile (zero rows past the request's last row).  Lane pairs walk the rows two apart; the
    // (node, query head of the group) pair of a row is stepped, not divided.
    bool q_issued = false, q_published = false;
    auto issue_q = [&]() {
      int node = (row0 + rbase) / p.group, g = (row0 + rbase) % p.group;
      for (int r = rbase; r < ROWS; r += 2) {
        const bool valid = row0 + r < rows_total;
        const __nv_bfloat16 *src =
            p.q + (((long long)b * p.t_max + (valid ? node : 0)) * p.n_q_heads + hk * p.group + (valid ? g : 0)) * kD + c * 8;
        cp_async_16(q_s + (c >> 3) * ROWS * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, valid);
        g += 2;
        while (g >= p.group) {
          g -= p.group;
          ++node;
        }
      }
      cp_async_commit();
      q_issued = true;
    };
    auto publish_q = [&]() {                    // Q has landed: publish it once
      if (q_issued && !q_published) {
        cp_async_wait<0>();
        fence_async_smem();
        mbar_arrive(bar_q);
        q_published = true;
      }
    };
    const int n_units = 2 * n_my;
    bool ok = true;
    auto issue_unit = [&](int u) {
      const int slot = u % kSlots;
      const int t = t_begin + (u >> 1);
      const uint32_t dst = ring_s + slot * kTileBytes;
      if (t * KT + KT <= L) {                   // whole tile inside the cached prefix: two TMA boxes
        if (lane == 0) {
          mbar_arrive_expect_tx(bar_full(slot), kTileBytes);
          const CUtensorMap *map = (u & 1) ? &vmap : &kmap;
          tma_load_5d(dst, map, bar_full(slot), 0, t * KT, hk, b, p.layer);
          tma_load_5d(dst + kPanelBytes, map, bar_full(slot), 64, t * KT, hk, b, p.layer);
        } else {
          mbar_arrive(bar_full(slot));
        }
      } else {                                  // prefix end and / or tree rows: cp.async with zero fill
        const __nv_bfloat16 *cbase = (u & 1) ? cv : ck, *tbase = (u & 1) ? tv : tk;
#pragma unroll 4
        for (int i = 0; i < KT / 2; ++i) {
          const int r = rbase + 2 * i;
          const int vj = t * KT + r;
          const __nv_bfloat16 *src = cbase;
          bool valid = false;
          if (vj < L) {
            src = cbase + (long long)vj * p.c_sp + c * 8;
            valid = true;
          } else if (vj < NK) {
            src = tbase + (vj - L) * kD + c * 8;
            valid = true;
          }
          cp_async_16(dst + panel + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, valid);
        }
        cp_async_commit();
        cp_async_wait<0>();                     // (this also completes the Q copies, if they were issued)
        fence_async_smem();
        if (q_issued && !q_published) {
          mbar_arrive(bar_q);
          q_published = true;
        }
        mbar_arrive(bar_full(slot));
      }
    };
    // K of the first tile, then Q (what S(0) needs), then the rest of the first ring
    const int n_first = min(n_units, kSlots);
    if (n_first > 0) issue_unit(0);
    if (n_my > 0 && !C::TMEM_AB) issue_q();
    for (int u = 1; u < n_first; ++u) issue_unit(u);
    for (int u = n_first; u < n_units && ok; ++u) {
      publish_q();                              // (all ring slots are in flight by now)
      ok = mbar_wait(bar_empty(u % kSlots), (u / kSlots - 1) & 1, fail);
      if (!ok) break;
      issue_unit(u);
    }
    publish_q();
    if (!ok) s_fail = 1;
  } else if (warp == 5) {
    // ================= MMA issuer (one thread) =================
    if (lane == 0) {
      constexpr uint32_t kIdescS = instr_desc(C::MMA_M, KT, false), kIdescO = instr_desc(C::MMA_M, kD, true);
      bool ok = true;
      auto wait_full = [&](int u) {
        if (ok) ok = mbar_wait(bar_full(u % kSlots), (u / kSlots) & 1, fail);
        fence_async_smem();
        tc_fence_after();
      };
      auto issue_s = [&](int it) {            // S(it) = Q K(it)^T into S buffer it & 1
        const int u = 2 * it;
        wait_full(u);
        if (!ok) return;
        const uint32_t kb = ring_s + (u % kSlots) * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t ka = kb + (ks >> 2) * kPanelBytes + (ks & 3) * 32;
          if (C::TMEM_AB) {            // Q from tensor memory: 16 head-dim entries = 8 columns per step
            umma_ts(tmem + (it & 1) * KT, tmem + C::Q_COL + ks * 8, smem_desc(ka, 16), kIdescS, ks > 0);
          } else {
            const uint32_t qa = q_s + (ks >> 2) * ROWS * 128 + (ks & 3) * 32;
            umma(tmem + (it & 1) * KT, smem_desc(qa, 16), smem_desc(ka, 16), kIdescS, ks > 0);
          }
        }
        umma_commit(bar_s(it & 1));
        umma_commit(bar_empty(u % kSlots));
      };
      if (n_my > 0) {
        ok = mbar_wait(bar_q, 0, fail);         // Q is in shared memory
        issue_s(0);
      }
      if (n_my > 1) issue_s(1);
      for (int it = 0; it < n_my && ok; ++it) {
        const int u = 2 * it + 1;
        const int pb = it % PB;
        ok = mbar_wait(bar_p(pb), (it / PB) & 1, fail);   // P(it) is in shared memory, S(it) has been read
        wait_full(u);
        if (!ok) break;
        const uint32_t vb = ring_s + (u % kSlots) * kTileBytes;
#pragma unroll
        for (int j = 0; j < KT / 16; ++j) {        // 16 keys per step: V rows 16 j ..
          if (C::TMEM_AB)              // P(it) lies over the first half of S(it): 8 columns per step
            umma_ts(tmem_o, tmem + (it & 1) * KT + j * 8, smem_desc(vb + j * 2048, kPanelBytes), kIdescO, (it > 0) || (j > 0));
          else                         // P panel j / 4 in shared memory
            umma(tmem_o, smem_desc(p_s + pb * C::P_ONE + (j >> 2) * ROWS * 128 + (j & 3) * 32, 16),
                 smem_desc(vb + j * 2048, kPanelBytes), kIdescO, (it > 0) || (j > 0));
        }
        umma_commit(bar_o(pb));
        umma_commit(bar_empty(u % kSlots));
        if (it + 2 < n_my) issue_s(it + 2);
      }
      if (!ok) s_fail = 1;
    }
  } else if (warp < n_soft && C::MMA_M == 64) {
    // ================= softmax, 64-row accumulators =================
    // Such an accumulator keeps only 16 rows in a warp's 32 tensor-memory lanes; read one row per
    // lane, half of every warp would idle.  The 16-lane load shape spreads the 16 rows over all 32
    // lanes instead (lane t: rows t/4 and t/4 + 8, two adjacent columns of every 8-column group),
    // so a quad shares a row: maxima and sums take two shuffles, every lane does half the work.
    const int gq = lane >> 2, tq = lane & 3;
    const int r_lo = 16 * warp + gq, r_hi = r_lo + 8;
    const int g_lo = row0 + r_lo, g_hi = row0 + r_hi;
    const unsigned long long mask_lo = g_lo < rows_total ? s_mask[g_lo / p.group] : 0ull;
    const unsigned long long mask_hi = g_hi < rows_total ? s_mask[g_hi / p.group] : 0ull;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;     // l: this lane's columns only
    const int row_src = 4 * (lane & 7);          // a lane that holds row (lane & 15) of this warp
    constexpr int NH = KT / 64;
    bool ok = true;
    for (int it = 0; it < n_my; ++it) {
      const int t = t_begin + it;
      ok = mbar_wait(bar_s(it & 1), (it >> 1) & 1, fail);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t ts = t_lane + (it & 1) * KT;
      uint32_t sr[NH][32];
#pragma unroll
      for (int h = 0; h < NH; ++h) tmem_ld_16rows_64cols(ts + h * 64, sr[h]);
      tmem_ld_wait();
      // the keys that hold the prefix end and / or the tree are masked
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const int key0 = t * KT + h * 64;
        if (key0 + 64 > L) {
          // bit j of vis_*: key key0 + j is visible to the row (every prefix key; tree keys by the
          // ancestor mask, whose bits at and above n are clear)
          const int rel0 = key0 - L;               // > -64
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
          for (int g = 0; g < 8; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const unsigned long long v = (e & 2) ? vis_hi : vis_lo;
              if (!((v >> (g * 8 + (e & 1))) & 1ull)) sr[h][4 * g + e] = 0xff800000u;     // -inf
            }
        }
      }
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          mx_lo = fmaxf(mx_lo, fmaxf(__uint_as_float(sr[h][4 * g]), __uint_as_float(sr[h][4 * g + 1])));
          mx_hi = fmaxf(mx_hi, fmaxf(__uint_as_float(sr[h][4 * g + 2]), __uint_as_float(sr[h][4 * g + 3])));
        }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      mx_lo *= p.scale_log2;                      // scale > 0, so the max commutes with it
      mx_hi *= p.scale_log2;
      const bool raise_lo = mx_lo > m_lo + kLazyMax, raise_hi = mx_hi > m_hi + kLazyMax;   // also the first finite maximum
      const float mn_lo = raise_lo ? mx_lo : m_lo, mn_hi = raise_hi ? mx_hi : m_hi;
      const float use_lo = mn_lo == -INFINITY ? 0.f : mn_lo, use_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const int pb = it % PB;
      if (it >= PB) {                             // this P buffer is free once P(it-PB) V(it-PB) is done
        ok = mbar_wait(bar_o(pb), (it / PB - 1) & 1, fail);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
      }
      if (it > 0 && __any_sync(0xffffffffu, raise_lo || raise_hi)) {
        if (PB > 1) {                             // O must be stable: wait for P(it-1) V(it-1) as well
          ok = mbar_wait(bar_o((it - 1) % PB), ((it - 1) / PB) & 1, fail);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
        }
        const float a_lo = fast_exp2(m_lo - use_lo), a_hi = fast_exp2(m_hi - use_hi);   // 1 for rows that keep their maximum
        l_lo *= a_lo;
        l_hi *= a_hi;
        // O is read one row per lane (lanes 0-15 of the warp): fetch that row's factor from its quad
        const float al = __shfl_sync(0xffffffffu, a_lo, row_src), ah = __shfl_sync(0xffffffffu, a_hi, row_src);
        const float alpha = lane >= 16 ? 1.f : ((lane & 8) ? ah : al);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t v[32];
          tmem_ld32(t_lane + C::O_COL + ch * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
          tmem_st32(t_lane + C::O_COL + ch * 32, v);
        }
        tmem_st_wait();
      }
      m_lo = mn_lo;
      m_hi = mn_hi;
      // P = exp2(S * scale - m) as bf16 to shared memory (rows of 128 bytes per 64 keys, 16-byte
      // chunks XORed with the row), row sums
      float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const uint32_t pl = p_s + pb * C::P_ONE + h * ROWS * 128 + r_lo * 128 + tq * 4;
        const uint32_t ph = p_s + pb * C::P_ONE + h * ROWS * 128 + r_hi * 128 + tq * 4;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sr[h][4 * g]), p.scale_log2, -use_lo));
          const float p1 = poly_exp2(fmaf(__uint_as_float(sr[h][4 * g + 1]), p.scale_log2, -use_lo));
          const float p2 = fast_exp2(fmaf(__uint_as_float(sr[h][4 * g + 2]), p.scale_log2, -use_hi));
          const float p3 = poly_exp2(fmaf(__uint_as_float(sr[h][4 * g + 3]), p.scale_log2, -use_hi));
          sum_lo += p0 + p1;
          sum_hi += p2 + p3;
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(pl + ((g ^ (r_lo & 7)) << 4)), "r"(pack_bf16(p0, p1)) : "memory");
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(ph + ((g ^ (r_hi & 7)) << 4)), "r"(pack_bf16(p2, p3)) : "memory");
        }
      }
      l_lo += sum_lo;
      l_hi += sum_hi;
      fence_async_smem();            // P was written with ordinary stores
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p(pb));
    }
    if (ok && n_my > 0) {
      ok = mbar_wait(bar_o((n_my - 1) % PB), ((n_my - 1) / PB) & 1, fail);   // the last P V product has completed
      tc_fence_after();
    }
    // hand the rows' state to the one-row-per-lane layout of the epilogue (lanes 0-15)
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    {
      const float ml = __shfl_sync(0xffffffffu, m_lo, row_src), mh = __shfl_sync(0xffffffffu, m_hi, row_src);
      const float ll = __shfl_sync(0xffffffffu, l_lo, row_src), lh = __shfl_sync(0xffffffffu, l_hi, row_src);
      m_run = (lane & 8) ? mh : ml;
      l_run = (lane & 8) ? lh : ll;
    }
    if (!ok) s_fail = 1;
  } else if (C::MMA_M == 128 && (warp & 3) < n_soft) {
    // ================= softmax, 128-row accumulators =================
    // Lane quadrant q of tensor memory (rows 32q .. 32q+31, one per lane) is served by two warps:
    // warp q takes the first half of a tile's keys, the warp of 6..9 with the same index modulo 4
    // the second half.  They agree on the rows' maxima through shared memory; each keeps the row
    // sums of its own keys, rescales its half of O's columns and writes its half of P.  No wait
    // below is followed by a break: a failed wait marks the request and the rest runs through, so
    // that both warps meet at every pair barrier.
    const int quad = warp & 3, half = warp >= 6 ? 1 : 0;
    const int row = 32 * quad + lane;
    const int grow = row0 + row;
    const unsigned long long my_mask = grow < rows_total ? s_mask[grow / p.group] : 0ull;
    constexpr int NV = KT / 2;                  // keys of a tile this thread handles
    constexpr int NC = NV / 32;
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory"); };
    float m_r = -INFINITY, l_r = 0.f;           // l_r: this thread's keys only
    bool ok = true;
    if (C::TMEM_AB && n_my > 0) {
      // Q into tensor memory, once: the row's 128 bf16 are 64 columns of pairs (the pair of head-dim
      // entries 2c, 2c+1 in column c, the lower one in the low half: as they lie in memory); this
      // warp writes the half `half` of its rows' columns.  Rows past the last one are zero.
      uint32_t qw[32];
      if (grow < rows_total) {
        const int node = grow / p.group, g = grow % p.group;
        const uint4 *src = reinterpret_cast<const uint4 *>(
            p.q + (((long long)b * p.t_max + node) * p.n_q_heads + hk * p.group + g) * kD + half * 64);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 w = ld_nc_16(src + i);
          qw[4 * i] = w.x;
          qw[4 * i + 1] = w.y;
          qw[4 * i + 2] = w.z;
          qw[4 * i + 3] = w.w;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) qw[i] = 0u;
      }
      tmem_st32(t_lane + C::Q_COL + half * 32, qw);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_q);
    }
    for (int it = 0; it < n_my; ++it) {
      const int t = t_begin + it;
      ok = ok && mbar_wait(bar_s(it & 1), (it >> 1) & 1, fail);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      const uint32_t ts = t_lane + (it & 1) * KT + half * NV;
      uint32_t sr[NC][32];
#pragma unroll
      for (int c = 0; c < NC; ++c) tmem_ld32(ts + 32 * c, sr[c]);
      tmem_ld_wait();
      const int key0 = t * KT + half * NV;
      if (key0 + NV > L) {                      // the prefix end and / or the tree: mask
        const int rel0 = key0 - L;              // > -NV
        unsigned long long vis;                 // bit j: key key0 + j is visible to this row
        if (rel0 >= 0) vis = rel0 < 64 ? my_mask >> rel0 : 0ull;
        else vis = (my_mask << -rel0) | ((1ull << -rel0) - 1ull);
#pragma unroll
        for (int c = 0; c < NC; ++c)
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (!((vis >> (32 * c + j)) & 1ull)) sr[c][j] = 0xff800000u;     // -inf
      }
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < NC; ++c)
#pragma unroll
        for (int j = 0; j < 32; j += 2)
          mx = fmaxf(mx, fmaxf(__uint_as_float(sr[c][j]), __uint_as_float(sr[c][j + 1])));
      mx *= p.scale_log2;                       // scale > 0, so the max commutes with it
      s_pair[it & 1][half][row] = mx;
      pair_sync();
      mx = fmaxf(mx, s_pair[it & 1][half ^ 1][row]);
      const bool raise = mx > m_r + kLazyMax;   // also true for the first finite maximum
      const float m_new = raise ? mx : m_r;
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      const int pb = it % PB;
      // a P buffer in shared memory is free once P(it-PB) V(it-PB) is done; in tensor memory P(it)
      // lies over S(it), which was only computed after P(it-2) V(it-2) (the products run in order)
      if (!C::TMEM_AB && it >= PB) {
        ok = ok && mbar_wait(bar_o(pb), (it / PB - 1) & 1, fail);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
      }
      if (it > 0 && __any_sync(0xffffffffu, raise)) {     // (the same decision in both warps of the pair)
        if (PB > 1) {                           // O must be stable: wait for P(it-1) V(it-1) as well
          ok = ok && mbar_wait(bar_o((it - 1) % PB), ((it - 1) / PB) & 1, fail);
          ok = __all_sync(0xffffffffu, ok);
          tc_fence_after();
        }
        const float alpha = fast_exp2(m_r - m_use);       // 1 for rows that keep their maximum
        l_r *= alpha;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {        // this warp's 64 of O's 128 columns
          uint32_t v[32];
          const uint32_t col = t_lane + C::O_COL + half * 64 + ch * 32;
          tmem_ld32(col, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
          tmem_st32(col, v);
        }
        tmem_st_wait();
      }
      m_r = m_new;
      // P = exp2(S * scale - m) as bf16, row sums
      float sum0 = 0.f, sum1 = 0.f;
      if (C::TMEM_AB) {
        // into tensor memory, over the first half of this S tile's columns (the other warp of the pair
        // has read its S by now: the pair met above): key pairs (2c, 2c+1) in column c of the tile
        uint32_t pw[NV / 2];
#pragma unroll
        for (int c = 0; c < NV / 2; ++c) {
          const int j = 2 * c;
          const float p0 = fast_exp2(fmaf(__uint_as_float(sr[j >> 5][j & 31]), p.scale_log2, -m_use));
          const float p1 = poly_exp2(fmaf(__uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]), p.scale_log2, -m_use));
          sum0 += p0;
          sum1 += p1;
          pw[c] = pack_bf16(p0, p1);
        }
        const uint32_t pcol = t_lane + (it & 1) * KT + half * (NV / 2);
        if constexpr (NV / 2 == 32) tmem_st32(pcol, reinterpret_cast<const uint32_t (&)[32]>(pw));
        else tmem_st16(pcol, reinterpret_cast<const uint32_t (&)[16]>(pw));
        tmem_st_wait();
      } else {
        constexpr int panel = KT == 128 ? 1 : 0;  // with 128-key tiles the second half is the second 64-key panel
        const uint32_t prow = p_s + pb * C::P_ONE + half * panel * ROWS * 128 + row * 128;
        const int chunk0 = KT == 128 ? 0 : half * 4;
#pragma unroll
        for (int cc = 0; cc < NV / 8; ++cc) {     // chunk: 8 keys of this row
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j = cc * 8 + e * 2;
            const float p0 = fast_exp2(fmaf(__uint_as_float(sr[j >> 5][j & 31]), p.scale_log2, -m_use));
            const float p1 = poly_exp2(fmaf(__uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]), p.scale_log2, -m_use));
            sum0 += p0;
            sum1 += p1;
            w[e] = pack_bf16(p0, p1);
          }
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(prow + (((chunk0 + cc) ^ (row & 7)) << 4)), "r"(w[0]),
                       "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
        }
        fence_async_smem();            // P was written with ordinary stores
      }
      l_r += sum0 + sum1;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p(pb));
    }
    if (n_my > 0) {
      ok = ok && mbar_wait(bar_o((n_my - 1) % PB), ((n_my - 1) / PB) & 1, fail);   // the last P V product has completed
      tc_fence_after();
    }
    // row sums: add the other warp's share (the buffer of the parity no tile is using)
    s_pair[n_my & 1][half][row] = l_r;
    pair_sync();
    l_run = l_r + s_pair[n_my & 1][half ^ 1][row];
    m_run = m_r;
    if (!ok) s_fail = 1;
  }
  __syncthreads();
  const bool ok = s_fail == 0;
  if (!ok && tid == 0) flag_status(p.dev_status, b, TWIG_DEV_INTERNAL);
  const bool have_o = n_my > 0 && warp < n_soft && ok;      // this thread's O row is in tensor memory

  if (n_splits == 1) {
    // ---- no key splits: every thread finishes and stores its own row ---------------
    if (have_o) {                           // warp-uniform: the tensor-memory loads need the whole warp
      const float inv = 1.f / l_run;
      const int node = row_valid ? gr / p.group : 0, g = row_valid ? gr % p.group : 0;
      const int h = hk * p.group + g;
      __nv_bfloat16 *dst = p.out + (((long long)b * p.t_max + node) * p.n_q_heads + h) * kD;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32(t_lane + C::O_COL + ch * 32, v);
        tmem_ld_wait();
        if (row_valid) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(v[8 * c]) * inv, __uint_as_float(v[8 * c + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(v[8 * c + 2]) * inv, __uint_as_float(v[8 * c + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(v[8 * c + 4]) * inv, __uint_as_float(v[8 * c + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(v[8 * c + 6]) * inv, __uint_as_float(v[8 * c + 7]) * inv);
            st_16(dst + ch * 32 + 8 * c, w);
          }
        }
      }
      if (p.lse && row_valid)
        p.lse[((long long)b * p.n_q_heads + h) * p.t_max + node] = (m_run + log2f(l_run)) * 0.6931471805599453f;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
    return;
  }

  // ---- merge the key splits of the cluster ----
  // Every CTA owns ROWS / n_splits rows.  Once all CTAs have left their key loops (the receive
  // buffer lies in the stage ring) each thread sends its row's (m, l) and O / l as scaled fp16 (see
  // row_scale: finer than the bf16 output whatever the magnitude of V) to the row's owner: asynchronous stores that the owner's barrier counts, plain stores for the CTA's
  // own share.  The owner waits for its bytes (bounded), combines and stores.
  const int rows_per = ROWS / n_splits;
  unsigned char *recv = smem + C::Q_BYTES + C::P_BYTES;      // [sender * rows_per + owned row][128] fp16
  const uint32_t recv_bar = smem_u32(&s_recv_bar);
  cluster.sync();                          // every CTA has left its key loop: the rings are free
  if (warp < 4) {
    const int rl_ = row_active ? row_local : 0;
    const int owner = rl_ / rows_per, lr = rl_ % rows_per;
    const int slot = split * rows_per + lr;
    const bool remote = owner != split;
    unsigned char *ro = recv + (size_t)slot * kD * 2;
    const uint32_t ro_c = map_to_cta(smem_u32(ro), owner), bar_c = map_to_cta(recv_bar, owner);
    // (a row that saw no key in this split carries m = -inf and counts for nothing)
    const bool seen = have_o && m_run > -INFINITY && l_run > 0.f;
    const float inv_l = seen ? 1.f / l_run : 0.f;
    float amax = 0.f;
    if (have_o) {                           // warp-uniform: the row's largest |O|
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32(t_lane + C::O_COL + ch * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(__uint_as_float(v[j])));
      }
    }
    float down, up;
    row_scale(amax * inv_l, down, up);
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      uint32_t v[32];
      if (have_o) {                         // warp-uniform
        tmem_ld32(t_lane + C::O_COL + ch * 32, v);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 0u;
      }
      if (row_active) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {       // 16-byte chunks (8 columns) are XOR-swizzled by the row to spread banks
          uint32_t h[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            h[e] = pack_f16(__uint_as_float(v[8 * i + 2 * e]) * inv_l * down, __uint_as_float(v[8 * i + 2 * e + 1]) * inv_l * down);
          const int off = ((ch * 4 + i) ^ (lr & 15)) << 4;
          if (remote) st_async_b32x4(ro_c + off, h[0], h[1], h[2], h[3], bar_c);
          else *reinterpret_cast<uint4 *>(ro + off) = make_uint4(h[0], h[1], h[2], h[3]);
        }
      }
    }
    if (row_active) {
      const float mm = seen ? m_run : -INFINITY, ll = seen ? l_run : 0.f;
      if (remote) st_async_f32x4(map_to_cta(smem_u32(r_ml + slot), owner), mm, ll, up, 0.f, bar_c);
      else r_ml[slot] = make_float4(mm, ll, up, 0.f);
    }
    __syncwarp();                           // the lanes' own-share stores come before lane 0's arrival
    if (lane == 0) mbar_arrive(recv_bar);
  }
  tc_fence_before();
  __syncthreads();                          // every tensor-memory load of this CTA is done
  if (warp == 5) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
  {
    // (bounded by the spin limit alone: a CTA whose own key loop failed must still stay until its
    // peers' stores have landed)
    const bool landed = mbar_wait(recv_bar, 0, &s_never);
    if (!landed) {                          // a peer never delivered: reported, not waited for
      if (tid == 0) flag_status(p.dev_status, b, TWIG_DEV_INTERNAL);
      return;
    }
  }

  {
    constexpr int TPR = kD / 4;                       // 32 threads per row, 4 columns each
    constexpr int RPP = C::THREADS / TPR;
    const int i4 = tid % TPR;
    for (int lr = tid / TPR; lr < rows_per; lr += RPP) {
      const int grow = row0 + split * rows_per + lr;
      if (grow >= rows_total || !ok) continue;
      float mv[8];
      float mstar = -INFINITY;
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        mv[sd] = sd < n_splits ? r_ml[sd * rows_per + lr].x : -INFINITY;
        mstar = fmaxf(mstar, mv[sd]);
      }
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float lsum = 0.f;
      const int off = (((i4 >> 1) ^ (lr & 15)) << 4) + (i4 & 1) * 8;
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        if (sd < n_splits) {
          const float4 ml = r_ml[sd * rows_per + lr];
          const float wl = fast_exp2(mv[sd] - mstar) * ml.y;
          lsum += wl;
          const float wgt = wl * ml.z;
          const uint2 raw = *reinterpret_cast<const uint2 *>(recv + (size_t)(sd * rows_per + lr) * kD * 2 + off);
          const float2 v01 = unpack_f16(raw.x), v23 = unpack_f16(raw.y);
          acc.x = fmaf(wgt, v01.x, acc.x);
          acc.y = fmaf(wgt, v01.y, acc.y);
          acc.z = fmaf(wgt, v23.x, acc.z);
          acc.w = fmaf(wgt, v23.y, acc.w);
        }
      }
      const float inv = 1.f / lsum;
      const int node = grow / p.group, g = grow % p.group;
      const int h = hk * p.group + g;
      uint2 packed;
      packed.x = pack_bf16(acc.x * inv, acc.y * inv);
      packed.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2 *>(p.out + (((long long)b * p.t_max + node) * p.n_q_heads + h) * kD + i4 * 4) = packed;
      if (p.lse && i4 == 0)
        p.lse[((long long)b * p.n_q_heads + h) * p.t_max + node] = (mstar + log2f(lsum)) * 0.6931471805599453f;
    }
  }
}

}  // namespace

// ---- tensor maps over the whole K and V cache: dims (d, pos, head, batch, layer) ----
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapKey {
  const void *k, *v;
  long long sl, sb, sh, sp;
  int n_layers, batch, heads, max_len, box_rows;
  bool operator==(const MapKey &o) const {
    return k == o.k && v == o.v && sl == o.sl && sb == o.sb && sh == o.sh && sp == o.sp && n_layers == o.n_layers &&
           batch == o.batch && heads == o.heads && max_len == o.max_len && box_rows == o.box_rows;
  }
};
struct MapEntry {
  MapKey key;
  alignas(64) CUtensorMap kmap;
  alignas(64) CUtensorMap vmap;
  bool valid = false;
};

static bool encode_cache_map(EncodeTiledFn fn, CUtensorMap *out, const void *base, const MapKey &key) {
  const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)key.max_len, (cuuint64_t)key.heads, (cuuint64_t)key.batch,
                              (cuuint64_t)key.n_layers};
  const cuuint64_t strides[4] = {(cuuint64_t)key.sp * 2, (cuuint64_t)key.sh * 2, (cuuint64_t)key.sb * 2,
                                 (cuuint64_t)key.sl * 2};
  const cuuint32_t box[5] = {64, (cuuint32_t)key.box_rows, 1, 1, 1};   // 128 bytes x KT rows: one swizzled panel
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Copies the (cached) pair of maps for this cache layout into `out`; false when none can be made.
// (The table is a small ring that other threads may overwrite as soon as the lock is gone, so
// the caller gets a copy, not a pointer into it.)
bool cache_maps(const AttnParams &p, int box_rows, CacheMaps *out) {
  static std::mutex mu;
  static EncodeTiledFn fn = nullptr;
  static bool fn_tried = false;
  static MapEntry table[16];
  static int next = 0;
  std::lock_guard<std::mutex> lock(mu);
  if (!fn_tried) {
    fn_tried = true;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  if (!fn) return false;
  // strides must be multiples of 16 bytes, and every dimension but the last needs stride * extent in range
  if (p.c_sp <= 0 || p.c_sh <= 0 || p.c_sb < 0 || p.c_sl < 0) return false;
  MapKey key{p.cache_k0, p.cache_v0, p.n_layers > 1 ? p.c_sl : p.c_sp, p.batch > 1 ? p.c_sb : p.c_sp, p.c_sh, p.c_sp,
             p.n_layers, p.batch, p.n_kv_heads, p.max_len, box_rows};
  if (p.n_kv_heads == 1) key.sh = key.sp;      // a stride of an extent-1 dimension is never used
  for (auto &e : table)
    if (e.valid && e.key == key) {
      out->kmap = e.kmap;
      out->vmap = e.vmap;
      return true;
    }
  MapEntry &e = table[next];
  next = (next + 1) % 16;
  e.valid = false;
  if (!encode_cache_map(fn, &e.kmap, p.cache_k0, key) || !encode_cache_map(fn, &e.vmap, p.cache_v0, key)) return false;
  e.key = key;
  e.valid = true;
  out->kmap = e.kmap;
  out->vmap = e.vmap;
  return true;
}

namespace {

template <int ROWS, int KT>
twig_status launch_umma(const AttnParams &p, const CacheMaps *maps, int batch, int n_splits, cudaStream_t st) {
  using C = UmmaCfg<ROWS, KT>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_attn_umma_kernel<ROWS, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, p.n_kv_heads * p.row_blocks, batch);
  cfg.blockDim = dim3(UmmaCfg<ROWS, KT>::THREADS);
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
  if (cudaLaunchKernelEx(&cfg, tree_attn_umma_kernel<ROWS, KT>, p, maps->kmap, maps->vmap) != cudaSuccess)
    return TWIG_ERR_CUDA;
  return TWIG_OK;
}

}  // namespace

twig_status launch_tree_attn_umma(AttnParams &p, int batch, int rows, cudaStream_t st) {
  const int rows_per_cta = rows <= 32 ? 32 : rows <= 64 ? 64 : 128;
  p.row_blocks = (rows + rows_per_cta - 1) / rows_per_cta;
  if ((long long)p.n_kv_heads * p.row_blocks > 65535) return TWIG_ERR_UNSUPPORTED;
  const int items = batch * p.n_kv_heads * p.row_blocks;
  // Few, long work items: 128-key tiles, one CTA per SM (larger MMA instructions, all of tensor
  // memory).  Many items, or short caches: 64-key tiles, two CTAs per SM.
  const bool wide = items <= 148 && ((rows_per_cta == 128 && p.max_len >= 1024) || (rows_per_cta == 64 && p.max_len >= 4096));
  const int kt = wide ? 128 : 64;
  CacheMaps cm;
  if (!cache_maps(p, kt, &cm)) return TWIG_ERR_UNSUPPORTED;
  const CacheMaps *maps = &cm;
  const int max_tiles = (p.max_len + p.t_max + kt - 1) / kt;
  const int n_splits = pick_splits(items, max_tiles, wide ? 1 : 2, p.forced_splits);
  if (wide) {
    if (rows_per_cta == 64) return launch_umma<64, 128>(p, maps, batch, n_splits, st);
    return launch_umma<128, 128>(p, maps, batch, n_splits, st);
  }
  switch (rows_per_cta) {
    case 32: return launch_umma<32, 64>(p, maps, batch, n_splits, st);
    case 64: return launch_umma<64, 64>(p, maps, batch, n_splits, st);
    default: return launch_umma<128, 64>(p, maps, batch, n_splits, st);
  }
}

}  // namespace twig
