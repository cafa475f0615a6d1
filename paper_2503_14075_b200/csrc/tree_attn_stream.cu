// Tree attention of the verification pass (Sec. 5.4, Appendix A, Algorithm 2; Eq. 2 with the
// tree's ancestor mask) as ONE persistent tcgen05 kernel per call.
//
// Work: a call is a list of items (request, kv head, block of query rows), each a run of key
// tiles (cached prefix followed by the tree's own rows).  The grid has one CTA per SM slot; a CTA's
// share of the call is a list of segments (item, tile range), found on the device from the
// requests' lengths.  Tensor memory, barriers and the K/V ring are set up once per CTA and run
// through all of its segments; the loaders run ahead across segment borders, so the ring never
// drains between items.  Two ways of sharing, chosen on the device:
//   whole items  when no item is large next to a CTA's share: the items, longest first, are dealt
//                out to the CTAs back and forth (c, 2G-1-c, 2G+c, ...), every segment is a whole item;
//   equal shares when items are long or few: all tiles of all items, in item order, form one
//                sequence and CTA c takes the c-th equal share (+-1 tile) of it.
//
// A segment that covers its whole item is finished on the spot.  An item that straddles CTAs is
// finished by whichever of them arrives last: each writes its partial (row maxima, row sums,
// normalised rows as scaled fp16) to the caller's scratch and takes a ticket on the item; the
// last ticket holder adds up the partials and stores.  Nobody waits for another CTA.  Tickets
// return to zero, which is what the next call expects to find.
//
// Warp roles (they only meet at mbarriers):
//   softmax warps   tcgen05.ld of S, running max / sum, P (bf16) to shared memory, epilogue;
//   loader warp     the only producer: K / V tiles that lie wholly in the cached prefix by TMA (two
//                   64-column boxes of a 5-D tensor map over the cache, 128-byte swizzle); the tile
//                   that holds the prefix end and the tree's rows, and the Q tile of every segment
//                   (one or two segments ahead), by 16-byte cp.async with zero fill, completed lazily
//                   so that the TMA requests behind them are not held up;
//   issuer          one thread issues S = Q K^T two tiles ahead (double-buffered S in tensor memory)
//                   and O += P V (accumulator in tensor memory).
// Every wait is bounded; if one runs out the request is flagged TWIG_DEV_INTERNAL.
#include "tcgen05_common.cuh"

namespace twig {

namespace {

// 64-row blocks: Q tiles in flight and ring slots (what two CTAs per SM leave room for)
#ifndef TWIG_STREAM64_QB
#define TWIG_STREAM64_QB 2
#define TWIG_STREAM64_SLOTS 4
#endif

constexpr int kD = 128;                 // head_dim
constexpr float kLazyMax = 8.f;         // raise the running max only beyond this (log2 units)
constexpr int kStreamMaxBatch = 256;    // requests per call on this path
constexpr int kMaxSlots = 6;

// ---- the CTA's share of the work, as segments -------------------------------------------
struct Seg {
  int b, hk, rb;          // request, kv head, row block
  int t0, t1, tiles;      // tile range of this segment, tiles of the item
  int L, n;               // cached length and tree nodes of the request
  int item;               // ticket index of the item
  int gstart;             // position of the item's first tile in the global sequence
};

struct SegIter {
  const int *cum, *sL, *sn;   // shared memory: first global tile of every request (cum[B] = total)
  const int *cum_items;       // whole-item mode: first item rank of every request in sorted order
  const unsigned char *order; // whole-item mode: requests, longest items first
  int n_kv_heads, group, row_blocks, rows, kt;
  int pos, end, b;            // equal shares: position in the global tile sequence
  int whole, round, cta, n_cta, n_items, j;     // whole items: dealing round, position in sorted order
  __device__ __forceinline__ void fill(Seg &s, int idx) {
    const int rbs = (s.n * group + rows - 1) / rows;
    s.hk = idx / rbs;
    s.rb = idx - s.hk * rbs;
    s.item = (s.b * n_kv_heads + s.hk) * row_blocks + s.rb;
  }
  __device__ __forceinline__ bool next(Seg &s) {
    if (whole) {
      // item ranks of this CTA: c, 2G-1-c, 2G+c, 4G-1-c, ... (increasing)
      const int r = (round & 1) ? (round + 1) * n_cta - 1 - cta : round * n_cta + cta;
      if (r >= n_items) return false;
      ++round;
      while (cum_items[j + 1] <= r) ++j;
      s.b = order[j];
      s.n = sn[s.b];
      s.L = sL[s.b];
      s.tiles = (s.L + s.n + kt - 1) / kt;
      s.t0 = 0;
      s.t1 = s.tiles;
      s.gstart = 0;
      fill(s, r - cum_items[j]);
      return true;
    }
    if (pos >= end) return false;
    while (cum[b + 1] <= pos) ++b;
    s.b = b;
    s.n = sn[b];
    s.L = sL[b];
    s.tiles = (s.L + s.n + kt - 1) / kt;
    const int off = pos - cum[b];
    const int idx = off / s.tiles;
    s.t0 = off - idx * s.tiles;
    s.t1 = min(s.tiles, s.t0 + (end - pos));
    s.gstart = pos - s.t0;
    fill(s, idx);
    pos += s.t1 - s.t0;
    return true;
  }
};

// Equal shares of `total` tiles over `g` CTAs: the first total % g CTAs take one tile more.
__device__ __forceinline__ int share_begin(int c, int total, int g) {
  const int q = total / g, r = total - q * g;
  return c * q + min(c, r);
}
__device__ __forceinline__ int share_owner(int x, int total, int g) {
  const int q = total / g, r = total - q * g;
  const int cut = r * (q + 1);
  return x < cut ? x / (q + 1) : r + (x - cut) / q;     // (x >= cut with x < total implies q >= 1)
}

template <int ROWS, int KT, int QB, int SLOTS_>
struct StreamCfg {
  static constexpr int SLOTS = SLOTS_;
  static constexpr int TILE_BYTES = KT * kD * 2;         // one K (or V) tile
  static constexpr int PANEL_BYTES = KT * 128;           // 64-column panel of a K/V tile
  static constexpr int Q_ONE = ROWS * kD * 2;            // two 64-column panels of ROWS x 128 B
  static constexpr int P_ONE = ROWS * KT * 2;            // KT/64 panels of ROWS x 128 B
  static constexpr bool TWO_PER_SM = KT == 64 && ROWS <= 64;
  static constexpr int P_BUFS = TWO_PER_SM ? 1 : 2;
  static constexpr int Q_BYTES = QB * Q_ONE, P_BYTES = P_BUFS * P_ONE, RING_BYTES = SLOTS * TILE_BYTES;
  static constexpr int SMEM_BYTES = Q_BYTES + P_BYTES + RING_BYTES;
  static constexpr uint32_t TMEM_COLS = KT == 64 ? 256 : 512;   // S: [0,KT) and [KT,2KT); O: [2KT, 2KT+128)
  static constexpr uint32_t O_COL = 2 * KT;
  static constexpr int MIN_CTAS = TWO_PER_SM ? 2 : 1;
  static constexpr int MMA_M = ROWS <= 64 ? 64 : 128;
  static constexpr int ROWS_PER_WARP = MMA_M == 64 ? 16 : 32;
  static constexpr int NSOFT = ROWS / ROWS_PER_WARP;             // warps of a softmax group that own rows
  static constexpr int SOFT_GROUPS = MMA_M == 128 ? 2 : 1;       // 128-row accumulators: two warps per lane quadrant
  // warps 0-3: softmax group 0 (the first NSOFT of them), 4: loader, 5: issuer,
  // 6-9: softmax group 1 (128-row accumulators only; warp w serves the lane quadrant w % 4)
  static constexpr int WARPS = 6 + 4 * (SOFT_GROUPS - 1);
  static constexpr int THREADS = 32 * WARPS;
  static constexpr int SOFT_THREADS = 32 * NSOFT * SOFT_GROUPS;
  // scratch slot of one partial result: ROWS rows of 128 fp16 (16 chunks of [ROWS][16 bytes]), then
  // (m, l, scale, -) per row
  static constexpr int SLOT_BYTES = ROWS * (kD * 2 + 16);
  static_assert(Q_ONE % 1024 == 0 && P_ONE % 1024 == 0, "swizzled tiles start on 1024 bytes");
  static_assert(SLOTS <= kMaxSlots && SLOTS >= 3, "ring depth");
  static_assert(NSOFT >= 1 && NSOFT <= 4, "softmax warps");
};

template <int ROWS, int KT, int QB, int SLOTS_>
__global__ void __launch_bounds__(StreamCfg<ROWS, KT, QB, SLOTS_>::THREADS, StreamCfg<ROWS, KT, QB, SLOTS_>::MIN_CTAS)
tree_attn_stream_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap,
                        const __grid_constant__ CUtensorMap vmap, unsigned int *tickets,
                        unsigned char *slots) {
  using C = StreamCfg<ROWS, KT, QB, SLOTS_>;
  constexpr int kTileBytes = C::TILE_BYTES, kPanelBytes = C::PANEL_BYTES, kSlots = C::SLOTS;
  constexpr int PB = C::P_BUFS, RPW = C::ROWS_PER_WARP, NSOFT = C::NSOFT;
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long s_mask[TWIG_MAX_NODES];
  __shared__ int s_par[TWIG_MAX_NODES];
  __shared__ int s_cum[kStreamMaxBatch + 1], s_L[kStreamMaxBatch], s_n[kStreamMaxBatch];
  __shared__ unsigned char s_badtree[kStreamMaxBatch], s_order[kStreamMaxBatch];
  __shared__ int s_cumi[kStreamMaxBatch + 1], s_whole;
  __shared__ float s_pair[C::SOFT_GROUPS == 2 ? 2 : 1][2][C::SOFT_GROUPS == 2 ? 128 : 1];
  // barriers: full[6], empty[6] (ring slots), s_ready[2], p_ready[2], o_done[2], q_ready[2], q_free[2], o_free
  __shared__ __align__(8) unsigned long long s_bar[2 * kMaxSlots + 11];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail, s_last[2];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = p.batch;

  const uint32_t q_s = smem_u32(smem);
  const uint32_t p_s = q_s + C::Q_BYTES;
  const uint32_t ring_s = p_s + C::P_BYTES;
  const uint32_t bars = smem_u32(s_bar);
  auto bar_full = [&](int slot) { return bars + 8 * slot; };
  auto bar_empty = [&](int slot) { return bars + 8 * (kMaxSlots + slot); };
  auto bar_s = [&](int buf) { return bars + 8 * (2 * kMaxSlots + buf); };
  auto bar_p = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 2 + buf); };
  auto bar_o = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 4 + buf); };
  auto bar_q = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 6 + buf); };
  auto bar_qfree = [&](int buf) { return bars + 8 * (2 * kMaxSlots + 8 + buf); };
  const uint32_t bar_ofree = bars + 8 * (2 * kMaxSlots + 10);

  // ---- what needs nothing from global memory comes first, while the preceding kernel of the
  // stream may still be draining: barriers and tensor memory ----
  if (tid == 0) {
    s_fail = 0;
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(bar_full(i), 1);        // lane 0 of the loader warp: with the TMA's byte count, or after its cp.async copies
      mbar_init(bar_empty(i), 1);       // one tcgen05.commit
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_s(i), 1);
      mbar_init(bar_p(i), NSOFT * C::SOFT_GROUPS);     // one arrival per softmax warp
      mbar_init(bar_o(i), 1);
      mbar_init(bar_q(i), 1);
      mbar_init(bar_qfree(i), 1);
    }
    mbar_init(bar_ofree, NSOFT);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {         // the two tensor maps (kernel parameters) into the descriptor cache
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&kmap)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&vmap)) : "memory");
  }
  // Without the early-prefix promise nothing is read before the preceding kernel has completed.
  // With it the lengths, the trees and the cached prefix are read at once; what may still be in the
  // making (Q and the tree's rows) is fetched by warps that wait first, and everything this kernel
  // writes is written after that data has arrived.
  if (!p.early_prefix) grid_dependency_sync();
  else asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- requests: validation, tiles per request, the global tile sequence ----
  // (lengths and parents are requested together: one round trip to memory)
  constexpr int kParRegs = 4;
  const int n_par = B * p.t_max;
  const bool par_in_regs = n_par <= kParRegs * C::THREADS;
  int par_reg[kParRegs];
  if (par_in_regs) {
#pragma unroll
    for (int j = 0; j < kParRegs; ++j) {
      const int idx = tid + j * C::THREADS;
      par_reg[j] = idx < n_par ? p.parent[idx] : -1;
    }
  }
  for (int b = tid; b < B; b += C::THREADS) {
    const int n = p.n_nodes[b], L = p.kv_len[b];
    int use = n;
    if (n < 0 || n > p.t_max) {
      use = 0;
      if (blockIdx.x == 0) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    } else if (n > 0 && (L < 0 || L > p.max_len)) {
      use = 0;
      if (blockIdx.x == 0) flag_status(p.dev_status, b, TWIG_DEV_OVERFLOW);
    }
    s_n[b] = use;
    s_L[b] = L;
    s_badtree[b] = 0;
  }
  __syncthreads();
  if (par_in_regs) {
#pragma unroll
    for (int j = 0; j < kParRegs; ++j) {
      const int idx = tid + j * C::THREADS;
      if (idx < n_par) {
        const int b = idx / p.t_max, i = idx - b * p.t_max;
        if (i < s_n[b] && ((i == 0) ? (par_reg[j] != -1) : (par_reg[j] < 0 || par_reg[j] >= i))) s_badtree[b] = 1;
      }
    }
  } else {
    for (int idx = tid; idx < n_par; idx += C::THREADS) {
      const int b = idx / p.t_max, i = idx - b * p.t_max;
      if (i < s_n[b]) {
        const int pr = p.parent[idx];
        if ((i == 0) ? (pr != -1) : (pr < 0 || pr >= i)) s_badtree[b] = 1;
      }
    }
  }
  __syncthreads();
  for (int b = tid; b < B; b += C::THREADS)
    if (s_badtree[b]) {
      if (blockIdx.x == 0) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
      s_n[b] = 0;
    }
  __syncthreads();
  // requests by the length of their items, longest first (equal lengths: lower index first)
  for (int b = tid; b < B; b += C::THREADS) {
    const int mine = s_n[b] > 0 ? (s_L[b] + s_n[b] + KT - 1) / KT : 0;
    int rank = 0;
    for (int o = 0; o < B; ++o) {
      const int other = s_n[o] > 0 ? (s_L[o] + s_n[o] + KT - 1) / KT : 0;
      rank += (other > mine || (other == mine && o < b)) ? 1 : 0;
    }
    s_order[rank] = (unsigned char)b;
  }
  __syncthreads();
  if (warp == 0) {
    // eight requests per lane: tiles of request b = (kv heads x row blocks) items of ceil((L + n) / KT)
    // tiles, in request order; items per request in sorted order
    constexpr int PER = kStreamMaxBatch / 32;
    int loc[PER], loci[PER];
    int sum = 0, sumi = 0, mx = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int b = lane * PER + j;
      int t = 0, it = 0;
      if (b < B) {
        const int n = s_n[b];
        if (n > 0) t = ((s_L[b] + n + KT - 1) / KT) * p.n_kv_heads * ((n * p.group + ROWS - 1) / ROWS);
        const int bs = s_order[b], ns = s_n[bs];
        if (ns > 0) {
          it = p.n_kv_heads * ((ns * p.group + ROWS - 1) / ROWS);
          mx = max(mx, (s_L[bs] + ns + KT - 1) / KT);
        }
      }
      loc[j] = sum;
      loci[j] = sumi;
      sum += t;
      sumi += it;
    }
    int inc = sum, inci = sumi;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, inc, o), yi = __shfl_up_sync(0xffffffffu, inci, o);
      if (lane >= o) {
        inc += y;
        inci += yi;
      }
      mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const int base = inc - sum, basei = inci - sumi;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int b = lane * PER + j;
      if (b < B) {
        s_cum[b] = base + loc[j];
        s_cumi[b] = basei + loci[j];
      }
    }
    if (lane == 31) {      // (requests past B count nothing)
      s_cum[B] = inc;
      s_cumi[B] = inci;
      // Whole items when every CTA gets one and none of them is long next to a CTA's share of the
      // tiles (an item that is not split costs its CTA up to its own length in imbalance; a split
      // costs a trip through scratch memory, a few tiles' worth).
      const int n_cta = (int)gridDim.x;
      int whole = inci >= n_cta && mx <= max(12, inc / (2 * n_cta));
      if (p.stream_policy == 1) whole = 0;
      if (p.stream_policy == 2) whole = 1;
      s_whole = whole;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t tmem_o = tmem + C::O_COL;
  volatile int *fail = &s_fail;
  const int total = s_cum[B];
  const int G = gridDim.x;
  const int g_begin = share_begin(blockIdx.x, total, G), g_end = share_begin(blockIdx.x + 1, total, G);
  auto make_iter = [&]() {
    SegIter it;
    it.cum = s_cum;
    it.sL = s_L;
    it.sn = s_n;
    it.cum_items = s_cumi;
    it.order = s_order;
    it.whole = s_whole;
    it.round = 0;
    it.cta = (int)blockIdx.x;
    it.n_cta = (int)gridDim.x;
    it.n_items = s_cumi[B];
    it.j = 0;
    it.n_kv_heads = p.n_kv_heads;
    it.group = p.group;
    it.row_blocks = p.row_blocks;
    it.rows = ROWS;
    it.kt = KT;
    it.pos = g_begin;
    it.end = g_end;
    it.b = 0;
    return it;
  };

  if (warp == 4) {
    // ================= loader warp: the only producer of the ring and of the Q tiles =================
    // Tiles that lie wholly inside the cached prefix come by TMA (lane 0: two 64-column boxes per
    // tile); the tile that holds the prefix end and / or the tree's rows, and the Q tile of every
    // segment, by 16-byte cp.async with zero fill from all lanes.  Those copies are not waited for on
    // the spot: up to two groups of them stay in flight while the warp goes on requesting tiles, and
    // they are completed (wait, proxy fence, arrival on their barriers) when a third group comes or
    // when the warp would block on a barrier anyway.  One producer per barrier: every parity wait
    // below is for the phase that directly precedes the next use.
    SegIter it = make_iter(), ahead = make_iter();
    Seg s, sa;
    int u = 0;
    bool ok = true;
    bool waited_dep = !p.early_prefix;               // Q and the tree's rows may still be in the making
    // groups in flight, oldest first: ring slots (or -1) and a Q buffer (or -1) whose barriers they complete
    int g_slot0[2] = {-1, -1}, g_slot1[2] = {-1, -1}, g_q[2] = {-1, -1};
    int n_groups = 0;
    auto arrive_group = [&](int g) {
      if (lane == 0) {
        if (g_slot0[g] >= 0) mbar_arrive(bar_full(g_slot0[g]));
        if (g_slot1[g] >= 0) mbar_arrive(bar_full(g_slot1[g]));
        if (g_q[g] >= 0) mbar_arrive(bar_q(g_q[g]));
      }
    };
    auto complete_oldest = [&]() {              // (with two groups in flight: the older one)
      if (n_groups == 2) cp_async_wait<1>();
      else cp_async_wait<0>();
      fence_async_smem();
      __syncwarp();
      arrive_group(0);
      g_slot0[0] = g_slot0[1];
      g_slot1[0] = g_slot1[1];
      g_q[0] = g_q[1];
      --n_groups;
    };
    auto complete_all = [&]() {
      while (n_groups > 0) complete_oldest();
    };
    auto open_group = [&](int slot0, int slot1, int qbuf) {     // after the copies were issued
      cp_async_commit();
      g_slot0[n_groups] = slot0;
      g_slot1[n_groups] = slot1;
      g_q[n_groups] = qbuf;
      ++n_groups;
    };
    // a wait that would block first completes what is in flight (nothing is lost by waiting there)
    auto wait_bar = [&](uint32_t bar, uint32_t parity) {
      bool ready = mbar_try_wait(bar, parity);
      ready = __all_sync(0xffffffffu, ready);
      if (ready) return;
      complete_all();
      ok = mbar_wait(bar, parity, fail);
      ok = __all_sync(0xffffffffu, ok);
    };
    const int c = lane & 15, rbase = lane >> 4;      // chunk c of rows rbase, rbase + 2, ...
    const uint32_t panel = (uint32_t)((c >> 3) * kPanelBytes);
    int q_next = 0;                                   // segments whose Q tile has been requested
    auto request_q = [&]() {                          // the Q tile of segment q_next, if there is one
      if (!ahead.next(sa)) {
        q_next = 1 << 30;
        return;
      }
      const int buf = q_next % QB;
      // the buffer's previous segment is done with it once all of its S products have completed
      if (q_next >= QB) wait_bar(bar_qfree(buf), (q_next / QB - 1) & 1);
      if (!ok) return;
      if (!waited_dep) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited_dep = true;
      }
      if (n_groups == 2) complete_oldest();
      // zero rows past the request's last row.  Lane pairs walk the rows two apart; the (node, query
      // head of the group) pair of a row is stepped, not divided.
      const uint32_t qb = q_s + buf * C::Q_ONE;
      const int row0 = sa.rb * ROWS, rows_total = sa.n * p.group;
      int node = (row0 + rbase) / p.group, g = (row0 + rbase) % p.group;
      for (int r = rbase; r < ROWS; r += 2) {
        const bool valid = row0 + r < rows_total;
        const __nv_bfloat16 *src =
            p.q + (((long long)sa.b * p.t_max + (valid ? node : 0)) * p.n_q_heads + sa.hk * p.group + (valid ? g : 0)) * kD + c * 8;
        cp_async_16(qb + (c >> 3) * ROWS * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, valid);
        g += 2;
        while (g >= p.group) {
          g -= p.group;
          ++node;
        }
      }
      open_group(-1, -1, buf);
      ++q_next;
    };
    for (int si = 0; ok && it.next(s); ++si) {
      if (si == 0) request_q();                       // Q of the first segment goes out before its tiles
      const __nv_bfloat16 *ck = p.cache_k + s.b * p.c_sb + s.hk * p.c_sh;
      const __nv_bfloat16 *cv = p.cache_v + s.b * p.c_sb + s.hk * p.c_sh;
      const __nv_bfloat16 *tk = p.tree_k + ((long long)s.b * p.n_kv_heads + s.hk) * p.t_max * kD;
      const __nv_bfloat16 *tv = p.tree_v + ((long long)s.b * p.n_kv_heads + s.hk) * p.t_max * kD;
      const int NK = s.L + s.n;
      for (int t = s.t0; t < s.t1 && ok; ++t, u += 2) {
        const bool pure = t * KT + KT <= s.L;
        if (!pure) {
          if (!waited_dep) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited_dep = true;
          }
          if (n_groups == 2) complete_oldest();
        }
        int slots_kv[2];
#pragma unroll 1
        for (int kv = 0; kv < 2 && ok; ++kv) {
          const int uu = u + kv, slot = uu % kSlots;
          slots_kv[kv] = slot;
          if (uu >= kSlots) wait_bar(bar_empty(slot), (uu / kSlots - 1) & 1);
          if (!ok) break;
          const uint32_t dst = ring_s + slot * kTileBytes;
          if (pure) {
            if (lane == 0) {
              mbar_arrive_expect_tx(bar_full(slot), kTileBytes);
              const CUtensorMap *map = kv ? &vmap : &kmap;
              tma_load_5d(dst, map, bar_full(slot), 0, t * KT, s.hk, s.b, p.layer);
              tma_load_5d(dst + kPanelBytes, map, bar_full(slot), 64, t * KT, s.hk, s.b, p.layer);
            }
          } else {
            const __nv_bfloat16 *cbase = kv ? cv : ck, *tbase = kv ? tv : tk;
#pragma unroll 4
            for (int i = 0; i < KT / 2; ++i) {
              const int r = rbase + 2 * i;
              const int vj = t * KT + r;
              const __nv_bfloat16 *src = cbase;
              bool valid = false;
              if (vj < s.L) {
                src = cbase + (long long)vj * p.c_sp + c * 8;
                valid = true;
              } else if (vj < NK) {
                src = tbase + (vj - s.L) * kD + c * 8;
                valid = true;
              }
              cp_async_16(dst + panel + r * 128 + (((c & 7) ^ (r & 7)) << 4), src, valid);
            }
          }
        }
        // (a wait that failed between the two halves leaves copies without a group: they are
        // committed and waited for below like the rest, their barrier is never completed)
        if (!pure) {
          if (ok) open_group(slots_kv[0], slots_kv[1], -1);
          else cp_async_commit();
        }
        // the next segments' Q tiles, as early as their buffers can be free: with two buffers after
        // this segment's first tile, with one after its last
        if (ok && (QB > 1 ? (q_next <= si + QB - 1 && t == s.t0) : (q_next <= si + 1 && t == s.t1 - 1))) request_q();
      }
    }
    if (ok) complete_all();
    else {
      // giving up: the copies and TMA requests already made still write into this CTA's shared memory,
      // so the CTA stays for longer than any of them can take before it leaves
      cp_async_wait<0>();
      s_fail = 1;
      unsigned long long t0, t1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
      do {
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
      } while (t1 - t0 < 100000ull);                 // 0.1 ms
    }
    // every CTA carries the dependency on its predecessor on to its successor
    if (!waited_dep) asm volatile("griddepcontrol.wait;" ::: "memory");
  } else if (warp == 5) {
    // ================= MMA issuer (one thread) =================
    if (lane == 0) {
      constexpr uint32_t kIdescS = instr_desc(C::MMA_M, KT, false), kIdescO = instr_desc(C::MMA_M, kD, true);
      bool ok = true;
      // two cursors over the CTA's tiles: S products run two tiles ahead of the P V products
      SegIter it_s = make_iter(), it_o = make_iter();
      Seg ss, so;
      bool have_s = it_s.next(ss), have_o = it_o.next(so);
      int ts = have_s ? ss.t0 : 0, to = have_o ? so.t0 : 0;     // tile within the segment
      int si_s = 0, si_o = 0;                                   // segment index of each cursor
      int gs = 0;                                               // running tile index of the S cursor
      auto wait_full = [&](int u) {
        if (ok) ok = mbar_wait(bar_full(u % kSlots), (u / kSlots) & 1, fail);
        fence_async_smem();
        tc_fence_after();
      };
      auto issue_s = [&]() {                  // S(gs) = Q K^T into S buffer gs & 1; advances the S cursor
        if (!have_s || !ok) return;
        const int qbuf = si_s % QB;
        if (ts == ss.t0) ok = mbar_wait(bar_q(qbuf), (si_s / QB) & 1, fail);     // the segment's Q has landed
        const int u = 2 * gs;
        wait_full(u);
        if (!ok) return;
        const uint32_t kb = ring_s + (u % kSlots) * kTileBytes;
        const uint32_t qb = q_s + qbuf * C::Q_ONE;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
          const uint32_t qa = qb + (ks >> 2) * ROWS * 128 + (ks & 3) * 32;
          const uint32_t ka = kb + (ks >> 2) * kPanelBytes + (ks & 3) * 32;
          umma(tmem + (gs & 1) * KT, smem_desc(qa, 16), smem_desc(ka, 16), kIdescS, ks > 0);
        }
        umma_commit(bar_s(gs & 1));
        umma_commit(bar_empty(u % kSlots));
        if (ts == ss.t1 - 1) umma_commit(bar_qfree(qbuf));       // the last product that reads this Q tile
        ++gs;
        if (++ts >= ss.t1) {
          have_s = it_s.next(ss);
          ts = ss.t0;
          ++si_s;
        }
      };
      issue_s();
      issue_s();
      for (int go = 0; have_o && ok; ++go) {
        const int u = 2 * go + 1;
        const int pb = go % PB;
        ok = mbar_wait(bar_p(pb), (go / PB) & 1, fail);   // P(go) is in shared memory, S(go) has been read
        wait_full(u);
        const bool first = to == so.t0;
        // the accumulator is overwritten: the previous segment's epilogue must have read it
        if (ok && first && si_o > 0) {
          ok = mbar_wait(bar_ofree, (si_o - 1) & 1, fail);
          tc_fence_after();
        }
        if (!ok) break;
        const uint32_t vb = ring_s + (u % kSlots) * kTileBytes;
#pragma unroll
        for (int j = 0; j < KT / 16; ++j)          // 16 keys per step: P panel j / 4, V rows 16 j ..
          umma(tmem_o, smem_desc(p_s + pb * C::P_ONE + (j >> 2) * ROWS * 128 + (j & 3) * 32, 16),
               smem_desc(vb + j * 2048, kPanelBytes), kIdescO, (!first) || (j > 0));
        umma_commit(bar_o(pb));
        umma_commit(bar_empty(u % kSlots));
        if (++to >= so.t1) {
          have_o = it_o.next(so);
          to = so.t0;
          ++si_o;
        }
        issue_s();
      }
      if (!ok) s_fail = 1;
    }
  } else if ((warp & 3) < NSOFT && (warp < 4 || warp >= 6)) {
    // ================= softmax warps =================
    const int quad = warp & 3, half = warp >= 6 ? 1 : 0;
    const int stid = (half * NSOFT + quad) * 32 + lane;              // index among the softmax threads
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);    // this warp's 32 tensor-memory lanes
    auto soft_sync = [&]() { asm volatile("bar.sync 5, %0;" ::"n"(C::SOFT_THREADS) : "memory"); };
    auto group0_sync = [&]() { asm volatile("bar.sync 6, %0;" ::"n"(32 * NSOFT) : "memory"); };
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory"); };
    // the row this thread owns in the epilogue (one row per lane; 64-row accumulators keep 16 rows
    // in lanes 0-15 of a warp's quadrant)
    const int row_local = C::MMA_M == 64 ? 16 * quad + lane : 32 * quad + lane;
    const bool row_active = half == 0 && lane < RPW;
    SegIter it = make_iter();
    Seg s;
    // A wait that runs out marks the CTA as failed (every later wait of every role then gives up at
    // once) but no softmax warp leaves its loops early: they all meet at the named barriers below, so
    // they all have to reach them.  A failed CTA stores nothing more.
    bool ok = true;
    auto check = [&](bool waited) {
      ok = __all_sync(0xffffffffu, ok && waited);
      if (!ok) s_fail = 1;
    };
    int gt = 0;            // running tile index of this CTA
    int mask_b = -1;       // request whose ancestor masks are in s_mask
    int n_partial = 0;     // partial segments so far (the ticket's hand-over word alternates)
    while (it.next(s)) {
      const int row0 = s.rb * ROWS, rows_total = s.n * p.group;
      const int n_it = s.t1 - s.t0;
      // ---- ancestor masks of the request, if this segment reaches past the prefix ----
      if (s.t1 * KT > s.L && mask_b != s.b) {
        soft_sync();                               // nobody still reads the previous request's masks
        if (stid < s.n) s_par[stid] = p.parent[(long long)s.b * p.t_max + stid];
        if (C::SOFT_THREADS < TWIG_MAX_NODES && stid + C::SOFT_THREADS < s.n)
          s_par[stid + C::SOFT_THREADS] = p.parent[(long long)s.b * p.t_max + stid + C::SOFT_THREADS];
        soft_sync();
        for (int i = stid; i < s.n; i += C::SOFT_THREADS) {
          unsigned long long m = 0;
          int x = i;
          while (x >= 0) {                         // parent[x] < x was checked for the whole request
            m |= 1ull << x;
            x = s_par[x];
          }
          s_mask[i] = m;
        }
        soft_sync();
        mask_b = s.b;
      }
      float m_run = -INFINITY, l_run = 0.f;        // of the row this thread owns in the epilogue

      if (C::MMA_M == 64) {
        // Such an accumulator keeps only 16 rows in a warp's 32 tensor-memory lanes; the 16-lane load
        // shape spreads them over all 32 lanes (lane t: rows t/4 and t/4 + 8, two adjacent columns of
        // every 8-column group), so a quad shares a row: maxima and sums take two shuffles.
        const int gq = lane >> 2, tq = lane & 3;
        const int r_lo = 16 * quad + gq, r_hi = r_lo + 8;
        const int g_lo = row0 + r_lo, g_hi = row0 + r_hi;
        const bool need_mask = s.t1 * KT > s.L;
        const unsigned long long mask_lo = (need_mask && g_lo < rows_total) ? s_mask[g_lo / p.group] : 0ull;
        const unsigned long long mask_hi = (need_mask && g_hi < rows_total) ? s_mask[g_hi / p.group] : 0ull;
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;     // l: this lane's columns only
        const int row_src = 4 * (lane & 7);          // a lane that holds row (lane & 15) of this warp
        constexpr int NH = KT / 64;
        for (int k = 0; k < n_it; ++k, ++gt) {
          const int t = s.t0 + k;
          check(ok && mbar_wait(bar_s(gt & 1), (gt >> 1) & 1, fail));
          tc_fence_after();
          const uint32_t ts = t_lane + (gt & 1) * KT;
          uint32_t sr[NH][32];
#pragma unroll
          for (int h = 0; h < NH; ++h) tmem_ld_16rows_64cols(ts + h * 64, sr[h]);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < NH; ++h) {
            const int key0 = t * KT + h * 64;
            if (key0 + 64 > s.L) {
              // bit j of vis_*: key key0 + j is visible to the row (every prefix key; tree keys by the
              // ancestor mask, whose bits at and above n are clear)
              const int rel0 = key0 - s.L;             // > -64
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
          const int pb = gt % PB;
          if (gt >= PB) {                             // this P buffer is free once P(gt-PB) V(gt-PB) is done
            check(ok && mbar_wait(bar_o(pb), (gt / PB - 1) & 1, fail));
            tc_fence_after();
          }
          if (k > 0 && __any_sync(0xffffffffu, raise_lo || raise_hi)) {
            if (PB > 1) {                             // O must be stable: wait for P(gt-1) V(gt-1) as well
              check(ok && mbar_wait(bar_o((gt - 1) % PB), ((gt - 1) / PB) & 1, fail));
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
        // hand the rows' state to the one-row-per-lane layout of the epilogue (lanes 0-15)
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        const float ml = __shfl_sync(0xffffffffu, m_lo, row_src), mh = __shfl_sync(0xffffffffu, m_hi, row_src);
        const float ll = __shfl_sync(0xffffffffu, l_lo, row_src), lh = __shfl_sync(0xffffffffu, l_hi, row_src);
        m_run = (lane & 8) ? mh : ml;
        l_run = (lane & 8) ? lh : ll;
      } else {
        // 128-row accumulators: lane quadrant q of tensor memory (rows 32q .. 32q+31, one per lane) is
        // served by two warps: the warp of group 0 takes the first half of a tile's keys, the warp of
        // group 1 the second half.  They agree on the rows' maxima through shared memory; each keeps
        // the row sums of its own keys, rescales its half of O's columns and writes its half of P.
        const int row = 32 * quad + lane;
        const int grow = row0 + row;
        const bool need_mask = s.t1 * KT > s.L;
        const unsigned long long my_mask = (need_mask && grow < rows_total) ? s_mask[grow / p.group] : 0ull;
        constexpr int NV = KT / 2;                  // keys of a tile this thread handles
        constexpr int NC = NV / 32;
        float m_r = -INFINITY, l_r = 0.f;           // l_r: this thread's keys only
        for (int k = 0; k < n_it; ++k, ++gt) {
          const int t = s.t0 + k;
          check(ok && mbar_wait(bar_s(gt & 1), (gt >> 1) & 1, fail));
          tc_fence_after();
          const uint32_t ts = t_lane + (gt & 1) * KT + half * NV;
          uint32_t sr[NC][32];
#pragma unroll
          for (int c = 0; c < NC; ++c) tmem_ld32(ts + 32 * c, sr[c]);
          tmem_ld_wait();
          const int key0 = t * KT + half * NV;
          if (key0 + NV > s.L) {                    // the prefix end and / or the tree: mask
            const int rel0 = key0 - s.L;            // > -NV
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
          s_pair[gt & 1][half][row] = mx;
          pair_sync();
          mx = fmaxf(mx, s_pair[gt & 1][half ^ 1][row]);
          const bool raise = mx > m_r + kLazyMax;   // also true for the first finite maximum
          const float m_new = raise ? mx : m_r;
          const float m_use = m_new == -INFINITY ? 0.f : m_new;
          const int pb = gt % PB;
          if (gt >= PB) {                           // this P buffer is free once P(gt-PB) V(gt-PB) is done
            check(ok && mbar_wait(bar_o(pb), (gt / PB - 1) & 1, fail));
            tc_fence_after();
          }
          if (k > 0 && __any_sync(0xffffffffu, raise)) {     // (the same decision in both warps of the pair)
            if (PB > 1) {                           // O must be stable: wait for P(gt-1) V(gt-1) as well
              check(ok && mbar_wait(bar_o((gt - 1) % PB), ((gt - 1) / PB) & 1, fail));
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
          // P = exp2(S * scale - m) as bf16 to shared memory, row sums
          float sum0 = 0.f, sum1 = 0.f;
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
          l_r += sum0 + sum1;
          fence_async_smem();            // P was written with ordinary stores
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p(pb));
        }
        // row sums: add the other warp's share (the buffer of the parity no tile is using)
        s_pair[gt & 1][half][row] = l_r;
        pair_sync();
        l_run = l_r + s_pair[gt & 1][half ^ 1][row];
        m_run = m_r;
        pair_sync();                     // both have read before the next segment writes these entries
      }

      // ---- the segment's last P V product has completed: epilogue (group 0; one row per lane) ----
      if (half == 0) {
        check(ok && mbar_wait(bar_o((gt - 1) % PB), ((gt - 1) / PB) & 1, fail));
        tc_fence_after();
        const int gr = row0 + row_local;
        const bool row_valid = ok && row_active && gr < rows_total;
        const int node = row_valid ? gr / p.group : 0, g = row_valid ? gr % p.group : 0;
        const int h = s.hk * p.group + g;
        __nv_bfloat16 *dst = p.out + (((long long)s.b * p.t_max + node) * p.n_q_heads + h) * kD;
        float *lse_dst = p.lse ? p.lse + ((long long)s.b * p.n_q_heads + h) * p.t_max + node : nullptr;
        const bool whole = s.t0 == 0 && s.t1 == s.tiles;
        if (whole) {
          const float inv = 1.f / l_run;
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
          if (lse_dst && row_valid) *lse_dst = (m_run + log2f(l_run)) * 0.6931471805599453f;
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_ofree);        // the accumulator may be overwritten
        } else {
          // ---- partial result of an item that straddles CTAs ----
          // the CTAs that share the item, and this CTA's scratch slot: 2c if the segment starts the
          // CTA's share, else 2c + 1
          const int c_first = share_owner(s.gstart, total, G), c_last = share_owner(s.gstart + s.tiles - 1, total, G);
          const int n_seg = c_last - c_first + 1;
          const int my_slot = 2 * (int)blockIdx.x + ((s.gstart + s.t0 == g_begin) ? 0 : 1);
          unsigned char *slot = slots + (size_t)my_slot * C::SLOT_BYTES;
          // rows go out as scaled fp16 of O / l (see row_scale)
          // (a row that saw no key in this segment carries m = -inf and counts for nothing)
          const bool seen = m_run > -INFINITY && l_run > 0.f;
          const float inv_l = seen ? 1.f / l_run : 0.f;
          float amax = 0.f;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t v[32];
            tmem_ld32(t_lane + C::O_COL + ch * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(__uint_as_float(v[j])));
          }
          amax *= inv_l;
          float down, up;
          row_scale(amax, down, up);
          // one factor where it is finite (a row sum below 2^-100 or so overflows it: then two steps)
          const float f1 = inv_l * down;
          const bool one_step = f1 < INFINITY;
          const float fa = one_step ? f1 : inv_l, fb = one_step ? 1.f : down;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t v[32];
            tmem_ld32(t_lane + C::O_COL + ch * 32, v);
            tmem_ld_wait();
            if (row_active && ok) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint4 w;
                w.x = pack_f16(__uint_as_float(v[8 * i]) * fa * fb, __uint_as_float(v[8 * i + 1]) * fa * fb);
                w.y = pack_f16(__uint_as_float(v[8 * i + 2]) * fa * fb, __uint_as_float(v[8 * i + 3]) * fa * fb);
                w.z = pack_f16(__uint_as_float(v[8 * i + 4]) * fa * fb, __uint_as_float(v[8 * i + 5]) * fa * fb);
                w.w = pack_f16(__uint_as_float(v[8 * i + 6]) * fa * fb, __uint_as_float(v[8 * i + 7]) * fa * fb);
                st_16(slot + ((size_t)(ch * 4 + i) * ROWS + row_local) * 16, w);
              }
            }
          }
          if (row_active && ok)
            *reinterpret_cast<float4 *>(slot + (size_t)ROWS * kD * 2 + row_local * 16) = make_float4(seen ? m_run : -INFINITY, seen ? l_run : 0.f, up, 0.f);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_ofree);        // the accumulator may be overwritten
          // ---- ticket: the last of the item's CTAs to get here finishes the item ----
          // (the barrier orders every thread's stores before thread 0's fence, which publishes them
          // device-wide before the ticket is taken)
          const int tk_par = n_partial & 1;
          ++n_partial;
          group0_sync();
          if (tid == 0) {
            int last = 0;
            if (ok) {
              __threadfence();
              const unsigned int old = atomicAdd(tickets + s.item, 1u);
              last = old == (unsigned int)(n_seg - 1);
              if (last) tickets[s.item] = 0u;           // nobody else touches it before the next call
              __threadfence();
            }
            s_last[tk_par] = last;
          }
          group0_sync();
          if (s_last[tk_par] != 0 && ok) {
            // ---- this CTA adds up the partials of the item's CTAs c_first..c_last ----
            // Two threads per row (64 columns each, lanes 16-31 of a warp help lanes 0-15 out with
            // 64-row accumulators); the partials are fetched four at a time so that a pass over them is
            // one round trip to L2: first their (m, l, scale), then the rows, 32 columns per pass.
            constexpr int TPR = C::MMA_M == 64 ? 2 : 1;            // threads per row
            const int mrow = C::MMA_M == 64 ? 16 * quad + (lane & 15) : row_local;
            const int chalf = C::MMA_M == 64 ? (lane >> 4) : 0;     // which half of the columns
            const int mg = row0 + mrow;
            const bool m_valid = mg < rows_total;
            const int m_node = m_valid ? mg / p.group : 0, m_h = s.hk * p.group + (m_valid ? mg % p.group : 0);
            __nv_bfloat16 *m_dst = p.out + (((long long)s.b * p.t_max + m_node) * p.n_q_heads + m_h) * kD;
            auto slot_of = [&](int c) {
              const int sl = 2 * c + ((c == c_first && s.gstart != share_begin(c, total, G)) ? 1 : 0);
              return slots + (size_t)sl * C::SLOT_BYTES;
            };
            auto stats_of = [&](int c) {
              return __ldcg(reinterpret_cast<const float4 *>(slot_of(c) + (size_t)ROWS * kD * 2 + mrow * 16));
            };
            float mstar = -INFINITY;
            for (int c0 = c_first; c0 <= c_last; c0 += 4) {
              float4 st[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) st[j] = stats_of(min(c0 + j, c_last));
#pragma unroll
              for (int j = 0; j < 4; ++j) mstar = fmaxf(mstar, st[j].x);
            }
            float lsum = 0.f;
            for (int c0 = c_first; c0 <= c_last; c0 += 4) {
              float4 st[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) st[j] = stats_of(min(c0 + j, c_last));
#pragma unroll
              for (int j = 0; j < 4; ++j)
                if (c0 + j <= c_last) lsum += fast_exp2(st[j].x - mstar) * st[j].y;
            }
            const float inv = 1.f / lsum;
#pragma unroll 1
            for (int pass = 0; pass < (kD / 32) / TPR; ++pass) {
              const int chunk0 = (chalf * ((kD / 32) / TPR) + pass) * 4;       // first of this pass's four 8-column chunks
              float acc[32];
#pragma unroll
              for (int j = 0; j < 32; ++j) acc[j] = 0.f;
              for (int c0 = c_first; c0 <= c_last; c0 += 4) {
                float4 st[4];
                uint4 raw[4][4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int c = min(c0 + j, c_last);
                  const unsigned char *sp = slot_of(c);
                  st[j] = __ldcg(reinterpret_cast<const float4 *>(sp + (size_t)ROWS * kD * 2 + mrow * 16));
#pragma unroll
                  for (int ch = 0; ch < 4; ++ch)
                    raw[j][ch] = __ldcg(reinterpret_cast<const uint4 *>(sp + ((size_t)(chunk0 + ch) * ROWS + mrow) * 16));
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  // share of the row sum, times the row's scale (nothing for a repeated last partial)
                  const float wgt = (c0 + j <= c_last) ? fast_exp2(st[j].x - mstar) * st[j].y * st[j].z * inv : 0.f;
#pragma unroll
                  for (int ch = 0; ch < 4; ++ch) {
                    const float2 a0 = unpack_f16(raw[j][ch].x), a1 = unpack_f16(raw[j][ch].y);
                    const float2 a2 = unpack_f16(raw[j][ch].z), a3 = unpack_f16(raw[j][ch].w);
                    acc[8 * ch + 0] = fmaf(wgt, a0.x, acc[8 * ch + 0]);
                    acc[8 * ch + 1] = fmaf(wgt, a0.y, acc[8 * ch + 1]);
                    acc[8 * ch + 2] = fmaf(wgt, a1.x, acc[8 * ch + 2]);
                    acc[8 * ch + 3] = fmaf(wgt, a1.y, acc[8 * ch + 3]);
                    acc[8 * ch + 4] = fmaf(wgt, a2.x, acc[8 * ch + 4]);
                    acc[8 * ch + 5] = fmaf(wgt, a2.y, acc[8 * ch + 5]);
                    acc[8 * ch + 6] = fmaf(wgt, a3.x, acc[8 * ch + 6]);
                    acc[8 * ch + 7] = fmaf(wgt, a3.y, acc[8 * ch + 7]);
                  }
                }
              }
              if (m_valid) {
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                  uint4 w;
                  w.x = pack_bf16(acc[8 * ch], acc[8 * ch + 1]);
                  w.y = pack_bf16(acc[8 * ch + 2], acc[8 * ch + 3]);
                  w.z = pack_bf16(acc[8 * ch + 4], acc[8 * ch + 5]);
                  w.w = pack_bf16(acc[8 * ch + 6], acc[8 * ch + 7]);
                  st_16(m_dst + 8 * (chunk0 + ch), w);
                }
              }
            }
            if (p.lse && m_valid && chalf == 0)
              p.lse[((long long)s.b * p.n_q_heads + m_h) * p.t_max + m_node] = (mstar + log2f(lsum)) * 0.6931471805599453f;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // a CTA whose waits ran out cannot tell which of its requests are affected: all of the call's are flagged
  if (s_fail)
    for (int b = tid; b < B; b += C::THREADS) flag_status(p.dev_status, b, TWIG_DEV_INTERNAL);
  if (warp == 5) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
}

// Scratch layout, the same for every shape so that the tickets never share bytes with the partial
// results of another call: [partial-result slots: 4 x SMs x 64 rows x 272 bytes][tickets: one per item].
// (Two CTAs per SM with 64-row slots and one CTA per SM with 128-row slots take the same space.)
size_t slot_region_bytes(int n_sm) { return (size_t)2 * (2 * n_sm) * 64 * (kD * 2 + 16); }

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      return 148;
  }
  return n;
}

template <int ROWS, int KT, int QB, int SLOTS>
twig_status launch_stream(const AttnParams &p, const CacheMaps &maps, int grid, unsigned int *tickets,
                          unsigned char *slots, cudaStream_t st) {
  using C = StreamCfg<ROWS, KT, QB, SLOTS>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_attn_stream_kernel<ROWS, KT, QB, SLOTS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(C::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, tree_attn_stream_kernel<ROWS, KT, QB, SLOTS>, p, maps.kmap, maps.vmap, tickets, slots) !=
      cudaSuccess)
    return TWIG_ERR_CUDA;
  return TWIG_OK;
}

}  // namespace

// Scratch of the persistent kernel: the partial-result slots, then one ticket per item (at most
// 2 x batch x n_q_heads items: a kv head's 64 x group rows in blocks of 32 or more).
size_t tree_attn_stream_workspace_bytes(int batch, int n_q_heads, int max_nodes) {
  (void)max_nodes;
  return slot_region_bytes(sm_count()) + (size_t)2 * batch * n_q_heads * sizeof(unsigned int);
}

twig_status launch_tree_attn_stream(AttnParams &p, int batch, int rows, cudaStream_t st) {
  if (batch > kStreamMaxBatch) return TWIG_ERR_UNSUPPORTED;
  const int n_sm = sm_count();
  // blocks of up to 64 query rows, 64-key tiles, two CTAs per SM; more rows per kv head (wide GQA
  // groups) become several row blocks that re-read their K / V tiles from L2
  const int rows_per_cta = rows <= 32 ? 32 : 64;
  const int kt = 64;
  const int grid = 2 * n_sm;
  p.row_blocks = (rows + rows_per_cta - 1) / rows_per_cta;
  const size_t items = (size_t)batch * p.n_kv_heads * p.row_blocks;
  const size_t slot_bytes = slot_region_bytes(n_sm);
  if (!p.ws || p.ws_bytes < slot_bytes + items * sizeof(unsigned int)) return TWIG_ERR_WORKSPACE;
  // the tile counts stay far inside 32 bits
  if ((double)items * ((double)(p.max_len + p.t_max) / kt + 1.0) > 1.0e9) return TWIG_ERR_UNSUPPORTED;
  CacheMaps maps;
  if (!cache_maps(p, kt, &maps)) return TWIG_ERR_UNSUPPORTED;
  unsigned char *slots = p.ws;
  unsigned int *tickets = reinterpret_cast<unsigned int *>(p.ws + slot_bytes);
  if (rows_per_cta == 32) return launch_stream<32, 64, 2, 5>(p, maps, grid, tickets, slots, st);
  return launch_stream<64, 64, TWIG_STREAM64_QB, TWIG_STREAM64_SLOTS>(p, maps, grid, tickets, slots, st);
}

}  // namespace twig
