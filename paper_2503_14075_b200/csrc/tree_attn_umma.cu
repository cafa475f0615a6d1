// Tree attention of the verification pass on the 5th-generation tensor cores
// (Sec. 5.4, Appendix A, Algorithm 2; Eq. 2 with the tree's ancestor mask).
//
// One CTA of 128 threads owns up to ROWS query rows (tree node x query head of
// one kv head) and a share of the key tiles; thread r owns row r, which is also
// lane r of tensor memory.  Per 64-key tile:
//   S = Q K^T     tcgen05.mma, M = 128, N = 64, K = 8 x 16, operands in shared memory
//   softmax step  tcgen05.ld of the row, running max / sum, P (bf16) back to shared memory
//   O_t = P V     tcgen05.mma, M = 128, N = 128, K = 4 x 16, V read MN-major (no transpose copy)
//   O += O_t      tcgen05.ld, rescaled accumulation in registers
// K and V tiles travel separately through a ring of five 16 KB slots, filled by 16-byte
// cp.async in the 128-byte-swizzled layout that the matrix descriptors name; a K slot is
// refilled as soon as its S product has completed, a V slot after its P V product, so four
// tiles (64 KB) per CTA are in flight while one is being consumed.  The instruction
// always multiplies 128 rows; rows past ROWS read whatever follows in shared memory
// and land in lanes nobody reads.
// Key splits of a cluster are merged through distributed shared memory exactly as
// in the mma.sync kernel (each CTA pushes its per-row partial to the row's owner).
#include <cooperative_groups.h>

#include "tree_attn.cuh"

namespace cg = cooperative_groups;

namespace twig {

namespace {

constexpr int kD = 128;          // head_dim
constexpr int kKT = 64;          // keys per tile
constexpr int kThreads = 128;
constexpr int kSlots = 5;                         // ring of K / V tiles (K0 V0 K1 V1 K2 ...)
constexpr int kTileBytes = kKT * kD * 2;          // one K (or V) tile: 16 KB
constexpr int kPanelBytes = kKT * 128;            // 64-column panel of a K/V tile
constexpr uint32_t kTmemCols = 256;               // S: columns [0,64), O tile: [128,256)
constexpr int kSpinLimit = 1 << 22;

// ---- descriptors -------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
// lbo_bytes is the distance between 64-element groups along the leading (MN) dimension
// and is only meaningful for MN-major operands.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffff) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;      // descriptor version of this architecture
  d |= (uint64_t)2 << 61;      // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Bounded wait on an mbarrier phase; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < kSpinLimit; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}

#define TWIG_R8(a, o) "=r"(a[o]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]), "=r"(a[o + 7])
// 32 consecutive fp32 columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : TWIG_R8(v, 0), TWIG_R8(v, 8), TWIG_R8(v, 16), TWIG_R8(v, 24)
      : "r"(taddr));
}
#undef TWIG_R8
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

template <int ROWS>
struct UmmaCfg {
  static constexpr int Q_BYTES = ROWS * kD * 2;          // two 64-column panels of ROWS x 128 B
  static constexpr int P_BYTES = ROWS * 128;             // ROWS x 64 keys bf16
  static constexpr int RING_BYTES = kSlots * kTileBytes;
  static constexpr int RECV_BYTES = ROWS * kD * 4;
  static_assert(RECV_BYTES <= RING_BYTES, "split-merge buffer must fit in the stage ring");
  static_assert(Q_BYTES % 1024 == 0 && P_BYTES % 1024 == 0, "swizzled tiles start on 1024 bytes");
  static constexpr int SMEM_BYTES = Q_BYTES + P_BYTES + RING_BYTES;
};

template <int ROWS>
__global__ void __launch_bounds__(kThreads, 2)
tree_attn_umma_kernel(const AttnParams p) {
  using C = UmmaCfg<ROWS>;
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ unsigned long long s_mask[TWIG_MAX_NODES];
  __shared__ int s_par[TWIG_MAX_NODES];
  __shared__ float r_m[ROWS], r_l[ROWS];
  __shared__ __align__(8) unsigned long long s_bar[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_bad;

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, n_splits = gridDim.x;
  const int hk = blockIdx.y / p.row_blocks, rb = blockIdx.y % p.row_blocks;
  const int b = blockIdx.z;

  // ---- per-request metadata; every exit below is uniform over the cluster ----
  const int n = p.n_nodes[b], L = p.kv_len[b];
  if (n == 0) return;
  const bool first = split == 0 && blockIdx.y == 0 && tid == 0;
  if (n < 0 || n > p.t_max) {
    if (first) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    return;
  }
  if (L < 0 || L > p.max_len) {
    if (first) flag_status(p.dev_status, b, TWIG_DEV_OVERFLOW);
    return;
  }
  const int rows_total = n * p.group, row0 = rb * ROWS;
  if (row0 >= rows_total) return;

  const uint32_t q_s = smem_u32(smem);
  const uint32_t p_s = q_s + C::Q_BYTES;
  const uint32_t ring_s = p_s + C::P_BYTES;

  const int NK = L + n;
  const int n_tiles = (NK + kKT - 1) / kKT;
  const int per = (n_tiles + n_splits - 1) / n_splits;
  const int t_begin = split * per;
  const int t_end = min(n_tiles, t_begin + per);

  const __nv_bfloat16 *ck = p.cache_k + b * p.c_sb + hk * p.c_sh;
  const __nv_bfloat16 *cv = p.cache_v + b * p.c_sb + hk * p.c_sh;
  const __nv_bfloat16 *tk = p.tree_k + ((long long)b * p.n_kv_heads + hk) * p.t_max * kD;
  const __nv_bfloat16 *tv = p.tree_v + ((long long)b * p.n_kv_heads + hk) * p.t_max * kD;

  // A thread copies chunk (tid & 15) of rows (tid >> 4) + 8 i, i = 0..7, of a K or V tile.
  // Unit u of this CTA is K (u even) or V (u odd) of its tile u / 2 and lives in slot u % kSlots.
  const int ld_c = tid & 15, ld_r0 = tid >> 4;
  const uint32_t ld_off0 = (uint32_t)((ld_c >> 3) * kPanelBytes + ld_r0 * 128 + (((ld_c & 7) ^ (ld_r0 & 7)) << 4));
  auto load_unit = [&](int u) {
    const int t = t_begin + (u >> 1);
    if (t >= t_end) return;
    const uint32_t dst = ring_s + (u % kSlots) * kTileBytes + ld_off0;
    const __nv_bfloat16 *cbase = (u & 1) ? cv : ck, *tbase = (u & 1) ? tv : tk;
    const int j0 = t * kKT + ld_r0;
    if (t * kKT + kKT <= L) {               // whole tile inside the cached prefix
      const __nv_bfloat16 *src = cbase + (long long)j0 * p.c_sp + ld_c * 8;
      const long long step = 8 * p.c_sp;
#pragma unroll
      for (int i = 0; i < 8; ++i)           // rows 8 apart keep (row & 7): same swizzle, +1024 bytes
        cp_async_16(dst + i * 1024, src + i * step, true);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int vj = j0 + 8 * i;
        const __nv_bfloat16 *src = cbase;
        bool valid = false;
        if (vj < L) {
          src = cbase + (long long)vj * p.c_sp + ld_c * 8;
          valid = true;
        } else if (vj < NK) {
          src = tbase + (vj - L) * kD + ld_c * 8;
          valid = true;
        }
        cp_async_16(dst + i * 1024, src, valid);
      }
    }
  };

  // ---- start the copies: Q (zero rows past the last row) and the first key tiles ----
#pragma unroll
  for (int i = 0; i < ROWS / 8; ++i) {
    const int r = ld_r0 + 8 * i;
    const int gr = row0 + r;
    const bool valid = gr < rows_total;
    const int node = valid ? gr / p.group : 0, g = valid ? gr % p.group : 0;
    const __nv_bfloat16 *src =
        p.q + (((long long)b * p.t_max + node) * p.n_q_heads + hk * p.group + g) * kD + ld_c * 8;
    cp_async_16(q_s + (ld_c >> 3) * ROWS * 128 + r * 128 + (((ld_c & 7) ^ (r & 7)) << 4), src, valid);
  }
  load_unit(0);
  cp_async_commit();              // this group also carries Q
#pragma unroll
  for (int u = 1; u < kSlots; ++u) {
    load_unit(u);
    cp_async_commit();
  }

  // ---- while they fly: parents, validation, ancestor masks ---------------------
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (tid < n) {
    const int pr = p.parent[(long long)b * p.t_max + tid];
    s_par[tid] = pr;
    if ((tid == 0) ? (pr != -1) : (pr < 0 || pr >= tid)) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (first) flag_status(p.dev_status, b, TWIG_DEV_BAD_TREE);
    cp_async_wait<0>();
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
  // tensor memory and the two completion barriers (S ready, O tile ready)
  const uint32_t bar_s = smem_u32(&s_bar[0]), bar_o = smem_u32(&s_bar[1]);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_s) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_o) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);     // this warp's 32 lanes
  const uint32_t tmem_s = tmem, tmem_o = tmem + 128;

  // ---- per-thread state: thread r owns row r ------------------------------------
  const bool warp_rows = warp * 32 < ROWS && row0 + warp * 32 < rows_total;   // warp-uniform
  const int gr = row0 + tid;
  const bool row_valid = tid < ROWS && gr < rows_total;
  const unsigned long long my_mask = row_valid ? s_mask[gr / p.group] : 0ull;
  float o[kD];
#pragma unroll
  for (int i = 0; i < kD; ++i) o[i] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;
  uint32_t ph_s = 0, ph_o = 0;
  constexpr uint32_t kIdescS = instr_desc(kKT, false), kIdescO = instr_desc(kD, true);
  bool ok = true;

  for (int t = t_begin; t < t_end; ++t) {
    const int it = t - t_begin;
    cp_async_wait<kSlots - 1>();   // this tile's K has landed (four later units may still be in flight)
    fence_async_smem();            // make the copied bytes visible to the tensor core's reads
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t kb = ring_s + ((2 * it) % kSlots) * kTileBytes;
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks) {
        const uint32_t qa = q_s + (ks >> 2) * ROWS * 128 + (ks & 3) * 32;
        const uint32_t ka = kb + (ks >> 2) * kPanelBytes + (ks & 3) * 32;
        umma(tmem_s, smem_desc(qa, 16), smem_desc(ka, 16), kIdescS, ks > 0);
      }
      umma_commit(bar_s);
    }
    float alpha = 1.f;
    if (ok) ok = mbar_wait(bar_s, ph_s);
    ph_s ^= 1;
    tc_fence_after();
    if (ok) load_unit(2 * it + kSlots);      // the K slot is free: S has been computed
    cp_async_commit();
    if (warp_rows && ok) {
      uint32_t sr[2][32];
      tmem_ld32(t_lane + 0, sr[0]);
      tmem_ld32(t_lane + 32, sr[1]);
      tmem_ld_wait();
      const int key0 = t * kKT;
      float mx = -INFINITY;
      if (key0 + kKT > L) {        // the tile that holds the prefix end and / or the tree
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int vj = key0 + h * 32 + j;
            const bool vis = vj < L || (vj < NK && ((my_mask >> (vj - L)) & 1ull));
            const float x = vis ? __uint_as_float(sr[h][j]) * p.scale_log2 : -INFINITY;
            sr[h][j] = __float_as_uint(x);
            mx = fmaxf(mx, x);
          }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float x = __uint_as_float(sr[h][j]) * p.scale_log2;
            sr[h][j] = __float_as_uint(x);
            mx = fmaxf(mx, x);
          }
      }
      const float m_new = fmaxf(m_run, mx);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;
      alpha = fast_exp2(m_run - m_use);
      m_run = m_new;
      float sum = 0.f;
      const uint32_t prow = p_s + tid * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {          // chunk c = keys 8c .. 8c+7 of this row
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = c * 8 + e * 2;
          const float p0 = fast_exp2(__uint_as_float(sr[j >> 5][j & 31]) - m_use);
          const float p1 = fast_exp2(__uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]) - m_use);
          sum += p0 + p1;
          w[e] = pack_bf16(p0, p1);
        }
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(prow + ((c ^ (tid & 7)) << 4)), "r"(w[0]), "r"(w[1]),
                     "r"(w[2]), "r"(w[3]) : "memory");
      }
      l_run = l_run * alpha + sum;
    }
    cp_async_wait<kSlots - 1>();   // this tile's V has landed
    fence_async_smem();            // ... and P was written with ordinary stores
    tc_fence_before();
    ok = __syncthreads_and(ok);
    if (tid == 0 && ok) {
      tc_fence_after();
      const uint32_t vb = ring_s + ((2 * it + 1) % kSlots) * kTileBytes;
#pragma unroll
      for (int j = 0; j < kKT / 16; ++j)
        umma(tmem_o, smem_desc(p_s + j * 32, 16), smem_desc(vb + j * 2048, kPanelBytes), kIdescO, j > 0);
      umma_commit(bar_o);
    }
    if (warp_rows && alpha != 1.f) {          // overlaps with the P V product
#pragma unroll
      for (int i = 0; i < kD; ++i) o[i] *= alpha;
    }
    if (ok) ok = mbar_wait(bar_o, ph_o);
    ph_o ^= 1;
    tc_fence_after();
    if (ok) load_unit(2 * it + kSlots + 1);  // the V slot is free: the O tile has been computed
    cp_async_commit();
    if (warp_rows && ok) {
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld32(t_lane + 128 + ch * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) o[ch * 32 + j] += __uint_as_float(v[j]);
      }
    }
    tc_fence_before();
    ok = __syncthreads_and(ok);     // S, the O tile and P are free again
    if (!ok) break;
  }
  cp_async_wait<0>();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  if (!ok && tid == 0) flag_status(p.dev_status, b, TWIG_DEV_INTERNAL);

  // ---- merge the key splits of the cluster (push to the row's owner, then reduce) ----
  const int rows_per = ROWS / n_splits;
  float *recv = reinterpret_cast<float *>(smem + C::Q_BYTES + C::P_BYTES);
  if (n_splits > 1) cluster.sync();        // every CTA has left its key loop: the rings are free
  if (tid < ROWS) {
    const int owner = tid / rows_per, lr = tid % rows_per;
    const int slot = split * rows_per + lr;
    float *ro = recv + (size_t)slot * kD, *rm = r_m + slot, *rl = r_l + slot;
    if (n_splits > 1) {
      ro = cluster.map_shared_rank(ro, owner);
      rm = cluster.map_shared_rank(rm, owner);
      rl = cluster.map_shared_rank(rl, owner);
    }
#pragma unroll
    for (int i = 0; i < kD / 4; ++i)        // float4 slots are XOR-swizzled by the row to spread banks
      *reinterpret_cast<float4 *>(ro + ((i ^ (lr & 31)) << 2)) = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
    *rm = m_run;
    *rl = l_run;
  }
  if (n_splits > 1) cluster.sync(); else __syncthreads();

  {
    constexpr int TPR = kD / 4;                       // 32 threads per row, one float4 each
    constexpr int RPP = kThreads / TPR;
    const int i4 = tid % TPR;
    for (int lr = tid / TPR; lr < rows_per; lr += RPP) {
      const int grow = row0 + split * rows_per + lr;
      if (grow >= rows_total || !ok) continue;
      float mv[8];
      float mstar = -INFINITY;
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        mv[sd] = sd < n_splits ? r_m[sd * rows_per + lr] : -INFINITY;
        mstar = fmaxf(mstar, mv[sd]);
      }
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float lsum = 0.f;
      const int col = (i4 ^ (lr & 31)) << 2;
#pragma unroll
      for (int sd = 0; sd < 8; ++sd) {
        if (sd < n_splits) {
          const float wgt = fast_exp2(mv[sd] - mstar);
          lsum = fmaf(wgt, r_l[sd * rows_per + lr], lsum);
          const float4 v = *reinterpret_cast<const float4 *>(recv + (size_t)(sd * rows_per + lr) * kD + col);
          acc.x = fmaf(wgt, v.x, acc.x);
          acc.y = fmaf(wgt, v.y, acc.y);
          acc.z = fmaf(wgt, v.z, acc.z);
          acc.w = fmaf(wgt, v.w, acc.w);
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

template <int ROWS>
twig_status launch_umma(const AttnParams &p, int batch, int n_splits, cudaStream_t st) {
  using C = UmmaCfg<ROWS>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tree_attn_umma_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, p.n_kv_heads * p.row_blocks, batch);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = n_splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, tree_attn_umma_kernel<ROWS>, p) != cudaSuccess) return TWIG_ERR_CUDA;
  return TWIG_OK;
}

}  // namespace

twig_status launch_tree_attn_umma(AttnParams &p, int batch, int rows, cudaStream_t st) {
  const int rows_per_cta = rows <= 32 ? 32 : rows <= 64 ? 64 : 128;
  p.row_blocks = (rows + rows_per_cta - 1) / rows_per_cta;
  if ((long long)p.n_kv_heads * p.row_blocks > 65535) return TWIG_ERR_UNSUPPORTED;
  const int max_tiles = (p.max_len + p.t_max + kKT - 1) / kKT;
  const int n_splits = pick_splits(batch * p.n_kv_heads * p.row_blocks, max_tiles);
  switch (rows_per_cta) {
    case 32: return launch_umma<32>(p, batch, n_splits, st);
    case 64: return launch_umma<64>(p, batch, n_splits, st);
    default: return launch_umma<128>(p, batch, n_splits, st);
  }
}

}  // namespace twig
