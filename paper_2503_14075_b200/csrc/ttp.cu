// Twig-guided token pruning (TTP): importance scores, TopR selection and the
// gather that compacts the kept rows of the KV cache.
//
// Scores follow Eq. 3 / Eq. 5 (row of the last prompt token in the attention
// map of the last twig layer) and Eq. 7 (softmax over the visual tokens, mean
// over heads).  TopR is Eq. 3's selection with the lower index winning ties
// and sequence order kept.  The gather applies the pruned token list to the
// cached K/V rows of every layer; position ids travel with their rows.
#include "twig_common.cuh"

namespace twig {

constexpr int kScoreThreads = 256;
constexpr int kScoreKeysPerCta = 128;
constexpr int kScoreWarps = kScoreThreads / 32;   // every warp of the logits stage writes one partial (max, sum) per head
constexpr int kMaxGroup = 16;   // query heads per kv head
constexpr int kMaxQHeads = 128;
constexpr int kTopkThreads = 1024;

// per-request layout check shared by the three stages
__device__ __forceinline__ bool layout_ok(int lp, int vs, int nv, int k_max_len, int m_max) {
  return lp >= 0 && lp <= k_max_len && vs >= 0 && nv >= 0 && nv <= m_max && vs <= lp &&
         nv <= lp - vs;
}

// ---------------------------------------------------------------------------
// Stage 1a: scaled logits of the last prompt query against every key in scope.
// One CTA = 128 keys of one kv head; the G query heads of the group share the
// key read.  D/8 lanes cover one key row (16 bytes each).
// ---------------------------------------------------------------------------
// GATED (Eq. 7): q is multiplied element-wise by q_gate and every key row by the row of k_gate at the
// same place (k_gate has K's strides), in fp32, before the dot product.
template <int D, bool GATED>
__global__ void __launch_bounds__(kScoreThreads)
ttp_logits_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k,
                  const __nv_bfloat16 *__restrict__ q_gate, const __nv_bfloat16 *__restrict__ k_gate,
                  long long ksb, long long ksh, long long ksp, int k_max_len,
                  const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                  const int *__restrict__ n_vis, int n_q_heads, int group, int norm_scope,
                  float scale, float *__restrict__ logits, int lstride, float2 *__restrict__ stats,
                  int n_parts, int m_max, int *dev_status) {
  constexpr int LPK = D / 8;               // lanes per key row
  constexpr int KPP = kScoreThreads / LPK; // keys per pass of the CTA
  constexpr int PASSES = kScoreKeysPerCta / KPP;
  __shared__ float qs[kMaxGroup * D];

  grid_dependency_sync();
  const int b = blockIdx.z, hk = blockIdx.y;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b];
  if (!layout_ok(lp, vs, nv, k_max_len, m_max)) {
    if (threadIdx.x == 0 && blockIdx.x == 0 && hk == 0) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
    return;
  }
  const int lo = norm_scope ? vs : 0, hi = norm_scope ? vs + nv : lp;
  const int j0 = blockIdx.x * kScoreKeysPerCta;
  if (j0 >= hi || j0 + kScoreKeysPerCta <= lo) return;

  // the key rows are requested first: they are the long pole, q is staged while they fly
  const int sub = threadIdx.x % LPK, slot = threadIdx.x / LPK;
  const __nv_bfloat16 *kb = k + b * ksb + hk * ksh + sub * 8;
  const __nv_bfloat16 *gb = GATED ? k_gate + b * ksb + hk * ksh + sub * 8 : nullptr;
  uint4 kr[PASSES], gr[GATED ? PASSES : 1];
#pragma unroll
  for (int p = 0; p < PASSES; ++p) {
    const int j = j0 + p * KPP + slot;
    const bool in = j >= lo && j < hi;
    kr[p] = in ? ld_nc_16(kb + (long long)j * ksp) : make_uint4(0, 0, 0, 0);
    if (GATED) gr[p] = in ? ld_nc_16(gb + (long long)j * ksp) : make_uint4(0, 0, 0, 0);
  }
  for (int i = threadIdx.x; i < group * D; i += kScoreThreads) {
    const long long at = ((long long)b * n_q_heads + hk * group) * D + i;
    float v = __bfloat162float(q[at]) * scale;
    if (GATED) v *= __bfloat162float(q_gate[at]);
    qs[i] = v;
  }
  __syncthreads();

  // the (gated) key row of every pass as eight floats
  float kf[PASSES][8];
#pragma unroll
  for (int p = 0; p < PASSES; ++p) {
    kf[p][0] = bf16_lo(kr[p].x); kf[p][1] = bf16_hi(kr[p].x);
    kf[p][2] = bf16_lo(kr[p].y); kf[p][3] = bf16_hi(kr[p].y);
    kf[p][4] = bf16_lo(kr[p].z); kf[p][5] = bf16_hi(kr[p].z);
    kf[p][6] = bf16_lo(kr[p].w); kf[p][7] = bf16_hi(kr[p].w);
    if (GATED) {
      kf[p][0] *= bf16_lo(gr[p].x); kf[p][1] *= bf16_hi(gr[p].x);
      kf[p][2] *= bf16_lo(gr[p].y); kf[p][3] *= bf16_hi(gr[p].y);
      kf[p][4] *= bf16_lo(gr[p].z); kf[p][5] *= bf16_hi(gr[p].z);
      kf[p][6] *= bf16_lo(gr[p].w); kf[p][7] *= bf16_hi(gr[p].w);
    }
  }
  for (int g = 0; g < group; ++g) {
    const float4 qa = *reinterpret_cast<const float4 *>(qs + g * D + sub * 8);
    const float4 qb = *reinterpret_cast<const float4 *>(qs + g * D + sub * 8 + 4);
    float *lrow = logits + ((long long)b * n_q_heads + hk * group + g) * lstride;
    float a[PASSES];                       // the warp's logits of this head, -inf outside the scope
#pragma unroll
    for (int p = 0; p < PASSES; ++p) {
      float acc = kf[p][0] * qa.x;
      acc = fmaf(kf[p][1], qa.y, acc);
      acc = fmaf(kf[p][2], qa.z, acc);
      acc = fmaf(kf[p][3], qa.w, acc);
      acc = fmaf(kf[p][4], qb.x, acc);
      acc = fmaf(kf[p][5], qb.y, acc);
      acc = fmaf(kf[p][6], qb.z, acc);
      acc = fmaf(kf[p][7], qb.w, acc);
#pragma unroll
      for (int o = LPK / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      const int j = j0 + p * KPP + slot;
      const bool in = j >= lo && j < hi;
      if (sub == 0 && in) lrow[j] = acc;
      a[p] = in ? acc : -INFINITY;
    }
    // softmax statistics of the warp's keys (32 / LPK key rows per pass): the maximum and the sum of
    // exponentials relative to it, every lane of a row's group holding the row's logit; the next stage
    // merges the partials of a head.  No barrier and no tail: the CTA is done when its warps are.
    float mx = a[0];
#pragma unroll
    for (int p = 1; p < PASSES; ++p) mx = fmaxf(mx, a[p]);
#pragma unroll
    for (int o = 16; o >= LPK; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
#pragma unroll
    for (int p = 0; p < PASSES; ++p) sum += a[p] > -INFINITY ? expf(a[p] - mx) : 0.f;
#pragma unroll
    for (int o = 16; o >= LPK; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((threadIdx.x & 31) == 0)
      stats[((long long)b * n_q_heads + hk * group + g) * n_parts + blockIdx.x * kScoreWarps + (threadIdx.x >> 5)] =
          make_float2(mx, sum);
  }
}

// ---------------------------------------------------------------------------
// Stage 1b + 2: softmax per head, mean over heads -> scores; then exact TopR.
// mode bit 0: compute scores from the logits; bit 1: select.  Without bit 0 the scores are read from
// `scores`.  With the selection: one CTA of 1024 threads per request.  Scores alone: grid
// (slices, batch), any CTA size, every CTA takes a slice of the request's visual tokens (the
// per-head statistics are merged from the logits stage's per-warp partials by every CTA: cheap).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive block scan of `x` over 1024 threads; returns the block total in `total`
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t x, uint32_t *warp_sums, uint32_t &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = warp_sums[lane], winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    warp_sums[lane] = winc - w;
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  const uint32_t res = warp_sums[warp] + inc - x;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kTopkThreads)
ttp_finalize_topk_kernel(const float *__restrict__ logits, int lstride, const float2 *__restrict__ stats,
                         int n_parts, int n_q_heads, int k_max_len,
                         const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                         const int *__restrict__ n_vis, const int *__restrict__ keep, int norm_scope,
                         float *__restrict__ scores, int m_max, int *__restrict__ kept_idx, int r_max,
                         int *dev_status, int mode) {
  extern __shared__ uint32_t keys[];                 // [m_max] fp32 scores, then ordered keys
  __shared__ float h_max[kMaxQHeads], h_inv[kMaxQHeads];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t warp_sums[33];
  __shared__ uint32_t sel_digit, sel_remaining;

  // the kernel after this one (the gather of the fused call) may start on what does not depend on the
  // selection; this kernel itself reads its predecessor's output from here on
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = blockDim.x;
  const int nv = n_vis[b];
  float *sc = scores + (long long)b * m_max;

  if (mode & 1) {
    const int lp = prefix_len[b], vs = vis_start[b];
    if (!layout_ok(lp, vs, nv, k_max_len, m_max)) {
      if (tid == 0 && blockIdx.x == 0) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
      return;
    }
    const int lo = norm_scope ? vs : 0, hi = norm_scope ? vs + nv : lp;
    // partials of the logits stage that may hold keys of the scope: those of its chunks (none for an
    // empty scope); a partial without a key in scope is (-inf, 0)
    const int c_lo = lo / kScoreKeysPerCta, c_hi = hi > lo ? (hi - 1) / kScoreKeysPerCta : c_lo - 1;
    const int p_lo = c_lo * kScoreWarps, p_hi = (c_hi + 1) * kScoreWarps;        // [p_lo, p_hi)
    // a lane takes the partials p_lo + lane, + 32, ... of a head, eight of them in registers, and a warp
    // has two heads in flight: for scopes of up to 4096 keys every load of a pair of heads is one round trip
    constexpr int kHeadsInFlight = 2, kPartRegs = 8;
    for (int h0 = warp * kHeadsInFlight; h0 < n_q_heads; h0 += (nt / 32) * kHeadsInFlight) {
      float2 part[kHeadsInFlight][kPartRegs];
#pragma unroll
      for (int i = 0; i < kHeadsInFlight; ++i)
#pragma unroll
        for (int r = 0; r < kPartRegs; ++r) {
          const int h = h0 + i, c = p_lo + lane + 32 * r;
          part[i][r] = h < n_q_heads && c < p_hi ? stats[((long long)b * n_q_heads + h) * n_parts + c]
                                                 : make_float2(-INFINITY, 0.f);
        }
#pragma unroll
      for (int i = 0; i < kHeadsInFlight; ++i) {
        const int h = h0 + i;
        if (h >= n_q_heads) break;                   // (uniform in the warp)
        float mx = part[i][0].x;
#pragma unroll
        for (int r = 1; r < kPartRegs; ++r) mx = fmaxf(mx, part[i][r].x);
        for (int c = p_lo + lane + 32 * kPartRegs; c < p_hi; c += 32)
          mx = fmaxf(mx, stats[((long long)b * n_q_heads + h) * n_parts + c].x);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;                             // (exp(-inf - mx) = 0: partials without keys add nothing)
#pragma unroll
        for (int r = 0; r < kPartRegs; ++r) sum += part[i][r].y * expf(part[i][r].x - mx);
        for (int c = p_lo + lane + 32 * kPartRegs; c < p_hi; c += 32) {
          const float2 more = stats[((long long)b * n_q_heads + h) * n_parts + c];
          sum += more.y * expf(more.x - mx);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) {
          h_max[h] = mx;
          h_inv[h] = 1.f / sum;
        }
      }
    }
    __syncthreads();
    const float inv_h = 1.f / (float)n_q_heads;
    for (int m = blockIdx.x * nt + tid; m < m_max; m += gridDim.x * nt) {
      float acc = 0.f;
      if (m < nv) {
        const float *z = logits + (long long)b * n_q_heads * lstride + vs + m;
        int h = 0;
        for (; h + 32 <= n_q_heads; h += 32) {         // 32 heads' logits in flight: one round trip
          float zz[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) zz[i] = z[(long long)(h + i) * lstride];
#pragma unroll
          for (int i = 0; i < 32; ++i) acc += expf(zz[i] - h_max[h + i]) * h_inv[h + i];
        }
        for (; h + 8 <= n_q_heads; h += 8) {
          float zz[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) zz[i] = z[(long long)(h + i) * lstride];
#pragma unroll
          for (int i = 0; i < 8; ++i) acc += expf(zz[i] - h_max[h + i]) * h_inv[h + i];
        }
        for (; h < n_q_heads; ++h) acc += expf(z[(long long)h * lstride] - h_max[h]) * h_inv[h];
        acc *= inv_h;
      }
      sc[m] = acc;
      if (mode & 2) keys[m] = order_key(acc);
    }
  } else {
    if (nv < 0 || nv > m_max) {
      if (tid == 0) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
      return;
    }
    for (int m = tid; m < nv; m += kTopkThreads) keys[m] = order_key(sc[m]);
  }
  if (!(mode & 2)) return;
  const int R = keep[b];
  if (R < 0 || R > nv || R > r_max) {
    if (tid == 0) flag_status(dev_status, b, TWIG_DEV_BAD_KEEP);
    return;
  }
  int *out = kept_idx + (long long)b * r_max;
  for (int i = R + tid; i < r_max; i += kTopkThreads) out[i] = -1;
  if (R == 0) return;
  __syncthreads();

  // radix select, 8 bits per pass from the top: the R-th largest key
  uint32_t prefix = 0, mask = 0;
  uint32_t remaining = (uint32_t)R;
#pragma unroll 1
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    // (scores of one request are close to each other, so in the top passes nearly all keys share a
    // digit: the lanes of a warp that hold the same digit add their count with one atomic)
    for (int base = 0; base < nv; base += kTopkThreads) {
      const int m = base + tid;
      const uint32_t key = m < nv ? keys[m] : 0u;
      const bool cand = m < nv && (key & mask) == prefix;
      const uint32_t digit = cand ? (key >> shift) & 255u : 256u + (uint32_t)lane;     // non-candidates match nobody
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      if (cand && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      uint32_t c[8], mine = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        c[i] = hist[lane * 8 + i];
        mine += c[i];
      }
      uint32_t suf = mine;   // inclusive suffix sum over lanes (lane 31 = top digits)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += y;
      }
      uint32_t above = suf - mine;
      if (above < remaining && remaining <= suf) {
#pragma unroll
        for (int i = 7; i >= 0; --i) {
          if (above < remaining && remaining <= above + c[i]) {
            sel_digit = lane * 8 + i;
            sel_remaining = remaining - above;
          }
          above += c[i];
        }
      }
    }
    __syncthreads();
    prefix |= sel_digit << shift;
    mask |= 255u << shift;
    remaining = sel_remaining;
    __syncthreads();
  }
  const uint32_t tau = prefix, need_eq = remaining;

  // ordered compaction: keys above tau, plus the first need_eq keys equal to tau
  uint32_t run_gt = 0, run_eq = 0;
  for (int base = 0; base < nv; base += kTopkThreads) {
    const int m = base + tid;
    const uint32_t key = (m < nv) ? keys[m] : 0u;
    const uint32_t gt = (m < nv && key > tau), eq = (m < nv && key == tau);
    uint32_t total;
    const uint32_t ex = block_exclusive_scan(gt | (eq << 16), warp_sums, total);
    const uint32_t gt_before = run_gt + (ex & 0xffffu), eq_before = run_eq + (ex >> 16);
    if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = m;
    run_gt += total & 0xffffu;
    run_eq += total >> 16;
  }
}

// ---------------------------------------------------------------------------
// Stage 3: gather the rows of the pruned sequence, all layers and kv heads.
// One CTA = 64 rows of one (layer, kv head, request), K and V.  The rows of a request come in two
// kinds: text rows (before and after the image), whose source needs nothing but the request's
// layout, and kept visual rows, whose source is kept_idx.  blockIdx.y walks the text rows first
// (text_blocks blocks of 64) and the visual rows last (the remaining blocks), so that in the
// fused call, where the selection may still be running when this kernel starts, the CTAs that do
// not need it are scheduled first and leave without waiting; only the visual CTAs wait for it.
// ---------------------------------------------------------------------------
constexpr int kGatherThreads = 256;
constexpr int kGatherRows = 64;

template <int D>
__global__ void __launch_bounds__(kGatherThreads)
kv_gather_kernel(KvView src, KvViewMut dst, const int *__restrict__ kept_idx, int r_max,
                 const int *__restrict__ keep, const int *__restrict__ prefix_len,
                 const int *__restrict__ vis_start, const int *__restrict__ n_vis,
                 const int *__restrict__ pos_in, int *__restrict__ pos_out, int pos_stride,
                 int *__restrict__ new_len, int *dev_status, int text_blocks, int early_text) {
  constexpr int LPR = D / 8;                   // lanes per row
  constexpr int RPP = kGatherThreads / LPR;    // rows per pass
  constexpr int PASSES = kGatherRows / RPP;
  // early_text (the fused call): the kernels before this one in the stream are the call's own scoring
  // and selection, which write nothing this kernel reads except kept_idx; text CTAs then run without
  // waiting for them.  Otherwise nothing is read before the preceding kernel has completed.
  const bool visual = (int)blockIdx.y >= text_blocks;
  if (!early_text || visual) grid_dependency_sync();
  const int slice = blockIdx.x % (src.n_layers * src.n_kv_heads), b = blockIdx.x / (src.n_layers * src.n_kv_heads);
  const int layer = slice / src.n_kv_heads, h = slice % src.n_kv_heads;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b], kp = keep[b];
  const bool first = slice == 0 && blockIdx.y == 0 && threadIdx.x == 0;
  const int nl = lp - nv + kp;
  {
    int code = 0;
    if (!layout_ok(lp, vs, nv, src.max_len, TWIG_MAX_VISUAL)) code = TWIG_DEV_BAD_LAYOUT;
    else if (kp < 0 || kp > nv || kp > r_max) code = TWIG_DEV_BAD_KEEP;
    else if (nl > dst.max_len) code = TWIG_DEV_OVERFLOW;
    if (code != 0) {
      if (first) flag_status(dev_status, b, code);
      return;
    }
    if (first && new_len) new_len[b] = nl;
  }
  // this CTA's rows: index i0.. within its kind (text rows: the lp - nv rows outside the image)
  const int i0 = (visual ? (int)blockIdx.y - text_blocks : (int)blockIdx.y) * kGatherRows;
  const int n_kind = visual ? kp : lp - nv;
  if (i0 >= n_kind) return;

  const int sub = threadIdx.x % LPR, slot = threadIdx.x / LPR;
  const long long sbase = layer * src.stride_layer + b * src.stride_batch + h * src.stride_head + sub * 8;
  const long long dbase = layer * dst.stride_layer + b * dst.stride_batch + h * dst.stride_head + sub * 8;
  const int *kidx = kept_idx + (long long)b * r_max;

  int srow[PASSES], drow[PASSES];
  uint4 kr[PASSES], vr[PASSES];
#pragma unroll
  for (int p = 0; p < PASSES; ++p) {
    const int i = i0 + p * RPP + slot;
    int s = -1, j = 0;
    if (i < n_kind) {
      if (!visual) {                 // text row i: before the image it stays, after it moves up by the dropped tokens
        s = i < vs ? i : i + nv;
        j = i < vs ? i : i + kp;
      } else {
        const int kk = kidx[i];
        const int prev = i > 0 ? kidx[i - 1] : -1;
        if (kk < 0 || kk >= nv || kk <= prev) {
          if (sub == 0 && slice == 0) flag_status(dev_status, b, TWIG_DEV_BAD_INDEX);
        } else {
          s = vs + kk;
          j = vs + i;
        }
      }
    }
    srow[p] = s;
    drow[p] = j;
    if (s >= 0) {
      kr[p] = ld_nc_16(src.k + sbase + (long long)s * src.stride_pos);
      vr[p] = ld_nc_16(src.v + sbase + (long long)s * src.stride_pos);
    }
  }
#pragma unroll
  for (int p = 0; p < PASSES; ++p) {
    if (srow[p] >= 0) {
      st_16(dst.k + dbase + (long long)drow[p] * dst.stride_pos, kr[p]);
      st_16(dst.v + dbase + (long long)drow[p] * dst.stride_pos, vr[p]);
      if (slice == 0 && sub == 0 && pos_in && pos_out)
        pos_out[(long long)b * pos_stride + drow[p]] = pos_in[(long long)b * pos_stride + srow[p]];
    }
  }
}

// ---------------------------------------------------------------------------
// Stage 3 in place (dst is src).  Rows only ever move to lower positions (the source of row j is
// idx[j] >= j), so a slice can be compacted where it lies if ONE CTA owns it and works through
// ascending chunks of rows, loading a whole chunk before it stores any row of it: a chunk's stores
// land below every row a later chunk reads, and the rows a chunk overwrites are either its own
// sources (already in registers) or rows nobody needs any more.  Independent CTAs on one slice
// would race, so the grid is one CTA per (layer, kv head, K or V, request).  Rows that stay where
// they are (the text before the image, kept tokens at the head of the image) are not touched.
// The kept list is validated in full before the first store: an in-place pass cannot be undone.
// ---------------------------------------------------------------------------
constexpr int kInplacePasses = 8;      // 16-byte loads in flight per thread

__device__ __forceinline__ uint4 ld_cg_16(const void *p) {
  uint4 r;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

template <int D>
__global__ void __launch_bounds__(kGatherThreads)
kv_compact_inplace_kernel(KvViewMut kv, const int *__restrict__ kept_idx, int r_max,
                          const int *__restrict__ keep, const int *__restrict__ prefix_len,
                          const int *__restrict__ vis_start, const int *__restrict__ n_vis, int *pos,
                          int pos_stride, int *__restrict__ new_len, int *dev_status) {
  constexpr int LPR = D / 8;                   // lanes per row
  constexpr int RPP = kGatherThreads / LPR;    // rows per pass
  constexpr int CHUNK = RPP * kInplacePasses;  // rows per chunk
  const int b = blockIdx.z, which = blockIdx.y;
  const int layer = blockIdx.x / kv.n_kv_heads, h = blockIdx.x % kv.n_kv_heads;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b], kp = keep[b];
  const bool first = blockIdx.x == 0 && which == 0 && threadIdx.x == 0;
  if (!layout_ok(lp, vs, nv, kv.max_len, TWIG_MAX_VISUAL)) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
    return;
  }
  if (kp < 0 || kp > nv || kp > r_max) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_KEEP);
    return;
  }
  const int *kidx = kept_idx + (long long)b * r_max;
  int bad = 0;
  for (int i = threadIdx.x; i < kp; i += kGatherThreads) {
    const int kk = kidx[i], prev = i > 0 ? kidx[i - 1] : -1;
    bad |= (kk < 0 || kk >= nv || kk <= prev) ? 1 : 0;
  }
  if (__syncthreads_or(bad)) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_INDEX);
    return;
  }
  const int nl = lp - nv + kp;
  if (first && new_len) new_len[b] = nl;
  auto source = [&](int j) { return j < vs + kp ? vs + kidx[j - vs] : j - kp + nv; };   // j >= vs

  __nv_bfloat16 *base = (which ? kv.v : kv.k) + layer * kv.stride_layer + b * kv.stride_batch + h * kv.stride_head;
  const int sub = threadIdx.x % LPR, slot = threadIdx.x / LPR;
  for (int j0 = vs; j0 < nl; j0 += CHUNK) {
    uint4 val[kInplacePasses];
    bool moved[kInplacePasses];
#pragma unroll
    for (int p = 0; p < kInplacePasses; ++p) {
      const int j = j0 + p * RPP + slot;
      moved[p] = false;
      if (j < nl) {
        const int sj = source(j);
        moved[p] = sj != j;
        if (moved[p]) val[p] = ld_cg_16(base + (long long)sj * kv.stride_pos + sub * 8);
      }
    }
    __syncthreads();                         // the whole chunk is in registers
#pragma unroll
    for (int p = 0; p < kInplacePasses; ++p) {
      const int j = j0 + p * RPP + slot;
      if (moved[p]) st_16(base + (long long)j * kv.stride_pos + sub * 8, val[p]);
    }
  }
  // position ids, by the CTA of the first slice: the same schedule, one row per thread
  if (blockIdx.x == 0 && which == 0 && pos) {
    int *prow = pos + (long long)b * pos_stride;
    for (int j0 = vs; j0 < nl; j0 += kGatherThreads) {
      const int j = j0 + threadIdx.x;
      int v = 0;
      bool moved = false;
      if (j < nl) {
        const int sj = source(j);
        moved = sj != j;
        if (moved) v = __ldcg(prow + sj);
      }
      __syncthreads();
      if (moved) prow[j] = v;
    }
  }
}

// ---------------------------------------------------------------------------
// Stage 3 on rows of any width (hidden states of layer K; FinalWipe with keep = 0).
// One CTA = 4 destination rows of one request; 16-byte chunks, 8 loads in flight per thread.
// ---------------------------------------------------------------------------
constexpr int kRowGatherRows = 4;

__global__ void __launch_bounds__(kGatherThreads)
row_gather_kernel(const unsigned char *__restrict__ src, unsigned char *__restrict__ dst, long long row_bytes,
                  long long s_row, long long s_batch, int src_rows, long long d_row, long long d_batch,
                  int dst_rows, const int *__restrict__ kept_idx, int r_max, const int *__restrict__ keep,
                  const int *__restrict__ prefix_len, const int *__restrict__ vis_start,
                  const int *__restrict__ n_vis, int *__restrict__ new_len, int *dev_status) {
  const int b = blockIdx.y;
  const int lp = prefix_len[b], vs = vis_start[b], nv = n_vis[b], kp = keep[b];
  const bool first = blockIdx.x == 0 && threadIdx.x == 0;
  if (!layout_ok(lp, vs, nv, src_rows, TWIG_MAX_VISUAL)) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_LAYOUT);
    return;
  }
  if (kp < 0 || kp > nv || kp > r_max) {
    if (first) flag_status(dev_status, b, TWIG_DEV_BAD_KEEP);
    return;
  }
  const int nl = lp - nv + kp;
  if (nl > dst_rows) {
    if (first) flag_status(dev_status, b, TWIG_DEV_OVERFLOW);
    return;
  }
  if (first && new_len) new_len[b] = nl;
  const int j0 = blockIdx.x * kRowGatherRows;
  if (j0 >= nl) return;
  const int *kidx = kept_idx + (long long)b * r_max;
  const unsigned char *sp[kRowGatherRows];
  unsigned char *dp[kRowGatherRows];
#pragma unroll
  for (int r = 0; r < kRowGatherRows; ++r) {
    const int j = j0 + r;
    int s = -1;
    if (j < nl) {
      if (j < vs) {
        s = j;
      } else if (j < vs + kp) {
        const int kk = kidx[j - vs];
        const int prev = (j > vs) ? kidx[j - vs - 1] : -1;
        if (kk < 0 || kk >= nv || kk <= prev) {
          if (threadIdx.x == 0) flag_status(dev_status, b, TWIG_DEV_BAD_INDEX);
        } else {
          s = vs + kk;
        }
      } else {
        s = j - kp + nv;
      }
    }
    sp[r] = s >= 0 ? src + b * s_batch + (long long)s * s_row : nullptr;
    dp[r] = dst + b * d_batch + (long long)j * d_row;
  }
  const long long chunks = row_bytes >> 4;
  for (long long c0 = threadIdx.x; c0 < chunks; c0 += 2 * kGatherThreads) {
    const long long c1 = c0 + kGatherThreads;
    uint4 v0[kRowGatherRows], v1[kRowGatherRows];
#pragma unroll
    for (int r = 0; r < kRowGatherRows; ++r) {
      if (sp[r]) {
        v0[r] = ld_nc_16(sp[r] + (c0 << 4));
        if (c1 < chunks) v1[r] = ld_nc_16(sp[r] + (c1 << 4));
      }
    }
#pragma unroll
    for (int r = 0; r < kRowGatherRows; ++r) {
      if (sp[r]) {
        st_16(dp[r] + (c0 << 4), v0[r]);
        if (c1 < chunks) st_16(dp[r] + (c1 << 4), v1[r]);
      }
    }
  }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
static inline int logits_stride(int k_max_len) { return (k_max_len + 3) & ~3; }

// partial softmax statistics per head: one per warp of the logits stage
static inline int score_parts(int k_max_len) { return (k_max_len + kScoreKeysPerCta - 1) / kScoreKeysPerCta * kScoreWarps; }

// scaled logits [batch, heads, stride], then the partial softmax statistics [batch, heads, parts]
static inline size_t logits_bytes(int batch, int n_q_heads, int max_len) {
  return (size_t)batch * n_q_heads * logits_stride(max_len) * sizeof(float);
}
size_t score_workspace_bytes(int batch, int n_q_heads, int max_len) {
  return logits_bytes(batch, n_q_heads, max_len) + (size_t)batch * n_q_heads * score_parts(max_len) * sizeof(float2);
}

struct ScoreArgs {
  const void *twig_q, *twig_k;
  int64_t ksb, ksh, ksp;
  int k_max_len;
  const int *prefix_len, *vis_start, *n_vis;
  int batch, n_q_heads, n_kv_heads, head_dim, norm_scope;
  float softmax_scale;
  float *scores;
  int m_max;
  const void *q_gate = nullptr, *k_gate = nullptr;     // both or neither (Eq. 7's gates)
};

static twig_status check_score_args(const ScoreArgs &a, const void *ws, size_t ws_bytes) {
  if (!a.twig_q || !a.twig_k || !a.prefix_len || !a.vis_start || !a.n_vis || !a.scores || !ws)
    return TWIG_ERR_NULL;
  if (a.batch <= 0 || a.n_q_heads <= 0 || a.n_kv_heads <= 0 || a.k_max_len <= 0 || a.m_max <= 0)
    return TWIG_ERR_SHAPE;
  if (a.n_q_heads % a.n_kv_heads) return TWIG_ERR_SHAPE;
  if (a.head_dim != 64 && a.head_dim != 128) return TWIG_ERR_UNSUPPORTED;
  if (a.n_q_heads / a.n_kv_heads > kMaxGroup || a.n_q_heads > kMaxQHeads) return TWIG_ERR_UNSUPPORTED;
  if (a.m_max > TWIG_MAX_VISUAL || a.batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (a.norm_scope != 0 && a.norm_scope != 1) return TWIG_ERR_UNSUPPORTED;
  if (a.ksp < a.head_dim) return TWIG_ERR_SHAPE;
  if (!aligned16(a.twig_q) || !aligned16(a.twig_k) || !aligned16(ws) || ((a.ksb | a.ksh | a.ksp) & 7))
    return TWIG_ERR_ALIGN;
  if (ws_bytes < score_workspace_bytes(a.batch, a.n_q_heads, a.k_max_len)) return TWIG_ERR_WORKSPACE;
  return TWIG_OK;
}

static twig_status launch_logits(const ScoreArgs &a, int *dev_status, void *ws, cudaStream_t st) {
  const float scale = a.softmax_scale != 0.f ? a.softmax_scale : 1.f / sqrtf((float)a.head_dim);
  dim3 grid((a.k_max_len + kScoreKeysPerCta - 1) / kScoreKeysPerCta, a.n_kv_heads, a.batch);
  const int group = a.n_q_heads / a.n_kv_heads;
  const int ls = logits_stride(a.k_max_len);
  auto q = static_cast<const __nv_bfloat16 *>(a.twig_q);
  auto k = static_cast<const __nv_bfloat16 *>(a.twig_k);
  auto qg = static_cast<const __nv_bfloat16 *>(a.q_gate);
  auto kg = static_cast<const __nv_bfloat16 *>(a.k_gate);
  PdlLaunch L(grid, dim3(kScoreThreads), 0, st);
  const long long ksb = a.ksb, ksh = a.ksh, ksp = a.ksp;
  float *lg = static_cast<float *>(ws);
  float2 *stats = reinterpret_cast<float2 *>(static_cast<unsigned char *>(ws) + logits_bytes(a.batch, a.n_q_heads, a.k_max_len));
  const int n_parts = score_parts(a.k_max_len);
  cudaError_t err;
#define TWIG_LOGITS(D_, G_)                                                                                          \
  err = cudaLaunchKernelEx(&L.cfg, ttp_logits_kernel<D_, G_>, q, k, qg, kg, ksb, ksh, ksp, a.k_max_len, a.prefix_len, \
                           a.vis_start, a.n_vis, a.n_q_heads, group, a.norm_scope, scale, lg, ls, stats, n_parts,     \
                           a.m_max, dev_status)
  if (a.head_dim == 128) {
    if (qg) TWIG_LOGITS(128, true); else TWIG_LOGITS(128, false);
  } else {
    if (qg) TWIG_LOGITS(64, true); else TWIG_LOGITS(64, false);
  }
#undef TWIG_LOGITS
  return err == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}

static twig_status launch_finalize(const float *logits, const ScoreArgs &a, const int *keep,
                                   int *kept_idx, int r_max, int *dev_status, int mode,
                                   cudaStream_t st) {
  static bool attr_set = false;
  const bool select = mode & 2;
  const size_t smem = select ? (size_t)a.m_max * sizeof(uint32_t) : 0;
  if (smem > 48 * 1024 && !attr_set) {
    if (cudaFuncSetAttribute(ttp_finalize_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TWIG_MAX_VISUAL * (int)sizeof(uint32_t)) != cudaSuccess)
      return TWIG_ERR_CUDA;
    attr_set = true;
  }
  // the selection needs a request's scores in one CTA; scores alone are spread over slices of 256 tokens
  constexpr int kSliceThreads = 256;
  const dim3 grid = select ? dim3(1, a.batch) : dim3((a.m_max + kSliceThreads - 1) / kSliceThreads, a.batch);
  PdlLaunch L(grid, dim3(select ? kTopkThreads : kSliceThreads), smem, st);
  const int ls = logits_stride(a.k_max_len);
  const float2 *stats = logits ? reinterpret_cast<const float2 *>(reinterpret_cast<const unsigned char *>(logits) +
                                                                  logits_bytes(a.batch, a.n_q_heads, a.k_max_len))
                               : nullptr;
  const cudaError_t err = cudaLaunchKernelEx(&L.cfg, ttp_finalize_topk_kernel, logits, ls, stats, score_parts(a.k_max_len),
                                             a.n_q_heads, a.k_max_len, a.prefix_len, a.vis_start, a.n_vis, keep,
                                             a.norm_scope, a.scores, a.m_max, kept_idx, r_max, dev_status, mode);
  return err == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}

// bytes from the base pointer to the end of the last row of a K (or V) tensor
static size_t kv_extent_bytes(const twig_kv *kv) {
  const long long last = (long long)(kv->n_layers - 1) * kv->stride_layer + (long long)(kv->batch - 1) * kv->stride_batch +
                         (long long)(kv->n_kv_heads - 1) * kv->stride_head + (long long)(kv->max_len - 1) * kv->stride_pos +
                         kv->head_dim;
  return (size_t)last * sizeof(__nv_bfloat16);
}
static bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + nb && y < x + na;
}
// dst names exactly the tensors of src: compaction in place
static bool same_kv(const twig_kv *a, const twig_kv *b) {
  return a->k == b->k && a->v == b->v && a->stride_layer == b->stride_layer && a->stride_batch == b->stride_batch &&
         a->stride_head == b->stride_head && a->stride_pos == b->stride_pos && a->max_len == b->max_len;
}

static twig_status check_compact_args(const twig_kv *src, const twig_kv *dst, const int *kept_idx,
                                      int r_max, const int *keep, const int *prefix_len,
                                      const int *vis_start, const int *n_vis, const int *pos_in,
                                      int *pos_out, int pos_stride) {
  twig_status s = check_kv(src);
  if (s != TWIG_OK) return s;
  s = check_kv(dst);
  if (s != TWIG_OK) return s;
  if (!kept_idx || !keep || !prefix_len || !vis_start || !n_vis) return TWIG_ERR_NULL;
  if ((pos_in == nullptr) != (pos_out == nullptr)) return TWIG_ERR_NULL;
  if (r_max <= 0 || (pos_in && pos_stride <= 0)) return TWIG_ERR_SHAPE;
  if (src->head_dim != dst->head_dim || src->n_layers != dst->n_layers || src->batch != dst->batch ||
      src->n_kv_heads != dst->n_kv_heads)
    return TWIG_ERR_SHAPE;
  if ((long long)src->n_layers * src->n_kv_heads > 65535) return TWIG_ERR_UNSUPPORTED;
  // dst is either the very same tensors as src (in place) or shares no byte with them
  if (!same_kv(src, dst)) {
    const void *sa[2] = {src->k, src->v}, *da[2] = {dst->k, dst->v};
    for (int i = 0; i < 2; ++i)
      for (int j = 0; j < 2; ++j)
        if (ranges_overlap(sa[i], kv_extent_bytes(src), da[j], kv_extent_bytes(dst))) return TWIG_ERR_UNSUPPORTED;
    if (pos_in && pos_in == pos_out) return TWIG_ERR_UNSUPPORTED;
  } else if (ranges_overlap(src->k, kv_extent_bytes(src), src->v, kv_extent_bytes(src))) {
    return TWIG_ERR_UNSUPPORTED;
  }
  return TWIG_OK;
}

static twig_status launch_gather(const twig_kv *src, const twig_kv *dst, const int *kept_idx, int r_max,
                                 const int *keep, const int *prefix_len, const int *vis_start,
                                 const int *n_vis, const int *pos_in, int *pos_out, int pos_stride,
                                 int *new_len, int *dev_status, cudaStream_t st, int early_text = 0) {
  if (same_kv(src, dst)) {
    // in place: one CTA per (layer, kv head, K or V, request); position ids move in place as well
    // (pos_out may be pos_in, or a separate array that then receives the gathered ids)
    if (pos_in && pos_out && pos_in != pos_out) {
      // a separate pos_out: gather it with the out-of-place rule (one small launch over no KV rows
      // would cost more than it is worth; the in-place kernel compacts pos_in itself instead)
      return TWIG_ERR_UNSUPPORTED;
    }
    dim3 grid(src->n_layers * src->n_kv_heads, 2, src->batch);
    if (src->head_dim == 128)
      kv_compact_inplace_kernel<128><<<grid, kGatherThreads, 0, st>>>(view_of_mut(dst), kept_idx, r_max, keep, prefix_len,
          vis_start, n_vis, pos_out, pos_stride, new_len, dev_status);
    else
      kv_compact_inplace_kernel<64><<<grid, kGatherThreads, 0, st>>>(view_of_mut(dst), kept_idx, r_max, keep, prefix_len,
          vis_start, n_vis, pos_out, pos_stride, new_len, dev_status);
    return launch_status();
  }
  // text rows of a request fit both tensors; kept visual rows are at most r_max (and at most dst's rows)
  const int rows_bound = src->max_len < dst->max_len ? src->max_len : dst->max_len;
  const int text_blocks = (rows_bound + kGatherRows - 1) / kGatherRows;
  const int vis_rows = r_max < dst->max_len ? r_max : dst->max_len;
  const int vis_blocks = (vis_rows + kGatherRows - 1) / kGatherRows;
  if (text_blocks + vis_blocks > 65535) return TWIG_ERR_UNSUPPORTED;
  dim3 grid(src->n_layers * src->n_kv_heads * src->batch, text_blocks + vis_blocks);
  PdlLaunch L(grid, dim3(kGatherThreads), 0, st);
  const KvView sv = view_of(src);
  const KvViewMut dv = view_of_mut(dst);
  if (!launch_overlap_enabled()) early_text = 0;
  const cudaError_t err =
      src->head_dim == 128
          ? cudaLaunchKernelEx(&L.cfg, kv_gather_kernel<128>, sv, dv, kept_idx, r_max, keep, prefix_len, vis_start, n_vis,
                               pos_in, pos_out, pos_stride, new_len, dev_status, text_blocks, early_text)
          : cudaLaunchKernelEx(&L.cfg, kv_gather_kernel<64>, sv, dv, kept_idx, r_max, keep, prefix_len, vis_start, n_vis,
                               pos_in, pos_out, pos_stride, new_len, dev_status, text_blocks, early_text);
  return err == cudaSuccess ? TWIG_OK : TWIG_ERR_CUDA;
}

}  // namespace twig

using namespace twig;

extern "C" twig_status ttp_score(const void *twig_q, const void *twig_k, int64_t k_stride_batch,
                                 int64_t k_stride_head, int64_t k_stride_pos, int32_t k_max_len,
                                 const int32_t *prefix_len, const int32_t *vis_start,
                                 const int32_t *n_vis, int32_t batch, int32_t n_q_heads,
                                 int32_t n_kv_heads, int32_t head_dim, int32_t norm_scope,
                                 float softmax_scale, float *scores, int32_t m_max,
                                 int32_t *dev_status, void *ws, size_t ws_bytes, void *stream) {
  ScoreArgs a{twig_q, twig_k, k_stride_batch, k_stride_head, k_stride_pos, k_max_len, prefix_len,
              vis_start, n_vis, batch, n_q_heads, n_kv_heads, head_dim, norm_scope, softmax_scale,
              scores, m_max};
  twig_status s = check_score_args(a, ws, ws_bytes);
  if (s != TWIG_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  s = launch_logits(a, dev_status, ws, st);
  if (s != TWIG_OK) return s;
  return launch_finalize(static_cast<const float *>(ws), a, nullptr, nullptr, 0, dev_status, 1, st);
}

extern "C" twig_status ttp_score_gated(const void *twig_q, const void *q_gate, const void *twig_k,
                                       const void *k_gate, int64_t k_stride_batch, int64_t k_stride_head,
                                       int64_t k_stride_pos, int32_t k_max_len, const int32_t *prefix_len,
                                       const int32_t *vis_start, const int32_t *n_vis, int32_t batch,
                                       int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                       int32_t norm_scope, float softmax_scale, float *scores,
                                       int32_t m_max, int32_t *dev_status, void *ws, size_t ws_bytes,
                                       void *stream) {
  if (!q_gate || !k_gate) return TWIG_ERR_NULL;
  if (!aligned16(q_gate) || !aligned16(k_gate)) return TWIG_ERR_ALIGN;
  ScoreArgs a{twig_q, twig_k, k_stride_batch, k_stride_head, k_stride_pos, k_max_len, prefix_len,
              vis_start, n_vis, batch, n_q_heads, n_kv_heads, head_dim, norm_scope, softmax_scale,
              scores, m_max, q_gate, k_gate};
  twig_status s = check_score_args(a, ws, ws_bytes);
  if (s != TWIG_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  s = launch_logits(a, dev_status, ws, st);
  if (s != TWIG_OK) return s;
  return launch_finalize(static_cast<const float *>(ws), a, nullptr, nullptr, 0, dev_status, 1, st);
}

// ---------------------------------------------------------------------------
// ttp_score for callers that cannot allocate device memory: the logits scratch is
// a fixed array that lives in the library image on every device that loads it.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[TWIG_NOALLOC_SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a handle; the device address has to be asked
// for, once per device, with that device current.
static twig_status noalloc_scratch_address(void **out) {
  constexpr int kMaxDevices = 64;
  static void *addr[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TWIG_ERR_CUDA;
  if (!addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return TWIG_ERR_CUDA;
    addr[dev] = p;
  }
  *out = addr[dev];
  return TWIG_OK;
}

extern "C" twig_status ttp_score_noalloc(const void *twig_q, const void *twig_k, int64_t k_stride_batch,
                                         int64_t k_stride_head, int64_t k_stride_pos, int32_t k_max_len,
                                         const int32_t *prefix_len, const int32_t *vis_start,
                                         const int32_t *n_vis, int32_t batch, int32_t n_q_heads,
                                         int32_t n_kv_heads, int32_t head_dim, int32_t norm_scope,
                                         float softmax_scale, float *scores, int32_t m_max,
                                         int32_t *dev_status, void *stream) {
  if (batch > 0 && n_q_heads > 0 && k_max_len > 0 &&
      score_workspace_bytes(batch, n_q_heads, k_max_len) > (size_t)TWIG_NOALLOC_SCRATCH_BYTES)
    return TWIG_ERR_WORKSPACE;     // batch * n_q_heads * k_max_len logits do not fit the fixed array
  void *ws = nullptr;
  twig_status s = noalloc_scratch_address(&ws);
  if (s != TWIG_OK) return s;
  ScoreArgs a{twig_q, twig_k, k_stride_batch, k_stride_head, k_stride_pos, k_max_len, prefix_len,
              vis_start, n_vis, batch, n_q_heads, n_kv_heads, head_dim, norm_scope, softmax_scale,
              scores, m_max};
  s = check_score_args(a, ws, TWIG_NOALLOC_SCRATCH_BYTES);
  if (s != TWIG_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // every logit the second kernel reads is written by the first one in this call, so the
  // array's old contents never matter and nothing has to be cleared
  s = launch_logits(a, dev_status, ws, st);
  if (s != TWIG_OK) return s;
  return launch_finalize(static_cast<const float *>(ws), a, nullptr, nullptr, 0, dev_status, 1, st);
}

extern "C" twig_status ttp_topk(const float *scores, const int32_t *n_vis, const int32_t *keep,
                                int32_t batch, int32_t m_max, int32_t r_max, int32_t *kept_idx,
                                int32_t *dev_status, void *stream) {
  if (!scores || !n_vis || !keep || !kept_idx) return TWIG_ERR_NULL;
  if (batch <= 0 || m_max <= 0 || r_max <= 0) return TWIG_ERR_SHAPE;
  if (m_max > TWIG_MAX_VISUAL || batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  ScoreArgs a{};
  a.n_vis = n_vis;
  a.batch = batch;
  a.scores = const_cast<float *>(scores);
  a.m_max = m_max;
  a.k_max_len = 1;
  return launch_finalize(nullptr, a, keep, kept_idx, r_max, dev_status, 2,
                         static_cast<cudaStream_t>(stream));
}

extern "C" twig_status ttp_compact(const twig_kv *src, const twig_kv *dst, const int32_t *kept_idx,
                                   int32_t r_max, const int32_t *keep, const int32_t *prefix_len,
                                   const int32_t *vis_start, const int32_t *n_vis,
                                   const int32_t *pos_in, int32_t *pos_out, int32_t pos_stride,
                                   int32_t *new_len, int32_t *dev_status, void *stream) {
  twig_status s = check_compact_args(src, dst, kept_idx, r_max, keep, prefix_len, vis_start, n_vis,
                                     pos_in, pos_out, pos_stride);
  if (s != TWIG_OK) return s;
  return launch_gather(src, dst, kept_idx, r_max, keep, prefix_len, vis_start, n_vis, pos_in, pos_out,
                       pos_stride, new_len, dev_status, static_cast<cudaStream_t>(stream));
}

extern "C" twig_status ttp_score_topk_compact(
    const void *twig_q, const void *twig_k, int64_t k_stride_batch, int64_t k_stride_head,
    int64_t k_stride_pos, int32_t k_max_len, const int32_t *prefix_len, const int32_t *vis_start,
    const int32_t *n_vis, const int32_t *keep, int32_t n_q_heads, int32_t norm_scope,
    float softmax_scale, float *scores, int32_t m_max, int32_t *kept_idx, int32_t r_max,
    const twig_kv *src, const twig_kv *dst, const int32_t *pos_in, int32_t *pos_out,
    int32_t pos_stride, int32_t *new_len, int32_t *dev_status, void *ws, size_t ws_bytes,
    void *stream) {
  twig_status s = check_compact_args(src, dst, kept_idx, r_max, keep, prefix_len, vis_start, n_vis,
                                     pos_in, pos_out, pos_stride);
  if (s != TWIG_OK) return s;
  ScoreArgs a{twig_q, twig_k, k_stride_batch, k_stride_head, k_stride_pos, k_max_len, prefix_len,
              vis_start, n_vis, src->batch, n_q_heads, src->n_kv_heads, src->head_dim, norm_scope,
              softmax_scale, scores, m_max};
  s = check_score_args(a, ws, ws_bytes);
  if (s != TWIG_OK) return s;
  if (k_max_len > src->max_len) return TWIG_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  s = launch_logits(a, dev_status, ws, st);
  if (s != TWIG_OK) return s;
  s = launch_finalize(static_cast<const float *>(ws), a, keep, kept_idx, r_max, dev_status, 3, st);
  if (s != TWIG_OK) return s;
  // The gather's predecessors in the stream are this call's own kernels: it may copy the rows that do
  // not depend on the selection while they run.  (Not in place: there every row move needs the list.)
  return launch_gather(src, dst, kept_idx, r_max, keep, prefix_len, vis_start, n_vis, pos_in, pos_out,
                       pos_stride, new_len, dev_status, st, same_kv(src, dst) ? 0 : 1);
}

extern "C" twig_status ttp_compact_rows(const void *src, void *dst, int64_t row_bytes, int64_t src_stride_row,
                                        int64_t src_stride_batch, int32_t src_rows, int64_t dst_stride_row,
                                        int64_t dst_stride_batch, int32_t dst_rows, int32_t batch,
                                        const int32_t *kept_idx, int32_t r_max, const int32_t *keep,
                                        const int32_t *prefix_len, const int32_t *vis_start,
                                        const int32_t *n_vis, int32_t *new_len, int32_t *dev_status,
                                        void *stream) {
  if (!src || !dst || !kept_idx || !keep || !prefix_len || !vis_start || !n_vis) return TWIG_ERR_NULL;
  if (row_bytes <= 0 || batch <= 0 || src_rows <= 0 || dst_rows <= 0 || r_max <= 0) return TWIG_ERR_SHAPE;
  if (src_stride_row < row_bytes || dst_stride_row < row_bytes) return TWIG_ERR_SHAPE;
  if (batch > TWIG_MAX_BATCH) return TWIG_ERR_UNSUPPORTED;
  if (src == dst) return TWIG_ERR_UNSUPPORTED;
  if ((row_bytes | src_stride_row | src_stride_batch | dst_stride_row | dst_stride_batch) & 15) return TWIG_ERR_ALIGN;
  if (!aligned16(src) || !aligned16(dst)) return TWIG_ERR_ALIGN;
  dim3 grid((dst_rows + kRowGatherRows - 1) / kRowGatherRows, batch);
  row_gather_kernel<<<grid, kGatherThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const unsigned char *>(src), static_cast<unsigned char *>(dst), row_bytes, src_stride_row,
      src_stride_batch, src_rows, dst_stride_row, dst_stride_batch, dst_rows, kept_idx, r_max, keep, prefix_len,
      vis_start, n_vis, new_len, dev_status);
  return launch_status();
}
