/*
 * twig.h — C ABI of the B200 (sm_100a) kernels for the inference hot path of
 * TwigVLM / TwigVLM++ ("Growing a Multi-head Twig via Distillation and
 * Reinforcement Learning to Accelerate Large Vision-Language Models").
 *
 * Three calls make up the path:
 *   ttp_score_topk_compact   twig-guided token pruning (Sec. 4.2 "TTP", Eq. 3, Eq. 5, Eq. 7/8)
 *   tree_verify_attention    tree attention of the verification pass (Sec. 5.4, Appendix A, Algorithm 2)
 *   tree_accept_compact      tree traversal / acceptance + bonus token + KV append (Sec. 5.4, Appendix A)
 * The three stages of the first call are exported on their own as well.
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 * Pointers: every data pointer is DEVICE memory unless marked "host".  The
 *   twig_kv descriptor structs themselves are host memory, read during the
 *   call.  The caller owns every buffer; the library allocates nothing.
 * dtype: K, V, Q and attention outputs are bf16 (2 bytes); scores and lse are
 *   fp32; all lengths, indices and token ids are int32.
 * Layout: head_dim is contiguous and is 64 or 128.  Strides are in ELEMENTS.
 *   Base pointers and row strides must make every row 16-byte aligned.
 *   q-head h reads kv-head h / (n_q_heads / n_kv_heads).
 * Stream: `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   Calls enqueue work and return; they never synchronise, and they read
 *   per-request metadata (lengths, parents, tokens) on the device.
 * Errors: anything the host can check returns a twig_status != TWIG_OK and
 *   launches nothing.  Data-dependent faults (a parent index out of range,
 *   keep > n_vis, a cache that would overflow ...) set dev_status[b] to a
 *   TWIG_DEV_* code and skip request b; kernels never trap or spin.
 *   dev_status (int32 [batch], may be NULL) is only ever written with
 *   non-zero codes: clear it before the call if you want to read it after.
 * Positions: K is cached after the rotary embedding, so rows are moved
 *   verbatim and kept tokens keep their ORIGINAL position ids (pos_ids are
 *   carried through the gather, never recomputed).
 */
#ifndef TWIG_H_
#define TWIG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TWIG_OK = 0,
  TWIG_ERR_NULL = 1,        /* a required pointer is NULL                          */
  TWIG_ERR_SHAPE = 2,       /* a size is non-positive or inconsistent               */
  TWIG_ERR_UNSUPPORTED = 3, /* head_dim not 64/128, t_max > 64, n_vis bound > max  */
  TWIG_ERR_WORKSPACE = 4,   /* ws_bytes < twig_workspace_bytes(...)                 */
  TWIG_ERR_CUDA = 5,        /* a CUDA runtime call failed (launch error)            */
  TWIG_ERR_ALIGN = 6        /* a pointer or stride breaks the 16-byte row rule      */
} twig_status;

/* per-request device status codes (written to dev_status[b]) */
enum {
  TWIG_DEV_OK = 0,
  TWIG_DEV_BAD_LAYOUT = 1, /* vis_start/n_vis/prefix_len inconsistent or out of bounds */
  TWIG_DEV_BAD_KEEP = 2,   /* keep < 0 or keep > n_vis                                 */
  TWIG_DEV_BAD_INDEX = 3,  /* kept_idx not strictly ascending within [0, n_vis)        */
  TWIG_DEV_BAD_TREE = 4,   /* n_nodes out of [0, t_max] or parent[i] not in [-1, i)    */
  TWIG_DEV_OVERFLOW = 5,   /* kv_len < 0 or kv_len + rows to append > max_len          */
  TWIG_DEV_INTERNAL = 6    /* a bounded on-chip wait ran out; the request's output is not written */
};

#define TWIG_MAX_NODES 64      /* draft-tree nodes per request (root included)      */
#define TWIG_MAX_VISUAL 16384  /* visual tokens per request                         */
#define TWIG_MAX_BATCH 4096    /* requests per call                                 */

/* One K/V tensor family: element (l, b, h, pos, c) of K is at
 * k[l*stride_layer + b*stride_batch + h*stride_head + pos*stride_pos + c]. */
typedef struct {
  void *k, *v;             /* device, bf16 */
  int64_t stride_layer, stride_batch, stride_head, stride_pos;
  int32_t n_layers, batch, n_kv_heads, head_dim, max_len;
} twig_kv;

const char *twig_status_str(twig_status s);

/* Bytes of device scratch the calls below need for these bounds (max_len is
 * the longest prompt / cache length any of them will see). */
size_t twig_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim, int32_t max_len,
                            int32_t max_nodes);

/* ---- TTP stage 1: importance score of every visual token -----------------
 * Eq. 3 / Eq. 5 (attention map of the last twig layer, row of the last prompt
 * token) and Eq. 7 (P-Head score).  For query head h:
 *   p_h = softmax_j( twig_q[b,h] . twig_k[b, h/G, j] * softmax_scale ),
 *   scores[b, m] = (1/n_q_heads) * sum_h p_h[vis_start[b] + m],  m < n_vis[b].
 * norm_scope 0: the softmax runs over j in [0, prefix_len[b]) (the last
 * query's full causal row); 1: over the visual span only (Eq. 7; scores sum
 * to 1).  softmax_scale 0 means 1/sqrt(head_dim).
 *   twig_q   [batch, n_q_heads, head_dim] contiguous (post-rotary, post-gate)
 *   twig_k   rows at twig_k + b*k_stride_batch + h*k_stride_head + j*k_stride_pos
 *   k_max_len  host bound on prefix_len (sizes the grid and the scratch)
 *   scores   [batch, m_max] fp32 out; entries m >= n_vis[b] are set to 0
 * Scratch: ws/ws_bytes from twig_workspace_bytes(batch, n_q_heads, head_dim, k_max_len, .).
 */
twig_status ttp_score(const void *twig_q, const void *twig_k, int64_t k_stride_batch,
                      int64_t k_stride_head, int64_t k_stride_pos, int32_t k_max_len,
                      const int32_t *prefix_len, const int32_t *vis_start, const int32_t *n_vis,
                      int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                      int32_t norm_scope, float softmax_scale, float *scores, int32_t m_max,
                      int32_t *dev_status, void *ws, size_t ws_bytes, void *stream);

/* ---- P-Head score with its gates applied in the kernel ----------------------
 * Eq. 7: s = (1/H) sum_h softmax( (G_q(x_q)^(h) * q^(h)) . (G_k(X_k)^(h) * K^(h))^T / sqrt(d_h) ), the
 * products element-wise.  ttp_score on q_gate * twig_q and k_gate * twig_k, the products formed in
 * fp32 inside the kernel (the gated tensors are never written).  The gates themselves (a linear
 * layer and an activation each) are inputs.
 *   q_gate  [batch, n_q_heads, head_dim] bf16, like twig_q
 *   k_gate  bf16, same strides and extent as twig_k (entry (b, h_kv, j, c) gates K's entry there)
 * Everything else as in ttp_score; Eq. 7 normalises over the visual span: norm_scope = 1.
 */
twig_status ttp_score_gated(const void *twig_q, const void *q_gate, const void *twig_k,
                            const void *k_gate, int64_t k_stride_batch, int64_t k_stride_head,
                            int64_t k_stride_pos, int32_t k_max_len, const int32_t *prefix_len,
                            const int32_t *vis_start, const int32_t *n_vis, int32_t batch,
                            int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                            int32_t norm_scope, float softmax_scale, float *scores, int32_t m_max,
                            int32_t *dev_status, void *ws, size_t ws_bytes, void *stream);

/* ---- Multi-query pruning guide (FastV's form of the TopR argument) ----------
 * Eq. 3: "sum_{i=M+1}^{M+N} A[i, 1:M]", the attention the textual tokens after the image pay to
 * every visual token, A the causal attention map averaged over heads:
 *   scores[b, m] = (1/n_q_heads) sum_h sum_i softmax_{j <= t_i}(q_text[b,h,i] . twig_k[b,h/G,j] * scale)[vis_start[b] + m],
 * i < N_b = prefix_len[b] - vis_start[b] - n_vis[b], t_i = vis_start[b] + n_vis[b] + i (text token i's
 * prompt position).  With one text token this is ttp_score with norm_scope 0.
 *   q_text  [batch, n_q_heads, n_text_max, head_dim] bf16 contiguous; rows i >= N_b are ignored.
 *           N_b > n_text_max is reported as TWIG_DEV_BAD_LAYOUT (scores of that request: 0)
 *   twig_k, strides, k_max_len, prefix_len, vis_start, n_vis, scores, m_max: as in ttp_score
 * Scratch: ttp_multiquery_workspace_bytes(batch, n_q_heads, n_text_max, m_max, k_max_len) bytes (it
 * holds one fp16 per (head, text row, key) between the kernels of the call: 2 * batch * n_q_heads *
 * n_text_max' * k_max_len' bytes plus statistics, the primes rounded up to 64 rows and 128 keys);
 * no initial contents are assumed.  softmax_scale must be positive (0: 1/sqrt(head_dim)).  The
 * result is reproducible from run to run (partial sums are added in a fixed order).
 */
size_t ttp_multiquery_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t n_text_max, int32_t m_max,
                                      int32_t k_max_len);
twig_status ttp_score_multiquery(const void *q_text, int32_t n_text_max, const void *twig_k,
                                 int64_t k_stride_batch, int64_t k_stride_head, int64_t k_stride_pos,
                                 int32_t k_max_len, const int32_t *prefix_len, const int32_t *vis_start,
                                 const int32_t *n_vis, int32_t batch, int32_t n_q_heads,
                                 int32_t n_kv_heads, int32_t head_dim, float softmax_scale,
                                 float *scores, int32_t m_max, int32_t *dev_status, void *ws,
                                 size_t ws_bytes, void *stream);

/* ---- ttp_score without any caller-provided or allocated scratch --------------
 * (No counterpart in the paper: this is a deployment convenience.)
 * Some hosts of this library may not allocate device memory at the point where
 * they prune: a serving process that handed all device memory to its own pool
 * at start-up, a plugin that is given tensors and a stream but no allocator, a
 * latency-critical loop that must stay clear of cudaMalloc because it
 * synchronises the device.  For them this variant of ttp_score keeps the fp32
 * logits scratch in a fixed array inside the library image,
 * TWIG_NOALLOC_SCRATCH_BYTES long; every GPU that loads the library holds that
 * much memory until the process exits.  Same arguments, results and errors as
 * ttp_score, minus ws / ws_bytes; it calls no allocator of any kind.
 * Limit: batch * n_q_heads * round_up(k_max_len, 4) * 4 bytes must fit in the
 * array, otherwise TWIG_ERR_WORKSPACE is returned and nothing is launched.
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.
 * All calls on a device share the one array.  It keeps the previous call's
 * logits, which is harmless (each call overwrites what it reads), but two calls
 * whose kernels overlap on the GPU (different streams) race on it: serialise
 * them, or give the concurrent ones their own scratch through ttp_score.
 */
#define TWIG_NOALLOC_SCRATCH_BYTES (4u << 20)
twig_status ttp_score_noalloc(const void *twig_q, const void *twig_k, int64_t k_stride_batch,
                              int64_t k_stride_head, int64_t k_stride_pos, int32_t k_max_len,
                              const int32_t *prefix_len, const int32_t *vis_start,
                              const int32_t *n_vis, int32_t batch, int32_t n_q_heads,
                              int32_t n_kv_heads, int32_t head_dim, int32_t norm_scope,
                              float softmax_scale, float *scores, int32_t m_max,
                              int32_t *dev_status, void *stream);

/* ---- TTP stage 2: TopR of Eq. 3 --------------------------------------------
 * kept_idx[b, 0..keep[b]) = indices of the keep[b] largest scores[b, 0..n_vis[b]),
 * equal scores resolved to the LOWER index, written in ascending index order
 * (sequence order is kept); entries past keep[b] are set to -1.  The choice is
 * exact on the fp32 bit patterns.  Scores must not be NaN.
 *   kept_idx [batch, r_max] int32 out;  m_max <= TWIG_MAX_VISUAL.
 */
twig_status ttp_topk(const float *scores, const int32_t *n_vis, const int32_t *keep, int32_t batch,
                     int32_t m_max, int32_t r_max, int32_t *kept_idx, int32_t *dev_status,
                     void *stream);

/* ---- TTP stage 3: prune the KV cache (Eq. 5 applied to cached rows) --------
 * New sequence of request b = [0, vis_start) ++ (vis_start + kept_idx[b, :keep])
 * ++ [vis_start + n_vis, prefix_len).  For every layer and kv head,
 * dst row j = src row idx[j] (bytes copied verbatim), pos_out[b, j] =
 * pos_in[b, idx[j]], new_len[b] = prefix_len - n_vis + keep.  keep = 0 drops
 * every visual token (the FinalWipe form); keep = n_vis is the identity.
 * pos_in/pos_out ([batch, pos_stride], may both be NULL) and new_len (may be
 * NULL) are int32.
 * Aliasing: dst either shares no byte with src (rows past new_len of dst are
 * left as they were), or names the very same tensors (same k, v, strides and
 * max_len): the cache is then compacted IN PLACE, which saves the second copy
 * of the KV cache; pos_out must then be pos_in (or both NULL).  Rows only move
 * to lower positions, so one CTA per (layer, kv head) slice moves them chunk by
 * chunk in ascending order; rows that stay where they are are not touched and
 * rows past new_len keep their old contents.  Any other overlap of dst and src
 * is refused with TWIG_ERR_UNSUPPORTED.  In place, a kept_idx list that is not
 * strictly ascending within [0, n_vis) is detected before anything moves
 * (TWIG_DEV_BAD_INDEX, request untouched).
 */
twig_status ttp_compact(const twig_kv *src, const twig_kv *dst, const int32_t *kept_idx,
                        int32_t r_max, const int32_t *keep, const int32_t *prefix_len,
                        const int32_t *vis_start, const int32_t *n_vis, const int32_t *pos_in,
                        int32_t *pos_out, int32_t pos_stride, int32_t *new_len,
                        int32_t *dev_status, void *stream);

/* ---- TTP stage 3 on hidden states: Eq. 5 in the paper's literal form -------------
 * The paper prunes the token sequence X^(K) that leaves layer K (and, with FinalWipe,
 * drops every visual token after layer K_f: keep = 0).  Same index list as ttp_compact,
 * applied to rows of any width: dst row j of request b = src row idx_b[j], bytes verbatim.
 *   src, dst   device; row (b, i) at base + b*stride_batch + i*stride_row (strides in BYTES)
 *   row_bytes  bytes per row, a multiple of 16 (e.g. d_model * 2); rows must be 16-byte aligned
 *   src_rows / dst_rows   rows available per request in src / dst (bounds for the checks)
 * new_len (may be NULL) receives prefix_len - n_vis + keep.  dst must not overlap src.
 */
twig_status ttp_compact_rows(const void *src, void *dst, int64_t row_bytes, int64_t src_stride_row,
                             int64_t src_stride_batch, int32_t src_rows, int64_t dst_stride_row,
                             int64_t dst_stride_batch, int32_t dst_rows, int32_t batch,
                             const int32_t *kept_idx, int32_t r_max, const int32_t *keep,
                             const int32_t *prefix_len, const int32_t *vis_start,
                             const int32_t *n_vis, int32_t *new_len, int32_t *dev_status,
                             void *stream);

/* ---- TTP, all three stages (Sec. 4.2, Algorithm 1 "pruning", Algorithm 2) --
 * Arguments as above; scores and kept_idx are outputs the caller may inspect. */
twig_status ttp_score_topk_compact(
    const void *twig_q, const void *twig_k, int64_t k_stride_batch, int64_t k_stride_head,
    int64_t k_stride_pos, int32_t k_max_len, const int32_t *prefix_len, const int32_t *vis_start,
    const int32_t *n_vis, const int32_t *keep, int32_t n_q_heads, int32_t norm_scope,
    float softmax_scale, float *scores, int32_t m_max, int32_t *kept_idx, int32_t r_max,
    const twig_kv *src, const twig_kv *dst, const int32_t *pos_in, int32_t *pos_out,
    int32_t pos_stride, int32_t *new_len, int32_t *dev_status, void *ws, size_t ws_bytes,
    void *stream);

/* ---- Tree attention of the verification pass, one layer per call ------------
 * Sec. 5.4 / Appendix A ("topology-aware causal mask so that each node attends
 * only to its ancestors"), Eq. 2.  Node i < n_nodes[b] of request b, head h:
 *   keys/values = cache rows [0, kv_len[b]) of layer `layer`, kv head h/G,
 *                 followed by tree rows j with j an ancestor of i or i itself;
 *   out[b,i,h,:] = softmax(q[b,i,h] . k * softmax_scale) @ v   (fp32 accumulate, bf16 out)
 *   lse[b,h,i]   = log sum exp of the visible scaled logits    (optional)
 *   q, out   [batch, t_max, n_q_heads, head_dim] bf16 contiguous
 *   tree_k/v [batch, n_kv_heads, t_max, head_dim] bf16 contiguous (this layer's draft-tree K/V)
 *   parent   [batch, t_max] int32; parent[b,0] = -1, parent[b,i] in [0, i)
 *   lse      [batch, n_q_heads, t_max] fp32 or NULL
 * t_max <= TWIG_MAX_NODES.  Rows of nodes >= n_nodes[b] are not written.
 * softmax_scale 0 means 1/sqrt(head_dim).  ws may be NULL when ws_bytes is 0: the kernels this call
 * chooses from combine key splits on chip and need no scratch (the persistent kernel of
 * tree_verify_attention_ex does).
 */
twig_status tree_verify_attention(const void *q, const void *tree_k, const void *tree_v,
                                  const twig_kv *cache, int32_t layer, const int32_t *kv_len,
                                  const int32_t *n_nodes, const int32_t *parent, int32_t t_max,
                                  int32_t n_q_heads, float softmax_scale, void *out, float *lse,
                                  int32_t *dev_status, void *ws, size_t ws_bytes, void *stream);

/* tree_verify_attention with per-call flags (the call above is this one with flags = 0).
 *
 * TWIG_ATTN_EARLY_PREFIX: the caller promises that the kernel which precedes this call in its stream
 *   writes neither kv_len, n_nodes, parent nor cache rows below kv_len (true when that kernel is
 *   another layer's attention or a projection of the same verification step; false right after
 *   tree_accept_compact or ttp_compact, which write kv_len).  The kernel then reads the lengths and
 *   starts fetching the cached prefix while the preceding kernel is still draining; q, tree_k and
 *   tree_v are still read only after it has completed.  Results do not change when the promise holds.
 * TWIG_ATTN_EARLY_QUERY (with TWIG_ATTN_EARLY_PREFIX): the second promise, that the preceding kernel does
 *   not write q, tree_k or tree_v either.  The small-call kernel then waits for nothing before it
 *   computes and only orders its stores after the preceding kernel, so consecutive calls overlap
 *   almost entirely.  In a model the layers of a verification step cannot make this promise (a
 *   layer's q is computed from the previous layer's output): it exists to measure what the launch
 *   chain costs, and for callers whose q is staged ahead of time.
 * TWIG_ATTN_PLAIN_LAUNCH: launch without programmatic stream serialization (see twig_set_launch_overlap).
 * TWIG_ATTN_KERNEL(k): run exactly kernel k, a testing and tuning control (all kernels compute the
 *   same function).  TWIG_ATTN_KERNEL_AUTO picks by shape; _MMA is the mma.sync kernel (any shape);
 *   _TCGEN05 the tcgen05 kernel whose key splits are the CTAs of a cluster; _STREAM the persistent
 *   tcgen05 kernel (needs ws, below).  The tcgen05 kernels need head_dim 128 and a cache layout that a
 *   tensor map can describe; a named kernel that cannot run the call returns TWIG_ERR_UNSUPPORTED (or
 *   TWIG_ERR_WORKSPACE); only the automatic choice moves on to another kernel.
 * TWIG_ATTN_SPLITS(n): force n = 1, 2, 4 or 8 key splits per cluster in the _MMA and _TCGEN05 kernels.
 * TWIG_ATTN_STREAM_SHARES / _WHOLE: how the persistent kernel shares the work between its CTAs: equal
 *   shares of all key tiles (items may straddle CTAs) or whole items dealt out longest first; by
 *   default the kernel picks from the lengths it finds on the device.  A testing control.
 *
 * Scratch of the persistent kernel.  One CTA per SM slot walks an equal share of all (request, kv head,
 * row block, key tile) work; a work item that straddles two CTAs is finished by whichever of them
 * arrives last, through ws: per-item arrival counters followed by per-CTA partial results.
 *   size      tree_attention_workspace_bytes(batch, n_q_heads, max_nodes) (twig_workspace_bytes is
 *             at least that large)
 *   contents  the first call that uses a buffer must find it ZERO-FILLED (cudaMemset once after
 *             allocation); every call leaves its counters at zero again.  Nothing else may write
 *             the buffer between calls: do not pass the buffer that ttp_score uses.
 *   sharing   calls whose kernels may overlap on the GPU need a buffer each.
 * The automatic choice does not take the persistent kernel (on the shapes measured so far the
 * cluster kernel is faster); ws is only read when TWIG_ATTN_KERNEL_STREAM is named.
 */
#define TWIG_ATTN_EARLY_PREFIX 1u
#define TWIG_ATTN_KERNEL_AUTO 0u
#define TWIG_ATTN_KERNEL_MMA 1u
#define TWIG_ATTN_KERNEL_TCGEN05 2u
#define TWIG_ATTN_KERNEL_STREAM 3u
#define TWIG_ATTN_KERNEL(k) ((uint32_t)(k) << 1)
#define TWIG_ATTN_PLAIN_LAUNCH (1u << 4)
#define TWIG_ATTN_EARLY_QUERY (1u << 5)
#define TWIG_ATTN_SPLITS(n) ((uint32_t)(n) << 8)
#define TWIG_ATTN_STREAM_SHARES (1u << 12)
#define TWIG_ATTN_STREAM_WHOLE (2u << 12)
twig_status tree_verify_attention_ex(const void *q, const void *tree_k, const void *tree_v,
                                     const twig_kv *cache, int32_t layer, const int32_t *kv_len,
                                     const int32_t *n_nodes, const int32_t *parent, int32_t t_max,
                                     int32_t n_q_heads, float softmax_scale, void *out, float *lse,
                                     int32_t *dev_status, void *ws, size_t ws_bytes, void *stream,
                                     uint32_t flags);
size_t tree_attention_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t max_nodes);

/* Launch overlap (default on): tree_verify_attention and tree_accept_compact launch their kernels
 * with programmatic stream serialization, so the next kernel of the stream is scheduled while the
 * current one drains; each kernel waits on the device for its predecessor before it reads anything,
 * so results do not change.  0 switches it off for the whole process (an atomic flag; a testing
 * control, not meant to be toggled while other threads are launching).  Returns the previous value. */
int32_t twig_set_launch_overlap(int32_t on);

/* ---- Draft-side token tree ---------------------------------------------------
 * Sec. 4.3 and the appendix's "Tree-based self-speculative decoding": the tree is rooted at the last
 * accepted token and grown level by level with an expansion width E, a selection width K and a
 * depth D; level 1 holds the root's top-E tokens, at every later level the K best nodes of the level
 * before are expanded into their top-E tokens; the finished tree is cut to N_max nodes.  The draft
 * model runs between these calls (its logits are inputs).  A node's score is the log of the joint
 * probability of its root-to-node path; "best" is by score, equal scores to the lower node id, equal
 * logits to the lower token id.  Logits must not be NaN.
 *
 * Tree state of request b: node_tok / node_parent / node_score [batch, cap], node 0 the root, nodes in
 * creation order (level 1 at 1..E, each later level after it).  tree_reset writes the roots (node 0:
 * token -1, parent -1, score 0); so does an expansion with level_base == 1, so a caller that starts
 * every tree with such a call needs no tree_reset.
 *
 * tree_expand_level: row r of logits ([batch, rows, vocab] at (b*rows + r)*row_stride ELEMENTS, bf16 or
 *   fp32, rows 16-byte aligned) is the draft distribution after node src_node[b, r] (-1: unused row);
 *   its n_children (<= 16) most probable tokens become nodes level_base + r*n_children + e, best
 *   first, with score = score[src] + log softmax(row)[token].  level_base = first node id of the new
 *   level (1 for level 1); every src must be older than level_base (else TWIG_DEV_BAD_TREE).
 * tree_select_expansion: expand_node[b, 0..n_select) = ids of the n_select best nodes among
 *   level_lo..level_hi-1, ascending: the src_node of the next tree_expand_level.  n_select may not
 *   exceed the level's size (TWIG_ERR_SHAPE), so that every row of the next level has a node.
 * tree_finalize: keeps the root and the n_max - 1 best of the nodes 1..n_built-1 (a set closed under
 *   parents, since a child's score never exceeds its parent's), renumbers them in creation order and
 *   writes parent / draft_tok [batch, t_max] (root: parent -1, token -1; unused entries -1 / 0) and
 *   n_nodes[b]: the arrays tree_verify_attention and tree_accept_compact take.  kept_node (optional)
 *   [batch, t_max]: the state id of every kept node.  n_max <= t_max <= TWIG_MAX_NODES; cap <= 6144.
 * tree_grow_level: one level in one launch: tree_expand_level, then, for every request, in the CTA
 *   that finishes the request's last row, the step that consumes the new level
 *   (level_hi = level_base + rows*n_children):
 *     n_select > 0:  tree_select_expansion over level_base..level_hi-1 into expand_node [batch, n_select]
 *                    (n_max, parent, draft_tok, n_nodes, kept_node, t_max are not used);
 *     n_select == 0: tree_finalize with n_built = level_hi (expand_node is not used).
 *   Same results as the two calls one after the other.  A tree of depth D is D calls.
 *   ticket [batch] int32 (device): zero-filled by the caller before its first use, left zero by every
 *   call; written only by these calls; one array per stream that builds trees concurrently.
 */
twig_status tree_reset(int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                       int32_t batch, void *stream);
twig_status tree_expand_level(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                              int32_t rows, const int32_t *src_node, int32_t n_children, int32_t level_base,
                              int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                              int32_t batch, int32_t *dev_status, void *stream);
twig_status tree_select_expansion(const float *node_score, int32_t cap, int32_t level_lo, int32_t level_hi,
                                  int32_t n_select, int32_t *expand_node, int32_t batch,
                                  int32_t *dev_status, void *stream);
twig_status tree_finalize(const int32_t *node_tok, const int32_t *node_parent, const float *node_score,
                          int32_t cap, int32_t n_built, int32_t n_max, int32_t *parent, int32_t *draft_tok,
                          int32_t *n_nodes, int32_t *kept_node, int32_t t_max, int32_t batch,
                          int32_t *dev_status, void *stream);
twig_status tree_grow_level(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                            int32_t rows, const int32_t *src_node, int32_t n_children, int32_t level_base,
                            int32_t *node_tok, int32_t *node_parent, float *node_score, int32_t cap,
                            int32_t batch, int32_t n_select, int32_t *expand_node, int32_t n_max,
                            int32_t *parent, int32_t *draft_tok, int32_t *n_nodes, int32_t *kept_node,
                            int32_t t_max, int32_t *ticket, int32_t *dev_status, void *stream);

/* ---- Chain drafting with early exit (sequence self-speculative decoding) ------
 * Appendix A, "Self-speculative decoding", and Algorithm 1's draft loop: in every iteration the draft
 * model predicts up to delta = 5 tokens one after another and stops early once the probability of
 * the token it has just predicted falls below theta = 0.6; that token still counts as drafted.  The
 * draft model runs between the calls; chain_draft_step takes one draft distribution per request:
 *   token = argmax_v logits[b, v] (lowest id among equal logits), prob = softmax(logits[b])[token],
 *   node n = n_nodes[b] is appended to the request's chain: parent[b, n] = n - 1,
 *   draft_tok[b, n] = token, tok_prob[b, n] = prob (optional), n_nodes[b] = n + 1;
 *   the request stops drafting (active[b] = 0) once it holds max_draft draft tokens or prob < threshold.
 * Requests with active[b] == 0 are left alone, so a batch is driven through max_draft calls without
 * reading anything back; afterwards n_nodes[b] - 1 is the request's draft length.  The arrays are
 * the ones tree_verify_attention and tree_accept_compact take (a chain is a tree whose node i has
 * parent i - 1; node 0, the root, is the last accepted token).  chain_draft_reset starts an
 * iteration: n_nodes = 1, parent[b, 0] = -1, draft_tok[b, 0] = -1, active = 1.
 *   logits   [batch, vocab] at logits + b*row_stride (ELEMENTS), bf16 (logits_fp32 = 0) or fp32; rows
 *            16-byte aligned; must not be NaN
 *   parent, draft_tok [batch, t_max] int32; tok_prob [batch, t_max] fp32 or NULL; n_nodes, active [batch]
 *   max_draft + 1 <= t_max <= TWIG_MAX_NODES (TWIG_ERR_SHAPE otherwise); threshold >= 0
 * The probability is formed in fp32 (one pass: running maximum and sum of exponentials).
 */
twig_status chain_draft_reset(int32_t *parent, int32_t *draft_tok, float *tok_prob, int32_t *n_nodes,
                              int32_t *active, int32_t t_max, int32_t batch, void *stream);
twig_status chain_draft_step(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                             int32_t max_draft, float threshold, int32_t *parent, int32_t *draft_tok,
                             float *tok_prob, int32_t *n_nodes, int32_t *active, int32_t t_max,
                             int32_t batch, int32_t *dev_status, void *stream);

/* ---- Greedy target token of every tree node (input of tree_accept_compact) -----
 * Algorithm 2 ("argmax(tgt_probs[...])"), Sec. 5.4: base_argmax[b, i] = the index of the largest of
 * logits[b, i, 0..vocab), the LOWEST index among equal values, for i < n_nodes[b]; other entries
 * are left untouched.  Logits must not be NaN.
 *   logits      [batch, t_max, vocab] at logits + (b*t_max + i)*row_stride (ELEMENTS), bf16
 *               (logits_fp32 = 0) or fp32 (logits_fp32 = 1); rows 16-byte aligned
 *   base_argmax [batch, t_max] int32 out
 */
twig_status tree_base_argmax(const void *logits, int32_t logits_fp32, int64_t row_stride, int32_t vocab,
                             const int32_t *n_nodes, int32_t batch, int32_t t_max,
                             int32_t *base_argmax, int32_t *dev_status, void *stream);

/* ---- Acceptance + bonus token + KV append, all layers in one call ------------
 * Sec. 5.4 / Appendix A / Algorithm 2.  Node 0 is the last accepted token and is
 * always accepted; child c is accepted iff its parent is and
 * draft_tok[b,c] == base_argmax[b,parent[c]] (base_argmax[b,u] is the target's
 * greedy token after consuming node u).  The winner is the accepted node of
 * greatest depth (lowest index among equals);
 *   path[b, 0..accept_len[b]] = root..winner, remaining entries -1,
 *   accept_len[b] = depth(winner)   (accepted draft tokens, root excluded),
 *   bonus_tok[b]  = base_argmax[b, winner].
 * Then for every layer l and kv head: cache row kv_len[b] + j = tree row
 * path[b, j] (j <= accept_len[b]) and kv_len[b] += accept_len[b] + 1.
 *   tree_k_all/v_all [n_layers, batch, n_kv_heads, t_max, head_dim] bf16 contiguous
 *   path [batch, d_max]; d_max must be >= the deepest level count (<= t_max)
 * Requests with n_nodes[b] == 0 are idle: nothing is written for them.
 * Two calls that are in flight at once on one device must not share a batch
 * slot b (the completion ticket of slot b is library state).
 */
twig_status tree_accept_compact(const int32_t *parent, const int32_t *draft_tok,
                                const int32_t *base_argmax, const int32_t *n_nodes, int32_t t_max,
                                int32_t d_max, const void *tree_k_all, const void *tree_v_all,
                                const twig_kv *cache, int32_t *kv_len, int32_t *accept_len,
                                int32_t *path, int32_t *bonus_tok, int32_t *dev_status,
                                void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TWIG_H_ */
