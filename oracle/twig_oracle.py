"""fp64 CPU oracle for the TwigVLM / TwigVLM++ inference hot path.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, exact-definition
implementation used to check the CUDA library; nothing in the product path
may import it, and it imports nothing from the product.  All floating-point
inputs are float64 arrays (bf16 values widened exactly by the caller); all
arithmetic is float64; softmax is the two-pass textbook form (max, then
sum); there is no tiling, no online rescaling and no key splitting.
``numpy.matmul`` is the only library primitive used.

Parity pins (tests/test_oracle_*.py): every function below is pinned by
closed forms, invariants the paper states, reductions to a library routine
(causal scaled-dot-product attention in float64) or brute force on tiny
inputs.  ``ttp_scores`` has no paper-printed numeric example to compare with
(the paper prints no score values): its pins are closed forms and
invariants only.

Readings of the paper where it leaves a choice (each is also a test):
  * scoring query = the last prompt token; heads are averaged (Eq. 7).
  * norm_scope 0: softmax over the whole causal row of that query (it sees
    every prompt key), then the visual columns are sliced (Eq. 2/3/5);
    norm_scope 1: softmax over the visual keys only (Eq. 7).
  * TopR ties go to the lower index; kept tokens stay in sequence order.
  * a tree node attends to the whole KV prefix, its ancestors and itself.
  * node 0 (root) is the last accepted token; it is always accepted.
  * child c is accepted iff draft_tok[c] == base_argmax[parent[c]] and its
    parent is accepted; the winner is the deepest accepted node (lowest index
    among equals); the bonus token is base_argmax[winner] (Sec. 5.4,
    Appendix A, Algorithm 2).
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# Eq. 4 / Eq. 6: average number of retained visual tokens
# --------------------------------------------------------------------------
def avg_retained_tokens(M: int, K: int, R: int, L: int, K_f=None) -> float:
    """Eq. 4 (K_f None): [M*K + R*(L-K)]/L.  Eq. 6: [M*K + R*(K_f-K)]/L."""
    upper = L if K_f is None else K_f
    return (M * K + R * (upper - K)) / L


# --------------------------------------------------------------------------
# O1: visual-token importance scores (Eq. 3/5 attention-map reading, Eq. 7)
# --------------------------------------------------------------------------
def ttp_scores(q, k, prefix_len, vis_start, n_vis, norm_scope=0, scale=None):
    """q [B,Hq,d], k [B,Hkv,Lmax,d] float64 -> s [B,Mmax] float64 (0 beyond n_vis).

    For request b and query head h (KV head h // G, G = Hq/Hkv):
      z_j = (q[b,h] . k[b,h//G,j]) * scale over the scope,
      p = softmax(z),  s[b,m] = mean_h p_h[vis_start + m].
    Scope: norm_scope 0 -> j in [0, prefix_len); 1 -> j in the visual span.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    m_max = int(np.max(n_vis)) if B else 0
    s = np.zeros((B, m_max), dtype=np.float64)
    for b in range(B):
        lp, vs, m = int(prefix_len[b]), int(vis_start[b]), int(n_vis[b])
        if m == 0:
            continue
        lo, hi = (0, lp) if norm_scope == 0 else (vs, vs + m)
        for h in range(Hq):
            z = np.matmul(k[b, h // G, lo:hi, :], q[b, h, :]) * scale
            e = np.exp(z - np.max(z))
            p = e / np.sum(e)
            s[b, :m] += p[vs - lo: vs - lo + m]
        s[b, :m] /= Hq
    return s


def ttp_scores_gated(q, q_gate, k, k_gate, prefix_len, vis_start, n_vis, norm_scope=1, scale=None):
    """Eq. 7, written out: for head h (KV head h // G) and key j of the scope
      z_j = sum_c (q_gate[b,h,c] * q[b,h,c]) * (k_gate[b,h//G,j,c] * k[b,h//G,j,c]) / sqrt(d),
    p = softmax_j(z), s[b,m] = mean_h p_h[visual token m].  q, q_gate [B,Hq,d]; k, k_gate
    [B,Hkv,Lmax,d].  Eq. 7 normalises over the visual tokens (norm_scope 1)."""
    q, q_gate = np.asarray(q, dtype=np.float64), np.asarray(q_gate, dtype=np.float64)
    k, k_gate = np.asarray(k, dtype=np.float64), np.asarray(k_gate, dtype=np.float64)
    B, Hq, d = q.shape
    G = Hq // k.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    m_max = int(np.max(n_vis)) if B else 0
    s = np.zeros((B, m_max), dtype=np.float64)
    for b in range(B):
        lp, vs, m = int(prefix_len[b]), int(vis_start[b]), int(n_vis[b])
        if m == 0:
            continue
        lo, hi = (0, lp) if norm_scope == 0 else (vs, vs + m)
        for h in range(Hq):
            gq = q_gate[b, h] * q[b, h]                               # [d]
            gk = k_gate[b, h // G, lo:hi] * k[b, h // G, lo:hi]       # [scope, d]
            z = np.sum(gk * gq[None, :], axis=1) * scale
            e = np.exp(z - np.max(z))
            s[b, :m] += (e / np.sum(e))[vs - lo: vs - lo + m]
        s[b, :m] /= Hq
    return s


def text_to_visual_scores(q_text, k, prefix_len, vis_start, n_vis, scale=None):
    """Eq. 3's guide "sum_{i=M+1}^{M+N} A[i, 1:M]": attention that the textual tokens after the
    image pay to every visual token, with A the causal attention map averaged over heads.
    q_text [B,Hq,Nmax,d]: row i is the query at prompt position vis_start + n_vis + i
    (N_b = prefix_len - vis_start - n_vis of them); k [B,Hkv,Lmax,d].  For head h and query i at
    position t: p = softmax_{j <= t}(q . k_j * scale);  s[b,m] = (1/Hq) sum_h sum_i p[vis_start + m]."""
    q_text = np.asarray(q_text, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    B, Hq, _, d = q_text.shape
    G = Hq // k.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    m_max = int(np.max(n_vis)) if B else 0
    s = np.zeros((B, m_max), dtype=np.float64)
    for b in range(B):
        lp, vs, m = int(prefix_len[b]), int(vis_start[b]), int(n_vis[b])
        for h in range(Hq):
            for i in range(lp - vs - m):
                t = vs + m + i
                z = np.matmul(k[b, h // G, :t + 1, :], q_text[b, h, i, :]) * scale
                e = np.exp(z - np.max(z))
                s[b, :m] += (e / np.sum(e))[vs:vs + m]
        s[b, :m] /= Hq
    return s


# --------------------------------------------------------------------------
# O2: TopR with the lowest-index tie rule (Eq. 3)
# --------------------------------------------------------------------------
def topk_lowest_index(s, R: int):
    """Indices of the R largest entries of s; among equal values the lower
    index wins; returned ascending."""
    s = np.asarray(s)
    order = sorted(range(len(s)), key=lambda m: (-s[m], m))
    return np.array(sorted(order[:R]), dtype=np.int32)


# --------------------------------------------------------------------------
# O3: pruned sequence and the row gather (Eq. 3 / Eq. 5 applied to KV rows)
# --------------------------------------------------------------------------
def prune_index_list(prefix_len: int, vis_start: int, n_vis: int, kept):
    """text before the image, kept visual tokens (ascending), text after."""
    kept = [int(x) for x in kept]
    return np.array(list(range(vis_start)) + [vis_start + m for m in kept]
                    + list(range(vis_start + n_vis, prefix_len)), dtype=np.int64)


def gather_compact(src_k, src_v, pos_in, prefix_len, vis_start, n_vis, kept_list, dst_k, dst_v, pos_out):
    """dst[l,b,h,j,:] = src[l,b,h,idx_b[j],:], pos_out[b,j] = pos_in[b,idx_b[j]].

    Arrays of any dtype (bit patterns are moved verbatim); dst/pos_out are
    updated in place, rows >= new_len are left as they were.  Returns new_len.
    dst may be src itself (compaction in place): rows are assigned in ascending
    order and idx_b[j] >= j, so a row is read before anything is written over it.
    """
    B = src_k.shape[1]
    new_len = np.zeros(B, dtype=np.int32)
    for b in range(B):
        idx = prune_index_list(int(prefix_len[b]), int(vis_start[b]), int(n_vis[b]), kept_list[b])
        n = len(idx)
        new_len[b] = n
        for j in range(n):
            dst_k[:, b, :, j, :] = src_k[:, b, :, idx[j], :]
            dst_v[:, b, :, j, :] = src_v[:, b, :, idx[j], :]
            pos_out[b, j] = pos_in[b, idx[j]]
    return new_len


def gather_rows(src, prefix_len, vis_start, n_vis, kept_list, dst):
    """Eq. 5 in its literal form: prune a [B, L, ...] token sequence (the layer-K hidden
    states X^(K)).  dst[b, j] = src[b, idx_b[j]]; rows >= new_len stay as they were.
    kept_list[b] = [] removes every visual token (FinalWipe after layer K_f)."""
    B = src.shape[0]
    new_len = np.zeros(B, dtype=np.int32)
    for b in range(B):
        idx = prune_index_list(int(prefix_len[b]), int(vis_start[b]), int(n_vis[b]), kept_list[b])
        new_len[b] = len(idx)
        for j, i in enumerate(idx):
            dst[b, j] = src[b, i]
    return new_len


# --------------------------------------------------------------------------
# O4: tree-masked verification attention (Sec. 5.4, Appendix A, Eq. 2)
# --------------------------------------------------------------------------
def ancestors_or_self(parent, i: int):
    """Root path of node i, root first.  A parent array must have parent[0] = -1
    and parent[x] in [0, x) for x > 0; anything else is rejected."""
    out = []
    x = int(i)
    while x >= 0:
        out.append(x)
        p = int(parent[x])
        if not (-1 <= p < x) or (x == 0) != (p == -1):
            raise ValueError(f"invalid parent array: parent[{x}] = {p}")
        x = p
    return out[::-1]


def tree_mask(parent, n_nodes: int, kv_len: int):
    """Topology-aware causal mask of one request: visible[i, j] for node i over
    the key sequence (cache rows 0..kv_len-1, then tree nodes 0..n_nodes-1)."""
    vis = np.zeros((n_nodes, kv_len + n_nodes), dtype=bool)
    vis[:, :kv_len] = True
    for i in range(n_nodes):
        for a in ancestors_or_self(parent, i):
            vis[i, kv_len + a] = True
    return vis


def masked_attention(q_rows, keys, vals, visible, scale):
    """Eq. 2 with mask: softmax over the visible keys of (q.k)*scale, times V.
    q_rows [n,d], keys/vals [m,d], visible [n,m] bool.  Returns (out [n,d], lse [n])."""
    z = np.matmul(q_rows, keys.T) * scale
    z = np.where(visible, z, -np.inf)
    zmax = np.max(z, axis=1, keepdims=True)
    e = np.exp(z - zmax)
    se = np.sum(e, axis=1, keepdims=True)
    return np.matmul(e / se, vals), (zmax + np.log(se))[:, 0]


def tree_attention(q, tree_k, tree_v, cache_k, cache_v, kv_len, n_nodes, parent, scale=None,
                   samples=None):
    """q [B,T,Hq,d]; tree_k/v [B,Hkv,T,d]; cache_k/v [B,Hkv,Lmax,d] (one layer).

    Node i of request b, head h: keys/values are cache rows [0, kv_len[b]) of
    KV head h//G followed by the tree rows, of which only i's ancestors and i
    itself are visible; out = softmax(q.k * scale) @ v, lse = log-sum-exp of
    the visible scaled logits.
    Returns out [B,T,Hq,d] and lse [B,Hq,T]; rows of nodes >= n_nodes[b] are 0.
    With ``samples`` (a list of (b, i, h)) only those rows are computed.
    """
    q = np.asarray(q, dtype=np.float64)
    B, T, Hq, d = q.shape
    Hkv = tree_k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((B, T, Hq, d), dtype=np.float64)
    lse = np.zeros((B, Hq, T), dtype=np.float64)

    def head_inputs(b, h):
        L, n = int(kv_len[b]), int(n_nodes[b])
        g = h // G
        keys = np.concatenate([cache_k[b, g, :L, :], tree_k[b, g, :n, :]], axis=0).astype(np.float64)
        vals = np.concatenate([cache_v[b, g, :L, :], tree_v[b, g, :n, :]], axis=0).astype(np.float64)
        return keys, vals

    if samples is not None:
        for (b, i, h) in samples:
            keys, vals = head_inputs(b, h)
            vis = tree_mask(parent[b], int(n_nodes[b]), int(kv_len[b]))
            o, l = masked_attention(q[b, i:i + 1, h, :], keys, vals, vis[i:i + 1], scale)
            out[b, i, h, :] = o[0]
            lse[b, h, i] = l[0]
        return out, lse

    for b in range(B):
        n = int(n_nodes[b])
        if n == 0:
            continue
        vis = tree_mask(parent[b], n, int(kv_len[b]))
        for h in range(Hq):
            keys, vals = head_inputs(b, h)
            o, l = masked_attention(q[b, :n, h, :], keys, vals, vis, scale)
            out[b, :n, h, :] = o
            lse[b, h, :n] = l
    return out, lse


# --------------------------------------------------------------------------
# O5: greedy tree acceptance (Sec. 5.4, Appendix A, Algorithm 2)
# --------------------------------------------------------------------------
def tree_accept(parent, draft_tok, base_argmax, n_nodes: int):
    """One request.  Returns (accept_len, path, bonus).

    A node is accepted when every edge (u -> c) on its root path has
    draft_tok[c] == base_argmax[u].  The winner is the accepted node of
    greatest depth, lowest index among equals; path = root..winner;
    accept_len = depth(winner) (draft tokens accepted, root excluded);
    bonus = base_argmax[winner].
    """
    best, best_depth = 0, 0
    for i in range(int(n_nodes)):
        chain = ancestors_or_self(parent, i)
        ok = all(int(draft_tok[c]) == int(base_argmax[u]) for u, c in zip(chain[:-1], chain[1:]))
        depth = len(chain) - 1
        if ok and depth > best_depth:
            best, best_depth = i, depth
    path = ancestors_or_self(parent, best)
    return best_depth, np.array(path, dtype=np.int32), int(base_argmax[best])


def base_argmax(logits, n_nodes):
    """Algorithm 2, "argmax(tgt_probs[...])": the target's greedy token after every tree node.
    logits [B, T, V]; returns int32 [B, T] with the LOWEST index among equal maxima and 0 for
    nodes >= n_nodes[b] (softmax is monotonic, so probabilities and logits agree)."""
    logits = np.asarray(logits, dtype=np.float64)
    B, T, V = logits.shape
    out = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        for i in range(int(n_nodes[b])):
            best, best_v = 0, logits[b, i, 0]
            for v in range(1, V):
                if logits[b, i, v] > best_v:
                    best, best_v = v, logits[b, i, v]
            out[b, i] = best
    return out


# --------------------------------------------------------------------------
# Draft-side token tree (Sec. 4.3 "tree-based SSD", Appendix "Tree-based self-speculative decoding")
# --------------------------------------------------------------------------
def topk_tokens(logits_row, E: int):
    """The E most probable tokens of one draft distribution, most probable first (equal logits:
    lower token id first), with their log-probabilities log softmax(logits)[token]."""
    x = np.asarray(logits_row, dtype=np.float64)
    order = sorted(range(len(x)), key=lambda v: (-x[v], v))[:E]
    mx = np.max(x)
    lse = mx + np.log(np.sum(np.exp(x - mx)))
    return np.array(order, dtype=np.int32), np.array([x[v] - lse for v in order], dtype=np.float64)


def select_top_nodes(score, lo: int, hi: int, K: int):
    """Node ids of the K highest scores among nodes lo..hi-1 (all of them if fewer), equal scores to
    the lower id; returned ascending."""
    ids = sorted(range(lo, hi), key=lambda i: (-score[i], i))[:K]
    return sorted(ids)


def build_token_tree(level_logits, E: int, K: int, n_max: int):
    """The token tree of one request, level by level.  level_logits[l] is [rows_l, V]: row r of
    level 0 is the draft distribution after the root (one row); row r of level l >= 1 is the draft
    distribution after the r-th node selected for expansion at that level (ascending node id).
    Level 1: the top-E tokens are the root's children.  Level l > 1: the K nodes of level l-1 with
    the highest score are expanded into E children each.  A node's score is the log of the joint
    probability of its root-to-node path (root: 0).  Finally the root and the n_max - 1 other nodes
    with the highest scores are kept (equal scores: lower id, i.e. the ancestor first, so the kept
    set is closed under parents) and renumbered in creation order.
    Returns (parent [n], token [n] (root: -1), score [n], kept_old_ids [n]) of the pruned tree and
    the full tree's (parent, token, score) for inspection."""
    tok, par, sc = [-1], [-1], [0.0]
    level_lo, level_hi = 0, 1
    expand = [0]
    for l, logits in enumerate(level_logits):
        logits = np.asarray(logits)
        assert logits.shape[0] >= len(expand)
        new_lo = len(tok)
        for r, u in enumerate(expand):
            t, lp = topk_tokens(logits[r], E)
            for e in range(len(t)):
                tok.append(int(t[e]))
                par.append(u)
                sc.append(sc[u] + float(lp[e]))
        level_lo, level_hi = new_lo, len(tok)
        expand = select_top_nodes(sc, level_lo, level_hi, K)
    keep = [0] + select_top_nodes(sc, 1, len(tok), max(0, n_max - 1))
    new_id = {old: i for i, old in enumerate(keep)}
    for old in keep[1:]:
        if par[old] not in new_id:
            raise ValueError("kept set is not closed under parents")
    parent = np.array([-1] + [new_id[par[old]] for old in keep[1:]], dtype=np.int32)
    token = np.array([tok[old] for old in keep], dtype=np.int32)
    score = np.array([sc[old] for old in keep], dtype=np.float64)
    full = (np.array(par, dtype=np.int32), np.array(tok, dtype=np.int32), np.array(sc, dtype=np.float64))
    return parent, token, score, np.array(keep, dtype=np.int32), full


# --------------------------------------------------------------------------
# O6: append the accepted nodes' K/V rows to the cache
# --------------------------------------------------------------------------
def chain_draft(step_logits, delta: int, theta: float):
    """Draft loop of sequence self-speculative decoding for one request (Appendix A, "Self-speculative
    decoding"; Algorithm 1): step_logits[i] is the draft distribution of step i (in the real loop it
    depends on the tokens drafted before; here the rows are given).  Every step appends the greedy token
    (lowest id among equal logits) and its probability; drafting stops once delta tokens are drafted or
    the probability of the token just appended is below theta (that token stays in the draft).
    Returns (tokens, probabilities)."""
    toks, probs = [], []
    for x in step_logits:
        x = np.asarray(x, dtype=np.float64)
        tok = 0
        for v in range(1, len(x)):
            if x[v] > x[tok]:
                tok = v
        e = np.exp(x - x[tok])
        prob = float(e[tok] / e.sum())
        toks.append(tok)
        probs.append(prob)
        if len(toks) >= delta or prob < theta:
            break
    return toks, probs


def accept_compact(tree_k, tree_v, cache_k, cache_v, kv_len, paths):
    """tree_k/v [Nl,B,Hkv,T,d]; cache_k/v [Nl,B,Hkv,Lmax,d] updated in place:
    cache[l,b,h,kv_len[b]+j,:] = tree[l,b,h,path_b[j],:]; returns new kv_len."""
    B = cache_k.shape[1]
    new_len = np.array(kv_len, dtype=np.int32).copy()
    for b in range(B):
        base = int(kv_len[b])
        for j, node in enumerate(paths[b]):
            cache_k[:, b, :, base + j, :] = tree_k[:, b, :, int(node), :]
            cache_v[:, b, :, base + j, :] = tree_v[:, b, :, int(node), :]
        new_len[b] = base + len(paths[b])
    return new_len
