"""Pins for the CPU oracle: closed forms, invariants the paper states,
reductions to library routines and brute force on tiny inputs.  No GPU."""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- Eq. 4 / Eq. 6
def test_eq6_paper_printed_values():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "eq6_pruning_settings.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 8
    for M, L, K, R, Kf, printed, _ in rows:
        val = O.avg_retained_tokens(int(M), int(K), int(R), int(L), int(Kf))
        assert int(math.floor(val + 0.5)) == int(printed), (K, R, Kf, val)


def test_eq4_is_eq6_without_finalwipe():
    assert O.avg_retained_tokens(576, 2, 30, 32) == O.avg_retained_tokens(576, 2, 30, 32, K_f=32)
    assert O.avg_retained_tokens(576, 2, 30, 32) == pytest.approx(64.125)
    # keeping everything retains M tokens on average
    assert O.avg_retained_tokens(576, 5, 576, 32) == 576


# ---------------------------------------------------------------- O1 scores
def _rand_scores_case(seed, B=2, Hq=4, Hkv=2, d=8, lens=((3, 7, 2), (0, 5, 4))):
    rng = np.random.default_rng(seed)
    lp = [a + m + c for a, m, c in lens]
    q = rng.standard_normal((B, Hq, d))
    k = rng.standard_normal((B, Hkv, max(lp), d))
    return q, k, np.array(lp), np.array([a for a, _, _ in lens]), np.array([m for _, m, _ in lens])


def test_scores_hand_computed_single_head():
    # d = 2, scale = 1/sqrt(2); logits ln2, 0, 0 -> softmax (1/2, 1/4, 1/4)
    q = np.array([[[1.0, 0.0]]])
    kv = np.array([[math.sqrt(2) * math.log(2), 0.0], [0.0, 3.0], [0.0, -1.0]])
    s = O.ttp_scores(q, kv[None, None], [3], [0], [3], norm_scope=1)
    assert np.allclose(s[0], [0.5, 0.25, 0.25], atol=1e-15)
    # one text key (logit 0) in front: full-row softmax (1/5 | 2/5, 1/5, 1/5)
    kt = np.concatenate([[[0.0, 5.0]], kv])
    s0 = O.ttp_scores(q, kt[None, None], [4], [1], [3], norm_scope=0)
    assert np.allclose(s0[0], [0.4, 0.2, 0.2], atol=1e-15)
    s1 = O.ttp_scores(q, kt[None, None], [4], [1], [3], norm_scope=1)
    assert np.allclose(s1[0], [0.5, 0.25, 0.25], atol=1e-15)


def test_scores_equal_keys_closed_form():
    q, k, lp, vs, nv = _rand_scores_case(1)
    k[:] = k[:, :, :1, :]          # every key identical per (b, kv head)
    s0 = O.ttp_scores(q, k, lp, vs, nv, 0)
    s1 = O.ttp_scores(q, k, lp, vs, nv, 1)
    for b in range(2):
        assert np.allclose(s0[b, :nv[b]], 1.0 / lp[b], atol=1e-15)
        assert np.allclose(s1[b, :nv[b]], 1.0 / nv[b], atol=1e-15)
        assert np.all(s0[b, nv[b]:] == 0)


def test_scores_match_library_softmax_and_normalisation():
    q, k, lp, vs, nv = _rand_scores_case(2)
    for scope in (0, 1):
        s = O.ttp_scores(q, k, lp, vs, nv, scope)
        for b in range(2):
            ref = np.zeros(nv[b])
            text_mass = 0.0
            for h in range(4):
                lo, hi = (0, lp[b]) if scope == 0 else (vs[b], vs[b] + nv[b])
                z = k[b, h // 2, lo:hi] @ q[b, h] / math.sqrt(8)
                p = scipy.special.softmax(z)
                ref += p[vs[b] - lo: vs[b] - lo + nv[b]] / 4
                text_mass += (1.0 - p[vs[b] - lo: vs[b] - lo + nv[b]].sum()) / 4
            assert np.allclose(s[b, :nv[b]], ref, atol=1e-14)
            # "a normalized score over visual tokens" (Eq. 7) in the visual-only scope
            if scope == 1:
                assert abs(s[b].sum() - 1.0) < 1e-12
            else:
                assert abs(s[b].sum() - (1.0 - text_mass)) < 1e-12


def test_scores_one_hot_and_gqa_head_mapping():
    # Hq = 4, Hkv = 2 (G = 2): query heads 0,1 -> kv head 0; 2,3 -> kv head 1.
    d = 4
    q = np.zeros((1, 4, d))
    for h in range(4):
        q[0, h, h % d] = 1.0
    k = np.zeros((1, 2, 6, d))
    # kv head 0: key 1 aligned with q head 0, key 2 with q head 1
    k[0, 0, 1, 0] = 1e3
    k[0, 0, 2, 1] = 1e3
    # kv head 1: key 4 aligned with q head 2, key 5 with q head 3
    k[0, 1, 4, 2] = 1e3
    k[0, 1, 5, 3] = 1e3
    s = O.ttp_scores(q, k, [6], [0], [6], 1)
    assert np.allclose(s[0], [0, .25, .25, 0, .25, .25], atol=1e-12)


def test_scores_permutation_equivariance_and_scale():
    q, k, lp, vs, nv = _rand_scores_case(3, lens=((2, 9, 3), (2, 9, 3)))
    perm = np.random.default_rng(0).permutation(9)
    k2 = k.copy()
    k2[:, :, 2:11] = k[:, :, 2 + perm]
    for scope in (0, 1):
        s, s2 = O.ttp_scores(q, k, lp, vs, nv, scope), O.ttp_scores(q, k2, lp, vs, nv, scope)
        assert np.allclose(s2, s[:, perm], atol=1e-15)
    # explicit scale argument == default 1/sqrt(d); zero scale -> uniform
    assert np.allclose(O.ttp_scores(q, k, lp, vs, nv, 1, scale=1 / math.sqrt(8)), O.ttp_scores(q, k, lp, vs, nv, 1))
    assert np.allclose(O.ttp_scores(q, k, lp, vs, nv, 0, scale=0.0), 1.0 / 14)


# ---------------------------------------------------------------- O2 top-k
def _rank_rule(s, R):
    """Independent definition: m is kept iff fewer than R entries beat it, where
    j beats m when s_j > s_m, or s_j == s_m and j < m."""
    M = len(s)
    return [m for m in range(M)
            if sum(1 for j in range(M) if s[j] > s[m] or (s[j] == s[m] and j < m)) < R]


def test_topk_exhaustive_binary_vectors():
    for M in range(1, 10):
        for bits in itertools.product((0.0, 1.0), repeat=M):
            for R in (0, 1, M // 2, M):
                assert list(O.topk_lowest_index(bits, R)) == _rank_rule(bits, R)


def test_topk_closed_forms_and_library_sort():
    M = 37
    assert list(O.topk_lowest_index(np.ones(M), 5)) == [0, 1, 2, 3, 4]
    assert list(O.topk_lowest_index(np.arange(M)[::-1].astype(float), 5)) == [0, 1, 2, 3, 4]
    assert list(O.topk_lowest_index(np.arange(M).astype(float), 5)) == list(range(M - 5, M))
    assert list(O.topk_lowest_index(np.random.default_rng(0).random(M), M)) == list(range(M))
    rng = np.random.default_rng(5)
    for _ in range(50):
        s = rng.integers(0, 6, size=M).astype(np.float32) / 7      # many exact ties
        R = int(rng.integers(0, M + 1))
        lib = np.sort(np.argsort(-s, kind="stable")[:R])
        assert list(O.topk_lowest_index(s, R)) == list(lib) == _rank_rule(s, R)


# ---------------------------------------------------------------- O3 gather
def _tagged_cache(nl, B, H, L, d):
    """Row payload = its own coordinates, so a moved row identifies its source."""
    k = np.zeros((nl, B, H, L, d), dtype=np.int64)
    for l, b, h, j in itertools.product(range(nl), range(B), range(H), range(L)):
        k[l, b, h, j, :] = ((l * 10 + b) * 10 + h) * 1000 + j
    return k


def test_gather_tagged_rows_and_lengths():
    nl, B, H, L, d = 2, 2, 2, 12, 3
    k = _tagged_cache(nl, B, H, L, d)
    v = -k
    pos = np.tile(np.arange(L, dtype=np.int32) + 100, (B, 1))
    lp, vs, nv = [12, 10], [2, 0], [6, 7]
    kept = [[1, 4, 5], [0, 6]]
    dk, dv, po = np.full_like(k, -7), np.full_like(v, -7), np.full_like(pos, -7)
    new_len = O.gather_compact(k, v, pos, lp, vs, nv, kept, dk, dv, po)
    assert list(new_len) == [12 - 6 + 3, 10 - 7 + 2]
    want = [[0, 1, 3, 6, 7, 8, 9, 10, 11], [0, 6, 7, 8, 9]]
    for b in range(B):
        n = new_len[b]
        assert list(O.prune_index_list(lp[b], vs[b], nv[b], kept[b])) == want[b]
        assert list(dk[0, b, 0, :n, 0] % 1000) == want[b]
        for l, h in itertools.product(range(nl), range(H)):
            assert np.array_equal(dk[l, b, h, :n], k[l, b, h, want[b]])
            assert np.array_equal(dv[l, b, h, :n], v[l, b, h, want[b]])
        assert list(po[b, :n]) == [100 + j for j in want[b]]       # original positions kept
        assert np.all(np.diff(po[b, :n]) > 0)
        assert np.all(dk[:, b, :, n:] == -7) and np.all(po[b, n:] == -7)


def test_gather_keep_all_is_identity_and_keep_none_is_text_only():
    nl, B, H, L, d = 1, 1, 2, 9, 2
    k = _tagged_cache(nl, B, H, L, d)
    pos = np.arange(L, dtype=np.int32)[None]
    dk, dv, po = np.zeros_like(k), np.zeros_like(k), np.zeros_like(pos)
    n = O.gather_compact(k, k, pos, [9], [2], [5], [list(range(5))], dk, dv, po)
    assert n[0] == 9 and np.array_equal(dk, k) and np.array_equal(po, pos)
    dk[:] = 0
    n = O.gather_compact(k, k, pos, [9], [2], [5], [[]], dk, dv, po)
    assert n[0] == 4 and list(dk[0, 0, 0, :4, 0] % 1000) == [0, 1, 7, 8]


def test_gather_in_place_equals_gather_into_a_copy():
    """Compaction in place (dst is src) must give what the gather into a separate buffer gives,
    whatever the kept list: every source row is still intact when its turn comes.  Lists whose
    rows move by one position (kept = [0, 2, 3]) are the ones an unordered copy would get wrong."""
    nl, B, H, L, d = 2, 1, 2, 14, 2
    rng = np.random.default_rng(5)
    lists = [[0, 2, 3], [1, 2, 3, 4, 5], [], [0, 1, 2], [5], list(range(6)), [0, 1, 4, 5]]
    lists += [sorted(rng.choice(6, size=int(rng.integers(0, 7)), replace=False).tolist()) for _ in range(40)]
    for kept in lists:
        for vs in (0, 3):
            k = _tagged_cache(nl, B, H, L, d)
            v = -k
            pos = (np.arange(L, dtype=np.int32) * 7 + 1)[None]
            lp = [vs + 6 + 4]
            dk, dv, po = k.copy(), v.copy(), pos.copy()           # rows past new_len: what was there
            n_out = O.gather_compact(k, v, pos, lp, [vs], [6], [kept], dk, dv, po)
            ik, iv, ip = k.copy(), v.copy(), pos.copy()
            n_in = O.gather_compact(ik, iv, ip, lp, [vs], [6], [kept], ik, iv, ip)
            assert list(n_in) == list(n_out) == [lp[0] - 6 + len(kept)]
            assert np.array_equal(ik, dk) and np.array_equal(iv, dv) and np.array_equal(ip, po), kept
            if len(kept) == 6:                                        # keep-all: nothing moves
                assert np.array_equal(ik, k) and np.array_equal(ip, pos)


def test_gather_rows_hidden_states_and_finalwipe():
    B, L, D = 2, 11, 5
    x = np.arange(B * L * D, dtype=np.int64).reshape(B, L, D)
    lp, vs, nv = [11, 9], [3, 0], [6, 4]
    dst = np.full_like(x, -1)
    n = O.gather_rows(x, lp, vs, nv, [[0, 5], [1, 2, 3]], dst)
    assert list(n) == [7, 8]
    assert np.array_equal(dst[0, :7], x[0, [0, 1, 2, 3, 8, 9, 10]]) and np.all(dst[0, 7:] == -1)
    assert np.array_equal(dst[1, :8], x[1, [1, 2, 3, 4, 5, 6, 7, 8]])
    # FinalWipe: no visual token survives; keep-all: identity
    dst[:] = -1
    n = O.gather_rows(x, lp, vs, nv, [[], []], dst)
    assert list(n) == [5, 5] and np.array_equal(dst[0, :5], x[0, [0, 1, 2, 9, 10]])
    n = O.gather_rows(x, lp, vs, nv, [list(range(6)), list(range(4))], dst)
    assert list(n) == lp and np.array_equal(dst[0], x[0]) and np.array_equal(dst[1, :9], x[1, :9])


# ---------------------------------------------------------------- O4 tree attention
def _attn_case(seed, B=2, T=6, Hq=4, Hkv=2, d=8, Lmax=11, kv_len=(7, 11), gain=1.0):
    rng = np.random.default_rng(seed)
    return dict(q=rng.standard_normal((B, T, Hq, d)) * gain,
                tree_k=rng.standard_normal((B, Hkv, T, d)), tree_v=rng.standard_normal((B, Hkv, T, d)),
                cache_k=rng.standard_normal((B, Hkv, Lmax, d)), cache_v=rng.standard_normal((B, Hkv, Lmax, d)),
                kv_len=np.array(kv_len))


def _brute_tree_attention(c, n_nodes, parent, b, i, h):
    """Scalar loops straight from the definition, no shared helper."""
    G = c["q"].shape[2] // c["tree_k"].shape[1]
    g, d = h // G, c["q"].shape[3]
    visible = []
    for j in range(int(c["kv_len"][b])):
        visible.append((c["cache_k"][b, g, j], c["cache_v"][b, g, j]))
    for j in range(int(n_nodes[b])):
        x, is_anc = i, False
        while x != -1:
            if x == j:
                is_anc = True
            x = int(parent[b][x])
        if is_anc:
            visible.append((c["tree_k"][b, g, j], c["tree_v"][b, g, j]))
    logits = [sum(c["q"][b, i, h, t] * kk[t] for t in range(d)) / math.sqrt(d) for kk, _ in visible]
    mx = max(logits)
    w = [math.exp(z - mx) for z in logits]
    tot = sum(w)
    out = [sum(w[n] * visible[n][1][t] for n in range(len(visible))) / tot for t in range(d)]
    return np.array(out), mx + math.log(tot), len(visible)


def test_tree_attention_brute_force_random_trees():
    for seed in range(4):
        c = _attn_case(seed)
        rng = np.random.default_rng(100 + seed)
        parent = np.stack([synth.random_tree(rng, 6, 3), synth.random_tree(rng, 6, 4)])
        n_nodes = np.array([6, 5])
        out, lse = O.tree_attention(parent=parent, n_nodes=n_nodes, **c)
        for b, h in itertools.product(range(2), range(4)):
            for i in range(n_nodes[b]):
                o, l, _ = _brute_tree_attention(c, n_nodes, parent, b, i, h)
                assert np.allclose(out[b, i, h], o, atol=1e-13)
                assert abs(lse[b, h, i] - l) < 1e-13
        assert np.all(out[1, 5] == 0)                     # padded node untouched
        # sampled evaluation equals the full one
        smp = [(0, 3, 1), (1, 4, 3)]
        o2, l2 = O.tree_attention(parent=parent, n_nodes=n_nodes, samples=smp, **c)
        for (b, i, h) in smp:
            assert np.allclose(o2[b, i, h], out[b, i, h], atol=1e-14) and abs(l2[b, h, i] - lse[b, h, i]) < 1e-14


def test_chain_tree_is_causal_attention_library():
    """A chain-shaped tree is ordinary causal attention of T appended tokens."""
    c = _attn_case(7, gain=3.0)
    B, T, Hq, d = c["q"].shape
    parent = np.stack([synth.chain_tree(T)] * B)
    out, _ = O.tree_attention(parent=parent, n_nodes=np.array([T, T]), **c)
    for b in range(B):
        L = int(c["kv_len"][b])
        kk = np.concatenate([c["cache_k"][b, :, :L], c["tree_k"][b]], axis=1)      # [Hkv, L+T, d]
        vv = np.concatenate([c["cache_v"][b, :, :L], c["tree_v"][b]], axis=1)
        kk, vv = np.repeat(kk, 2, axis=0), np.repeat(vv, 2, axis=0)                  # GQA expand
        qq = np.concatenate([np.zeros((Hq, L, d)), c["q"][b].transpose(1, 0, 2)], axis=1)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(qq), torch.from_numpy(kk), torch.from_numpy(vv), is_causal=True).numpy()
        assert np.allclose(out[b].transpose(1, 0, 2), ref[:, L:], atol=1e-12)


def test_single_node_tree_is_plain_decode():
    c = _attn_case(8, T=1)
    out, lse = O.tree_attention(parent=np.array([[-1], [-1]]), n_nodes=np.array([1, 1]), **c)
    for b, h in itertools.product(range(2), range(4)):
        L = int(c["kv_len"][b])
        kk = np.concatenate([c["cache_k"][b, h // 2, :L], c["tree_k"][b, h // 2]])
        vv = np.concatenate([c["cache_v"][b, h // 2, :L], c["tree_v"][b, h // 2]])
        z = kk @ c["q"][b, 0, h] / math.sqrt(8)
        assert np.allclose(out[b, 0, h], scipy.special.softmax(z) @ vv, atol=1e-13)
        assert abs(lse[b, h, 0] - scipy.special.logsumexp(z)) < 1e-13


def test_tree_attention_closed_forms():
    c = _attn_case(9)
    B, T, Hq, d = c["q"].shape
    rng = np.random.default_rng(1)
    parent = np.stack([synth.random_tree(rng, T, 4), synth.star_tree(T)])
    n_nodes = np.array([T, T])
    # all V rows equal v  ->  out == v
    c1 = dict(c)
    c1["cache_v"] = np.ones_like(c["cache_v"]) * 0.375
    c1["tree_v"] = np.ones_like(c["tree_v"]) * 0.375
    out, _ = O.tree_attention(parent=parent, n_nodes=n_nodes, **c1)
    assert np.allclose(out, 0.375, atol=1e-14)
    # all K equal -> uniform weights over exactly L + depth + 1 visible rows:
    # with V = 1 on cache rows and 0 on tree rows, out = L / (L + depth + 1)
    c2 = dict(c)
    c2["cache_k"] = np.zeros_like(c["cache_k"]) + 0.5
    c2["tree_k"] = np.zeros_like(c["tree_k"]) + 0.5
    c2["cache_v"] = np.ones_like(c["cache_v"])
    c2["tree_v"] = np.zeros_like(c["tree_v"])
    out, lse = O.tree_attention(parent=parent, n_nodes=n_nodes, **c2)
    for b in range(B):
        dep = synth.node_depths(parent[b])
        L = int(c["kv_len"][b])
        for i in range(T):
            assert np.allclose(out[b, i], L / (L + dep[i] + 1), atol=1e-14)
    # star tree: each node sees prefix + root + itself only
    out, _ = O.tree_attention(parent=parent, n_nodes=n_nodes, **c)
    c3 = {k: v.copy() for k, v in c.items()}
    c3["tree_k"][1, :, 2] += 5.0       # node 2 of the star is no ancestor of nodes 1, 3, 4, 5
    c3["tree_v"][1, :, 2] -= 3.0
    out3, _ = O.tree_attention(parent=parent, n_nodes=n_nodes, **c3)
    for i in (0, 1, 3, 4, 5):
        assert np.array_equal(out3[1, i], out[1, i])          # bit-identical
    assert not np.allclose(out3[1, 2], out[1, 2])


def test_tree_attention_prefix_permutation_and_lse_merge():
    c = _attn_case(10, gain=2.0)
    B, T, Hq, d = c["q"].shape
    rng = np.random.default_rng(2)
    parent = np.stack([synth.random_tree(rng, T, 3), synth.random_tree(rng, T, 5)])
    n_nodes = np.array([T, T])
    out, lse = O.tree_attention(parent=parent, n_nodes=n_nodes, **c)
    # softmax weights sum to one: out over V == 1 is 1 (checked above); lse finite
    assert np.all(np.isfinite(lse))
    # permuting the valid prefix rows changes nothing
    c2 = {k: v.copy() for k, v in c.items()}
    for b in range(B):
        L = int(c["kv_len"][b])
        perm = rng.permutation(L)
        c2["cache_k"][b, :, :L] = c["cache_k"][b][:, perm]
        c2["cache_v"][b, :, :L] = c["cache_v"][b][:, perm]
    out2, lse2 = O.tree_attention(parent=parent, n_nodes=n_nodes, **c2)
    assert np.allclose(out2, out, atol=1e-12) and np.allclose(lse2, lse, atol=1e-12)
    # rows past kv_len are never read
    c4 = {k: v.copy() for k, v in c.items()}
    c4["cache_k"][0, :, 7:] = np.nan
    c4["cache_v"][0, :, 7:] = np.nan
    out4, _ = O.tree_attention(parent=parent, n_nodes=n_nodes, **c4)
    assert np.array_equal(out4, out)
    # attention over a key set split in two, merged by log-sum-exp, equals the unsplit result
    b, h, i = 1, 2, 4
    L = int(c["kv_len"][b])
    vis = O.tree_mask(parent[b], T, L)[i:i + 1]
    keys = np.concatenate([c["cache_k"][b, h // 2, :L], c["tree_k"][b, h // 2]])
    vals = np.concatenate([c["cache_v"][b, h // 2, :L], c["tree_v"][b, h // 2]])
    cut = 5
    sc = 1 / math.sqrt(d)
    o1, l1 = O.masked_attention(c["q"][b, i:i + 1, h], keys[:cut], vals[:cut], vis[:, :cut], sc)
    o2, l2 = O.masked_attention(c["q"][b, i:i + 1, h], keys[cut:], vals[cut:], vis[:, cut:], sc)
    lt = np.logaddexp(l1, l2)
    merged = o1 * np.exp(l1 - lt)[:, None] + o2 * np.exp(l2 - lt)[:, None]
    assert np.allclose(merged[0], out[b, i, h], atol=1e-13) and abs(lt[0] - lse[b, h, i]) < 1e-13


# ---------------------------------------------------------------- O5 acceptance
def _greedy_level_traversal(parent, tok, tgt, n):
    """The paper's wording: walk down from the root, at each level take a child
    whose token equals the target's prediction, stop when none matches."""
    cur, path = 0, [0]
    while True:
        nxt = [c for c in range(1, n) if parent[c] == cur and tok[c] == tgt[cur]]
        if not nxt:
            return len(path) - 1, path, int(tgt[cur])
        cur = nxt[0]
        path.append(cur)


def test_accept_equals_level_traversal_when_siblings_distinct():
    rng = np.random.default_rng(11)
    for trial in range(300):
        n = int(rng.integers(1, 13))
        parent = synth.random_tree(rng, n, int(rng.integers(1, 6)))
        tok, tgt = synth.draft_and_target_tokens(rng, parent, 0.7)
        a, path, bonus = O.tree_accept(parent, tok, tgt, n)
        a2, path2, bonus2 = _greedy_level_traversal(parent, tok, tgt, n)
        assert (a, list(path), bonus) == (a2, path2, bonus2)
        assert path[0] == 0 and len(path) == a + 1


def test_accept_brute_force_with_duplicate_siblings():
    rng = np.random.default_rng(12)
    for trial in range(300):
        n = int(rng.integers(1, 11))
        parent = synth.random_tree(rng, n, int(rng.integers(1, 5)))
        tok, tgt = synth.draft_and_target_tokens(rng, parent, 0.8, per_child=True)
        a, path, bonus = O.tree_accept(parent, tok, tgt, n)
        # brute force: accepted set by top-down propagation, then the deepest / lowest index
        ok = [False] * n
        ok[0] = True
        dep = synth.node_depths(parent)
        for c in range(1, n):
            ok[c] = ok[parent[c]] and tok[c] == tgt[parent[c]]
        best = max((i for i in range(n) if ok[i]), key=lambda i: (dep[i], -i))
        assert a == dep[best] and path[-1] == best and bonus == tgt[best]
        for u, c in zip(path[:-1], path[1:]):
            assert parent[c] == u


def test_accept_special_cases_and_statistics():
    T = 6
    chain = synth.chain_tree(T)
    tgt = np.arange(10, 10 + T)
    tok = np.concatenate([[999], tgt[:-1]])              # every draft token matches
    assert O.tree_accept(chain, tok, tgt, T)[0] == T - 1
    assert O.tree_accept(chain, tok, tgt, T)[2] == tgt[T - 1]
    a, path, bonus = O.tree_accept(chain, tok + 1, tgt, T)       # nothing matches
    assert (a, list(path), bonus) == (0, [0], tgt[0])
    a, path, bonus = O.tree_accept(chain, tok, tgt, 3)           # only the first 3 nodes exist
    assert a == 2 and bonus == tgt[2]
    # a match below a mismatch does not count (stop at the first mismatch)
    tok2 = tok.copy()
    tok2[2] += 1
    assert O.tree_accept(chain, tok2, tgt, T)[0] == 1
    # chain of D levels, match probability p per edge: E[accept_len] = sum_{k=1}^{D-1} p^k
    rng = np.random.default_rng(13)
    D, p, n_trials = 5, 0.6, 20000
    tot = 0
    for _ in range(n_trials):
        tk, tg = synth.draft_and_target_tokens(rng, synth.chain_tree(D), p)
        tot += O.tree_accept(synth.chain_tree(D), tk, tg, D)[0]
    want = sum(p ** k for k in range(1, D))
    assert abs(tot / n_trials - want) < 0.03


def test_invalid_parent_arrays_are_rejected():
    for bad in ([0, 0], [-1, 1], [-1, 0, 2], [-1, -1]):
        with pytest.raises(ValueError):
            O.ancestors_or_self(np.array(bad), len(bad) - 1)


def test_speculative_decoding_is_lossless_with_toy_target():
    """With a deterministic toy target next = f(sequence), draft-tree verification
    must emit exactly the greedy sequence of f, whatever the drafts are."""
    def f(seq):
        x = 1469598103934665603
        for t in seq:
            x = ((x ^ (t + 1)) * 1099511628211) % (1 << 64)
        return int(x % 50)

    rng = np.random.default_rng(14)
    prompt = [3, 1, 4]
    greedy = list(prompt)
    for _ in range(60):
        greedy.append(f(greedy))
    seq = list(prompt) + [f(prompt)]                 # last accepted token = tree root
    while len(seq) < len(greedy):
        n = int(rng.integers(1, 12))
        parent = synth.random_tree(rng, n, int(rng.integers(1, 5)))
        tok = np.zeros(n, dtype=np.int64)
        tgt = np.zeros(n, dtype=np.int64)
        tok[0] = seq[-1]
        for i in range(n):
            if i > 0:
                pref = seq[:-1] + [int(tok[a]) for a in O.ancestors_or_self(parent, int(parent[i]))]
                tok[i] = f(pref) if rng.random() < 0.6 else int(rng.integers(0, 50))
            tgt[i] = f(seq[:-1] + [int(tok[a]) for a in O.ancestors_or_self(parent, i)])
        a, path, bonus = O.tree_accept(parent, tok, tgt, n)
        seq += [int(tok[x]) for x in path[1:]] + [bonus]
    assert seq[:len(greedy)] == greedy


def test_gated_scores_brute_force_and_reductions():
    """Eq. 7: against a loop-by-loop evaluation on a tiny case; gates of one give the ungated
    score; a gate can be moved between q and K; a key whose gate is zero gets the uniform share
    of a zero logit."""
    import math
    rng = np.random.default_rng(17)
    B, Hq, Hkv, L, d = 2, 4, 2, 9, 8
    q, gq = rng.standard_normal((B, Hq, d)), rng.uniform(0.2, 1.5, (B, Hq, d))
    k, gk = rng.standard_normal((B, Hkv, L, d)), rng.uniform(0.2, 1.5, (B, Hkv, L, d))
    lp, vs, nv = [9, 7], [2, 1], [5, 4]
    got = O.ttp_scores_gated(q, gq, k, gk, lp, vs, nv)
    for b in range(B):
        want = [0.0] * nv[b]
        for h in range(Hq):
            z = []
            for m in range(nv[b]):
                j = vs[b] + m
                z.append(sum(gq[b, h, c] * q[b, h, c] * gk[b, h // 2, j, c] * k[b, h // 2, j, c] for c in range(d)) / math.sqrt(d))
            den = sum(math.exp(x) for x in z)
            for m in range(nv[b]):
                want[m] += math.exp(z[m]) / den / Hq
        assert np.allclose(got[b, :nv[b]], want, rtol=1e-12, atol=1e-15)
        assert abs(got[b, :nv[b]].sum() - 1.0) < 1e-12
    one_q, one_k = np.ones_like(q), np.ones_like(k)
    assert np.allclose(O.ttp_scores_gated(q, one_q, k, one_k, lp, vs, nv, norm_scope=0), O.ttp_scores(q, k, lp, vs, nv, 0), rtol=1e-12)
    assert np.allclose(O.ttp_scores_gated(q, one_q, k, one_k, lp, vs, nv, norm_scope=1), O.ttp_scores(q, k, lp, vs, nv, 1), rtol=1e-12)
    # the same product whichever side carries the factor
    assert np.allclose(got, O.ttp_scores(q * gq, k * gk, lp, vs, nv, 1), rtol=1e-12)
    g0 = gk.copy()
    g0[:, :, 3, :] = 0.0                      # key 3: logit 0 in every head
    z0 = O.ttp_scores_gated(q, gq, k, g0, [9, 9], [0, 0], [9, 9])
    k0 = k.copy()
    k0[:, :, 3, :] = 0.0
    assert np.allclose(z0, O.ttp_scores_gated(q, gq, k0, gk, [9, 9], [0, 0], [9, 9]), rtol=1e-12)


def test_text_to_visual_scores_pins():
    """Eq. 3's multi-query guide: brute force on a tiny case; one query at the last prompt position
    is the single-query score over the full causal row; causality (a key after a query's position
    does not reach that query's share); each query spreads at most 1 over the visual tokens."""
    import math
    rng = np.random.default_rng(23)
    B, Hq, Hkv, L, d, N = 2, 4, 2, 12, 8, 4
    k = rng.standard_normal((B, Hkv, L, d))
    qt = rng.standard_normal((B, Hq, N, d))
    lp, vs, nv = [12, 9], [3, 2], [5, 6]          # 4 and 1 text tokens after the image
    got = O.text_to_visual_scores(qt, k, lp, vs, nv)
    for b in range(B):
        want = [0.0] * nv[b]
        for h in range(Hq):
            for i in range(lp[b] - vs[b] - nv[b]):
                t = vs[b] + nv[b] + i
                z = [sum(qt[b, h, i, c] * k[b, h // 2, j, c] for c in range(d)) / math.sqrt(d) for j in range(t + 1)]
                den = sum(math.exp(x) for x in z)
                for m in range(nv[b]):
                    want[m] += math.exp(z[vs[b] + m]) / den / Hq
        assert np.allclose(got[b, :nv[b]], want, rtol=1e-12, atol=1e-15)
        assert got[b, :nv[b]].sum() <= (lp[b] - vs[b] - nv[b]) + 1e-12
        assert np.all(got[b, nv[b]:] == 0)
    # request 1 has exactly one text token after the image, at the last prompt position
    single = O.ttp_scores(qt[1:2, :, 0, :], k[1:2], [9], [2], [6], norm_scope=0)
    assert np.allclose(got[1, :6], single[0, :6], rtol=1e-12)
    # causality: the last key (position 11) is seen by request 0's last query only
    k2 = k.copy()
    k2[0, :, 11, :] += 3.0
    got2 = O.text_to_visual_scores(qt, k2, lp, vs, nv)
    first3 = O.text_to_visual_scores(qt[:, :, :3], k, [11, 9], vs, nv)      # prompt cut before its last token
    first3_2 = O.text_to_visual_scores(qt[:, :, :3], k2, [11, 9], vs, nv)
    assert np.allclose(first3, first3_2, rtol=0, atol=0)
    assert np.allclose(got2[0] - first3_2[0], O.text_to_visual_scores(qt, k2, lp, vs, nv)[0] - first3[0], rtol=1e-12)
    assert not np.allclose(got2[0], got[0])


def test_base_argmax_library_and_ties():
    rng = np.random.default_rng(31)
    x = rng.integers(-3, 4, size=(2, 5, 40)).astype(np.float64)          # many exact ties
    got = O.base_argmax(x, [5, 3])
    assert np.array_equal(got[0], np.argmax(x[0], axis=-1))               # numpy: first occurrence
    assert np.array_equal(got[1, :3], np.argmax(x[1, :3], axis=-1)) and np.all(got[1, 3:] == 0)
    y = np.zeros((1, 2, 9))
    y[0, 0, [4, 7]] = 2.5
    y[0, 1, 8] = 1e-300
    assert O.base_argmax(y, [2]).tolist() == [[4, 8]]
    # the argmax of the logits is the argmax of the probabilities the paper's pseudocode uses
    import scipy.special as sp
    z = rng.standard_normal((1, 4, 50))
    assert np.array_equal(O.base_argmax(z, [4]), O.base_argmax(sp.softmax(z, axis=-1), [4]))


def test_token_tree_pins():
    """Tree builder: enumeration of every path of a tiny vocabulary; chain and full-tree limits;
    tie rules; closure under parents."""
    import itertools, math
    rng = np.random.default_rng(29)
    V, E, K, D = 5, 2, 2, 3
    levels = [rng.standard_normal((1, V))] + [rng.standard_normal((K, V)) for _ in range(D - 1)]
    parent, token, score, keep, (fpar, ftok, fsc) = O.build_token_tree(levels, E, K, n_max=100)
    # (a) sizes: 1 + E + (D-1) K E, nothing pruned
    assert len(fpar) == 1 + E + (D - 1) * K * E == len(parent)
    # (b) every node's score is the log joint probability of its path, recomputed with plain math
    def softmax(row):
        m = max(row)
        z = [math.exp(x - m) for x in row]
        return [x / sum(z) for x in z]
    # replay: which row fed which node
    row_of = {0: (0, 0)}                      # node -> (level, row) of the distribution after it
    lo, hi = 1, 1 + E
    for l in range(1, D):
        sel = sorted(sorted(range(lo, hi), key=lambda i: (-fsc[i], i))[:K])
        for r, u in enumerate(sel):
            row_of[u] = (l, r)
        lo, hi = hi, hi + K * E
    for i in range(1, len(fpar)):
        l, r = row_of[int(fpar[i])]
        p = softmax(list(levels[l][r]))
        assert math.isclose(fsc[i], fsc[fpar[i]] + math.log(p[ftok[i]]), rel_tol=1e-12, abs_tol=1e-12)
        # children of a node are its top-E tokens
        sibs = [int(ftok[j]) for j in range(1, len(fpar)) if fpar[j] == fpar[i]]
        assert sorted(sibs, key=lambda v: (-levels[l][r][v], v)) == sorted(range(V), key=lambda v: (-levels[l][r][v], v))[:E]
    # (c) pruning to n_max keeps the root and the n_max - 1 highest joint probabilities, parents included
    for n_max in (1, 2, 4, 7):
        p2, t2, s2, keep2, _ = O.build_token_tree(levels, E, K, n_max)
        best = sorted(range(1, len(fsc)), key=lambda i: (-fsc[i], i))[:n_max - 1]
        assert sorted(keep2.tolist()) == sorted([0] + best)
        assert p2[0] == -1 and all(0 <= p2[i] < i for i in range(1, len(p2)))
        for i in range(1, len(p2)):
            assert keep2[p2[i]] == fpar[keep2[i]]          # the renumbered parent is the old parent
    # (d) E = K = 1: the chain of greedy tokens of the rows
    chain = O.build_token_tree([lv[:1] for lv in levels], 1, 1, 100)
    assert chain[0].tolist() == [-1, 0, 1, 2] and chain[1].tolist() == [-1] + [int(np.argmax(lv[0])) for lv in levels]
    # (e) ties: equal logits go to the lower token id, equal scores to the lower node id
    flat = [np.zeros((1, 4)), np.zeros((2, 4))]
    p3, t3, s3, keep3, (fp3, ft3, fs3) = O.build_token_tree(flat, 2, 2, 4)
    assert ft3.tolist() == [-1, 0, 1, 0, 1, 0, 1] and fp3.tolist() == [-1, 0, 0, 1, 1, 2, 2]
    assert keep3.tolist() == [0, 1, 2, 3]                    # level 1 (higher score) first, then the lowest id
    # (f) top-E log-probabilities against scipy
    import scipy.special as sp
    x = rng.standard_normal(50)
    t, lp = O.topk_tokens(x, 5)
    assert t.tolist() == np.argsort(-x, kind="stable")[:5].tolist()
    assert np.allclose(lp, sp.log_softmax(x)[t], rtol=1e-12)


# ---------------------------------------------------------------- O6 accept-compact
def test_accept_compact_tail_rows_and_canaries():
    nl, B, H, T, L, d = 2, 2, 2, 5, 12, 3
    tree = _tagged_cache(nl, B, H, T, d) + 500
    cache = _tagged_cache(nl, B, H, L, d)
    ck, cv = cache.copy(), -cache
    before_k, before_v = ck.copy(), cv.copy()
    kv_len = np.array([4, 7])
    paths = [[0, 2, 3], [0]]
    new_len = O.accept_compact(tree, -tree, ck, cv, kv_len, paths)
    assert list(new_len) == [7, 8]
    for b in range(B):
        base = kv_len[b]
        for j, node in enumerate(paths[b]):
            assert np.array_equal(ck[:, b, :, base + j], tree[:, b, :, node])
            assert np.array_equal(cv[:, b, :, base + j], -tree[:, b, :, node])
        assert np.array_equal(ck[:, b, :, :base], before_k[:, b, :, :base])
        assert np.array_equal(ck[:, b, :, new_len[b]:], before_k[:, b, :, new_len[b]:])
        assert np.array_equal(cv[:, b, :, new_len[b]:], before_v[:, b, :, new_len[b]:])


# ---------------------------------------------------------------- chain drafting with early exit
def test_chain_draft_hand_case_and_limits():
    """Appendix A: up to delta = 5 draft tokens, stop once the predicted token's probability is below
    theta = 0.6; Algorithm 1 appends the token before it tests the probability, so the token that
    triggers the exit is part of the draft."""
    lg = lambda p: np.log(np.asarray(p, dtype=np.float64))
    rows = [lg([0.1, 0.7, 0.2]), lg([0.8, 0.1, 0.1]), lg([0.3, 0.2, 0.5]), lg([0.9, 0.05, 0.05]), lg([0.9, 0.05, 0.05]),
            lg([0.9, 0.05, 0.05])]
    toks, probs = O.chain_draft(rows, 5, 0.6)
    assert toks == [1, 0, 2] and np.allclose(probs, [0.7, 0.8, 0.5], atol=1e-12)      # 0.5 < 0.6: kept, then stop
    toks, probs = O.chain_draft(rows, 5, 0.0)                                          # no early exit: delta tokens
    assert toks == [1, 0, 2, 0, 0] and len(probs) == 5
    toks, _ = O.chain_draft(rows, 2, 0.0)
    assert toks == [1, 0]
    toks, probs = O.chain_draft(rows, 5, 1.5)                                          # nothing is confident enough
    assert toks == [1] and abs(probs[0] - 0.7) < 1e-12
    # a probability equal to the threshold is not below it
    toks, _ = O.chain_draft([lg([0.5, 0.5]), lg([0.25, 0.75]), lg([0.4, 0.6])], 5, 0.5)
    assert toks == [0, 1, 1]                       # (and equal logits go to the lower token id)
    # shifting a row's logits changes nothing
    toks2, probs2 = O.chain_draft([r + 3.25 for r in rows], 5, 0.6)
    assert toks2 == [1, 0, 2] and np.allclose(probs2, [0.7, 0.8, 0.5], atol=1e-12)


def test_chain_draft_against_library_softmax():
    from scipy.special import softmax
    rng = np.random.default_rng(21)
    for trial in range(50):
        V, delta = int(rng.integers(2, 40)), int(rng.integers(1, 7))
        theta = float(rng.uniform(0.05, 0.9))
        rows = rng.standard_normal((8, V)) * rng.uniform(0.5, 4.0)
        toks, probs = O.chain_draft(rows, delta, theta)
        want_t, want_p = [], []
        for r in rows:
            p = softmax(r)
            want_t.append(int(np.argmax(p)))
            want_p.append(float(p.max()))
            if len(want_t) >= delta or want_p[-1] < theta:
                break
        assert toks == want_t and np.allclose(probs, want_p, rtol=1e-12)
        assert 1 <= len(toks) <= delta and all(p >= theta for p in probs[:-1])


# ---------------------------------------------------------------- generator sanity
def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.140625], dtype=np.float32)
    b = synth.f32_to_bf16(x)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 ties upward to 1 + 2^-6
    assert list(synth.bf16_to_f32(b)) == [1.0, 1.0, 1.015625, -2.5, 0.0, 3.140625]
    r = synth.normal_bf16(np.random.default_rng(0), (1000,), 64)
    assert np.array_equal(synth.f32_to_bf16(synth.bf16_to_f32(r)), r)


def test_generator_tree_shapes():
    p = synth.fixed_branching_tree([4, 2, 1, 1], 26)
    dep = synth.node_depths(p)
    assert len(p) == 26 and [int((dep == l).sum()) for l in range(5)] == [1, 4, 8, 8, 5]
    rng = np.random.default_rng(0)
    for T, D in ((8, 3), (64, 8), (64, 6), (20, 6)):
        p = synth.random_tree(rng, T, D)
        assert p[0] == -1 and all(-1 < p[i] < i for i in range(1, T))
        assert synth.node_depths(p).max() == D - 1
    for i in range(1, 6):
        wl = synth.workload(i)
        assert len(wl.keep) == wl.batch == len(wl.n_nodes)
    assert synth.workload(2).prefix_len == [675] and synth.workload(2).pruned_len == [163]
