"""GPU parity: the draft-side token tree (top-E expansion, top-K selection, pruning to N_max)."""
import numpy as np
import pytest
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth
from gpu_common import DEV, MAX_ABS_TOL, REL_L2_TOL, dev_bf16, dev_i32, f64, host_bits, max_abs, rel_l2_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tw():
    from paper_2503_14075_b200 import twig
    return twig


def gpu_tree(tw, level_logits_dev, E, K, n_max, t_max):
    """Drives the four entry points for a whole batch; returns host arrays."""
    B = level_logits_dev[0].shape[0]
    D = len(level_logits_dev)
    cap = 1 + E + (D - 1) * K * E
    st = tw.TreeState(B, cap, DEV)
    st.tok.fill_(-77)
    st.parent.fill_(-77)
    st.score.fill_(float("nan"))
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_reset(st)
    src = torch.zeros((B, 1), dtype=torch.int32, device=DEV)
    lo, hi = 0, 1
    for l in range(D):
        rows = level_logits_dev[l].shape[1]
        if src.shape[1] < rows:                       # unused rows
            pad = torch.full((B, rows - src.shape[1]), -1, dtype=torch.int32, device=DEV)
            src = torch.cat([src, pad], dim=1).contiguous()
        tw.tree_expand_level(level_logits_dev[l], src, E, hi, st, dev_status=status)
        lo, hi = hi, hi + (1 if l == 0 else K) * E
        if l + 1 < D:
            src = torch.full((B, K), -5, dtype=torch.int32, device=DEV)
            tw.tree_select_expansion(st, lo, min(hi, cap), src, dev_status=status)
    parent = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
    tok = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
    n_nodes = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    kept = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
    tw.tree_finalize(st, cap, n_max, parent, tok, n_nodes, kept_node=kept, dev_status=status)
    torch.cuda.synchronize()
    return (parent.cpu().numpy(), tok.cpu().numpy(), n_nodes.cpu().numpy(), kept.cpu().numpy(), status.cpu().numpy(),
            st.score.cpu().numpy())


def gpu_tree_grown(tw, level_logits_dev, E, K, n_max, t_max, repeats=2):
    """The same trees with one launch per level (tree_grow_level), no tree_reset, and the state reused
    `repeats` times (the per-request tickets must come back to zero)."""
    B = level_logits_dev[0].shape[0]
    D = len(level_logits_dev)
    cap = 1 + E + (D - 1) * K * E
    st = tw.TreeState(B, cap, DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    for _ in range(repeats):
        st.tok.fill_(-77)
        st.parent.fill_(-77)
        st.score.fill_(float("nan"))
        parent = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
        tok = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
        n_nodes = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        kept = torch.full((B, t_max), -9, dtype=torch.int32, device=DEV)
        src = torch.zeros((B, 1), dtype=torch.int32, device=DEV)
        hi = 1
        for l in range(D):
            if l + 1 < D:
                nxt = torch.full((B, K), -5, dtype=torch.int32, device=DEV)
                tw.tree_grow_level(level_logits_dev[l], src, E, hi, st, expand_node=nxt, dev_status=status)
                src = nxt
            else:
                tw.tree_grow_level(level_logits_dev[l], src, E, hi, st, n_max=n_max, parent=parent, draft_tok=tok,
                                   n_nodes=n_nodes, kept_node=kept, dev_status=status)
            hi += (1 if l == 0 else K) * E
        torch.cuda.synchronize()
        assert not st.ticket.any()
    return (parent.cpu().numpy(), tok.cpu().numpy(), n_nodes.cpu().numpy(), kept.cpu().numpy(), status.cpu().numpy(),
            st.score.cpu().numpy())


BUILDERS = {"calls": gpu_tree, "one-launch-per-level": gpu_tree_grown}


@pytest.mark.parametrize("builder", list(BUILDERS))
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("cfg", [(10, 10, 4, 60, 64, 32000), (3, 2, 3, 7, 8, 1003), (16, 4, 2, 64, 64, 4096), (1, 1, 5, 6, 6, 77)],
                         ids=["paper-default", "small-ragged", "wide", "chain"])
def test_token_tree_matches_oracle(tw, cfg, dtype, builder):
    E, K, D, n_max, t_max, V = cfg
    B = 3
    rng = synth.rng_for(7, 21)
    stride = (V + 7) // 8 * 8
    host, dev = [], []
    for l in range(D):
        rows = 1 if l == 0 else K
        x = (rng.standard_normal((B, rows, V)) * 3.0).astype(np.float32)
        if dtype == "bf16":
            bits = synth.f32_to_bf16(x)
            padded = np.full((B, rows, stride), 0x7F7F, dtype=bits.dtype)          # a huge value nobody may read
            padded[..., :V] = bits
            dev.append(dev_bf16(padded)[..., :V])
            host.append(synth.bf16_to_f64(bits))
        else:
            padded = np.full((B, rows, stride), 3e38, dtype=np.float32)
            padded[..., :V] = x
            dev.append(torch.from_numpy(padded).to(DEV)[..., :V])
            host.append(x.astype(np.float64))
    parent, tok, n_nodes, kept, status, score = BUILDERS[builder](tw, dev, E, K, n_max, t_max)
    assert not status.any()
    for b in range(B):
        p_o, t_o, s_o, keep_o, (fp, ft, fs) = O.build_token_tree([h[b] for h in host], E, K, n_max)
        # (scores are fp32 on the GPU and fp64 in the oracle; the seeded rows have no near-ties at a selection
        # boundary, exact ties are covered by test_token_tree_ties)
        n = len(p_o)
        assert n_nodes[b] == n
        assert np.array_equal(kept[b, :n], keep_o)
        assert np.array_equal(parent[b, :n], p_o) and np.array_equal(tok[b, :n], t_o)
        assert np.all(parent[b, n:] == -1) and np.all(tok[b, n:] == 0) and np.all(kept[b, n:] == -1)
        assert np.allclose(score[b, :len(fs)], fs, rtol=0, atol=2e-4 * D)


@pytest.mark.parametrize("builder", list(BUILDERS))
@pytest.mark.parametrize("V", [64, 4096])
def test_token_tree_ties(tw, V, builder):
    """Equal logits go to the lower token id, equal scores to the lower node id (exact ties: rows that are
    bit-identical give bit-identical scores).  With 4096 equal logits the kernel's short candidate list
    overflows and the selection runs over the whole row."""
    E, K, D, n_max, t_max = 2, 2, 2, 4, 8
    flat = [torch.zeros((1, 1, V), dtype=torch.float32, device=DEV), torch.zeros((1, K, V), dtype=torch.float32, device=DEV)]
    parent, tok, n_nodes, kept, status, _ = BUILDERS[builder](tw, flat, E, K, n_max, t_max)
    p_o, t_o, _, keep_o, _ = O.build_token_tree([np.zeros((1, V)), np.zeros((K, V))], E, K, n_max)
    assert not status.any() and n_nodes[0] == 4
    assert kept[0, :4].tolist() == keep_o.tolist() == [0, 1, 2, 3]
    assert parent[0, :4].tolist() == p_o.tolist() and tok[0, :4].tolist() == t_o.tolist() == [-1, 0, 1, 0]


def test_tree_feeds_verification(tw):
    """The finalised arrays are valid inputs of the verification side: parents precede children."""
    E, K, D, n_max, t_max, V = 4, 3, 3, 20, 32, 512
    rng = synth.rng_for(7, 22)
    dev = [torch.from_numpy(rng.standard_normal((2, 1 if l == 0 else K, V)).astype(np.float32)).to(DEV) for l in range(D)]
    parent, tok, n_nodes, kept, status, _ = gpu_tree(tw, dev, E, K, n_max, t_max)
    assert not status.any()
    for b in range(2):
        n = int(n_nodes[b])
        assert n == n_max and parent[b, 0] == -1
        assert all(0 <= parent[b, i] < i for i in range(1, n))
        O.tree_mask(parent[b, :n], n, 5)               # the oracle accepts it as a tree


def test_draft_verify_accept_chain(tw):
    """The device arrays flow from one entry point into the next without touching the host: token tree ->
    target tokens -> tree attention -> acceptance + KV append, against the same chain of oracle functions."""
    E, K, D, n_max, t_max, V = 3, 2, 3, 10, 16, 512
    B, Hq, Hkv, d, nl, L0 = 2, 4, 2, 128, 2, 70
    rng = synth.rng_for(7, 23)
    levels = [rng.standard_normal((B, 1 if l == 0 else K, V)).astype(np.float32) * 2 for l in range(D)]
    parent_d, tok_d, n_d = (torch.zeros((B, t_max), dtype=torch.int32, device=DEV), torch.zeros((B, t_max), dtype=torch.int32, device=DEV),
                            torch.zeros(B, dtype=torch.int32, device=DEV))
    cap = 1 + E + (D - 1) * K * E
    st = tw.TreeState(B, cap, DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_reset(st)
    src, lo, hi = torch.zeros((B, 1), dtype=torch.int32, device=DEV), 0, 1
    for l in range(D):
        tw.tree_expand_level(torch.from_numpy(levels[l]).to(DEV), src, E, hi, st, dev_status=status)
        lo, hi = hi, hi + (1 if l == 0 else K) * E
        if l + 1 < D:
            src = torch.zeros((B, K), dtype=torch.int32, device=DEV)
            tw.tree_select_expansion(st, lo, hi, src, dev_status=status)
    tw.tree_finalize(st, cap, n_max, parent_d, tok_d, n_d, dev_status=status)
    # oracle trees; target logits that follow one root-to-leaf path of each tree and then diverge
    trees = [O.build_token_tree([lv[b] for lv in levels], E, K, n_max) for b in range(B)]
    tgt = rng.standard_normal((B, t_max, V)).astype(np.float32)
    planted = []
    for b in range(B):
        par, tk = trees[b][0], trees[b][1]
        u, depth = 0, 0
        for _ in range(2 + b):                                  # follow up to 2 (request 0) or 3 (request 1) levels
            kids = [i for i in range(len(par)) if par[i] == u]
            if not kids:
                break
            tgt[b, u, tk[kids[-1]]] = 40.0                       # the target agrees with the last child
            u, depth = kids[-1], depth + 1
        planted.append(depth)
    assert min(planted) >= 1
    tgt_d = torch.from_numpy(tgt).to(DEV)
    base_d = torch.zeros((B, t_max), dtype=torch.int32, device=DEV)
    tw.tree_base_argmax(tgt_d, n_d, base_d, dev_status=status)
    # verification inputs
    q = synth.normal_bf16(rng, (nl, B, t_max, Hq, d), d, d ** 0.5)
    tkv = [synth.normal_bf16(rng, (nl, B, Hkv, t_max, d), d, d ** 0.5) for _ in range(2)]
    cache = [synth.normal_bf16(rng, (nl, B, Hkv, L0 + t_max, d), d, d ** 0.5) for _ in range(2)]
    kv_len = np.array([L0, L0 - 9], dtype=np.int32)
    ck, cv = dev_bf16(cache[0]), dev_bf16(cache[1])
    kvl = dev_i32(kv_len)
    q_d, tk_d, tv_d = dev_bf16(q), dev_bf16(tkv[0]), dev_bf16(tkv[1])
    out = torch.zeros((nl, B, t_max, Hq, d), dtype=torch.bfloat16, device=DEV)
    kvc = tw.KV.of(ck, cv)
    for layer in range(nl):
        tw.tree_verify_attention(q_d[layer], tk_d[layer], tv_d[layer], kvc, layer, kvl, n_d, parent_d, out[layer], dev_status=status)
    alen = torch.zeros(B, dtype=torch.int32, device=DEV)
    path = torch.full((B, t_max), -7, dtype=torch.int32, device=DEV)
    bonus = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_accept_compact(parent_d, tok_d, base_d, n_d, tk_d, tv_d, kvc, kvl, alen, path, bonus, dev_status=status)
    torch.cuda.synchronize()
    assert not status.cpu().numpy().any()
    # the same chain on the CPU
    base_o = O.base_argmax(tgt.astype(np.float64), [len(t[0]) for t in trees])
    ok_, ov_ = cache[0].copy(), cache[1].copy()
    paths = []
    for b in range(B):
        par, tk = trees[b][0], trees[b][1]
        n = len(par)
        assert n_d.cpu().numpy()[b] == n and np.array_equal(parent_d.cpu().numpy()[b, :n], par)
        a, pth, bt = O.tree_accept(par, tk, base_o[b], n)
        assert a == planted[b]                                   # the planted path is what gets accepted
        assert alen.cpu().numpy()[b] == a and bonus.cpu().numpy()[b] == bt
        assert path.cpu().numpy()[b, :a + 1].tolist() == pth.tolist()
        paths.append(pth.tolist())
    par_pad = np.full((B, t_max), -1, dtype=np.int32)
    for b in range(B):
        par_pad[b, :len(trees[b][0])] = trees[b][0]
    n_list = [len(t[0]) for t in trees]
    for layer in range(nl):
        want, _ = O.tree_attention(f64(q[layer]), f64(tkv[0][layer]), f64(tkv[1][layer]), f64(cache[0][layer]),
                                   f64(cache[1][layer]), kv_len, n_list, par_pad)
        got = f64(host_bits(out[layer]))
        for b in range(B):
            n = n_list[b]
            assert max_abs(got[b, :n], want[b, :n]) <= MAX_ABS_TOL
            assert rel_l2_rows(got[b, :n].reshape(-1, d), want[b, :n].reshape(-1, d)) <= REL_L2_TOL
    new_len = O.accept_compact(tkv[0], tkv[1], ok_, ov_, kv_len, paths)
    assert np.array_equal(kvl.cpu().numpy(), new_len)
    assert np.array_equal(host_bits(ck), ok_) and np.array_equal(host_bits(cv), ov_)


def test_unused_expansion_rows_are_never_selected(tw):
    """A row with src_node = -1 leaves children with score -inf, which the selection in the same launch
    ranks after every real node."""
    B, V, E, K = 2, 300, 3, 3
    rng = synth.rng_for(7, 24)
    st = tw.TreeState(B, 1 + E + K * E, DEV)
    st.score.fill_(7.0)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    lv1 = torch.from_numpy(rng.standard_normal((B, 1, V)).astype(np.float32)).to(DEV)
    lv2 = torch.from_numpy(rng.standard_normal((B, K, V)).astype(np.float32)).to(DEV)
    src = torch.zeros((B, 1), dtype=torch.int32, device=DEV)
    nxt = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    tw.tree_grow_level(lv1, src, E, 1, st, expand_node=nxt, dev_status=status)
    torch.cuda.synchronize()
    assert nxt.cpu().tolist() == [[1, 2, 3]] * B
    nxt[1, 1] = -1                                   # request 1 expands only nodes 1 and 3
    nxt2 = torch.zeros((B, 2 * E), dtype=torch.int32, device=DEV)
    tw.tree_grow_level(lv2, nxt, E, 1 + E, st, expand_node=nxt2, dev_status=status)
    torch.cuda.synchronize()
    score = st.score.cpu().numpy()
    lo = 1 + E
    assert np.all(np.isneginf(score[1, lo + E:lo + 2 * E])) and np.all(np.isfinite(score[0, lo:lo + K * E]))
    assert np.all(np.isfinite(score[1, lo:lo + E])) and np.all(np.isfinite(score[1, lo + 2 * E:lo + 3 * E]))
    assert nxt2.cpu().numpy()[1].tolist() == list(range(lo, lo + E)) + list(range(lo + 2 * E, lo + 3 * E))
    assert not status.cpu().numpy().any() and not st.ticket.any()


def test_next_row_entry_points_report_bad_arguments(tw):
    """Host-side argument checks return an error and launch nothing; device-side checks set dev_status and
    leave the outputs of that request untouched.  (None of these cases can read or write out of bounds.)"""
    from paper_2503_14075_b200.twig import TwigError
    B, V, E, K = 2, 256, 4, 2
    st = tw.TreeState(B, 1 + E + K * E, DEV)
    tw.tree_reset(st)
    logits = torch.zeros((B, 1, V), dtype=torch.float32, device=DEV)
    root = torch.zeros((B, 1), dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    # more children than the state can hold
    with pytest.raises(TwigError) as e:
        tw.tree_expand_level(logits, root, 16, 1, st)
    assert e.value.code == 2          # TWIG_ERR_SHAPE
    # more children per node than the kernel supports
    with pytest.raises(TwigError) as e:
        tw.tree_expand_level(logits, root, 17, 1, tw.TreeState(B, 64, DEV))
    assert e.value.code == 3          # TWIG_ERR_UNSUPPORTED
    # selection wider than the level
    tw.tree_expand_level(logits, root, E, 1, st, dev_status=status)
    with pytest.raises(TwigError) as e:
        tw.tree_select_expansion(st, 1, 1 + E, torch.zeros((B, E + 1), dtype=torch.int32, device=DEV))
    assert e.value.code == 2
    # a source node that is not older than the level (request 1): flagged on the device, request 0 is built
    src = torch.tensor([[1, 2], [1, 7]], dtype=torch.int32, device=DEV)
    lv2 = torch.zeros((B, K, V), dtype=torch.float32, device=DEV)
    tw.tree_expand_level(lv2, src, E, 1 + E, st, dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 4]                      # TWIG_DEV_BAD_TREE
    assert st.parent.cpu().numpy()[0, 1 + E:1 + E + K * E].tolist() == [1] * E + [2] * E
    # target tokens: a node count beyond t_max is flagged, nothing is written for that request
    out = torch.full((B, 3), -5, dtype=torch.int32, device=DEV)
    status.zero_()
    tw.tree_base_argmax(torch.zeros((B, 3, V), dtype=torch.float32, device=DEV), dev_i32([3, 4]), out, dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 4] and out.cpu().numpy()[1].tolist() == [-5, -5, -5]
    # multi-query guide: more text tokens after the image than q_text holds
    qt = torch.zeros((1, 4, 2, 128), dtype=torch.bfloat16, device=DEV)
    k = torch.zeros((1, 4, 32, 128), dtype=torch.bfloat16, device=DEV)
    sc = torch.full((1, 8), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.zeros(tw.ttp_multiquery_workspace_bytes(1, 4, 2, 8, 32), dtype=torch.uint8, device=DEV)
    st1 = torch.zeros(1, dtype=torch.int32, device=DEV)
    tw.ttp_score_multiquery(qt, k, dev_i32([20]), dev_i32([4]), dev_i32([8]), sc, ws, dev_status=st1)   # 8 text tokens > 2
    torch.cuda.synchronize()
    assert st1.cpu().tolist() == [1] and np.all(sc.cpu().numpy() == 0)        # TWIG_DEV_BAD_LAYOUT, scores zeroed
