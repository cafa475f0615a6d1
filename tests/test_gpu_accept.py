"""GPU parity: tree acceptance + KV append, and the whole prune -> verify loop."""
import numpy as np
import pytest
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth
from gpu_common import DEV, REL_L2_TOL, dev_bf16, dev_i32, f64, host_bits, rel_l2_rows

pytestmark = pytest.mark.gpu
CANARY = 0x7FC1


@pytest.fixture(scope="module")
def tw():
    from paper_2503_14075_b200 import twig
    return twig


def _wl(nl, B, Hq, Hkv, d, n_nodes, depth, p=0.6):
    return synth.Workload(9, "test", nl, B, Hq, Hkv, d, [0] * B, [0] * B, [0] * B, [0] * B, list(n_nodes),
                          list(depth), p)


def run_accept(tw, ver, cache_k, cache_v, kv_len, d_max=None):
    B, T = ver["parent"].shape
    d_max = d_max or T
    ck, cv = dev_bf16(cache_k), dev_bf16(cache_v)
    kvl = dev_i32(kv_len)
    alen = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    path = torch.full((B, d_max), -7, dtype=torch.int32, device=DEV)
    bonus = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_accept_compact(dev_i32(ver["parent"]), dev_i32(ver["draft_tok"]), dev_i32(ver["base_argmax"]),
                           dev_i32(ver["n_nodes"]), dev_bf16(ver["tree_k"]), dev_bf16(ver["tree_v"]),
                           tw.KV.of(ck, cv), kvl, alen, path, bonus, dev_status=status)
    torch.cuda.synchronize()
    return (host_bits(ck), host_bits(cv), kvl.cpu().numpy(), alen.cpu().numpy(), path.cpu().numpy(),
            bonus.cpu().numpy(), status.cpu().numpy())


def oracle_accept(ver, cache_k, cache_v, kv_len):
    B = ver["parent"].shape[0]
    ok, ov = cache_k.copy(), cache_v.copy()
    alen, paths, bonus = [], [], []
    for b in range(B):
        n = int(ver["n_nodes"][b])
        if n == 0:
            alen.append(None)
            paths.append([])
            bonus.append(None)
            continue
        a, p, bt = O.tree_accept(ver["parent"][b], ver["draft_tok"][b], ver["base_argmax"][b], n)
        alen.append(a)
        paths.append(p.tolist())
        bonus.append(bt)
    new_len = O.accept_compact(ver["tree_k"], ver["tree_v"], ok, ov, kv_len, paths)
    return ok, ov, new_len, alen, paths, bonus


CASES = [
    ("c1", 1, 1, 4, 4, 64, [8], [3], 0.6, False),
    ("c2-shape", 4, 1, 8, 8, 128, [26], [5], 0.6, False),
    ("hetero", 3, 6, 4, 4, 128, [16, 32, 1, 0, 9, 27], [4, 6, 1, 2, 3, 6], 0.7, False),
    ("dup-siblings", 2, 8, 2, 2, 128, [20] * 8, [5] * 8, 0.8, True),
    ("deep64", 2, 2, 4, 2, 128, [64, 64], [64, 8], 0.95, False),
    ("gqa-d64", 5, 3, 12, 3, 64, [13, 64, 2], [3, 6, 2], 0.65, False),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_accept_compact_bit_exact(tw, case):
    name, nl, B, Hq, Hkv, d, n_nodes, depth, p, per_child = case
    wl = _wl(nl, B, Hq, Hkv, d, n_nodes, depth, p)
    for trial in range(4):
        rng = synth.rng_for(9, 200 + trial)
        ver = synth.make_verify_inputs(wl, rng, per_child=per_child)
        if name == "c2-shape":
            ver["parent"][0, :26] = synth.fixed_branching_tree([4, 2, 1, 1], 26)
        if name == "deep64" and trial % 2 == 0:
            ver["parent"][0] = synth.chain_tree(64)
            ver["draft_tok"][0, 1:] = ver["base_argmax"][0, :-1]          # whole chain accepted
        kv_len = rng.integers(0, 50, size=B).astype(np.int32)
        max_len = 50 + 64 + 3
        ck = np.full((nl, B, Hkv, max_len, d), CANARY, dtype=np.uint16)
        cv = ck.copy()
        gk, gv, glen, galen, gpath, gbonus, status = run_accept(tw, ver, ck, cv, kv_len)
        ok, ov, onew, oalen, opaths, obonus = oracle_accept(ver, ck, cv, kv_len)
        assert not status.any()
        for b in range(B):
            if oalen[b] is None:                    # idle request: nothing written
                assert galen[b] == -7 and gbonus[b] == -7 and np.all(gpath[b] == -7) and glen[b] == kv_len[b]
                continue
            assert galen[b] == oalen[b] and gbonus[b] == obonus[b]
            assert gpath[b, :oalen[b] + 1].tolist() == opaths[b] and np.all(gpath[b, oalen[b] + 1:] == -1)
            assert glen[b] == onew[b] == kv_len[b] + oalen[b] + 1
        assert np.array_equal(gk, ok) and np.array_equal(gv, ov)      # appended rows + untouched canaries


def test_accept_two_calls_in_a_row_and_status(tw):
    wl = _wl(2, 3, 4, 4, 128, [10, 10, 10], [4, 4, 4])
    rng = synth.rng_for(9, 300)
    ver = synth.make_verify_inputs(wl, rng)
    ver["parent"][1, 5] = 7                       # not an earlier node
    ck = np.full((2, 3, 4, 40, 128), CANARY, dtype=np.uint16)
    kv_len = np.array([5, 5, 38], dtype=np.int32)  # request 2 overflows unless nothing is accepted
    ver["draft_tok"][2, 1:] = ver["base_argmax"][2, ver["parent"][2, 1:]]       # accept a full path
    gk, gv, glen, galen, gpath, gbonus, status = run_accept(tw, ver, ck, ck.copy(), kv_len)
    assert status.tolist() == [0, tw.DEV_BAD_TREE, tw.DEV_OVERFLOW]
    assert glen.tolist()[1:] == [5, 38] and np.all(gk[:, 1:] == CANARY)
    # the completion ticket returned to zero: a second call behaves like the first
    gk2, _, glen2, galen2, _, _, status2 = run_accept(tw, ver, ck, ck.copy(), kv_len)
    assert np.array_equal(gk2, gk) and np.array_equal(glen2, glen) and galen2[0] == galen[0]


def test_prune_then_verify_loop_matches_oracle(tw):
    """The whole path on the tiny configuration plus a 7B-shaped 2-layer slice: prune, then
    several verify steps (attention in every layer, acceptance, append), GPU and oracle each
    keeping their own cache."""
    for index, nl, steps in ((1, 1, 6), (2, 2, 5)):
        wl = synth.workload(index)
        rng = synth.rng_for(index, 400)
        pre = synth.make_prefill(wl, rng, n_layers=nl)
        B, Hq, Hkv, d, T = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max
        max_len = max(wl.pruned_len) + steps * T + 8
        sk, sv = dev_bf16(pre["cache_k"]), dev_bf16(pre["cache_v"])
        dk = torch.zeros((nl, B, Hkv, max_len, d), dtype=torch.bfloat16, device=DEV)
        dv = torch.zeros_like(dk)
        scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=DEV)
        kept = torch.zeros((B, max(wl.keep)), dtype=torch.int32, device=DEV)
        kv_len = torch.zeros(B, dtype=torch.int32, device=DEV)
        status = torch.zeros(B, dtype=torch.int32, device=DEV)
        k = dev_bf16(pre["twig_k"])
        ws = torch.empty(tw.twig_workspace_bytes(B, Hq, d, k.shape[2], T), dtype=torch.uint8, device=DEV)
        cache = tw.KV.of(dk, dv)
        tw.ttp_score_topk_compact(dev_bf16(pre["twig_q"]), k, dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]),
                                  dev_i32(pre["n_vis"]), dev_i32(pre["keep"]), scores, kept, tw.KV.of(sk, sv), cache,
                                  ws, new_len=kv_len, dev_status=status)
        torch.cuda.synchronize()
        # oracle side: same selection rule applied to the GPU's fp32 scores
        s = scores.cpu().numpy()
        kept_lists = [O.topk_lowest_index(s[b, :wl.n_vis[b]], wl.keep[b]).tolist() for b in range(B)]
        ok = np.zeros((nl, B, Hkv, max_len, d), dtype=np.uint16)
        ov = ok.copy()
        opos = np.zeros_like(pre["pos_ids"])
        olen = O.gather_compact(pre["cache_k"], pre["cache_v"], pre["pos_ids"], pre["prefix_len"], pre["vis_start"],
                                pre["n_vis"], kept_lists, ok, ov, opos)
        assert np.array_equal(kv_len.cpu().numpy(), olen)
        alen = torch.zeros(B, dtype=torch.int32, device=DEV)
        path = torch.zeros((B, T), dtype=torch.int32, device=DEV)
        bonus = torch.zeros(B, dtype=torch.int32, device=DEV)
        out = torch.zeros((B, T, Hq, d), dtype=torch.bfloat16, device=DEV)
        for step in range(steps):
            ver = synth.make_verify_inputs(wl, rng, n_layers=nl, gain=d ** 0.5)
            par, nn = dev_i32(ver["parent"]), dev_i32(ver["n_nodes"])
            tk, tv = dev_bf16(ver["tree_k"]), dev_bf16(ver["tree_v"])
            for layer in range(nl):
                tw.tree_verify_attention(dev_bf16(ver["q"][layer]), tk[layer], tv[layer], cache, layer, kv_len, nn,
                                         par, out, dev_status=status)
                want, _ = O.tree_attention(f64(ver["q"][layer]), f64(ver["tree_k"][layer]), f64(ver["tree_v"][layer]),
                                           f64(ok[layer]), f64(ov[layer]), olen, ver["n_nodes"], ver["parent"])
                got = f64(host_bits(out))
                for b in range(B):
                    n = wl.n_nodes[b]
                    assert rel_l2_rows(got[b, :n], want[b, :n]) <= REL_L2_TOL
            tw.tree_accept_compact(par, dev_i32(ver["draft_tok"]), dev_i32(ver["base_argmax"]), nn, tk, tv, cache,
                                   kv_len, alen, path, bonus, dev_status=status)
            paths = []
            for b in range(B):
                a, p, bt = O.tree_accept(ver["parent"][b], ver["draft_tok"][b], ver["base_argmax"][b], wl.n_nodes[b])
                paths.append(p.tolist())
                assert int(alen[b]) == a and int(bonus[b]) == bt
            olen = O.accept_compact(ver["tree_k"], ver["tree_v"], ok, ov, olen, paths)
            assert np.array_equal(kv_len.cpu().numpy(), olen)
        torch.cuda.synchronize()
        assert not status.cpu().numpy().any()
        assert np.array_equal(host_bits(dk), ok) and np.array_equal(host_bits(dv), ov)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("vocab", [32000, 32003, 7])
def test_base_argmax_bit_exact(tw, dtype, vocab):
    """Greedy target token per tree node: lowest index on ties (bf16 rounding makes ties common)."""
    rng = np.random.default_rng(41)
    B, T = 3, 9
    n_nodes = [9, 4, 0]
    x = rng.standard_normal((B, T, vocab)).astype(np.float32)
    x[0, 1, :] = 0.25                                   # all equal -> index 0
    if vocab > 10:
        x[0, 2, [5, vocab - 1]] = 9.0                   # tie between far-apart indices
        x[1, 0, vocab - 1] = 11.0                       # winner in the ragged tail
    stride = (vocab + 7) // 8 * 8                       # rows start on 16 bytes
    if dtype == "bf16":
        bits = synth.f32_to_bf16(x)
        padded = np.full((B, T, stride), 0x7F7F, dtype=bits.dtype)   # padding holds a huge value
        padded[..., :vocab] = bits
        dev = dev_bf16(padded)[..., :vocab]
        ref_in = synth.bf16_to_f64(bits)
    else:
        padded = np.full((B, T, stride), 3e38, dtype=np.float32)
        padded[..., :vocab] = x
        dev = torch.from_numpy(padded).to(DEV)[..., :vocab]
        ref_in = x.astype(np.float64)
    out = torch.full((B, T), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_base_argmax(dev, dev_i32(n_nodes), out, dev_status=status)
    torch.cuda.synchronize()
    want = O.base_argmax(ref_in, n_nodes)
    got = out.cpu().numpy()
    assert not status.cpu().numpy().any()
    for b in range(B):
        assert np.array_equal(got[b, :n_nodes[b]], want[b, :n_nodes[b]])
        assert np.all(got[b, n_nodes[b]:] == -5)
