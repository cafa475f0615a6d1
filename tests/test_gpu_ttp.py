"""GPU parity: twig-guided token pruning (scores, TopR, KV gather) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth
from gpu_common import (DEV, MAX_ABS_TOL, REL_L2_TOL, dev_bf16, dev_i32, f64, host_bits, max_abs,
                        rel_l2_rows)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tw():
    from paper_2503_14075_b200 import twig
    return twig


def _small_workload(B, Hq, Hkv, d, lens, keep, index=9):
    return synth.Workload(index, "test", 2, B, Hq, Hkv, d, [a for a, _, _ in lens], [m for _, m, _ in lens],
                          [c for _, _, c in lens], list(keep), [8] * B, [3] * B, 0.6)


WORKLOADS = {
    "c1": lambda: synth.workload(1),
    "c2": lambda: synth.workload(2),
    "c3": lambda: synth.workload(3),      # the heterogeneous batch of 16
    "c4": lambda: synth.workload(4),      # 3008-token prompts, 2880 visual tokens
    "c5": lambda: synth.workload(5),      # 28 query heads on 4 kv heads
    "hetero": lambda: _small_workload(5, 8, 8, 128, [(35, 576, 40), (20, 300, 0), (0, 129, 7), (3, 1, 1), (10, 0, 5)],
                                      [64, 300, 1, 0, 0]),
    "gqa64": lambda: _small_workload(3, 12, 4, 64, [(17, 333, 9), (1, 1025, 130), (0, 64, 0)], [33, 128, 64]),
    "gqa7": lambda: _small_workload(2, 28, 4, 128, [(128, 1024, 128), (5, 200, 3)], [128, 7]),
}


def _run_scores(tw, pre, scope, wl):
    B = wl.batch
    m_max = max(1, int(pre["n_vis"].max()))
    q, k = dev_bf16(pre["twig_q"]), dev_bf16(pre["twig_k"])
    scores = torch.full((B, m_max), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, wl.head_dim, k.shape[2], 64), dtype=torch.uint8, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_score(q, k, dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]), dev_i32(pre["n_vis"]), scores, ws,
                 norm_scope=scope, dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * B
    return scores.cpu().numpy()


@pytest.mark.parametrize("name", list(WORKLOADS))
@pytest.mark.parametrize("scope", [0, 1])
@pytest.mark.parametrize("gain_mult", [1.0, "sharp", "sharp4"])
def test_scores_match_oracle(tw, name, scope, gain_mult):
    wl = WORKLOADS[name]()
    gain = {1.0: 1.0, "sharp": wl.head_dim ** 0.5, "sharp4": 2.0 * wl.head_dim ** 0.5}[gain_mult]
    pre = synth.make_prefill(wl, synth.rng_for(wl.index, 1), n_layers=1, gain=gain)
    got = _run_scores(tw, pre, scope, wl)
    want = O.ttp_scores(f64(pre["twig_q"]), f64(pre["twig_k"]), pre["prefix_len"], pre["vis_start"], pre["n_vis"], scope)
    for b in range(wl.batch):
        m = pre["n_vis"][b]
        assert max_abs(got[b, :m], want[b, :m]) <= MAX_ABS_TOL
        assert rel_l2_rows(got[b, :m].astype(np.float64), want[b, :m]) <= REL_L2_TOL
        assert np.all(got[b, m:] == 0)
        if scope == 1 and m > 0:
            assert abs(float(got[b, :m].astype(np.float64).sum()) - 1.0) < 1e-4


@pytest.mark.parametrize("name", ["c1", "hetero", "gqa64", "gqa7"])
@pytest.mark.parametrize("scope", [1, 0])
def test_gated_scores_match_oracle(tw, name, scope):
    """Eq. 7 with the gates applied inside the kernel."""
    wl = WORKLOADS[name]()
    rng = synth.rng_for(wl.index, 11)
    pre = synth.make_prefill(wl, rng, n_layers=1, gain=wl.head_dim ** 0.5)
    qg, kg = synth.gate_bf16(rng, pre["twig_q"].shape), synth.gate_bf16(rng, pre["twig_k"].shape)
    B = wl.batch
    m_max = max(1, int(pre["n_vis"].max()))
    q, k = dev_bf16(pre["twig_q"]), dev_bf16(pre["twig_k"])
    scores = torch.full((B, m_max), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, wl.head_dim, k.shape[2], 64), dtype=torch.uint8, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_score_gated(q, dev_bf16(qg), k, dev_bf16(kg), dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]),
                       dev_i32(pre["n_vis"]), scores, ws, norm_scope=scope, dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * B
    got = scores.cpu().numpy()
    want = O.ttp_scores_gated(f64(pre["twig_q"]), f64(qg), f64(pre["twig_k"]), f64(kg), pre["prefix_len"], pre["vis_start"],
                              pre["n_vis"], scope)
    ungated = O.ttp_scores(f64(pre["twig_q"]), f64(pre["twig_k"]), pre["prefix_len"], pre["vis_start"], pre["n_vis"], scope)
    for b in range(B):
        m = pre["n_vis"][b]
        assert max_abs(got[b, :m], want[b, :m]) <= MAX_ABS_TOL
        assert rel_l2_rows(got[b, :m].astype(np.float64), want[b, :m]) <= REL_L2_TOL
        assert np.all(got[b, m:] == 0)
        if m > 1:      # the gates matter on these inputs: the ungated score is far outside the tolerance
            assert rel_l2_rows(ungated[b, :m], want[b, :m]) > 10 * REL_L2_TOL


@pytest.mark.parametrize("name", ["c1", "c2", "hetero", "gqa64", "gqa7"])
@pytest.mark.parametrize("gain_mult", [1.0, "sharp"])
def test_multiquery_scores_match_oracle(tw, name, gain_mult):
    """Eq. 3's guide: attention from the text tokens after the image to the visual tokens."""
    wl = WORKLOADS[name]()
    gain = {1.0: 1.0, "sharp": wl.head_dim ** 0.5}[gain_mult]
    rng = synth.rng_for(wl.index, 12)
    pre = synth.make_prefill(wl, rng, n_layers=1, gain=gain)
    B, Hq, d = wl.batch, wl.n_q_heads, wl.head_dim
    n_text = [int(pre["prefix_len"][b] - pre["vis_start"][b] - pre["n_vis"][b]) for b in range(B)]
    n_max = max(1, max(n_text)) + 3                     # a few rows nobody may read
    qt = synth.normal_bf16(rng, (B, Hq, n_max, d), d, gain)
    for b in range(B):
        qt[b, :, n_text[b]:, :] = 0x7FC1                # NaN past the last text token
    m_max = max(1, int(pre["n_vis"].max()))
    scores = torch.full((B, m_max), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.full((tw.ttp_multiquery_workspace_bytes(B, Hq, n_max, m_max, pre["twig_k"].shape[2]) // 4,), float("nan"), dtype=torch.float32,
                    device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    args = (dev_bf16(qt), dev_bf16(pre["twig_k"]), dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]),
            dev_i32(pre["n_vis"]), scores, ws)
    tw.ttp_score_multiquery(*args, dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * B
    got = scores.cpu().numpy()
    qt_clean = qt.copy()
    for b in range(B):
        qt_clean[b, :, n_text[b]:, :] = 0
    want = O.text_to_visual_scores(f64(qt_clean), f64(pre["twig_k"]), pre["prefix_len"], pre["vis_start"], pre["n_vis"])
    for b in range(B):
        m = pre["n_vis"][b]
        scale = max(1, n_text[b])                       # up to n_text probabilities add up in an entry
        assert max_abs(got[b, :m], want[b, :m]) <= MAX_ABS_TOL * scale
        if m > 0 and n_text[b] > 0:
            assert rel_l2_rows(got[b, :m].astype(np.float64), want[b, :m]) <= REL_L2_TOL
        assert np.all(got[b, m:] == 0)
    # same bits on a second run (fixed summation order)
    scores2 = torch.full_like(scores, -2.0)
    tw.ttp_score_multiquery(*args[:5], scores2, ws, dev_status=status)
    torch.cuda.synchronize()
    assert torch.equal(scores, scores2)


@pytest.mark.parametrize("d", [64, 128])
def test_multiquery_many_text_rows(tw, d):
    """More text tokens than one 64-row block, a causal edge that crosses 128-key chunks, requests
    of different layouts in one call, keys past the prompt poisoned (nobody may see them)."""
    B, Hq, Hkv = 3, 4, 2
    vis_start = np.array([5, 0, 130], dtype=np.int32)
    n_vis = np.array([300, 70, 129], dtype=np.int32)
    n_text = [150, 64, 1]
    prefix_len = (vis_start + n_vis + np.array(n_text)).astype(np.int32)
    L_max = int(prefix_len.max()) + 9
    rng = synth.rng_for(9, 31)
    gain = d ** 0.5                                     # logits of order one
    k = synth.normal_bf16(rng, (B, Hkv, L_max, d), d, gain)
    for b in range(B):
        k[b, :, prefix_len[b]:, :] = 0x7FC1             # NaN past the prompt
    n_max = max(n_text) + 2
    qt = synth.normal_bf16(rng, (B, Hq, n_max, d), d, gain)
    for b in range(B):
        qt[b, :, n_text[b]:, :] = 0x7FC1
    m_max = int(n_vis.max())
    scores = torch.full((B, m_max), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.full((tw.ttp_multiquery_workspace_bytes(B, Hq, n_max, m_max, L_max) // 4,), float("nan"),
                    dtype=torch.float32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_score_multiquery(dev_bf16(qt), dev_bf16(k), dev_i32(prefix_len), dev_i32(vis_start), dev_i32(n_vis), scores, ws,
                            dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * B
    got = scores.cpu().numpy()
    qt_clean, k_clean = qt.copy(), k.copy()
    for b in range(B):
        qt_clean[b, :, n_text[b]:, :] = 0
        k_clean[b, :, prefix_len[b]:, :] = 0
    want = O.text_to_visual_scores(f64(qt_clean), f64(k_clean), prefix_len, vis_start, n_vis)
    for b in range(B):
        m = n_vis[b]
        assert np.all(np.isfinite(got[b]))
        assert max_abs(got[b, :m], want[b, :m]) <= MAX_ABS_TOL * n_text[b]
        assert rel_l2_rows(got[b, :m].astype(np.float64), want[b, :m]) <= REL_L2_TOL
        assert np.all(got[b, m:] == 0)


def _run_topk(tw, s, n_vis, keep, r_max=None):
    B, m_max = s.shape
    r_max = r_max or max(1, int(max(keep)))
    kept = torch.full((B, r_max), -9, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_topk(torch.from_numpy(s).to(DEV), dev_i32(n_vis), dev_i32(keep), kept, dev_status=status)
    torch.cuda.synchronize()
    return kept.cpu().numpy(), status.cpu().numpy()


def test_topk_bit_exact_adversarial():
    from paper_2503_14075_b200 import twig as tw
    rng = np.random.default_rng(3)
    cases = []
    for M in (1, 2, 31, 32, 33, 576, 1023, 1024, 1025, 2880, 5000, 16384):
        for kind in ("random", "ties", "binary", "zeros", "increasing", "decreasing", "signed", "denormal"):
            if kind == "random":
                s = rng.random(M, dtype=np.float32)
            elif kind == "ties":
                s = (rng.integers(0, 5, M) / 7).astype(np.float32)
            elif kind == "binary":
                s = rng.integers(0, 2, M).astype(np.float32)
            elif kind == "zeros":
                s = np.zeros(M, dtype=np.float32)
            elif kind == "increasing":
                s = np.arange(M, dtype=np.float32)
            elif kind == "decreasing":
                s = np.arange(M, dtype=np.float32)[::-1].copy()
            elif kind == "signed":
                s = rng.standard_normal(M).astype(np.float32)
                s[3::11] = 0.0
            else:
                s = (rng.integers(0, 4, M).astype(np.float32) * np.float32(1e-45))
            for R in sorted({0, 1, M // 3, M - 1, M} - {-1}):
                cases.append((s, R))
    m_max = 16384
    for i in range(0, len(cases), 16):
        chunk = cases[i:i + 16]
        s = np.zeros((len(chunk), m_max), dtype=np.float32)
        for j, (v, _) in enumerate(chunk):
            s[j, :len(v)] = v
        n_vis = [len(v) for v, _ in chunk]
        keep = [R for _, R in chunk]
        kept, status = _run_topk(tw, s, n_vis, keep, r_max=m_max)
        assert not status.any()
        for j, (v, R) in enumerate(chunk):
            want = O.topk_lowest_index(v, R)
            assert np.array_equal(kept[j, :R], want), (len(v), R)
            assert np.all(kept[j, R:] == -1)


def test_topk_given_gpu_scores_c2_and_c4_sizes(tw):
    for wl_i, scope in ((2, 0), (2, 1), (4, 0)):
        wl = synth.workload(wl_i)
        pre = synth.make_prefill(wl, synth.rng_for(wl_i, 2), n_layers=1)
        if wl_i == 4:       # only the twig tensors matter here
            pre["cache_k"] = pre["cache_v"] = None
        s = _run_scores(tw, pre, scope, wl)
        kept, status = _run_topk(tw, s, pre["n_vis"], pre["keep"])
        assert not status.any()
        for b in range(wl.batch):
            assert np.array_equal(kept[b, :wl.keep[b]], O.topk_lowest_index(s[b, :wl.n_vis[b]], wl.keep[b]))


def test_topk_bad_keep_sets_status(tw):
    s = np.random.default_rng(0).random((3, 40), dtype=np.float32)
    kept, status = _run_topk(tw, s, [40, 40, 10], [5, 41, 11], r_max=64)
    assert status.tolist() == [0, tw.DEV_BAD_KEEP, tw.DEV_BAD_KEEP]
    assert np.array_equal(kept[0, :5], O.topk_lowest_index(s[0], 5))
    assert np.all(kept[1] == -9) and np.all(kept[2] == -9)          # skipped requests are untouched


def _compact_case(tw, wl, pre, kept_lists, canary=0x7FC1):
    nl = pre["cache_k"].shape[0]
    B, Hkv, d = wl.batch, wl.n_kv_heads, wl.head_dim
    r_max = max(1, max(len(k) for k in kept_lists))
    kept = np.full((B, r_max), -1, dtype=np.int32)
    for b, kl in enumerate(kept_lists):
        kept[b, :len(kl)] = kl
    keep = np.array([len(k) for k in kept_lists], dtype=np.int32)
    dst_len = max(1, max(lp - m + r for lp, m, r in zip(wl.prefix_len, wl.n_vis, keep))) + 5
    sk, sv = dev_bf16(pre["cache_k"]), dev_bf16(pre["cache_v"])
    dk = torch.full((nl, B, Hkv, dst_len, d), 0, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    dv = dk.clone()
    dk.view(torch.int16).fill_(canary)
    dv.view(torch.int16).fill_(canary)
    lmax = pre["pos_ids"].shape[1]
    pos_in = dev_i32(pre["pos_ids"] * 3 + 1)
    pos_out = torch.full((B, lmax), -5, dtype=torch.int32, device=DEV)
    new_len = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_compact(tw.KV.of(sk, sv), tw.KV.of(dk, dv), dev_i32(kept), dev_i32(keep), dev_i32(pre["prefix_len"]),
                   dev_i32(pre["vis_start"]), dev_i32(pre["n_vis"]), pos_in, pos_out, new_len, status)
    torch.cuda.synchronize()
    # oracle on the same bits
    ok = np.full((nl, B, Hkv, dst_len, d), canary, dtype=np.uint16)
    ov = ok.copy()
    opos = np.full((B, lmax), -5, dtype=np.int32)
    onew = O.gather_compact(pre["cache_k"], pre["cache_v"], pre["pos_ids"] * 3 + 1, pre["prefix_len"],
                            pre["vis_start"], pre["n_vis"], kept_lists, ok, ov, opos)
    return (host_bits(dk), host_bits(dv), pos_out.cpu().numpy(), new_len.cpu().numpy(), status.cpu().numpy(),
            ok, ov, opos, onew)


@pytest.mark.parametrize("name", ["c1", "hetero", "gqa64", "c2"])
def test_compact_byte_exact(tw, name):
    wl = WORKLOADS[name]()
    nl = 3 if name != "c2" else 2
    pre = synth.make_prefill(wl, synth.rng_for(wl.index, 3), n_layers=nl)
    rng = np.random.default_rng(4)
    kept_lists = [sorted(rng.choice(m, size=r, replace=False).tolist()) if r else [] for m, r in zip(wl.n_vis, wl.keep)]
    gk, gv, gpos, gnew, status, ok, ov, opos, onew = _compact_case(tw, wl, pre, kept_lists)
    assert not status.any()
    assert np.array_equal(gnew, onew)
    assert np.array_equal(gk, ok) and np.array_equal(gv, ov)          # moved rows and untouched canaries
    assert np.array_equal(gpos, opos)


def _compact_in_place_case(tw, wl, pre, kept_lists):
    """Compaction in place on the device against the oracle's gather with dst = src on a copy
    of the same bits: the whole cache is compared, so rows that must not move are checked too."""
    B = wl.batch
    r_max = max(1, max(len(k) for k in kept_lists))
    kept = np.full((B, r_max), -1, dtype=np.int32)
    for b, kl in enumerate(kept_lists):
        kept[b, :len(kl)] = kl
    keep = np.array([len(k) for k in kept_lists], dtype=np.int32)
    ck, cv = dev_bf16(pre["cache_k"]), dev_bf16(pre["cache_v"])
    pos = dev_i32(pre["pos_ids"] * 3 + 1)
    new_len = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    cache = tw.KV.of(ck, cv)
    tw.ttp_compact(cache, cache, dev_i32(kept), dev_i32(keep), dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]),
                   dev_i32(pre["n_vis"]), pos, pos, new_len, status)
    torch.cuda.synchronize()
    ok, ov, opos = pre["cache_k"].copy(), pre["cache_v"].copy(), (pre["pos_ids"] * 3 + 1).astype(np.int32)
    onew = O.gather_compact(ok, ov, opos, pre["prefix_len"], pre["vis_start"], pre["n_vis"], kept_lists, ok, ov, opos)
    return host_bits(ck), host_bits(cv), pos.cpu().numpy(), new_len.cpu().numpy(), status.cpu().numpy(), ok, ov, opos, onew


@pytest.mark.parametrize("name", ["c1", "hetero", "gqa64", "c2"])
def test_compact_in_place_byte_exact(tw, name):
    wl = WORKLOADS[name]()
    nl = 3 if name != "c2" else 2
    pre = synth.make_prefill(wl, synth.rng_for(wl.index, 3), n_layers=nl)
    rng = np.random.default_rng(4)
    kept_lists = [sorted(rng.choice(m, size=r, replace=False).tolist()) if r else [] for m, r in zip(wl.n_vis, wl.keep)]
    gk, gv, gpos, gnew, status, ok, ov, opos, onew = _compact_in_place_case(tw, wl, pre, kept_lists)
    assert not status.any()
    assert np.array_equal(gnew, onew)
    assert np.array_equal(gk, ok) and np.array_equal(gv, ov) and np.array_equal(gpos, opos)


def test_compact_in_place_adversarial_lists(tw):
    """Kept lists whose rows move by a single position, lists longer than a chunk of the kernel,
    keep-all (nothing may move) and keep-none."""
    wl = _small_workload(6, 4, 4, 128, [(3, 6, 5), (0, 400, 30), (7, 400, 0), (2, 300, 300), (5, 70, 9), (0, 33, 2)],
                         [3, 399, 1, 150, 70, 0])
    pre = synth.make_prefill(wl, synth.rng_for(9, 8), n_layers=2)
    kept = [[0, 2, 3], [i for i in range(400) if i != 7], [399], list(range(150, 300)), list(range(70)), []]
    gk, gv, gpos, gnew, status, ok, ov, opos, onew = _compact_in_place_case(tw, wl, pre, kept)
    assert not status.any() and np.array_equal(gnew, onew)
    assert np.array_equal(gk, ok) and np.array_equal(gv, ov) and np.array_equal(gpos, opos)
    assert np.array_equal(gk[:, 4], pre["cache_k"][:, 4])            # keep-all: the request's cache is untouched


def test_compact_in_place_refuses_bad_lists_before_moving_anything(tw):
    wl = _small_workload(2, 4, 4, 64, [(5, 20, 4), (5, 20, 4)], [3, 3])
    pre = synth.make_prefill(wl, synth.rng_for(9, 6), n_layers=1)
    gk, gv, gpos, gnew, status, ok, ov, opos, onew = _compact_in_place_case(tw, wl, pre, [[1, 2, 3], [1, 2, 3]])
    assert not status.any()
    B = 2
    ck, cv = dev_bf16(pre["cache_k"]), dev_bf16(pre["cache_v"])
    cache = tw.KV.of(ck, cv)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.ttp_compact(cache, cache, dev_i32([[1, 2, 3], [4, 2, 9]]), dev_i32([3, 3]), dev_i32(pre["prefix_len"]),
                   dev_i32(pre["vis_start"]), dev_i32(pre["n_vis"]), dev_status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, tw.DEV_BAD_INDEX]
    assert np.array_equal(host_bits(ck)[:, 1], pre["cache_k"][:, 1])      # the bad request's cache is untouched
    # partial overlap of source and destination is refused on the host
    half = tw.KV.of(ck[:, :, :, 1:], cv[:, :, :, 1:])
    with pytest.raises(tw.TwigError) as e:
        tw.ttp_compact(cache, half, dev_i32([[1, 2, 3], [1, 2, 3]]), dev_i32([3, 3]), dev_i32(pre["prefix_len"]),
                       dev_i32(pre["vis_start"]), dev_i32(pre["n_vis"]))
    assert e.value.code == 3


def test_compact_keep_all_identity_and_keep_none(tw):
    wl = _small_workload(2, 4, 4, 128, [(5, 70, 9), (0, 33, 2)], [70, 0])
    pre = synth.make_prefill(wl, synth.rng_for(9, 5), n_layers=2)
    gk, gv, gpos, gnew, status, ok, ov, opos, onew = _compact_case(tw, wl, pre, [list(range(70)), []])
    assert not status.any() and gnew.tolist() == [84, 2]
    assert np.array_equal(gk[:, 0, :, :84], pre["cache_k"][:, 0, :, :84])      # keep-all: identical copy
    assert np.array_equal(gk[:, 1, :, :2], pre["cache_k"][:, 1, :, 33:35])     # keep-none: text rows only
    assert np.array_equal(gk, ok) and np.array_equal(gv, ov) and np.array_equal(gpos, opos)


def test_compact_bad_inputs_set_status(tw):
    wl = _small_workload(3, 4, 4, 64, [(5, 20, 4), (5, 20, 4), (5, 20, 4)], [3, 3, 3])
    pre = synth.make_prefill(wl, synth.rng_for(9, 6), n_layers=1)
    pre["n_vis"][2] = 40                                              # visual span leaves the prompt
    out = _compact_case(tw, wl, pre, [[1, 2, 3], [4, 2, 9], [1, 2, 3]])
    status = out[4]
    assert status.tolist() == [0, tw.DEV_BAD_INDEX, tw.DEV_BAD_LAYOUT]


@pytest.mark.parametrize("name,scope", [("c1", 0), ("c1", 1), ("c2", 0), ("hetero", 1), ("gqa7", 0)])
def test_fused_prune_matches_stage_chain(tw, name, scope):
    wl = WORKLOADS[name]()
    nl = 2
    pre = synth.make_prefill(wl, synth.rng_for(wl.index, 7), n_layers=nl)
    B, Hkv, d = wl.batch, wl.n_kv_heads, wl.head_dim
    m_max, r_max = max(1, max(wl.n_vis)), max(1, max(wl.keep))
    q, k = dev_bf16(pre["twig_q"]), dev_bf16(pre["twig_k"])
    sk, sv = dev_bf16(pre["cache_k"]), dev_bf16(pre["cache_v"])
    dst_len = max(wl.pruned_len) + 3
    dk = torch.zeros((nl, B, Hkv, dst_len, d), dtype=torch.bfloat16, device=DEV)
    dv = torch.zeros_like(dk)
    scores = torch.zeros((B, m_max), dtype=torch.float32, device=DEV)
    kept = torch.zeros((B, r_max), dtype=torch.int32, device=DEV)
    lmax = pre["pos_ids"].shape[1]
    pos_out = torch.full((B, lmax), -1, dtype=torch.int32, device=DEV)
    new_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, d, k.shape[2], 64), dtype=torch.uint8, device=DEV)
    tw.ttp_score_topk_compact(q, k, dev_i32(pre["prefix_len"]), dev_i32(pre["vis_start"]), dev_i32(pre["n_vis"]),
                              dev_i32(pre["keep"]), scores, kept, tw.KV.of(sk, sv), tw.KV.of(dk, dv), ws,
                              pos_in=dev_i32(pre["pos_ids"]), pos_out=pos_out, new_len=new_len, norm_scope=scope,
                              dev_status=status)
    torch.cuda.synchronize()
    assert not status.cpu().numpy().any()
    s = scores.cpu().numpy()
    want_s = O.ttp_scores(f64(pre["twig_q"]), f64(pre["twig_k"]), pre["prefix_len"], pre["vis_start"], pre["n_vis"], scope)
    kept_lists = []
    overlap = []
    for b in range(B):
        m, r = wl.n_vis[b], wl.keep[b]
        assert max_abs(s[b, :m], want_s[b, :m]) <= MAX_ABS_TOL
        assert rel_l2_rows(s[b, :m].astype(np.float64), want_s[b, :m]) <= REL_L2_TOL
        want_idx = O.topk_lowest_index(s[b, :m], r)              # bit-exact given the same fp32 scores
        assert np.array_equal(kept.cpu().numpy()[b, :r], want_idx)
        kept_lists.append(want_idx.tolist())
        full = set(O.topk_lowest_index(want_s[b, :m], r).tolist())
        if r > 0:
            overlap.append(len(full & set(want_idx.tolist())) / r)
    ok = np.zeros((nl, B, Hkv, dst_len, d), dtype=np.uint16)
    ov = ok.copy()
    opos = np.full((B, lmax), -1, dtype=np.int32)
    onew = O.gather_compact(pre["cache_k"], pre["cache_v"], pre["pos_ids"], pre["prefix_len"], pre["vis_start"],
                            pre["n_vis"], kept_lists, ok, ov, opos)
    assert np.array_equal(new_len.cpu().numpy(), onew)
    assert np.array_equal(host_bits(dk), ok) and np.array_equal(host_bits(dv), ov)
    assert np.array_equal(pos_out.cpu().numpy(), opos)
    assert min(overlap) > 0.8        # informational: near-ties may flip between fp32 and fp64 scores


@pytest.mark.parametrize("width", [4096, 1000 * 8, 8])
def test_compact_rows_hidden_states_and_finalwipe(tw, width):
    """Eq. 5 on rows of any width (layer-K hidden states), and keep = 0 (FinalWipe)."""
    rng = np.random.default_rng(21)
    lens = [(35, 576, 64), (3, 100, 0), (0, 7, 9)]
    B = len(lens)
    lp = [a + m + c for a, m, c in lens]
    x = rng.integers(0, 1 << 16, size=(B, max(lp), width), dtype=np.uint16)
    for kept_lists in ([sorted(rng.choice(m, size=min(m, 64), replace=False).tolist()) for _, m, _ in lens],
                       [[] for _ in lens]):
        r_max = max(1, max(len(k) for k in kept_lists))
        kept = np.full((B, r_max), -1, dtype=np.int32)
        for b, kl in enumerate(kept_lists):
            kept[b, :len(kl)] = kl
        keep = [len(k) for k in kept_lists]
        src = dev_bf16(x)
        dst_rows = max(l - m + k for l, (_, m, _), k in zip(lp, lens, keep)) + 2
        dst = torch.zeros((B, dst_rows, width), dtype=torch.int16, device=DEV)
        dst.fill_(0x7FC1)
        dst = dst.view(torch.bfloat16)
        new_len = torch.full((B,), -1, dtype=torch.int32, device=DEV)
        status = torch.zeros(B, dtype=torch.int32, device=DEV)
        tw.ttp_compact_rows(src, dst, dev_i32(kept), dev_i32(keep), dev_i32(lp), dev_i32([a for a, _, _ in lens]),
                            dev_i32([m for _, m, _ in lens]), new_len=new_len, dev_status=status)
        torch.cuda.synchronize()
        want = np.full((B, dst_rows, width), 0x7FC1, dtype=np.uint16)
        wlen = O.gather_rows(x, lp, [a for a, _, _ in lens], [m for _, m, _ in lens], kept_lists, want)
        assert not status.cpu().numpy().any()
        assert np.array_equal(new_len.cpu().numpy(), wlen)
        assert np.array_equal(host_bits(dst), want)
