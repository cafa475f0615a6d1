"""GPU parity: tree-masked verification attention against the oracle."""
import zlib

import numpy as np
import pytest
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth
from gpu_common import (DEV, MAX_ABS_TOL, REL_L2_TOL, dev_bf16, dev_i32, f64, host_bits, max_abs,
                        rel_l2_rows)

pytestmark = pytest.mark.gpu
CANARY = 0x7FC1          # a bf16 NaN pattern: untouched rows are recognisable, stray reads poison


@pytest.fixture(scope="module")
def tw():
    from paper_2503_14075_b200 import twig
    return twig


_WS = {}


def stream_ws(tw, B, Hq, T):
    """Scratch of the persistent kernel: zero-filled once, then only ever passed to attention calls
    (which leave it zeroed), so one buffer per size serves the whole test session."""
    need = tw.tree_attention_workspace_bytes(B, Hq, T)
    if need not in _WS:
        _WS[need] = torch.zeros(need, dtype=torch.uint8, device=DEV)
    return _WS[need]


# kernels under test: (id, kernel, work sharing of the persistent kernel: 0 its own choice, 1 equal shares, 2 whole items)
KERNELS = [("mma", 1), ("tcgen05", 2), ("stream", 3), ("stream-shares", (3, 1)), ("stream-whole", (3, 2))]
KERNEL_IDS = [k[0] for k in KERNELS]
KERNEL_VALS = [k[1] for k in KERNELS]


def run_attention(tw, wl, ver, cache_k, cache_v, kv_len, layer=0, max_len=None, lse=True, path=0, splits=0,
                  early=False):
    """cache_k/v: uint16 [Nl,B,Hkv,Lmax,d].  Returns (out bits [B,T,Hq,d], lse [B,Hq,T], status).
    path: 0 automatic, 1 mma.sync kernel, 2 tcgen05 kernel (cluster splits), 3 persistent tcgen05 kernel,
    (3, policy) the persistent kernel with its work sharing forced.
    A named kernel is the kernel that runs (the library refuses, it never substitutes)."""
    policy = 0
    if isinstance(path, tuple):
        path, policy = path
    B, T, Hq, d = ver["q"].shape[1:]
    ws = stream_ws(tw, B, Hq, T) if path == 3 else None
    ck, cv = dev_bf16(cache_k), dev_bf16(cache_v)
    out = torch.zeros((B, T, Hq, d), dtype=torch.int16, device=DEV)
    out.fill_(CANARY)
    out = out.view(torch.bfloat16)
    lse_t = torch.full((B, Hq, T), -123.0, dtype=torch.float32, device=DEV) if lse else None
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.tree_verify_attention(dev_bf16(ver["q"][layer]), dev_bf16(ver["tree_k"][layer]), dev_bf16(ver["tree_v"][layer]),
                             tw.KV.of(ck, cv), layer, dev_i32(kv_len), dev_i32(ver["n_nodes"]), dev_i32(ver["parent"]),
                             out, lse=lse_t, dev_status=status, ws=ws,
                             flags=tw.attn_flags(kernel=path, splits=splits, early_prefix=early, stream_policy=policy))
    torch.cuda.synchronize()
    if ws is not None:      # the call leaves its arrival counters (the tail of the buffer) at zero
        n_tail = tw.tree_attention_workspace_bytes(B, Hq, T) - tw.tree_attention_workspace_bytes(1, 1, T) + 8
        assert not ws[-n_tail:].any()
    return host_bits(out), (lse_t.cpu().numpy() if lse else None), status.cpu().numpy()


def oracle_attention(ver, cache_k, cache_v, kv_len, layer=0, samples=None):
    return O.tree_attention(f64(ver["q"][layer]), f64(ver["tree_k"][layer]), f64(ver["tree_v"][layer]),
                            f64(cache_k[layer]), f64(cache_v[layer]), kv_len, ver["n_nodes"], ver["parent"],
                            samples=samples)


def check(got_bits, got_lse, want, want_lse, n_nodes, tag=""):
    got = f64(got_bits)
    B = got.shape[0]
    for b in range(B):
        n = int(n_nodes[b])
        assert np.all(got_bits[b, n:] == CANARY), tag            # padded nodes are not written
        if n == 0:
            continue
        assert not np.isnan(got[b, :n]).any(), tag
        assert max_abs(got[b, :n], want[b, :n]) <= MAX_ABS_TOL * max(1.0, np.abs(want[b, :n]).max()), tag
        assert rel_l2_rows(got[b, :n], want[b, :n]) <= REL_L2_TOL, (tag, rel_l2_rows(got[b, :n], want[b, :n]))
        if got_lse is not None:
            assert max_abs(got_lse[b, :, :n], want_lse[b, :, :n]) <= 1e-3 * max(1.0, np.abs(want_lse[b]).max()), tag


def _wl(B, Hq, Hkv, d, n_nodes, depth, index=9):
    return synth.Workload(index, "test", 1, B, Hq, Hkv, d, [0] * B, [0] * B, [0] * B, [0] * B, list(n_nodes),
                          list(depth), 0.6)


SHAPES = [
    # name, B, Hq, Hkv, d, n_nodes, depth, kv_len
    ("c1", 1, 4, 4, 64, [8], [3], [64]),
    ("t1-decode", 2, 4, 4, 128, [1, 1], [1, 1], [130, 1]),
    ("rows32", 2, 8, 8, 128, [26, 17], [5, 4], [163, 291]),
    ("rows64", 2, 4, 4, 128, [64, 33], [8, 6], [448, 700]),
    ("gqa-rows128", 2, 8, 2, 128, [30, 32], [6, 5], [257, 64]),
    ("gqa7-rows448", 1, 14, 2, 128, [64], [6], [384]),
    ("d64-rows64", 3, 6, 3, 64, [32, 5, 20], [6, 2, 4], [0, 100, 513]),
    ("empty-prefix", 1, 4, 4, 128, [9], [4], [0]),
    ("idle-request", 3, 4, 4, 128, [12, 0, 7], [3, 2, 3], [77, 50, 200]),
    ("long-rows64", 2, 4, 4, 128, [64, 40], [8, 6], [4100, 130]),
    ("long-gqa-rows128", 1, 8, 2, 128, [31], [5], [1500]),
]


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
@pytest.mark.parametrize("gain_name", ["timing", "sharp", "sharp4"])
@pytest.mark.parametrize("path", KERNEL_VALS, ids=KERNEL_IDS)
def test_tree_attention_matches_oracle(tw, shape, gain_name, path):
    name, B, Hq, Hkv, d, n_nodes, depth, kv_len = shape
    if path != 1 and d != 128:
        pytest.skip("the tcgen05 kernels cover head_dim 128")
    gain = {"timing": 1.0, "sharp": d ** 0.5, "sharp4": 2.0 * d ** 0.5}[gain_name]   # logit std 1/d, 1, 4
    wl = _wl(B, Hq, Hkv, d, n_nodes, depth)
    rng = synth.rng_for(9, zlib.crc32(name.encode()) % 1000)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1, gain=gain)
    max_len = max(kv_len) + 70
    ck, cv = synth.make_cache(wl, rng, max_len, n_layers=1, gain=gain)
    for b in range(B):                       # rows past kv_len must never be read
        ck[0, b, :, kv_len[b]:] = CANARY
        cv[0, b, :, kv_len[b]:] = CANARY
    got, lse, status = run_attention(tw, wl, ver, ck, cv, kv_len, path=path)
    assert not status.any()
    want, want_lse = oracle_attention(ver, ck, cv, np.array(kv_len))
    check(got, lse, want, want_lse, ver["n_nodes"], name)


@pytest.mark.parametrize("path", KERNEL_VALS, ids=KERNEL_IDS)
@pytest.mark.parametrize("kind", ["chain", "star"])
def test_special_trees(tw, kind, path):
    T = 20
    wl = _wl(2, 4, 4, 128, [T, T], [T, 2])
    rng = synth.rng_for(9, 77)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1, gain=128 ** 0.5)
    ver["parent"][:] = synth.chain_tree(T) if kind == "chain" else synth.star_tree(T)
    ck, cv = synth.make_cache(wl, rng, 300, n_layers=1, gain=128 ** 0.5)
    kv_len = [190, 3]
    got, lse, status = run_attention(tw, wl, ver, ck, cv, kv_len, path=path)
    want, want_lse = oracle_attention(ver, ck, cv, np.array(kv_len))
    check(got, lse, want, want_lse, ver["n_nodes"], kind)


@pytest.mark.parametrize("path", KERNEL_VALS, ids=KERNEL_IDS)
def test_bad_tree_and_overflow_set_status(tw, path):
    wl = _wl(4, 4, 4, 128, [6, 6, 6, 6], [3, 3, 3, 3])
    rng = synth.rng_for(9, 78)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1)
    ver["parent"][1, 3] = 3            # parent must be an earlier node
    ver["parent"][2, 0] = 0            # root must have parent -1
    ck, cv = synth.make_cache(wl, rng, 64, n_layers=1)
    got, lse, status = run_attention(tw, wl, ver, ck, cv, [10, 10, 10, 65], path=path)
    assert status.tolist() == [0, tw.DEV_BAD_TREE, tw.DEV_BAD_TREE, tw.DEV_OVERFLOW]
    assert np.all(got[1:] == CANARY)                                   # skipped requests untouched
    good = {k: (v[:, :1] if k in ("q", "tree_k", "tree_v") else v[:1]) for k, v in ver.items()}
    want, want_lse = oracle_attention(good, ck[:, :1], cv[:, :1], np.array([10]))      # the valid request only
    check(got[:1], lse[:1], want, want_lse, good["n_nodes"])


FULL = [
    # workload, kv lengths to test (pruned prompt ... final length)
    (2, [163, 291]),
    (3, None),
    (4, [448, 1472]),
    (5, [384, 8128]),
]


@pytest.mark.parametrize("path", KERNEL_VALS, ids=KERNEL_IDS)
@pytest.mark.parametrize("index,lens", FULL, ids=["c2", "c3", "c4", "c5"])
def test_full_size_configs(tw, index, lens, path):
    """Full-size shapes of the benchmark configurations, one layer, every output row
    against the oracle (timing distribution), plus sampled rows of a sharp variant."""
    wl = synth.workload(index)
    rng = synth.rng_for(index, 11)
    if lens is None:      # heterogeneous: pruned prompt + part of the generation target
        lens_list = [[p + g // 2 for p, g in zip(wl.pruned_len, wl.gen_target)]]
    else:
        lens_list = [[l] * wl.batch for l in lens]
    max_len = max(max(l) for l in lens_list) + 64
    for gain, sampled in ((1.0, False), (wl.head_dim ** 0.5, True)):
        ver = synth.make_verify_inputs(wl, rng, n_layers=1, gain=gain)
        ck, cv = synth.make_cache(wl, rng, max_len, n_layers=1, gain=gain)
        for kv_len in lens_list:
            got, lse, status = run_attention(tw, wl, ver, ck, cv, kv_len, path=path)
            assert not status.any()
            if not sampled:
                want, want_lse = oracle_attention(ver, ck, cv, np.array(kv_len))
                check(got, lse, want, want_lse, ver["n_nodes"], f"c{index} L={kv_len[0]}")
            else:
                srng = np.random.default_rng(index)
                smp = [(int(srng.integers(wl.batch)), 0, 0)]
                for _ in range(24):
                    b = int(srng.integers(wl.batch))
                    smp.append((b, int(srng.integers(wl.n_nodes[b])), int(srng.integers(wl.n_q_heads))))
                want, want_lse = O.tree_attention(f64(ver["q"][0]), f64(ver["tree_k"][0]), f64(ver["tree_v"][0]),
                                                  _F64View(ck[0]), _F64View(cv[0]), np.array(kv_len), ver["n_nodes"],
                                                  ver["parent"], samples=smp)
                g = f64(got)
                for (b, i, h) in smp:
                    assert rel_l2_rows(g[b, i, h][None], want[b, i, h][None]) <= REL_L2_TOL
                    assert abs(lse[b, h, i] - want_lse[b, h, i]) <= 1e-3 * max(1.0, abs(want_lse[b, h, i]))


class _F64View:
    """Lazily widens slices of a bf16 bit-pattern array (avoids a full fp64 copy of a big cache)."""

    def __init__(self, bits):
        self.bits = bits

    def __getitem__(self, idx):
        return synth.bf16_to_f64(self.bits[idx])


EARLY = [(SHAPES[0], 1), (SHAPES[2], 1), (SHAPES[6], 1), (SHAPES[2], 3), (SHAPES[3], 3), (SHAPES[5], 3)]


@pytest.mark.parametrize("shape,path", EARLY, ids=[f"{s[0]}-{'mma' if k == 1 else 'stream'}" for s, k in EARLY])
def test_early_prefix_gives_the_same_bits(tw, shape, path):
    """With the early-prefix promise kept (nothing before the call writes lengths or cache), the kernel
    fetches the prefix under its predecessor and must return identical bits."""
    name, B, Hq, Hkv, d, n_nodes, depth, kv_len = shape
    wl = _wl(B, Hq, Hkv, d, n_nodes, depth)
    rng = synth.rng_for(9, 321)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1, gain=d ** 0.5)
    ck, cv = synth.make_cache(wl, rng, max(kv_len) + 70, n_layers=1, gain=d ** 0.5)
    ref, ref_lse, st0 = run_attention(tw, wl, ver, ck, cv, kv_len, path=path)
    got, got_lse, st1 = run_attention(tw, wl, ver, ck, cv, kv_len, path=path, early=True)
    # several calls back to back on one stream: each fetches its prefix under the one before
    B_, T, Hq_, d_ = ver["q"].shape[1:]
    dck, dcv = dev_bf16(ck), dev_bf16(cv)
    cache = tw.KV.of(dck, dcv)
    q, tk, tv = dev_bf16(ver["q"][0]), dev_bf16(ver["tree_k"][0]), dev_bf16(ver["tree_v"][0])
    kvl, nn, par = dev_i32(kv_len), dev_i32(ver["n_nodes"]), dev_i32(ver["parent"])
    outs = [torch.zeros((B_, T, Hq_, d_), dtype=torch.bfloat16, device=DEV) for _ in range(4)]
    ws = stream_ws(tw, B_, Hq_, T) if path == 3 else None
    for i, o in enumerate(outs):
        # (the second promise, that Q and the tree rows are final too, holds here as well: nothing in
        # the stream writes them; the small-call kernel then does not wait before it computes)
        tw.tree_verify_attention(q, tk, tv, cache, 0, kvl, nn, par, o, ws=ws,
                                 flags=tw.attn_flags(kernel=path, early_prefix=True, early_query=(i % 2 == 1)))
    torch.cuda.synchronize()
    assert not st0.any() and not st1.any()
    assert np.array_equal(got, ref) and np.array_equal(got_lse, ref_lse)
    for b in range(B):
        n = n_nodes[b]
        for o in outs:
            assert np.array_equal(host_bits(o)[b, :n], ref[b, :n])


def test_named_kernel_is_never_substituted(tw):
    """A kernel named in the flags either runs or the call fails on the host: the tcgen05 kernels do not
    take head_dim 64, the persistent one does not run without its scratch."""
    wl = _wl(1, 4, 4, 64, [8], [3])
    rng = synth.rng_for(9, 5)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1)
    ck, cv = synth.make_cache(wl, rng, 80, n_layers=1)
    for path in (2, 3):
        with pytest.raises(tw.TwigError) as e:
            run_attention(tw, wl, ver, ck, cv, [10], path=path)
        assert e.value.code == 3                   # TWIG_ERR_UNSUPPORTED
    wl = _wl(1, 4, 4, 128, [8], [3])
    ver = synth.make_verify_inputs(wl, rng, n_layers=1)
    ck, cv = synth.make_cache(wl, rng, 80, n_layers=1)
    B, T, Hq, d = ver["q"].shape[1:]
    out = torch.zeros((B, T, Hq, d), dtype=torch.bfloat16, device=DEV)
    args = (dev_bf16(ver["q"][0]), dev_bf16(ver["tree_k"][0]), dev_bf16(ver["tree_v"][0]),
            tw.KV.of(dev_bf16(ck), dev_bf16(cv)), 0, dev_i32([10]), dev_i32(ver["n_nodes"]), dev_i32(ver["parent"]), out)
    with pytest.raises(tw.TwigError) as e:
        tw.tree_verify_attention(*args, flags=tw.attn_flags(kernel=3))              # no scratch
    assert e.value.code == 4                       # TWIG_ERR_WORKSPACE
    small = torch.zeros(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(tw.TwigError) as e:
        tw.tree_verify_attention(*args, ws=small, flags=tw.attn_flags(kernel=3))
    assert e.value.code == 4
    with pytest.raises(tw.TwigError) as e:
        tw.tree_verify_attention(*args, flags=tw.attn_flags(kernel=1, splits=3))    # not a split count
    assert e.value.code == 3
    torch.cuda.synchronize()
    assert not out.any()                           # nothing was launched


@pytest.mark.parametrize("v_scale", [2.0 ** -17, 1.0, 2.0 ** 17], ids=["tinyV", "unitV", "largeV"])
@pytest.mark.parametrize("path,splits", [(1, 1), (1, 2), (1, 4), (1, 8), (2, 1), (2, 2), (2, 4), (2, 8), ((3, 1), 0),
                                         ((3, 2), 0)], ids=lambda v: str(v))
def test_key_splits_and_value_range(tw, path, splits, v_scale):
    """The result must not depend on how the keys are split between CTAs, nor on the magnitude of V:
    partial results cross between CTAs in a narrower format than they are accumulated in."""
    wl = _wl(2, 4, 4, 128, [30, 17], [6, 4])
    rng = synth.rng_for(9, 4242)
    ver = synth.make_verify_inputs(wl, rng, n_layers=1, gain=128 ** 0.5)
    kv_len = [700, 333]
    ck, cv = synth.make_cache(wl, rng, 800, n_layers=1, gain=128 ** 0.5)
    # (powers of two: exact in bf16; 2^17 is beyond what fp16 holds, 2^-17 far below its normal range)
    cv = synth.f32_to_bf16(synth.bf16_to_f32(cv) * np.float32(v_scale))
    ver["tree_v"] = synth.f32_to_bf16(synth.bf16_to_f32(ver["tree_v"]) * np.float32(v_scale))
    got, lse, status = run_attention(tw, wl, ver, ck, cv, kv_len, path=path, splits=splits)
    assert not status.any()
    want, want_lse = oracle_attention(ver, ck, cv, np.array(kv_len))
    g = f64(got)
    for b in range(2):
        n = int(ver["n_nodes"][b])
        assert rel_l2_rows(g[b, :n], want[b, :n]) <= REL_L2_TOL
        assert max_abs(g[b, :n], want[b, :n]) <= MAX_ABS_TOL * max(1.0, np.abs(want[b, :n]).max())
        assert max_abs(lse[b, :, :n], want_lse[b, :, :n]) <= 1e-3 * max(1.0, np.abs(want_lse[b]).max())
