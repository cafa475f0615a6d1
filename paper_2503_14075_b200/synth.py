"""Seeded synthetic inputs for the TwigVLM/TwigVLM++ inference hot path.

This module only draws random inputs (tensors, trees, token ids, request
shapes).  It holds none of the method's arithmetic: no attention, no top-k,
no acceptance rule.  Both the CUDA path's tests/bench and the CPU oracle's
tests are fed from here, so that they see identical bits.

bf16 tensors are carried on the host as ``numpy.uint16`` bit patterns
(numpy has no bf16 type); ``bf16_to_f64`` widens them exactly.

Shapes follow the paper's workloads: 576 visual tokens per image for
LLaVA-1.5, 2880 for the five-tile high-resolution model, 64/128/192 or 320
kept tokens, 32 layers, draft trees of at most 60-64 nodes, and a chain
acceptance rate near 57 % (Tables 1-2, Appendix A of the paper).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

SEED_BASE = 250314075
VOCAB = 32000


def rng_for(config: int, stream: int = 0) -> np.random.Generator:
    """PCG64 generator for (config, stream)."""
    return np.random.default_rng(SEED_BASE + 1000 * int(config) + int(stream))


# --------------------------------------------------------------------------
# bf16 <-> host formats
# --------------------------------------------------------------------------
def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_to_f32(b).astype(np.float64)


def normal_bf16(rng: np.random.Generator, shape, head_dim: int, gain: float = 1.0) -> np.ndarray:
    """iid N(0,1) * gain / sqrt(head_dim), rounded to bf16 (uint16 bits).

    gain=1 is the timing distribution; gain=sqrt(head_dim) (and 4x that) gives
    logits of order one, used by correctness tests so that a wrong mask or
    index changes outputs at O(1).
    """
    x = rng.standard_normal(size=shape, dtype=np.float32)
    x *= np.float32(gain / np.sqrt(head_dim))
    return f32_to_bf16(x)


# --------------------------------------------------------------------------
# draft trees (parent arrays; node 0 is the root, parent[0] = -1)
# --------------------------------------------------------------------------
def gate_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    """Gate values as a bounded activation would give them: 2 * sigmoid(N(0, 1)), in (0, 2), as bf16 bits."""
    x = rng.standard_normal(shape, dtype=np.float32)
    return f32_to_bf16((2.0 / (1.0 + np.exp(-x))).astype(np.float32))


def node_depths(parent: Sequence[int]) -> np.ndarray:
    dep = np.zeros(len(parent), dtype=np.int32)
    for i in range(1, len(parent)):
        dep[i] = dep[parent[i]] + 1
    return dep


def chain_tree(n_nodes: int) -> np.ndarray:
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def star_tree(n_nodes: int) -> np.ndarray:
    p = np.zeros(n_nodes, dtype=np.int32)
    p[0] = -1
    return p


def fixed_branching_tree(branching: Sequence[int], n_keep: Optional[int] = None) -> np.ndarray:
    """Full tree with the given per-level branching, in BFS order, truncated
    to its first ``n_keep`` nodes (the deepest leaves are the ones dropped)."""
    parent = [-1]
    level = [0]
    for br in branching:
        nxt = []
        for u in level:
            for _ in range(br):
                parent.append(u)
                nxt.append(len(parent) - 1)
        level = nxt
    parent = np.asarray(parent, dtype=np.int32)
    if n_keep is not None:
        parent = parent[:n_keep]
    return parent


def random_tree(rng: np.random.Generator, n_nodes: int, depth_levels: int) -> np.ndarray:
    """Random tree with exactly ``depth_levels`` levels (root included): nodes
    0..depth_levels-1 form a spine (a chain), every later node i draws
    parent[i] ~ U{j < i : depth(j) < depth_levels-1}."""
    if n_nodes <= 1:
        return np.full(n_nodes, -1, dtype=np.int32)
    depth_levels = max(2, min(depth_levels, n_nodes))
    parent = np.full(n_nodes, -1, dtype=np.int32)
    dep = np.zeros(n_nodes, dtype=np.int32)
    for i in range(1, n_nodes):
        if i < depth_levels:
            j = i - 1
        else:
            cand = np.nonzero(dep[:i] < depth_levels - 1)[0]
            j = int(cand[rng.integers(len(cand))])
        parent[i] = j
        dep[i] = dep[j] + 1
    return parent


def draft_and_target_tokens(rng: np.random.Generator, parent: np.ndarray, match_p: float,
                            per_child: bool = False):
    """Token ids for a draft tree and the target's greedy token after each node.

    base_argmax[u] ~ U[0, VOCAB) for every node u.  Default (per-parent): for
    every node with children, with probability ``match_p`` one uniformly chosen
    child carries base_argmax[u]; all other children carry distinct tokens that
    differ from it (siblings are distinct, as the children of a node are the
    top tokens of one distribution).  ``per_child=True`` makes every child match
    independently, so duplicate sibling tokens occur (correctness tests only).
    """
    n = len(parent)
    base_argmax = rng.integers(0, VOCAB, size=n, dtype=np.int64).astype(np.int32)
    draft_tok = rng.integers(0, VOCAB, size=n, dtype=np.int64).astype(np.int32)
    children: List[List[int]] = [[] for _ in range(n)]
    for i in range(1, n):
        children[int(parent[i])].append(i)
    for u in range(n):
        ch = children[u]
        if not ch:
            continue
        tgt = int(base_argmax[u])
        if per_child:
            for c in ch:
                if rng.random() < match_p:
                    draft_tok[c] = tgt
                else:
                    draft_tok[c] = (tgt + 1 + int(rng.integers(0, VOCAB - 1))) % VOCAB
            continue
        # distinct non-matching tokens: offsets 1.. from the target, shuffled
        offs = rng.choice(VOCAB - 1, size=len(ch), replace=False) + 1
        for c, o in zip(ch, offs):
            draft_tok[c] = (tgt + int(o)) % VOCAB
        if rng.random() < match_p:
            draft_tok[ch[int(rng.integers(len(ch)))]] = tgt
    return draft_tok, base_argmax


# --------------------------------------------------------------------------
# workloads (the five benchmark configurations)
# --------------------------------------------------------------------------
@dataclass
class Workload:
    """Shapes of one configuration; per-request lists have length ``batch``."""
    index: int
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    text_before: List[int]
    n_vis: List[int]
    text_after: List[int]
    keep: List[int]
    n_nodes: List[int]
    depth_levels: List[int]
    match_p: float
    branching: Optional[List[int]] = None      # fixed-branching tree, else random parents
    gen_target: List[int] = field(default_factory=list)   # tokens to emit per request
    final_kv_len: Optional[int] = None         # KV length the verify step is timed at

    @property
    def t_max(self) -> int:
        return max(self.n_nodes)

    @property
    def prefix_len(self) -> List[int]:
        return [a + m + c for a, m, c in zip(self.text_before, self.n_vis, self.text_after)]

    @property
    def pruned_len(self) -> List[int]:
        return [a + r + c for a, r, c in zip(self.text_before, self.keep, self.text_after)]

    def kv_row_bytes(self) -> int:
        """K+V bytes of one position of one layer of one request."""
        return 2 * self.n_kv_heads * self.head_dim * 2


def workload(index: int) -> Workload:
    """The configuration with the given 1-based index (c1..c5)."""
    if index == 1:
        return Workload(1, "c1-tiny", 1, 1, 4, 4, 64, [32], [144], [16], [16], [8], [3], 0.6,
                        gen_target=[16])
    if index == 2:
        return Workload(2, "c2-llava15-7b-b1", 32, 1, 32, 32, 128, [35], [576], [64], [64], [26], [5], 0.6,
                        branching=[4, 2, 1, 1], gen_target=[128])
    if index == 3:
        rng = rng_for(3, 99)
        B = 16
        prompt = rng.integers(20, 201, size=B)
        before = [int(min(35, p)) for p in prompt]
        after = [int(p) - b for p, b in zip(prompt, before)]
        keep = [(64, 128, 192)[i % 3] for i in range(B)]
        n_nodes = [int(x) for x in rng.integers(16, 33, size=B)]
        depth = [int(x) for x in rng.integers(3, 7, size=B)]
        gen = [int(x) for x in rng.integers(30, 513, size=B)]
        return Workload(3, "c3-llava15-7b-b16-hetero", 32, B, 32, 32, 128, before, [576] * B, after, keep,
                        n_nodes, depth, 0.7, gen_target=gen)
    if index == 4:
        B = 4
        return Workload(4, "c4-hires-b4", 32, B, 32, 32, 128, [64] * B, [2880] * B, [64] * B, [320] * B,
                        [64] * B, [8] * B, 0.6, gen_target=[1088] * B, final_kv_len=1536 - 64)
    if index == 5:
        B = 8
        return Workload(5, "c5-gqa-b8-long", 28, B, 28, 4, 128, [128] * B, [1024] * B, [128] * B, [128] * B,
                        [64] * B, [6] * B, 0.65, gen_target=[8192 - 384] * B, final_kv_len=8192 - 64)
    raise ValueError("workload index must be 1..5")


def make_tree(wl: Workload, rng: np.random.Generator, b: int) -> np.ndarray:
    if wl.branching is not None:
        return fixed_branching_tree(wl.branching, wl.n_nodes[b])
    return random_tree(rng, wl.n_nodes[b], wl.depth_levels[b])


def make_prefill(wl: Workload, rng: np.random.Generator, n_layers: Optional[int] = None,
                 gain: float = 1.0) -> dict:
    """Twig-layer query/keys of the prompt and the base model's unpruned KV
    cache (all bf16 bit patterns), plus per-request layout metadata."""
    nl = wl.n_layers if n_layers is None else n_layers
    B, Hq, Hkv, d = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    lp = wl.prefix_len
    lmax = max(lp)
    out = {
        "twig_q": normal_bf16(rng, (B, Hq, d), d, gain),
        "twig_k": normal_bf16(rng, (B, Hkv, lmax, d), d, gain),
        "cache_k": normal_bf16(rng, (nl, B, Hkv, lmax, d), d, gain),
        "cache_v": normal_bf16(rng, (nl, B, Hkv, lmax, d), d, gain),
        "pos_ids": np.tile(np.arange(lmax, dtype=np.int32), (B, 1)),
        "prefix_len": np.asarray(lp, dtype=np.int32),
        "vis_start": np.asarray(wl.text_before, dtype=np.int32),
        "n_vis": np.asarray(wl.n_vis, dtype=np.int32),
        "keep": np.asarray(wl.keep, dtype=np.int32),
    }
    return out


def make_verify_inputs(wl: Workload, rng: np.random.Generator, n_layers: Optional[int] = None,
                       gain: float = 1.0, per_child: bool = False) -> dict:
    """One verification step's inputs: per-layer tree queries and tree K/V,
    the parent arrays (padded with -1 beyond n_nodes) and the token ids."""
    nl = wl.n_layers if n_layers is None else n_layers
    B, Hq, Hkv, d, T = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max
    parent = np.full((B, T), -1, dtype=np.int32)
    draft = np.zeros((B, T), dtype=np.int32)
    tgt = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        p = make_tree(wl, rng, b)
        n = len(p)
        parent[b, :n] = p
        dt, ba = draft_and_target_tokens(rng, p, wl.match_p, per_child=per_child)
        draft[b, :n] = dt
        tgt[b, :n] = ba
    return {
        "q": normal_bf16(rng, (nl, B, T, Hq, d), d, gain),
        "tree_k": normal_bf16(rng, (nl, B, Hkv, T, d), d, gain),
        "tree_v": normal_bf16(rng, (nl, B, Hkv, T, d), d, gain),
        "parent": parent,
        "n_nodes": np.asarray(wl.n_nodes, dtype=np.int32),
        "draft_tok": draft,
        "base_argmax": tgt,
    }


def make_cache(wl: Workload, rng: np.random.Generator, max_len: int, n_layers: Optional[int] = None,
               gain: float = 1.0):
    """A KV cache of random rows, [n_layers, B, H_kv, max_len, d] for K and V."""
    nl = wl.n_layers if n_layers is None else n_layers
    shape = (nl, wl.batch, wl.n_kv_heads, max_len, wl.head_dim)
    return normal_bf16(rng, shape, wl.head_dim, gain), normal_bf16(rng, shape, wl.head_dim, gain)
