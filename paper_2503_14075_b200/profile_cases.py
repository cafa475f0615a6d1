"""Small, self-contained launches of each kernel for profiling (ncu) or quick timing.

  python -m paper_2503_14075_b200.profile_cases attn   --workload 4 --kv-len 1472 --layers 4 --iters 3
  python -m paper_2503_14075_b200.profile_cases gather --workload 4 --layers 2 --iters 3
  python -m paper_2503_14075_b200.profile_cases score  --workload 4 --iters 3
  python -m paper_2503_14075_b200.profile_cases accept --workload 2 --layers 32 --iters 3
  python -m paper_2503_14075_b200.profile_cases argmax --workload 4 --iters 3
  python -m paper_2503_14075_b200.profile_cases gscore --workload 4 --iters 3
  python -m paper_2503_14075_b200.profile_cases mqscore --workload 4 --iters 3

Every case holds well under a few GB on the device and launches a handful of kernels, so
that a profiler capture ends by itself.  Prints the mean launch time from CUDA events.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import synth, twig as tw

DEV = "cuda:0"


def _bf(x):
    return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(DEV).view(torch.bfloat16)


def _i32(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)


def _time(fn, iters):
    stream = torch.cuda.current_stream()
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(iters):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters


def case_attn(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 900)
    L = a.kv_len or wl.final_kv_len or max(wl.pruned_len)
    nl = a.layers
    ck, cv = synth.make_cache(wl, rng, L + wl.t_max, n_layers=nl)
    ver = synth.make_verify_inputs(wl, rng, n_layers=nl)
    ck, cv = _bf(ck), _bf(cv)
    q, tk, tv = _bf(ver["q"]), _bf(ver["tree_k"]), _bf(ver["tree_v"])
    par, nn = _i32(ver["parent"]), _i32(ver["n_nodes"])
    kvl = torch.full((wl.batch,), L, dtype=torch.int32, device=DEV)
    out = torch.zeros((wl.batch, wl.t_max, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16, device=DEV)
    cache = tw.KV.of(ck, cv)
    tw.twig_set_attention_path(a.path)
    tw.twig_set_attention_splits(a.splits)

    def run():
        for layer in range(nl):
            tw.tree_verify_attention(q[layer], tk[layer], tv[layer], cache, layer, kvl, nn, par, out)
    us = _time(run, a.iters) / nl
    by = sum(wl.kv_row_bytes() * (L + n) + 2 * n * wl.n_q_heads * wl.head_dim * 2 + 8 * n for n in wl.n_nodes)
    print(f"attn path={a.path} {wl.name} L={L}: {us:.2f} us/launch, {by / us / 1e3:.1f} GB/s algorithmic ({by} B/launch)")


def case_gather(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 901)
    nl = a.layers
    pre = synth.make_prefill(wl, rng, n_layers=nl)
    B = wl.batch
    sk, sv = _bf(pre["cache_k"]), _bf(pre["cache_v"])
    dk = torch.zeros((nl, B, wl.n_kv_heads, max(wl.pruned_len) + 8, wl.head_dim), dtype=torch.bfloat16, device=DEV)
    dv = torch.zeros_like(dk)
    kept = np.full((B, max(1, max(wl.keep))), -1, dtype=np.int32)
    for b in range(B):
        kept[b, :wl.keep[b]] = np.sort(rng.choice(wl.n_vis[b], wl.keep[b], replace=False))
    args = (tw.KV.of(sk, sv), tw.KV.of(dk, dv), _i32(kept), _i32(pre["keep"]), _i32(pre["prefix_len"]),
            _i32(pre["vis_start"]), _i32(pre["n_vis"]))
    us = _time(lambda: tw.ttp_compact(*args), a.iters)
    by = 2 * sum(wl.pruned_len) * wl.kv_row_bytes() * nl
    print(f"gather {wl.name} {nl} layers: {us:.2f} us/launch, {by / us / 1e3:.1f} GB/s algorithmic ({by} B/launch)")


def case_score(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 902)
    pre = synth.make_prefill(wl, rng, n_layers=1)
    B = wl.batch
    q, k = _bf(pre["twig_q"]), _bf(pre["twig_k"])
    scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=DEV)
    kept = torch.zeros((B, max(wl.keep)), dtype=torch.int32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, wl.head_dim, k.shape[2], 64), dtype=torch.uint8,
                     device=DEV)
    pl, vs, nv, kp = _i32(pre["prefix_len"]), _i32(pre["vis_start"]), _i32(pre["n_vis"]), _i32(pre["keep"])

    def run():
        tw.ttp_score(q, k, pl, vs, nv, scores, ws)
        tw.ttp_topk(scores, nv, kp, kept)
    us = _time(run, a.iters)
    by = sum(wl.n_kv_heads * lp * wl.head_dim * 2 for lp in wl.prefix_len)
    print(f"score+topk {wl.name}: {us:.2f} us per (score, topk) pair; K bytes {by}")


def case_accept(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 903)
    nl = a.layers
    ver = synth.make_verify_inputs(wl, rng, n_layers=nl)
    B, T = wl.batch, wl.t_max
    ck = torch.zeros((nl, B, wl.n_kv_heads, 256 + T, wl.head_dim), dtype=torch.bfloat16, device=DEV)
    cv = torch.zeros_like(ck)
    cache = tw.KV.of(ck, cv)
    tk, tv = _bf(ver["tree_k"]), _bf(ver["tree_v"])
    par, nn = _i32(ver["parent"]), _i32(ver["n_nodes"])
    dt, ba = _i32(ver["draft_tok"]), _i32(ver["base_argmax"])
    kvl = torch.zeros(B, dtype=torch.int32, device=DEV)
    alen = torch.zeros(B, dtype=torch.int32, device=DEV)
    path = torch.zeros((B, T), dtype=torch.int32, device=DEV)
    bonus = torch.zeros(B, dtype=torch.int32, device=DEV)

    def run():
        kvl.fill_(100)
        tw.tree_accept_compact(par, dt, ba, nn, tk, tv, cache, kvl, alen, path, bonus)
    us = _time(run, a.iters)
    print(f"accept {wl.name} {nl} layers: {us:.2f} us per (fill, accept) pair")


def case_argmax(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 904)
    B, T, V = wl.batch, wl.t_max, a.vocab
    logits = torch.from_numpy(rng.standard_normal((B, T, V), dtype=np.float32)).to(DEV).to(torch.bfloat16)
    nn = _i32(wl.n_nodes)
    out = torch.zeros((B, T), dtype=torch.int32, device=DEV)
    us = _time(lambda: tw.tree_base_argmax(logits, nn, out), a.iters)
    by = sum(wl.n_nodes) * V * 2
    print(f"argmax {wl.name} V={V}: {us:.2f} us/launch, {by / us / 1e3:.1f} GB/s algorithmic ({by} B/launch)")


def case_gscore(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 905)
    pre = synth.make_prefill(wl, rng, n_layers=1)
    B = wl.batch
    q, k = _bf(pre["twig_q"]), _bf(pre["twig_k"])
    qg, kg = _bf(synth.gate_bf16(rng, pre["twig_q"].shape)), _bf(synth.gate_bf16(rng, pre["twig_k"].shape))
    scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, wl.head_dim, k.shape[2], 64), dtype=torch.uint8,
                     device=DEV)
    pl, vs, nv = _i32(pre["prefix_len"]), _i32(pre["vis_start"]), _i32(pre["n_vis"])
    us = _time(lambda: tw.ttp_score_gated(q, qg, k, kg, pl, vs, nv, scores, ws), a.iters)
    by = 2 * sum(wl.n_kv_heads * n * wl.head_dim * 2 for n in wl.n_vis)
    print(f"gated score {wl.name}: {us:.2f} us per call (2 kernels), {by / us / 1e3:.1f} GB/s algorithmic ({by} B)")


def case_mqscore(a):
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 906)
    pre = synth.make_prefill(wl, rng, n_layers=1)
    B, n_txt = wl.batch, max(1, max(wl.text_after))
    k = _bf(pre["twig_k"])
    qt = _bf(synth.normal_bf16(rng, (B, wl.n_q_heads, n_txt, wl.head_dim), wl.head_dim))
    scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=DEV)
    ws = torch.empty(tw.ttp_multiquery_workspace_bytes(B, wl.n_q_heads, n_txt, max(wl.n_vis)), dtype=torch.uint8, device=DEV)
    pl, vs, nv = _i32(pre["prefix_len"]), _i32(pre["vis_start"]), _i32(pre["n_vis"])
    us = _time(lambda: tw.ttp_score_multiquery(qt, k, pl, vs, nv, scores, ws), a.iters)
    fl = sum(2 * wl.n_q_heads * wl.head_dim * c * (t + 2 * n + (c + 1) / 2)
             for t, n, c in zip(wl.text_before, wl.n_vis, wl.text_after))
    print(f"multi-query score {wl.name}: {us:.2f} us per call (2 kernels), {fl / us / 1e6:.1f} TFLOP/s algorithmic")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["attn", "gather", "score", "accept", "argmax", "gscore", "mqscore"])
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--kv-len", type=int, default=0)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--vocab", type=int, default=32000)
    ap.add_argument("--splits", type=int, default=0, help="force key splits (0 auto)")
    ap.add_argument("--path", type=int, default=0, help="attention kernel: 0 auto, 1 mma.sync, 2 tcgen05")
    a = ap.parse_args()
    {"attn": case_attn, "gather": case_gather, "score": case_score, "accept": case_accept, "argmax": case_argmax, "gscore": case_gscore,
     "mqscore": case_mqscore}[a.case](a)


if __name__ == "__main__":
    main()
