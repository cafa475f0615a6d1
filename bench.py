#!/usr/bin/env python
"""Benchmark of the TwigVLM/TwigVLM++ inference hot path on B200.

One bench "step" is one pass of the whole path over one batch of synthetic
requests: twig-guided pruning of the prompt's KV cache (score, TopR, gather over
all layers), then the tree-verification loop until every request has emitted its
target number of tokens (tree attention in each of the layers + acceptance and
KV append per verify step).  The metric is tree-verify steps per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_14075_b200 import replicas, synth  # noqa: E402

METRIC = "tree_verify_steps_per_s"
UNIT = "verify steps/s"
N_ROT = 4          # request replicas visited round-robin so that no launch finds its KV in L2
POOL = 8           # distinct per-step Q / tree-K/V sets per replica (cycled)
MAX_STEPS = 110    # bound on verify steps per request
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel (tree_attn_kernel,
# c2 shape, kv_len 227); set to None whenever that kernel changes after the capture
ATTN_TRAFFIC_NCU = 4414464


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax = float(f[2])
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------
class Replica:
    """One request of the workload with all of its device buffers."""

    def __init__(self, wl, stream_id, torch, tw, dev, max_len):
        self.wl = wl
        rng = synth.rng_for(wl.index, stream_id)
        B, Hq, Hkv, d, T, nl = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max, wl.n_layers

        def bf(x):
            return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev).view(torch.bfloat16)

        def i32(x):
            return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(dev)

        pre = synth.make_prefill(wl, rng)
        self.host_twig = (pre["twig_q"], pre["twig_k"])
        self.twig_q, self.twig_k = bf(pre["twig_q"]), bf(pre["twig_k"])
        self.src_k, self.src_v = bf(pre["cache_k"]), bf(pre["cache_v"])
        del pre["cache_k"], pre["cache_v"]
        self.prefix_len, self.vis_start = i32(pre["prefix_len"]), i32(pre["vis_start"])
        self.n_vis, self.keep = i32(pre["n_vis"]), i32(pre["keep"])
        self.pos_in = i32(pre["pos_ids"])
        self.pos_out = torch.zeros_like(self.pos_in)
        self.dst_k = torch.zeros((nl, B, Hkv, max_len, d), dtype=torch.bfloat16, device=dev)
        self.dst_v = torch.zeros_like(self.dst_k)
        self.src = tw.KV.of(self.src_k, self.src_v)
        self.cache = tw.KV.of(self.dst_k, self.dst_v)
        self.scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=dev)
        self.kept = torch.zeros((B, max(wl.keep)), dtype=torch.int32, device=dev)
        self.kv_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.status = torch.zeros(B, dtype=torch.int32, device=dev)
        self.ws = torch.empty(tw.twig_workspace_bytes(B, Hq, d, self.twig_k.shape[2], T), dtype=torch.uint8,
                              device=dev)
        # verify-step inputs: a pool of Q / tree K,V sets, and token ids for every step
        self.pool_host, self.q, self.tree_k, self.tree_v = [], [], [], []
        for _ in range(POOL):
            ver = synth.make_verify_inputs(wl, rng)
            self.pool_host.append((ver["q"], ver["tree_k"], ver["tree_v"]))
            self.q.append(bf(ver["q"]))
            self.tree_k.append(bf(ver["tree_k"]))
            self.tree_v.append(bf(ver["tree_v"]))
        self.parent_host, self.n_nodes_host = ver["parent"], ver["n_nodes"]
        self.parent, self.n_nodes = i32(ver["parent"]), i32(ver["n_nodes"])
        draft = np.zeros((MAX_STEPS, B, T), dtype=np.int32)
        tgt = np.zeros_like(draft)
        for s in range(MAX_STEPS):
            for b in range(B):
                n = wl.n_nodes[b]
                draft[s, b, :n], tgt[s, b, :n] = synth.draft_and_target_tokens(rng, ver["parent"][b, :n], wl.match_p)
        self.draft_host, self.tgt_host = draft, tgt
        self.draft, self.tgt = i32(draft), i32(tgt)
        self.out = torch.zeros((B, T, Hq, d), dtype=torch.bfloat16, device=dev)
        self.accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.path = torch.zeros((B, T), dtype=torch.int32, device=dev)
        self.bonus = torch.zeros(B, dtype=torch.int32, device=dev)
        self.n_steps = MAX_STEPS
        self.early_prefix = True
        self.attn_kernel, self.attn_splits, self.plain_launch = 0, 0, False
        # scratch of the persistent attention kernel: zero-filled once, used by the attention calls only
        self.attn_ws = torch.zeros(tw.tree_attention_workspace_bytes(B, Hq, T), dtype=torch.uint8, device=dev)

    def prune(self, tw):
        tw.ttp_score_topk_compact(self.twig_q, self.twig_k, self.prefix_len, self.vis_start, self.n_vis, self.keep,
                                  self.scores, self.kept, self.src, self.cache, self.ws, pos_in=self.pos_in,
                                  pos_out=self.pos_out, new_len=self.kv_len, dev_status=self.status)

    def attention_layers(self, tw, s, kv_len=None, q_ready=False):
        """The step's attention launches; kv_len: the lengths to read (default: the live ones); q_ready:
        also promise that Q and the tree rows are final (true here, where they are inputs; not in a model)."""
        slot = s % POOL
        q, tk, tv = self.q[slot], self.tree_k[slot], self.tree_v[slot]
        kv_len = self.kv_len if kv_len is None else kv_len
        for layer in range(self.wl.n_layers):
            # layer 0 follows the accept (or prune) kernel, which writes kv_len; the other layers follow
            # the previous layer's attention, which leaves lengths and cache alone
            flags = tw.attn_flags(kernel=self.attn_kernel, splits=self.attn_splits, plain_launch=self.plain_launch,
                                  early_prefix=layer > 0 and self.early_prefix,
                                  early_query=q_ready and layer > 0 and self.early_prefix)
            tw.tree_verify_attention(q[layer], tk[layer], tv[layer], self.cache, layer, kv_len, self.n_nodes,
                                     self.parent, self.out, dev_status=self.status, ws=self.attn_ws, flags=flags)

    def accept(self, tw, s):
        slot = s % POOL
        tw.tree_accept_compact(self.parent, self.draft[s], self.tgt[s], self.n_nodes, self.tree_k[slot],
                               self.tree_v[slot], self.cache, self.kv_len, self.accept_len, self.path, self.bonus,
                               dev_status=self.status)


def attn_bytes_per_launch(wl, kv_len):
    """Algorithmic bytes of one tree-attention layer-call: K and V rows of the prefix and
    of the tree, Q read, O written, parent ids."""
    tot = 0
    for b in range(wl.batch):
        n = wl.n_nodes[b]
        tot += wl.kv_row_bytes() * (int(kv_len[b]) + n) + 2 * n * wl.n_q_heads * wl.head_dim * 2 + 8 * n
    return int(tot)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2503_14075_b200 import build as _build
    _build.build()
    from paper_2503_14075_b200 import twig as tw

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    wl = synth.workload(args.workload)
    peaks = load_peaks()
    tw.twig_set_launch_overlap(0 if args.no_overlap else 1)
    max_len = ((max(wl.pruned_len) + max(wl.gen_target) + wl.t_max + 8 + 31) // 32) * 32

    reps = [Replica(wl, sid, torch, tw, dev, max_len) for sid in replicas.replica_streams(rank, N_ROT)]
    for rp in reps:
        rp.early_prefix = not args.no_early_prefix
        rp.attn_kernel, rp.attn_splits = args.attn_path, args.attn_splits
    stream = torch.cuda.current_stream()

    # ---- dry run: how many verify steps each request needs to emit its target ------------
    for rp in reps:
        rp.prune(tw)
        emitted, s = np.zeros(wl.batch, dtype=np.int64), 0
        lens = []
        while s < MAX_STEPS and np.any(emitted < np.asarray(wl.gen_target)):
            lens.append(rp.kv_len.cpu().numpy().copy())
            rp.attention_layers(tw, s)
            rp.accept(tw, s)
            emitted += rp.accept_len.cpu().numpy() + 1
            s += 1
        rp.n_steps, rp.lens, rp.emitted = s, lens, int(emitted.sum())
        assert not rp.status.cpu().numpy().any(), "device status set"
    torch.cuda.synchronize()
    total_verify = sum(rp.n_steps for rp in reps)
    max_s = max(rp.n_steps for rp in reps)
    attn_launches = total_verify * wl.n_layers
    attn_bytes = sum(attn_bytes_per_launch(wl, l) for rp in reps for l in rp.lens) * wl.n_layers

    # ---- CUDA graphs: one per (replica, verify step); each layer stays its own launch ----
    graphs = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        graphs = [[None] * rp.n_steps for rp in reps]
        with torch.cuda.stream(side):
            for r, rp in enumerate(reps):
                for s in range(rp.n_steps):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        rp.attention_layers(tw, s)
                        rp.accept(tw, s)
                    graphs[r][s] = g
        torch.cuda.synchronize()

    ev_pairs = []

    def one_step(record=False):
        for rp in reps:
            rp.prune(tw)
        for s in range(max_s):
            for r, rp in enumerate(reps):
                if s >= rp.n_steps:
                    continue
                if record:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                if graphs is not None:
                    graphs[r][s].replay()
                else:
                    rp.attention_layers(tw, s)
                    rp.accept(tw, s)
                if record:
                    e1.record(stream)
                    ev_pairs.append((e0, e1))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record(stream)
    for _ in range(args.steps):
        one_step(record=True)
    t1.record(stream)
    barrier()
    clocks = sampler.stop()
    # whole-job value: work summed over the ranks, time of the slowest rank
    job_steps, ms = replicas.combine(total_verify * args.steps, t0.elapsed_time(t1), dev)
    verify_ms = sum(a.elapsed_time(b) for a, b in ev_pairs)          # attention x layers + accept, per verify step
    value = job_steps / (ms * 1e-3)

    # ---- dominant kernel alone ---------------------------------------------------------------------
    # (a) launched one by one: the attention launches of every verify step between two events
    for rp in reps:
        rp.prune(tw)
    att_pairs = []
    for s in range(max_s):
        for rp in reps:
            if s >= rp.n_steps:
                continue
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            rp.attention_layers(tw, s)
            e1.record(stream)
            rp.accept(tw, s)
            att_pairs.append((e0, e1))
    torch.cuda.synchronize()
    att_ms = sum(a.elapsed_time(b) for a, b in att_pairs)
    att_us_per_launch = att_ms * 1e3 / attn_launches
    # (b) inside graphs, as the timed loop runs them, but the attention launches ALONE: one graph per
    # (replica, verify step) with the step's layers only, each reading that step's own lengths (a
    # snapshot taken in the dry run), replayed in the timed loop's order so that no launch finds its
    # cache in L2.  This is the figure the roofline uses when graphs are on.
    graph_us_per_launch = graph_us_q_ready = None
    if graphs is not None:
        for rp in reps:
            rp.len_at = [torch.from_numpy(np.ascontiguousarray(l, dtype=np.int32)).to(dev) for l in rp.lens]
        def time_attention_graphs(q_ready):
            att_graphs = [[None] * rp.n_steps for rp in reps]
            with torch.cuda.stream(side):
                for r, rp in enumerate(reps):
                    for s in range(rp.n_steps):
                        g = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(g, stream=side):
                            rp.attention_layers(tw, s, kv_len=rp.len_at[s], q_ready=q_ready)
                        att_graphs[r][s] = g
            torch.cuda.synchronize()

            def attention_only():
                for s in range(max_s):
                    for r, rp in enumerate(reps):
                        if s < rp.n_steps:
                            att_graphs[r][s].replay()
            attention_only()
            torch.cuda.synchronize()
            n_att_rep = 3
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(n_att_rep):
                attention_only()
            a1.record(stream)
            torch.cuda.synchronize()
            return a0.elapsed_time(a1) * 1e3 / (n_att_rep * attn_launches)
        graph_us_per_launch = time_attention_graphs(False)
        # benchmark-only: every launch also promises that its Q and tree rows are final, so consecutive
        # layers overlap almost entirely; in a model a layer's Q depends on the layer before
        graph_us_q_ready = time_attention_graphs(True)
    use_us = graph_us_per_launch if graph_us_per_launch is not None else att_us_per_launch
    bytes_per_launch = attn_bytes / attn_launches
    achieved = bytes_per_launch / (use_us * 1e-6) / 1e9
    roofline = {"kernel": "tree_attn_kernel", "bound": "hbm", "achieved": round(achieved, 1),
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(achieved / peaks["hbm_gbs"], 4),
                "peak_source": peaks["source"], "traffic": ATTN_TRAFFIC_NCU,
                "traffic_note": "dram read+write bytes of one launch at kv_len 227 (algorithmic 4571344 B there), "
                                "from the ncu capture summarised in profiles/kernels_ncu_full.md",
                "bytes_per_launch": int(bytes_per_launch), "us_per_launch": round(use_us, 3),
                "us_per_launch_source": ("graphs of the attention launches alone, replayed in the timed loop's order"
                                         if graph_us_per_launch is not None else "launched one by one between events"),
                "us_per_launch_direct": round(att_us_per_launch, 3),
                "us_per_launch_in_graph": None if graph_us_per_launch is None else round(graph_us_per_launch, 3),
                "us_per_launch_in_graph_q_ready_benchmark_only": None if graph_us_q_ready is None else round(graph_us_q_ready, 3),
                "note": "one launch = one layer of one verify step (3.5-5.6 MB): launch-latency sized"}

    # ---- prune latency (the third quantity of the metric) --------------------------------------
    # One ttp_score_topk_compact over all layers.  Launched directly the host's launch time shows in the
    # figure (three launches of a few microseconds each), so the call is also captured in a graph per
    # replica and replayed; both are reported, the replayed one is the device-side latency.
    def time_prune(fn):
        pr = []
        for _ in range(5):
            for i in range(len(reps)):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn(i)
                e1.record(stream)
                pr.append((e0, e1))
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in pr) * 1e3
    prune_us_direct = time_prune(lambda i: reps[i].prune(tw))
    prune_us = prune_us_direct
    prune_us_plain = None
    if graphs is not None:
        def prune_graphs():
            gs = []
            with torch.cuda.stream(side):
                for rp in reps:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        rp.prune(tw)
                    gs.append(g)
            torch.cuda.synchronize()
            return gs
        pg = prune_graphs()
        prune_us = time_prune(lambda i: pg[i].replay())
        # the same with plain launches (no programmatic stream serialization): what the overlap of the
        # gather's text rows with scoring and selection is worth
        prev = tw.twig_set_launch_overlap(0)
        pg = prune_graphs()
        prune_us_plain = time_prune(lambda i: pg[i].replay())
        tw.twig_set_launch_overlap(prev)
        del pg
    prune_bytes = 2 * max(wl.pruned_len) * wl.kv_row_bytes() * wl.n_layers + \
        wl.n_kv_heads * max(wl.prefix_len) * wl.head_dim * 2

    # ---- end to end through the public API with host buffers -----------------------------------
    e2e = run_e2e(torch, tw, wl, reps, stream, world, dev, dist if world > 1 else None, graphs[0] if graphs else None)

    out = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": bench_config(wl, {
            "verify_steps_per_bench_step": total_verify,
            "tokens_emitted_per_bench_step": sum(rp.emitted for rp in reps),
            "launch_mode": "direct" if graphs is None else "cuda-graph per verify step, one launch per layer",
            "l2": f"inputs larger than L2: {N_ROT} request replicas round-robin, >= {3 * 113} MB touched "
                  "between two uses of a buffer"}),
        "clocks": clocks, "gpu_launches": args.steps * (3 * N_ROT + total_verify * (wl.n_layers + 1)),
        "e2e": e2e, "roofline": roofline,
        "verify_us_per_step": round(verify_ms * 1e3 / (args.steps * total_verify), 2),
        "ttp_prune_latency_us": round(prune_us, 2),
        "ttp_prune_latency_us_direct_launches": round(prune_us_direct, 2),
        "ttp_prune_latency_us_without_launch_overlap": None if prune_us_plain is None else round(prune_us_plain, 2),
        "ttp_prune_gbs": round(prune_bytes / (prune_us * 1e-6) / 1e9, 1),
        "tokens_per_s": round(sum(rp.emitted for rp in reps) * args.steps * world / (ms * 1e-3), 1),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl)
    if rank == 0 and world == 1 and args.extra:
        out["other_kernels"] = extra_rooflines(torch, tw, peaks, dev)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(torch, tw, wl, reps, stream, world, dev, dist, step_graphs):
    """Same loop through the public API, every verify step's inputs (Q, tree K/V of all
    layers, tree and token ids) copied from pinned host memory and its result (accept
    length, path, bonus token) read back before the next step.  The prompt's KV cache is
    device-resident state, like the model weights.  The step's kernels are launched as in the
    device-resident loop: the captured graph of the step (one launch per layer + accept) where
    graphs are in use, one by one otherwise."""
    rp = reps[0]
    pin = []
    for (q, tk, tv) in rp.pool_host:
        pin.append(tuple(torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).pin_memory() for x in (q, tk, tv)))
    tq_pin = tuple(torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).pin_memory() for x in rp.host_twig)
    par_pin = torch.from_numpy(rp.parent_host).pin_memory()
    draft_pin = torch.from_numpy(rp.draft_host).pin_memory()
    tgt_pin = torch.from_numpy(rp.tgt_host).pin_memory()
    res_pin = torch.zeros((wl.batch, 2 + wl.t_max), dtype=torch.int32).pin_memory()
    res_dev = torch.zeros((wl.batch, 2 + wl.t_max), dtype=torch.int32, device=dev)
    stage = (torch.empty_like(rp.q[0]), torch.empty_like(rp.tree_k[0]), torch.empty_like(rp.tree_v[0]))
    h2d = d2h = 0

    def request():
        nonlocal h2d, d2h
        h2d = d2h = 0
        rp.twig_q.view(torch.int16).copy_(tq_pin[0], non_blocking=True)
        rp.twig_k.view(torch.int16).copy_(tq_pin[1], non_blocking=True)
        h2d += tq_pin[0].numel() * 2 + tq_pin[1].numel() * 2
        rp.prune(tw)
        for s in range(rp.n_steps):
            slot = s % POOL
            # (with graphs the copies land in the buffers the step's graph reads)
            d_q, d_tk, d_tv = (rp.q[slot], rp.tree_k[slot], rp.tree_v[slot]) if step_graphs else stage
            d_q.view(torch.int16).copy_(pin[slot][0], non_blocking=True)
            d_tk.view(torch.int16).copy_(pin[slot][1], non_blocking=True)
            d_tv.view(torch.int16).copy_(pin[slot][2], non_blocking=True)
            rp.parent.copy_(par_pin, non_blocking=True)
            rp.draft[s].copy_(draft_pin[s], non_blocking=True)
            rp.tgt[s].copy_(tgt_pin[s], non_blocking=True)
            h2d += 2 * (d_q.numel() + d_tk.numel() + d_tv.numel()) + 4 * (par_pin.numel() + 2 * draft_pin[s].numel())
            if step_graphs:
                step_graphs[s].replay()
            else:
                for layer in range(wl.n_layers):
                    tw.tree_verify_attention(d_q[layer], d_tk[layer], d_tv[layer], rp.cache, layer, rp.kv_len,
                                             rp.n_nodes, rp.parent, rp.out, dev_status=rp.status, ws=rp.attn_ws,
                                             flags=tw.attn_flags(kernel=rp.attn_kernel, splits=rp.attn_splits))
                tw.tree_accept_compact(rp.parent, rp.draft[s], rp.tgt[s], rp.n_nodes, d_tk, d_tv, rp.cache, rp.kv_len,
                                       rp.accept_len, rp.path, rp.bonus, dev_status=rp.status)
            res_dev[:, 0] = rp.accept_len
            res_dev[:, 1] = rp.bonus
            res_dev[:, 2:] = rp.path
            res_pin.copy_(res_dev, non_blocking=True)
            stream.synchronize()               # the host needs the accepted tokens to draft the next tree
            d2h += res_pin.numel() * 4

    request()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    n_req = 3
    t0 = time.perf_counter()
    for _ in range(n_req):
        request()
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3            # wall clock: the host waits for every step's result
    if dist is not None:
        tt = torch.tensor([ms], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms = float(tt.item())
    return {"value": round(rp.n_steps * n_req * world / (ms * 1e-3), 1), "unit": UNIT,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "timer": "host wall clock (time.perf_counter) around the requests",
            "note": "per bench step = one request; Q and tree K/V of all layers cross PCIe every verify step; "
                    + ("kernels replayed from the step's graph" if step_graphs else "kernels launched one by one")}


L2_BYTES = 126 * 1024 * 1024


def _time_attention(torch, tw, wl, kv_lens, nl, stream_id, dev, reps=20, kernel=0, early_prefix=False, splits=0):
    """Launch time (us: median and best over `reps` timed passes) of tree_verify_attention over `nl`
    resident layers visited in turn (nl = 0: as many as it takes for their KV to exceed twice the L2,
    so that no launch finds its cache in L2), plus the algorithmic bytes and flops of one launch.
    kernel: 0 automatic, 1 mma.sync, 2 tcgen05 with cluster splits, 3 persistent tcgen05."""
    rng = synth.rng_for(wl.index, stream_id)
    B, Hq, Hkv, d, T = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max
    by = attn_bytes_per_launch(wl, kv_lens)
    if nl <= 0:
        nl = int(min(40, max(2, -(-2 * L2_BYTES // by))))

    def bf(x):
        return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev).view(torch.bfloat16)

    ck, cv = synth.make_cache(wl, rng, max(kv_lens) + T, n_layers=nl)
    ck, cv = bf(ck), bf(cv)
    ver = synth.make_verify_inputs(wl, rng, n_layers=nl)
    q, tk, tv = bf(ver["q"]), bf(ver["tree_k"]), bf(ver["tree_v"])
    par = torch.from_numpy(ver["parent"]).to(dev)
    nn = torch.from_numpy(ver["n_nodes"]).to(dev)
    kvl = torch.from_numpy(np.asarray(kv_lens, dtype=np.int32)).to(dev)
    out = torch.zeros((B, T, Hq, d), dtype=torch.bfloat16, device=dev)
    ws = torch.zeros(tw.tree_attention_workspace_bytes(B, Hq, T), dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    cache = tw.KV.of(ck, cv)
    stream = torch.cuda.current_stream()
    # nothing but these launches runs in the stream, so the early-prefix promise holds for every launch
    flags = tw.attn_flags(kernel=kernel, early_prefix=early_prefix, splits=splits)

    def loop():
        for layer in range(nl):
            tw.tree_verify_attention(q[layer], tk[layer], tv[layer], cache, layer, kvl, nn, par, out,
                                     dev_status=status, ws=ws, flags=flags)
    for _ in range(3):
        loop()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    evs[0].record(stream)
    for r in range(reps):
        loop()
        evs[r + 1].record(stream)
    torch.cuda.synchronize()
    assert not status.cpu().numpy().any(), "device status set"
    per = sorted(evs[r].elapsed_time(evs[r + 1]) * 1e3 / nl for r in range(reps))
    flops = sum(4 * Hq * n * d * (int(l) + n) for n, l in zip(wl.n_nodes, kv_lens))
    return {"us": statistics.median(per), "us_best": per[0], "bytes": by, "flops": flops, "layers": nl, "reps": reps}


def extra_rooflines(torch, tw, peaks, dev):
    """HBM-sized launches of the bandwidth kernels on the larger configurations: tree attention
    for the heterogeneous batch (c3), the high-resolution shape (c4) and the GQA long-context
    shape (c5, tensor bound), and the pruning gather of c4."""
    res = {}

    def bf(x):
        return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev).view(torch.bfloat16)

    def hbm_entry(us, by):
        return {"bound": "hbm", "bytes_per_launch": by, "us_per_launch": round(us, 2),
                "achieved": round(by / us / 1e3, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(by / us / 1e3 / peaks["hbm_gbs"], 4)}

    def attn_entry(t, bound="hbm"):
        """Median of the timed passes is the figure; the best pass and, where the call was also timed
        with the early-prefix promise (the launches of a verification step other than its first may make
        it), that figure are reported beside it."""
        us, by, fl = t["us"], t["bytes"], t["flops"]
        e = hbm_entry(us, by)
        if bound == "tensor":
            e = {"bound": "tensor", "flops_per_launch": fl, "bytes_per_launch": by, "us_per_launch": round(us, 2),
                 "achieved": round(fl / us / 1e6, 1), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                 "frac": round(fl / us / 1e6 / peaks["bf16_tflops"], 4), "hbm_gbs": round(by / us / 1e3, 1)}
        e.update({"us_best": round(t["us_best"], 2), "reps": t["reps"], "layers_in_rotation": t["layers"]})
        return e

    def attn_both(wl_, lens_, sid, bound="hbm"):
        e = attn_entry(_time_attention(torch, tw, wl_, lens_, 0, sid, dev), bound)
        t2 = _time_attention(torch, tw, wl_, lens_, 0, sid, dev, early_prefix=True)
        e["us_per_launch_early_prefix"] = round(t2["us"], 2)
        num = t2["flops"] / 1e6 if bound == "tensor" else t2["bytes"] / 1e3
        e["frac_early_prefix"] = round(num / t2["us"] / (peaks["bf16_tflops"] if bound == "tensor" else peaks["hbm_gbs"]), 4)
        return e

    # c2's third launch mode: ONE launch for all 32 layers of a verify step, the layers standing in as
    # 32 requests of a batch (same shapes, same bytes: 32 x 4.6 MB).  Benchmark only: in a model layer l+1
    # needs layer l's output, so the layers cannot share a launch.
    wl2 = synth.workload(2)
    nl2 = wl2.n_layers
    wl2x = synth.Workload(2, "c2-all-layers-as-batch", 1, nl2, wl2.n_q_heads, wl2.n_kv_heads, wl2.head_dim,
                          wl2.text_before * nl2, wl2.n_vis * nl2, wl2.text_after * nl2, wl2.keep * nl2,
                          wl2.n_nodes * nl2, wl2.depth_levels * nl2, wl2.match_p, branching=wl2.branching)
    e = attn_entry(_time_attention(torch, tw, wl2x, [227] * nl2, 0, 505, dev))
    e["note"] = "benchmark-only: the 32 layers of one verify step as one launch (real layers depend on each other)"
    e["us_per_layer"] = round(e["us_per_launch"] / nl2, 3)
    res["tree_attn_c2_all_layers_one_launch"] = e

    wl3 = synth.workload(3)
    lens3 = [p + g // 2 for p, g in zip(wl3.pruned_len, wl3.gen_target)]      # half-way through generation
    res["tree_attn_c3_midway"] = attn_both(wl3, lens3, 501)
    wl = synth.workload(4)
    B, Hq, Hkv, d, T = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max
    res["tree_attn_c4_L1472"] = attn_both(wl, [wl.final_kv_len] * B, 500)
    # the same shape with a long cache (beyond the configuration's 1.5k): the kernel's steady state
    res["tree_attn_c4shape_L8128"] = attn_entry(_time_attention(torch, tw, wl, [8128] * B, 0, 504, dev))
    wl5 = synth.workload(5)
    for L5 in (384, 2048, wl5.final_kv_len):
        res[f"tree_attn_c5_L{L5}"] = attn_entry(_time_attention(torch, tw, wl5, [L5] * wl5.batch, 0, 502, dev), "tensor")
    rng = synth.rng_for(4, 503)
    stream = torch.cuda.current_stream()
    # pruning gather, 2 layers at a time of the B=4 x 3008-token prompt cache.  A chain of launches over
    # rotating source / destination sets: every read is cold (a source set is 394 MB) and the
    # write-backs of earlier launches' destinations are paid inside the timed region.
    nl, n_sets = 2, 3
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)  # noqa: E731
    pre = synth.make_prefill(wl, rng, n_layers=nl)
    kept = np.stack([np.sort(rng.choice(wl.n_vis[b], wl.keep[b], replace=False)) for b in range(B)]).astype(np.int32)
    meta = (i32(kept), i32(pre["keep"]), i32(pre["prefix_len"]), i32(pre["vis_start"]), i32(pre["n_vis"]))
    sets = []
    for i in range(n_sets):
        sk, sv = bf(pre["cache_k"]), bf(pre["cache_v"])
        if i:
            sk, sv = sk.roll(i, dims=3), sv.roll(i, dims=3)
        dk = torch.zeros((nl, B, Hkv, max(wl.pruned_len) + 8, d), dtype=torch.bfloat16, device=dev)
        sets.append((tw.KV.of(sk, sv), tw.KV.of(dk, torch.zeros_like(dk))))
    del pre
    n_chain = 12
    for i in range(n_sets):
        tw.ttp_compact(sets[i][0], sets[i][1], *meta)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(n_chain):
        tw.ttp_compact(sets[i % n_sets][0], sets[i % n_sets][1], *meta)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n_chain
    by = 2 * sum(wl.pruned_len) * wl.kv_row_bytes() * nl
    # the same compaction in place (dst = src): only rows after the first dropped token move; the
    # prompt caches are restored by a copy before each timed launch (outside the events)
    us_ip = []
    for i in range(6):
        srcs = sets[i % n_sets][0]
        backup_k, backup_v = srcs._keep[0].clone(), srcs._keep[1].clone()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        tw.ttp_compact(srcs, srcs, *meta)
        a1.record(stream)
        torch.cuda.synchronize()
        us_ip.append(a0.elapsed_time(a1) * 1e3)
        srcs._keep[0].copy_(backup_k)
        srcs._keep[1].copy_(backup_v)
        del backup_k, backup_v
    moved = 2 * sum(int((np.arange(wl.pruned_len[b]) != np.concatenate([np.arange(wl.text_before[b]), wl.text_before[b] + kept[b],
                    np.arange(wl.text_before[b] + wl.n_vis[b], wl.prefix_len[b])])).sum()) for b in range(B)) * wl.kv_row_bytes() * nl
    us_med = statistics.median(us_ip[1:])
    res["kv_gather_in_place_c4_2layers"] = {"bound": "hbm", "bytes_per_launch": int(moved), "us_per_launch": round(us_med, 2),
                                            "achieved": round(moved / us_med / 1e3, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                            "frac": round(moved / us_med / 1e3 / peaks["hbm_gbs"], 4),
                                            "note": "single launches on a cold cache; bytes = rows that move (read + write)"}
    res["kv_gather_c4_2layers"] = {"bound": "hbm", "bytes_per_launch": by, "us_per_launch": round(us, 2),
                                   "achieved": round(by / us / 1e3, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": round(by / us / 1e3 / peaks["hbm_gbs"], 4),
                                   "l2": f"chain of {n_chain} launches over {n_sets} rotating 394 MB source sets"}
    del sets
    # P-Head score with its gates applied in the kernel (Eq. 7) on the high-resolution prompts: K and the
    # key gates are each read once (2 x 98.6 MB, larger than L2 together), logits go through the scratch
    pre4 = synth.make_prefill(wl, rng, n_layers=1)
    q4, k4 = bf(pre4["twig_q"]), bf(pre4["twig_k"])
    qg4, kg4 = bf(synth.gate_bf16(rng, pre4["twig_q"].shape)), bf(synth.gate_bf16(rng, pre4["twig_k"].shape))
    sc4 = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=dev)
    ws4 = torch.empty(tw.twig_workspace_bytes(B, Hq, d, k4.shape[2], T), dtype=torch.uint8, device=dev)
    m4 = (i32(pre4["prefix_len"]), i32(pre4["vis_start"]), i32(pre4["n_vis"]))
    for _ in range(3):
        tw.ttp_score_gated(q4, qg4, k4, kg4, *m4, sc4, ws4)
    e0.record(stream)
    for _ in range(n_chain):
        tw.ttp_score_gated(q4, qg4, k4, kg4, *m4, sc4, ws4)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n_chain
    res["ttp_score_gated_c4"] = hbm_entry(us, int(2 * sum(Hkv * n * d * 2 for n in wl.n_vis)))
    res["ttp_score_gated_c4"]["launches"] = "logits + softmax/mean (2 kernels)"
    # multi-query guide of Eq. 3 on the same prompts: every text token after the image against the whole
    # prompt (K once per kv head is the algorithmic traffic; the two passes of the query blocks re-read it from L2)
    n_txt = max(wl.text_after)
    qt4 = bf(synth.normal_bf16(rng, (B, Hq, n_txt, d), d))
    wsm = torch.empty(tw.ttp_multiquery_workspace_bytes(B, Hq, n_txt, max(wl.n_vis), k4.shape[2]), dtype=torch.uint8, device=dev)
    for _ in range(3):
        tw.ttp_score_multiquery(qt4, k4, *m4, sc4, wsm)
    e0.record(stream)
    for _ in range(n_chain):
        tw.ttp_score_multiquery(qt4, k4, *m4, sc4, wsm)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n_chain
    # per head and text token i: the products with its a + n + i + 1 keys, formed once; a kernel that walks the
    # keys twice (statistics, then probabilities) forms the n visual products a second time
    fl = sum(2 * Hq * d * c * (a + n + (c + 1) / 2) for a, n, c in zip(wl.text_before, wl.n_vis, wl.text_after))
    fl2 = sum(2 * Hq * d * c * (a + 2 * n + (c + 1) / 2) for a, n, c in zip(wl.text_before, wl.n_vis, wl.text_after))
    res["ttp_score_multiquery_c4"] = hbm_entry(us, int(sum(Hkv * p * d * 2 for p in wl.prefix_len)))
    res["ttp_score_multiquery_c4"].update({"text_tokens": n_txt, "flops_per_launch": int(fl),
                                           "tflops": round(fl / us / 1e6, 1),
                                           "flops_two_pass_equivalent": int(fl2),
                                           "tflops_two_pass_equivalent": round(fl2 / us / 1e6, 1),
                                           "launches": "probabilities (tcgen05) + column sums + reduce (3 kernels)"})
    del pre4, q4, k4, qg4, kg4, qt4
    # greedy target token per tree node over the heterogeneous batch's trees (32000-entry bf16 rows);
    # six logits buffers in turn, 190 MB together, so that every read is cold
    V = 32000
    nn3 = i32(wl3.n_nodes)
    bufs = [torch.randn((wl3.batch, wl3.t_max, V), dtype=torch.bfloat16, device=dev) for _ in range(6)]
    arg = torch.zeros((wl3.batch, wl3.t_max), dtype=torch.int32, device=dev)
    for bfr in bufs:
        tw.tree_base_argmax(bfr, nn3, arg)
    e0.record(stream)
    for i in range(n_chain):
        tw.tree_base_argmax(bufs[i % 6], nn3, arg)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n_chain
    res["base_argmax_c3_V32000"] = hbm_entry(us, int(sum(wl3.n_nodes)) * V * 2)
    # the same chain replayed from a CUDA graph: what the device needs when the host is not in the way
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for bfr in bufs:
                tw.tree_base_argmax(bfr, nn3, arg)
    torch.cuda.synchronize()
    g.replay()
    reps = max(1, n_chain // 6)
    e0.record(stream)
    for _ in range(reps):
        g.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    us_g = e0.elapsed_time(e1) * 1e3 / (6 * reps)
    res["base_argmax_c3_V32000"]["us_per_launch_in_graph"] = round(us_g, 2)
    res["base_argmax_c3_V32000"]["frac_in_graph"] = round(int(sum(wl3.n_nodes)) * V * 2 / us_g / 1e3 / peaks["hbm_gbs"], 4)
    # draft-side token tree with the paper's settings (E = K = 10, D = 4, N_max = 60) for the heterogeneous
    # batch: 4 expansions (1 + 3 x 10 draft rows of 32000 bf16 logits per request), 3 selections, 1 pruning;
    # three sets of logits in turn (95 MB together with the argmax buffers evicted: cold reads)
    E_, K_, D_, NMAX = 10, 10, 4, 60
    Bt = wl3.batch
    cap = 1 + E_ + (D_ - 1) * K_ * E_
    state = tw.TreeState(Bt, cap, dev)
    lsets = [[torch.randn((Bt, 1 if l == 0 else K_, V), dtype=torch.bfloat16, device=dev) for l in range(D_)]
             for _ in range(3)]
    t_par = torch.zeros((Bt, 64), dtype=torch.int32, device=dev)
    t_tok, t_n = torch.zeros_like(t_par), torch.zeros(Bt, dtype=torch.int32, device=dev)
    root = torch.zeros((Bt, 1), dtype=torch.int32, device=dev)
    nxt = torch.zeros((Bt, K_), dtype=torch.int32, device=dev)

    def build_tree_calls(logit_levels):
        tw.tree_reset(state)
        src, lo, hi = root, 0, 1
        for l in range(D_):
            tw.tree_expand_level(logit_levels[l], src, E_, hi, state)
            lo, hi = hi, hi + (1 if l == 0 else K_) * E_
            if l + 1 < D_:
                tw.tree_select_expansion(state, lo, hi, nxt)
                src = nxt
        tw.tree_finalize(state, cap, NMAX, t_par, t_tok, t_n)

    def build_tree(logit_levels):
        # one launch per level: the level's last CTA of each request selects / prunes
        src, hi = root, 1
        for l in range(D_):
            if l + 1 < D_:
                tw.tree_grow_level(logit_levels[l], src, E_, hi, state, expand_node=nxt)
                src = nxt
            else:
                tw.tree_grow_level(logit_levels[l], src, E_, hi, state, n_max=NMAX, parent=t_par, draft_tok=t_tok,
                                   n_nodes=t_n)
            hi += (1 if l == 0 else K_) * E_

    def timed(fn):
        for ls in lsets:
            fn(ls)
        e0.record(stream)
        for i in range(n_chain):
            fn(lsets[i % 3])
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n_chain

    tree_bytes = int(Bt * (1 + (D_ - 1) * K_) * V * 2)
    us = timed(build_tree)
    res["tree_build_c3_E10_K10_D4"] = hbm_entry(us, tree_bytes)
    res["tree_build_c3_E10_K10_D4"]["launches"] = "4 (one per level: expansion + selection / pruning), launched one by one"
    # the same trees replayed from a CUDA graph (no host time between the launches)
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for ls in lsets:
                build_tree(ls)
    torch.cuda.synchronize()
    g.replay()
    e0.record(stream)
    for _ in range(max(1, n_chain // 3)):
        g.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    res["tree_build_c3_E10_K10_D4"]["us_per_tree_batch_in_graph"] = round(
        e0.elapsed_time(e1) * 1e3 / (3 * max(1, n_chain // 3)), 2)
    us = timed(build_tree_calls)
    res["tree_build_c3_E10_K10_D4_separate_calls"] = hbm_entry(us, tree_bytes)
    res["tree_build_c3_E10_K10_D4_separate_calls"]["launches"] = "1 reset + 4 expansions + 3 selections + 1 pruning, launched one by one"
    return res


# ----------------------------------------------------------------------------------
# single-kernel cases: small, self-contained launch sets for a profiler capture or a quick timing
#   python bench.py --case attn --workload 4 --kv-len 1472 --layers 2 --iters 3 [--attn-path 3] [--early-prefix]
#   python bench.py --case gather|score|accept|argmax|tree|gscore|mqscore --workload N [--layers n] [--iters k]
# Each holds well under a few GB on the device and launches a handful of kernels, so that a
# capture ends by itself.  Prints one JSON line.
# ----------------------------------------------------------------------------------
def run_case(a):
    import torch
    from paper_2503_14075_b200 import build as _build
    _build.build()
    from paper_2503_14075_b200 import twig as tw
    dev = "cuda:0"
    torch.cuda.set_device(0)
    wl = synth.workload(a.workload)
    rng = synth.rng_for(a.workload, 900)
    B, Hq, Hkv, d, T = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.t_max

    def bf(x):
        return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev).view(torch.bfloat16)

    def i32(x):
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(dev)

    def timed(fn):
        stream = torch.cuda.current_stream()
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(a.iters):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / a.iters

    out = {"case": a.case, "workload": wl.name}
    if a.case == "attn":
        if a.kv_len:
            lens = [a.kv_len] * B
        elif wl.index == 3:
            lens = [p + g // 2 for p, g in zip(wl.pruned_len, wl.gen_target)]
        else:
            lens = [wl.final_kv_len or max(wl.pruned_len)] * B
        t = _time_attention(torch, tw, wl, lens, a.layers, 900, dev, reps=a.iters, kernel=a.attn_path,
                            early_prefix=a.early_prefix, splits=a.attn_splits)
        out.update({"kernel": a.attn_path, "early_prefix": a.early_prefix, "kv_len": lens[0] if a.kv_len else "workload",
                    "us_per_launch": round(t["us"], 2), "us_best": round(t["us_best"], 2), "bytes_per_launch": t["bytes"],
                    "gbs": round(t["bytes"] / t["us"] / 1e3, 1), "tflops": round(t["flops"] / t["us"] / 1e6, 1),
                    "layers": t["layers"]})
    elif a.case == "gather":
        nl = a.layers or 2
        pre = synth.make_prefill(wl, rng, n_layers=nl)
        sk, sv = bf(pre["cache_k"]), bf(pre["cache_v"])
        kept = np.full((B, max(1, max(wl.keep))), -1, dtype=np.int32)
        for b in range(B):
            kept[b, :wl.keep[b]] = np.sort(rng.choice(wl.n_vis[b], wl.keep[b], replace=False))
        meta = (i32(kept), i32(pre["keep"]), i32(pre["prefix_len"]), i32(pre["vis_start"]), i32(pre["n_vis"]))
        if a.in_place:
            src = tw.KV.of(sk, sv)
            us = timed(lambda: tw.ttp_compact(src, src, *meta))
        else:
            dk = torch.zeros((nl, B, Hkv, max(wl.pruned_len) + 8, d), dtype=torch.bfloat16, device=dev)
            src, dst = tw.KV.of(sk, sv), tw.KV.of(dk, torch.zeros_like(dk))
            us = timed(lambda: tw.ttp_compact(src, dst, *meta))
        by = 2 * sum(wl.pruned_len) * wl.kv_row_bytes() * nl
        out.update({"layers": nl, "in_place": a.in_place, "us_per_launch": round(us, 2), "bytes_per_launch": by,
                    "gbs": round(by / us / 1e3, 1)})
    elif a.case in ("score", "gscore", "mqscore", "prune"):
        nl = (a.layers or wl.n_layers) if a.case == "prune" else 1
        pre = synth.make_prefill(wl, rng, n_layers=nl)
        q, k = bf(pre["twig_q"]), bf(pre["twig_k"])
        scores = torch.zeros((B, max(wl.n_vis)), dtype=torch.float32, device=dev)
        kept = torch.zeros((B, max(wl.keep)), dtype=torch.int32, device=dev)
        ws = torch.empty(tw.twig_workspace_bytes(B, Hq, d, k.shape[2], 64), dtype=torch.uint8, device=dev)
        pl, vs, nv, kp = i32(pre["prefix_len"]), i32(pre["vis_start"]), i32(pre["n_vis"]), i32(pre["keep"])
        if a.case == "score":
            def run():
                tw.ttp_score(q, k, pl, vs, nv, scores, ws)
                tw.ttp_topk(scores, nv, kp, kept)
            us = timed(run)
            out.update({"us_per_score_topk_pair": round(us, 2),
                        "k_bytes": int(sum(Hkv * lp * d * 2 for lp in wl.prefix_len))})
        elif a.case == "prune":
            sk, sv = bf(pre["cache_k"]), bf(pre["cache_v"])
            dk = torch.zeros((nl, B, Hkv, max(wl.pruned_len) + 8, d), dtype=torch.bfloat16, device=dev)
            src, dst = tw.KV.of(sk, sv), tw.KV.of(dk, torch.zeros_like(dk))
            us = timed(lambda: tw.ttp_score_topk_compact(q, k, pl, vs, nv, kp, scores, kept, src, dst, ws))
            out.update({"layers": nl, "us_per_call": round(us, 2)})
        elif a.case == "gscore":
            qg, kg = bf(synth.gate_bf16(rng, pre["twig_q"].shape)), bf(synth.gate_bf16(rng, pre["twig_k"].shape))
            us = timed(lambda: tw.ttp_score_gated(q, qg, k, kg, pl, vs, nv, scores, ws))
            by = 2 * sum(Hkv * n * d * 2 for n in wl.n_vis)
            out.update({"us_per_call": round(us, 2), "bytes": int(by), "gbs": round(by / us / 1e3, 1)})
        else:
            n_txt = max(1, max(wl.text_after))
            qt = bf(synth.normal_bf16(rng, (B, Hq, n_txt, d), d))
            wsm = torch.empty(tw.ttp_multiquery_workspace_bytes(B, Hq, n_txt, max(wl.n_vis), k.shape[2]), dtype=torch.uint8, device=dev)
            us = timed(lambda: tw.ttp_score_multiquery(qt, k, pl, vs, nv, scores, wsm))
            fl = sum(2 * Hq * d * c * (t + n + (c + 1) / 2) for t, n, c in zip(wl.text_before, wl.n_vis, wl.text_after))
            fl2 = sum(2 * Hq * d * c * (t + 2 * n + (c + 1) / 2) for t, n, c in zip(wl.text_before, wl.n_vis, wl.text_after))
            out.update({"us_per_call": round(us, 2), "tflops": round(fl / us / 1e6, 1),
                        "tflops_two_pass_equivalent": round(fl2 / us / 1e6, 1)})
    elif a.case == "accept":
        nl = a.layers or wl.n_layers
        ver = synth.make_verify_inputs(wl, rng, n_layers=nl)
        ck = torch.zeros((nl, B, Hkv, 256 + T, d), dtype=torch.bfloat16, device=dev)
        cache = tw.KV.of(ck, torch.zeros_like(ck))
        tk, tv = bf(ver["tree_k"]), bf(ver["tree_v"])
        par, nn = i32(ver["parent"]), i32(ver["n_nodes"])
        dt, ba = i32(ver["draft_tok"]), i32(ver["base_argmax"])
        kvl = torch.zeros(B, dtype=torch.int32, device=dev)
        alen, bonus = torch.zeros(B, dtype=torch.int32, device=dev), torch.zeros(B, dtype=torch.int32, device=dev)
        path = torch.zeros((B, T), dtype=torch.int32, device=dev)

        def run():
            kvl.fill_(100)
            tw.tree_accept_compact(par, dt, ba, nn, tk, tv, cache, kvl, alen, path, bonus)
        out.update({"layers": nl, "us_per_fill_accept_pair": round(timed(run), 2)})
    elif a.case == "argmax":
        V = 32000
        logits = torch.from_numpy(rng.standard_normal((B, T, V), dtype=np.float32)).to(dev).to(torch.bfloat16)
        nn = i32(wl.n_nodes)
        res = torch.zeros((B, T), dtype=torch.int32, device=dev)
        us = timed(lambda: tw.tree_base_argmax(logits, nn, res))
        by = sum(wl.n_nodes) * V * 2
        out.update({"us_per_launch": round(us, 2), "bytes": int(by), "gbs": round(by / us / 1e3, 1)})
    elif a.case == "tree":
        # the paper's tree settings (E = K = 10, D = 4, N_max = 60), one launch per level
        V, E_, K_, D_, NMAX = 32000, 10, 10, 4, 60
        cap = 1 + E_ + (D_ - 1) * K_ * E_
        state = tw.TreeState(B, cap, dev)
        levels = [torch.from_numpy(rng.standard_normal((B, 1 if l == 0 else K_, V), dtype=np.float32)).to(dev).to(torch.bfloat16)
                  for l in range(D_)]
        t_par = torch.zeros((B, 64), dtype=torch.int32, device=dev)
        t_tok, t_n = torch.zeros_like(t_par), torch.zeros(B, dtype=torch.int32, device=dev)
        root = torch.zeros((B, 1), dtype=torch.int32, device=dev)
        nxt = torch.zeros((B, K_), dtype=torch.int32, device=dev)

        def run():
            src, hi = root, 1
            for l in range(D_):
                if l + 1 < D_:
                    tw.tree_grow_level(levels[l], src, E_, hi, state, expand_node=nxt)
                    src = nxt
                else:
                    tw.tree_grow_level(levels[l], src, E_, hi, state, n_max=NMAX, parent=t_par, draft_tok=t_tok, n_nodes=t_n)
                hi += (1 if l == 0 else K_) * E_
        out.update({"us_per_tree_batch": round(timed(run), 2), "launches_per_tree_batch": D_})
    print(json.dumps(out))


# ----------------------------------------------------------------------------------
# CPU oracle arm
# ----------------------------------------------------------------------------------
def oracle_verify_steps(wl, host, n_steps, n_layers):
    """Runs the oracle: prune (all `n_layers`), then `n_steps` verify steps.  Returns seconds
    spent in the verify steps and in the prune."""
    from oracle import twig_oracle as O
    f64 = synth.bf16_to_f64
    pre, vers, draft, tgt = host["pre"], host["vers"], host["draft"], host["tgt"]
    B, Hkv, d, T = wl.batch, wl.n_kv_heads, wl.head_dim, wl.t_max
    max_len = max(wl.pruned_len) + n_steps * T + 8
    t0 = time.perf_counter()
    s = O.ttp_scores(f64(pre["twig_q"]), f64(pre["twig_k"]), pre["prefix_len"], pre["vis_start"], pre["n_vis"])
    kept = [O.topk_lowest_index(s[b, :wl.n_vis[b]], wl.keep[b]).tolist() for b in range(B)]
    ck = np.zeros((n_layers, B, Hkv, max_len, d), dtype=np.uint16)
    cv = ck.copy()
    pos = np.zeros_like(pre["pos_ids"])
    kv_len = O.gather_compact(pre["cache_k"][:n_layers], pre["cache_v"][:n_layers], pre["pos_ids"], pre["prefix_len"],
                              pre["vis_start"], pre["n_vis"], kept, ck, cv, pos)
    t_prune = time.perf_counter() - t0
    t0 = time.perf_counter()
    for st in range(n_steps):
        ver = vers[st % len(vers)]
        rows = int(max(kv_len))                      # only the rows in use are widened to fp64
        for layer in range(n_layers):
            O.tree_attention(f64(ver["q"][layer]), f64(ver["tree_k"][layer]), f64(ver["tree_v"][layer]),
                             f64(ck[layer][:, :, :rows]), f64(cv[layer][:, :, :rows]), kv_len, ver["n_nodes"], ver["parent"])
        paths = []
        for b in range(B):
            _, p, _ = O.tree_accept(ver["parent"][b], draft[st][b], tgt[st][b], wl.n_nodes[b])
            paths.append(p.tolist())
        kv_len = O.accept_compact(ver["tree_k"][:n_layers], ver["tree_v"][:n_layers], ck, cv, kv_len, paths)
    return time.perf_counter() - t0, t_prune


def oracle_host_inputs(wl, n_pool=2, n_tok=16, stream_id=100):
    rng = synth.rng_for(wl.index, stream_id)
    pre = synth.make_prefill(wl, rng)
    vers = [synth.make_verify_inputs(wl, rng) for _ in range(n_pool)]
    draft, tgt = [], []
    for _ in range(n_tok):
        dd = np.zeros((wl.batch, wl.t_max), dtype=np.int32)
        tt = np.zeros_like(dd)
        for b in range(wl.batch):
            n = wl.n_nodes[b]
            dd[b, :n], tt[b, :n] = synth.draft_and_target_tokens(rng, vers[0]["parent"][b, :n], wl.match_p)
        draft.append(dd)
        tgt.append(tt)
    return {"pre": pre, "vers": vers, "draft": draft, "tgt": tgt}


ORACLE_SAMPLE_STEPS = 8      # verify steps of one request per timed oracle sample (both CPU legs)


def oracle_sample(wl, host):
    """One timed sample of the oracle, single-threaded: the first ORACLE_SAMPLE_STEPS verify steps of one
    request, every layer each.  Returns (verify steps per second, seconds, seconds of the oracle prune)."""
    from threadpoolctl import threadpool_limits
    with threadpool_limits(limits=1):
        t, t_prune = oracle_verify_steps(wl, host, ORACLE_SAMPLE_STEPS, wl.n_layers)
    return ORACLE_SAMPLE_STEPS / t, t, t_prune


def oracle_sample_text(wl):
    return (f"first {ORACLE_SAMPLE_STEPS} verify steps of one request, all {wl.n_layers} layers each "
            "(numpy fp64, 1 thread)")


def cpu_baseline(wl):
    """The oracle as it stands on one host core, one bounded sample (the same sample the reference arm times)."""
    host = oracle_host_inputs(wl)
    value, t, t_prune = oracle_sample(wl, host)
    return {"value": round(value, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": oracle_sample_text(wl) + f", {t:.1f} s; oracle prune of the same request took {t_prune:.2f} s",
            "host_cores_available": os.cpu_count()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.workload(args.workload)
    host = oracle_host_inputs(wl)
    for _ in range(min(args.warmup, 1)):
        oracle_verify_steps(wl, host, 1, wl.n_layers)
    k = max(1, min(args.steps, 5))          # each step is one bounded sample; the whole run stays within minutes
    tot = 0.0
    for _ in range(k):
        _, t, _ = oracle_sample(wl, host)
        tot += t
    value = ORACLE_SAMPLE_STEPS * k / tot
    sample = oracle_sample_text(wl) + f" per step, {k} steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": k, "warmup": min(args.warmup, 1),
        "ms_per_step": round(tot / k * 1e3, 2), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": bench_config(wl, None),
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "kind": "oracle", "cores": 1, "sample": sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def bench_config(wl, extra):
    """The `config` object both arms print: the workload and its shape."""
    cfg = {"workload": wl.name, "requests_per_step": N_ROT, "layers": wl.n_layers, "heads": wl.n_q_heads,
           "head_dim": wl.head_dim, "tree_nodes": wl.t_max, "prefix": wl.prefix_len[0], "keep": wl.keep[0],
           "tokens_per_request": wl.gen_target[0]}
    if extra:
        cfg.update(extra)
    return cfg


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2)
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel directly instead of graph replay")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", dest="extra", action="store_false",
                    help="skip the HBM-sized launches of the attention and gather kernels")
    ap.add_argument("--no-early-prefix", action="store_true", help="do not prefetch the KV prefix under the previous layer")
    ap.add_argument("--no-overlap", action="store_true", help="plain launches (no programmatic stream serialization)")
    ap.add_argument("--attn-splits", type=int, default=0, help="force key splits per cluster (0 auto)")
    ap.add_argument("--attn-path", type=int, default=0,
                    help="tree-attention kernel: 0 auto, 1 mma.sync, 2 tcgen05 (cluster splits), 3 tcgen05 persistent")
    ap.add_argument("--case", default=None,
                    choices=["attn", "gather", "score", "prune", "accept", "argmax", "tree", "gscore", "mqscore"],
                    help="run one small single-kernel case (for a profiler capture) instead of the benchmark")
    ap.add_argument("--kv-len", type=int, default=0, help="--case attn: cache length of every request")
    ap.add_argument("--layers", type=int, default=0, help="--case: layers resident / per call (0: the case's default)")
    ap.add_argument("--iters", type=int, default=3, help="--case: timed repetitions")
    ap.add_argument("--early-prefix", action="store_true", help="--case attn: launch with the early-prefix promise")
    ap.add_argument("--in-place", action="store_true", help="--case gather: compact the cache in place")
    args = ap.parse_args()
    if args.case:
        run_case(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start one rank per GPU ourselves (replicas only, no data-path collective)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    world_env = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world_env and "WORLD_SIZE" in os.environ:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started {world_env} ranks; reporting {world_env}\n")
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
