"""The pins must catch plausible mistakes.  Each case plants one mistake in a copy of the
oracle's source (on the CPU, in memory), runs the pin tests against that copy and expects at
least one of them to fail."""
import os
import types

import pytest

import test_oracle_pins as pins

ORACLE_SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "twig_oracle.py")

MUTATIONS = [
    ("scores: scale dropped", "z = np.matmul(k[b, h // G, lo:hi, :], q[b, h, :]) * scale",
     "z = np.matmul(k[b, h // G, lo:hi, :], q[b, h, :])"),
    ("scores: heads summed, not averaged", "        s[b, :m] /= Hq\n", ""),
    ("scores: wrong kv head for a query head", "z = np.matmul(k[b, h // G, lo:hi, :]", "z = np.matmul(k[b, h % Hkv, lo:hi, :]"),
    ("scores: visual slice off by one", "p[vs - lo: vs - lo + m]", "p[vs - lo + 1: vs - lo + m + 1]"),
    ("scores: eq. 7 scope ignored", "lo, hi = (0, lp) if norm_scope == 0 else (vs, vs + m)", "lo, hi = (0, lp)"),
    ("gated scores: key gate dropped", "gk = k_gate[b, h // G, lo:hi] * k[b, h // G, lo:hi]", "gk = k[b, h // G, lo:hi]"),
    ("gated scores: query gate of another head", "gq = q_gate[b, h] * q[b, h]", "gq = q_gate[b, 0] * q[b, h]"),
    ("gated scores: gate of the wrong kv head", "gk = k_gate[b, h // G, lo:hi] *", "gk = k_gate[b, h % k.shape[1], lo:hi] *"),
    ("eq. 3 guide: not causal", "z = np.matmul(k[b, h // G, :t + 1, :], q_text[b, h, i, :]) * scale", "z = np.matmul(k[b, h // G, :lp, :], q_text[b, h, i, :]) * scale"),
    ("eq. 3 guide: query position off by one", "                t = vs + m + i\n", "                t = vs + m + i - 1\n"),
    ("eq. 3 guide: only the last text token", "for i in range(lp - vs - m):", "for i in range(lp - vs - m - 1, lp - vs - m):"),
    ("tree: conditional instead of joint probability", "sc.append(sc[u] + float(lp[e]))", "sc.append(float(lp[e]))"),
    ("tree: expansion picks the lowest scores", "ids = sorted(range(lo, hi), key=lambda i: (-score[i], i))[:K]", "ids = sorted(range(lo, hi), key=lambda i: (score[i], i))[:K]"),
    ("tree: children attached to the root", "                par.append(u)\n", "                par.append(0)\n"),
    ("tree: log-probability without the normaliser", "[x[v] - lse for v in order]", "[x[v] for v in order]"),
    ("top-k: ties to the higher index", "key=lambda m: (-s[m], m)", "key=lambda m: (-s[m], -m)"),
    ("top-k: smallest instead of largest", "key=lambda m: (-s[m], m)", "key=lambda m: (s[m], m)"),
    ("prune: text after the image dropped", "+ list(range(vis_start + n_vis, prefix_len))", ""),
    ("gather: rows assigned from the top down (breaks compaction in place)", "        for j in range(n):\n            dst_k[:, b, :, j, :]",
     "        for j in reversed(range(n)):\n            dst_k[:, b, :, j, :]"),
    ("prune: kept indices not offset", "[vis_start + m for m in kept]", "[m for m in kept]"),
    ("attention: node does not see itself", "    while x >= 0:\n        out.append(x)", "    while x >= 0:\n        out.append(x) if x != i or x == 0 else None"),
    ("attention: mask shifted by one key", "vis[i, kv_len + a] = True", "vis[i, min(kv_len + a + 1, kv_len + n_nodes - 1)] = True"),
    ("attention: prefix end off by one", "vis[:, :kv_len] = True", "vis[:, :max(kv_len - 1, 0)] = True"),
    ("attention: scale dropped", "z = np.matmul(q_rows, keys.T) * scale", "z = np.matmul(q_rows, keys.T)"),
    ("attention: lse without the max", "(zmax + np.log(se))[:, 0]", "(np.log(se))[:, 0]"),
    ("attention: wrong kv head", "        g = h // G\n", "        g = h % Hkv\n"),
    ("accept: any matching node counts", "ok = all(", "ok = any([True] if len(chain) == 1 else []) or any("),
    ("accept: compares with the node's own target", "int(base_argmax[u]) for u, c in zip(chain[:-1], chain[1:])",
     "int(base_argmax[c]) for u, c in zip(chain[:-1], chain[1:])"),
    ("accept: ties to the later node", "if ok and depth > best_depth:", "if ok and depth >= best_depth:"),
    ("accept: bonus from the root", "return best_depth, np.array(path, dtype=np.int32), int(base_argmax[best])",
     "return best_depth, np.array(path, dtype=np.int32), int(base_argmax[0])"),
    ("append: rows written one position late", "cache_k[:, b, :, base + j, :]", "cache_k[:, b, :, base + j + 1, :]"),
    ("append: length not advanced by the root", "new_len[b] = base + len(paths[b])", "new_len[b] = base + len(paths[b]) - 1"),
    ("argmax: ties to the higher index", "if logits[b, i, v] > best_v:", "if logits[b, i, v] >= best_v:"),
    ("chain draft: the token below the threshold is dropped", "        toks.append(tok)\n        probs.append(prob)\n        if len(toks) >= delta or prob < theta:\n            break",
     "        if prob < theta and toks:\n            break\n        toks.append(tok)\n        probs.append(prob)\n        if len(toks) >= delta or prob < theta:\n            break"),
    ("chain draft: a probability equal to the threshold exits", "if len(toks) >= delta or prob < theta:", "if len(toks) >= delta or prob <= theta:"),
    ("chain draft: one token too many", "if len(toks) >= delta or prob < theta:", "if len(toks) > delta or prob < theta:"),
    ("chain draft: ties to the higher token id", "            if x[v] > x[tok]:", "            if x[v] >= x[tok]:"),
    ("chain draft: probability without the normaliser", "prob = float(e[tok] / e.sum())", "prob = float(e[tok])"),
    ("eq. 6: K_f ignored", "upper = L if K_f is None else K_f", "upper = L"),
]

PIN_TESTS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_") and "generator" not in n and "bf16" not in n]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_pins_catch_planted_mistake(monkeypatch, name, old, new):
    src = open(ORACLE_SRC).read()
    assert src.count(old) >= 1, "mutation target not found: " + name
    mutant = types.ModuleType("twig_oracle_mutant")
    exec(compile(src.replace(old, new, 1), "twig_oracle_mutant.py", "exec"), mutant.__dict__)
    monkeypatch.setattr(pins, "O", mutant)
    caught = []
    for t in PIN_TESTS:
        try:
            t()
        except Exception as e:          # an assertion, or a crash caused by the mistake
            caught.append((t.__name__, type(e).__name__))
    assert caught, f"no pin noticed: {name}"
