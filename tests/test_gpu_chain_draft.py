"""GPU parity: chain drafting with early exit (sequence self-speculative decoding) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import twig_oracle as O
from paper_2503_14075_b200 import synth
from gpu_common import DEV, dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tw():
    from paper_2503_14075_b200 import twig
    return twig


def _rows_with_top_probability(rng, n_rows, vocab, probs, fp32):
    """Draft distributions whose most likely token has (about) the given probability: random logits
    with one entry raised.  Returned as the exact values the device sees (bf16 or fp32), widened."""
    x = rng.standard_normal((n_rows, vocab)).astype(np.float32)
    for r in range(n_rows):
        t = int(rng.integers(vocab))
        rest = np.delete(x[r].astype(np.float64), t)
        lse = np.log(np.exp(rest - rest.max()).sum()) + rest.max()
        x[r, t] = np.float32(lse + np.log(probs[r] / (1.0 - probs[r])))
    if fp32:
        return x, x.astype(np.float64)
    bits = synth.f32_to_bf16(x)
    return bits, synth.bf16_to_f64(bits)


@pytest.mark.parametrize("vocab", [32000, 32003, 7])
@pytest.mark.parametrize("fp32", [False, True], ids=["bf16", "fp32"])
def test_chain_draft_matches_oracle(tw, vocab, fp32):
    """The paper's settings (delta = 5, theta = 0.6) on a batch of 16 requests whose draft confidence
    sits well clear of the threshold (the decision is taken in fp32 on the device, in fp64 by the
    oracle), so that draft lengths 1..5 all occur."""
    B, T, delta, theta = 16, 8, 5, 0.6
    rng = synth.rng_for(9, 600 + vocab % 100 + int(fp32))
    # per step and request: confident (0.7 .. 0.97) or not (0.2 .. 0.5)
    conf = rng.uniform(0.7, 0.97, size=(delta, B))
    low = rng.uniform(0.2, 0.5, size=(delta, B))
    probs = np.where(rng.random((delta, B)) < 0.3, low, conf)
    probs[:, 0] = conf[:, 0]                 # one request drafts all delta tokens
    probs[0, 1] = low[0, 1]                  # one stops after its first token
    dev_rows, host_rows = [], []
    for s in range(delta):
        dev_x, host_x = _rows_with_top_probability(rng, B, vocab, probs[s], fp32)
        host_rows.append(host_x)
        pad = (-vocab) % 8                   # rows must start on 16 bytes
        if fp32:
            t = torch.zeros((B, vocab + pad), dtype=torch.float32, device=DEV)
            t[:, :vocab] = torch.from_numpy(dev_x).to(DEV)
        else:
            t = torch.zeros((B, vocab + pad), dtype=torch.int16, device=DEV)
            t[:, :vocab] = torch.from_numpy(dev_x.view(np.int16)).to(DEV)
            t = t.view(torch.bfloat16)
        dev_rows.append(t[:, :vocab])
    parent = torch.full((B, T), -7, dtype=torch.int32, device=DEV)
    tok = torch.full((B, T), -7, dtype=torch.int32, device=DEV)
    prob = torch.full((B, T), -7.0, dtype=torch.float32, device=DEV)
    n_nodes = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    active = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.chain_draft_reset(parent, tok, n_nodes, active, tok_prob=prob)
    for s in range(delta):
        tw.chain_draft_step(dev_rows[s], delta, theta, parent, tok, n_nodes, active, tok_prob=prob, dev_status=status)
    torch.cuda.synchronize()
    assert not status.cpu().numpy().any() and not active.cpu().numpy().any()
    parent, tok, prob, n_nodes = parent.cpu().numpy(), tok.cpu().numpy(), prob.cpu().numpy(), n_nodes.cpu().numpy()
    lengths = set()
    for b in range(B):
        want_t, want_p = O.chain_draft([host_rows[s][b] for s in range(delta)], delta, theta)
        n = len(want_t)
        lengths.add(n)
        assert n_nodes[b] == n + 1
        assert tok[b, 0] == -1 and parent[b, 0] == -1
        assert tok[b, 1:n + 1].tolist() == want_t
        assert parent[b, 1:n + 1].tolist() == list(range(n))            # a chain: node i hangs on node i - 1
        assert np.allclose(prob[b, 1:n + 1], want_p, rtol=2e-4)
        assert np.all(tok[b, n + 1:] == 0) and np.all(parent[b, n + 1:] == -1)      # nothing past the draft
    assert {1, delta} <= lengths


def test_chain_draft_ties_masked_logits_and_errors(tw):
    B, T, V = 4, 4, 64
    x = torch.full((B, V), -float("inf"), dtype=torch.float32, device=DEV)
    x[0, 5] = x[0, 9] = 1.0                 # two equal maxima: the lower id, probability 1/2
    x[1, 63] = 0.0                          # a single finite logit: probability 1
    x[2, :] = 0.0                           # all equal: token 0, probability 1/V
    x[3, 0], x[3, 1] = -1.0, 2.0
    parent = torch.zeros((B, T), dtype=torch.int32, device=DEV)
    tok, n_nodes, active = torch.zeros_like(parent), torch.zeros(B, dtype=torch.int32, device=DEV), torch.zeros(B, dtype=torch.int32, device=DEV)
    prob = torch.zeros((B, T), dtype=torch.float32, device=DEV)
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    tw.chain_draft_reset(parent, tok, n_nodes, active, tok_prob=prob)
    tw.chain_draft_step(x, 3, 0.6, parent, tok, n_nodes, active, tok_prob=prob, dev_status=status)
    torch.cuda.synchronize()
    assert tok[:, 1].tolist() == [5, 63, 0, 1]
    want = [O.chain_draft([x[b].cpu().numpy().astype(np.float64)], 3, 0.6)[1][0] for b in range(B)]
    assert np.allclose(prob[:, 1].cpu().numpy(), want, rtol=1e-5) and abs(want[0] - 0.5) < 1e-12
    assert active.tolist() == [0, 1, 0, 1]                 # 1/2 and 1/64 are below 0.6
    # a request that has stopped ignores further calls; one without room for another node is flagged
    for _ in range(3):
        tw.chain_draft_step(x, 3, 0.0, parent, tok, n_nodes, active, dev_status=status)
    torch.cuda.synchronize()
    assert n_nodes.tolist() == [2, 4, 2, 4] and not active.cpu().numpy().any() and not status.cpu().numpy().any()
    active.fill_(1)
    tw.chain_draft_step(x, 3, 0.0, parent, tok, n_nodes, active, dev_status=status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, tw.DEV_BAD_TREE, 0, tw.DEV_BAD_TREE] and n_nodes.tolist() == [3, 4, 3, 4]
    # host-side refusals: the root and max_draft tokens must fit t_max
    with pytest.raises(tw.TwigError) as e:
        tw.chain_draft_step(x, 4, 0.6, parent, tok, n_nodes, active)
    assert e.value.code == 2
