"""ttp_score_noalloc: the scoring call for hosts that may not allocate device memory
(a server whose memory pool already owns the whole device, a plugin that only receives
tensors, a loop that must avoid cudaMalloc's device synchronisation).  Its scratch is a fixed array inside the library, so the check here is
simply that it returns what ttp_score returns, on two calls in a row that leave different
contents in that shared array, and that an oversized request is refused on the host.

Collected last on purpose (file name), so a run that stops at the first failure has
already run every other test."""
import numpy as np
import pytest
import torch

from paper_2503_14075_b200 import synth
from gpu_common import DEV, MAX_ABS_TOL, REL_L2_TOL, dev_bf16, dev_i32, max_abs, rel_l2_rows

pytestmark = pytest.mark.gpu


def _both(tw, wl, stream_id, scope):
    pre = synth.make_prefill(wl, synth.rng_for(wl.index, stream_id), n_layers=1, gain=wl.head_dim ** 0.5)
    B, m_max = wl.batch, max(wl.n_vis)
    q, k = dev_bf16(pre["twig_q"]), dev_bf16(pre["twig_k"])
    meta = [dev_i32(pre[n]) for n in ("prefix_len", "vis_start", "n_vis")]
    ref = torch.full((B, m_max), -1.0, dtype=torch.float32, device=DEV)
    got = torch.full((B, m_max), -2.0, dtype=torch.float32, device=DEV)
    st_ref = torch.zeros(B, dtype=torch.int32, device=DEV)
    st_got = torch.zeros(B, dtype=torch.int32, device=DEV)
    ws = torch.empty(tw.twig_workspace_bytes(B, wl.n_q_heads, wl.head_dim, k.shape[2], 64), dtype=torch.uint8,
                     device=DEV)
    tw.ttp_score(q, k, *meta, ref, ws, norm_scope=scope, dev_status=st_ref)
    tw.ttp_score_noalloc(q, k, *meta, got, norm_scope=scope, dev_status=st_got)
    torch.cuda.synchronize()
    assert not st_ref.cpu().numpy().any() and not st_got.cpu().numpy().any()
    return ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)


def test_noalloc_scores_equal_ttp_score_on_two_calls_in_a_row():
    from paper_2503_14075_b200 import twig as tw
    big = synth.Workload(9, "noalloc-a", 1, 3, 12, 4, 64, [17, 1, 0], [333, 1025, 64], [9, 130, 0], [1, 1, 1],
                         [8] * 3, [3] * 3, 0.6)
    # first call: a long prompt fills a large part of the shared array; second call: a small
    # request of another shape reads only what it has written itself
    for wl, sid, scope in ((big, 1, 0), (synth.workload(1), 2, 1), (synth.workload(2), 3, 0)):
        ref, got = _both(tw, wl, sid, scope)
        for b in range(wl.batch):
            m = wl.n_vis[b]
            assert max_abs(got[b, :m], ref[b, :m]) <= MAX_ABS_TOL
            assert rel_l2_rows(got[b, :m], ref[b, :m]) <= REL_L2_TOL
            # both calls run the same two kernels on the same inputs (only the scratch differs), so the
            # scores are not just within tolerance of each other but the same bits
            assert np.array_equal(got[b, :m], ref[b, :m])
            assert np.all(got[b, m:] == 0)


def test_noalloc_refuses_requests_beyond_its_fixed_scratch():
    from paper_2503_14075_b200 import twig as tw
    B, Hq, d, L = 64, 32, 128, 2048                      # 64 * 32 * 2048 * 4 bytes = 16 MiB > 4 MiB
    assert B * Hq * L * 4 > tw.NOALLOC_SCRATCH_BYTES
    q = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV)
    k = torch.zeros((B, 1, 1, d), dtype=torch.bfloat16, device=DEV).expand(B, 32, L, d)   # never read
    meta = [torch.zeros(B, dtype=torch.int32, device=DEV) for _ in range(3)]
    scores = torch.zeros((B, 16), dtype=torch.float32, device=DEV)
    with pytest.raises(tw.TwigError) as e:
        tw.ttp_score_noalloc(q, k, *meta, scores)
    assert e.value.code == 4                             # TWIG_ERR_WORKSPACE, nothing launched
