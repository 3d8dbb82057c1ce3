"""The retrieval side of Algorithm 1 run as a loop on the GPU, every call through the library:
speculate from the caches, verify a stride of queries against the corpus, find the first
mismatch, put the retrieved documents into the caches, let OS^3 pick the next stride.

The language model is not part of this library, so the query stream is synthetic: every
request keeps asking about a small pool of documents of one cluster (noisy copies of them), which
is the temporal locality that makes speculation work. What is checked: every verification
retrieval equals the oracle's on a sample, caches stay sets, and, as the caches fill, more
speculations match and the scheduler moves to longer strides.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_speculate_verify_update_schedule():
    import paper_2401_14021_b200 as ralm
    N, d, R, C, k, s_max, rounds = 120_000, 256, 4, 256, 20, 8, 14
    x, assign = workloads.mixture_corpus(N, d, 64, seed=71, device=DEV)
    g = torch.Generator(device=DEV).manual_seed(72)
    # each request talks about 12 documents of one cluster
    pools = []
    for r in range(R):
        members = torch.nonzero(assign == (5 + 7 * r)).flatten()
        pools.append(members[torch.randperm(members.numel(), generator=g, device=DEV)[:12]])
    idx = ralm.Index(x, ralm.IP, max_s=R * s_max, max_k=k)
    cache = torch.full((R, C), -1, dtype=torch.int64, device=DEV)
    cursor = torch.zeros((R,), dtype=torch.int32, device=DEV)
    history = [[] for _ in range(R)]            # (matched, stride) of the last verifications, per request
    strides, matched_per_round = [], []
    stride = 1                                  # the scheduler starts at 1
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    xn = None
    for t in range(rounds):
        src = torch.stack([pool[torch.randint(0, pool.numel(), (stride,), generator=g, device=DEV)]
                           for pool in pools])                                    # [R][stride]
        rows = x[src.flatten()].float()
        noise = torch.randn(rows.shape, generator=g, device=DEV) * (0.1 * rows.norm(dim=1, keepdim=True) / d ** 0.5)
        q = (rows + noise).to(torch.float16).reshape(R, stride, d).contiguous()
        ev[0].record()
        spec, _ = ralm.cache_search(idx, cache, q, 1)                             # speculation step
        ev[1].record()
        retr, scores = ralm.search(idx, q.reshape(R * stride, d), k)              # batched verification
        retr = retr.reshape(R, stride, k).contiguous()
        m = ralm.verify(spec.reshape(R, stride).contiguous(), retr)
        ev[2].record()
        ralm.cache_update(cache, cursor, retr, k, N)                              # top-k update, every retrieved list
        torch.cuda.synchronize()
        assert idx.device_status() == 0
        m_host = m.tolist()
        step_hits = (spec.reshape(R, stride) == retr[:, :, 0]).float().mean().item()   # per speculation step
        matched_per_round.append(step_hits)
        # first_mismatch is consistent with the step-wise comparison
        for r in range(R):
            eq = (spec[r, :, 0] == retr[r, :, 0]).tolist()
            assert m_host[r] == (eq.index(False) if False in eq else stride)
        strides.append(stride)
        # the verification retrieval is the exact one (checked on request 0's first query)
        if t in (0, rounds - 1):
            xn = x.cpu().numpy() if xn is None else xn
            o_ids, _ = oracle.search(xn, q[0, :1].cpu().numpy(), oracle.IP, k)
            assert retr[0, 0, 0].item() == o_ids[0, 0] == src[0, 0].item()
        # caches stay sets
        for r in range(R):
            held = cache[r][cache[r] >= 0]
            assert held.unique().numel() == held.numel()
        # OS^3: gamma from the last five verifications of request 0, a and b from the events
        for r in range(R):
            history[r] = (history[r] + [(m_host[r], stride)])[-5:]
        a = ev[0].elapsed_time(ev[1]) / stride
        b = ev[1].elapsed_time(ev[2])
        stride = ralm.os3_stride([h[0] for h in history[0]], [h[1] for h in history[0]], a, b, s_max=s_max)
        assert 1 <= stride <= s_max
    assert strides[0] == 1
    assert matched_per_round[0] == 0.0                         # empty caches: nothing to speculate from
    assert np.mean(matched_per_round[-4:]) > 0.6               # warm caches: most speculations match
    assert max(strides[4:]) > 1                                # and the scheduler lengthens the stride
    print("strides", strides, "matched fraction", [round(v, 2) for v in matched_per_round])
