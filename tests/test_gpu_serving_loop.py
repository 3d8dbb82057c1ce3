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


def test_serving_step_replays_from_a_cuda_graph():
    """The whole retrieval step (cache lookup, batched search, verify, cache update) issues only
    stream-ordered work, so it can be captured once in a CUDA graph and replayed with new queries
    in the same buffers, which is how a launch-bound serving loop would run it. Every replay is
    compared with the oracle, integer-valued data so that ids and scores are exact."""
    import paper_2401_14021_b200 as ralm
    from oracle.cache_update import cache_update as oracle_cache_update
    N, d, R, C, k, stride = 60_000, 64, 4, 64, 5, 4
    x = workloads.integer_valued((N, d), seed=1801, lo=-3, hi=3, device=DEV)
    xn = x.cpu().numpy()
    idx = ralm.Index(x, ralm.IP, max_s=R * stride, max_k=k)
    q = torch.zeros((R, stride, d), dtype=torch.float16, device=DEV)
    cache = torch.full((R, C), -1, dtype=torch.int64, device=DEV)
    cursor = torch.zeros((R,), dtype=torch.int32, device=DEV)
    spec = torch.empty((R, stride, 1), dtype=torch.int64, device=DEV)
    spec_scores = torch.empty((R, stride, 1), dtype=torch.float32, device=DEV)
    ids = torch.empty((R * stride, k), dtype=torch.int64, device=DEV)
    scores = torch.empty((R * stride, k), dtype=torch.float32, device=DEV)
    first_mismatch = torch.empty((R,), dtype=torch.int32, device=DEV)

    def step(st):
        ralm.cache_search(idx, cache, q, 1, spec, spec_scores, st)
        ralm.search(idx, q.view(R * stride, d), k, ids, scores, st)
        ralm.verify(spec.view(R, stride), ids.view(R, stride, k), 1, first_mismatch, st)
        ralm.cache_update(cache, cursor, ids.view(R, stride, k), k, N, stream=st)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(side)                                   # first use outside the capture (module load)
    side.synchronize()
    cache.fill_(-1)
    cursor.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
        step(torch.cuda.current_stream())
    o_cache, o_cursor = cache.cpu().numpy(), cursor.cpu().numpy()
    for t in range(3):
        # (the third round repeats the first round's queries: their documents are cached by then)
        q.copy_(workloads.integer_valued((R, stride, d), seed=1810 + t % 2, lo=-3, hi=3, device=DEV))
        graph.replay()
        torch.cuda.synchronize()
        assert idx.device_status() == 0
        qn = q.cpu().numpy()
        o_spec, _ = oracle.cache_search(xn, o_cache, qn, oracle.IP, 1)
        o_ids, o_scores = oracle.search(xn, qn.reshape(R * stride, d), oracle.IP, k)
        o_m = oracle.verify(o_spec.reshape(R, stride), o_ids.reshape(R, stride, k))
        o_cache, o_cursor = oracle_cache_update(o_cache, o_cursor, o_ids.reshape(R, stride, k), k, N=N)
        assert np.array_equal(spec.cpu().numpy(), o_spec)
        assert np.array_equal(ids.cpu().numpy(), o_ids)
        assert np.array_equal(scores.cpu().numpy(), o_scores.astype(np.float32))
        assert np.array_equal(first_mismatch.cpu().numpy(), o_m)
        assert np.array_equal(cache.cpu().numpy(), o_cache)
        assert np.array_equal(cursor.cpu().numpy(), o_cursor)
    assert o_m.max() > 0                          # the repeated queries found their documents cached
    idx.close()
