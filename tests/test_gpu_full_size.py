"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot rank 21 M or 50 M rows in seconds, so the check is sampled, in a way that
still catches a missed row: the oracle ranks a SUB-CORPUS made of (a) seeded random chunks of
rows, the first rows and the ragged tail and (b) every row the GPU returned. If the GPU's
lists are the top-k of the whole corpus they are also the top-k of any sub-corpus that contains
them, so the oracle's ranking of the sub-corpus must reproduce them (ids by the near-tie rule,
scores within tolerance); a sampled row that the GPU wrongly left out shows up as a mismatch.
Rank 0 must also be the row each query was copied from.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import Counts, check_lists

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ralm():
    import paper_2401_14021_b200 as ralm
    return ralm


def _sampled_parity(x, q, ids, scores, metric, k, n_chunks, chunk_rows, seed, query_sel=None):
    N = x.shape[0]
    sel = list(range(q.shape[0])) if query_sel is None else list(query_sel)
    g = torch.Generator().manual_seed(seed)
    starts = (torch.randint(0, max(1, N // chunk_rows), (n_chunks,), generator=g) * chunk_rows).tolist()
    starts += [0, max(0, N - chunk_rows + 1)]
    rows = torch.cat([torch.arange(s0, min(N, s0 + chunk_rows)) for s0 in sorted(set(starts))])
    gi, gs = ids.cpu(), scores.cpu().numpy()
    returned = gi[sel].flatten()
    sub_rows = torch.unique(torch.cat([rows, returned[returned >= 0]]))     # ascending: id order is kept
    xs = x[sub_rows.to(x.device)].cpu().numpy()
    qn = q.cpu().numpy()[sel]
    o_local, o_scores = oracle.search(xs, qn, metric, k)
    o_ids = np.where(o_local >= 0, sub_rows.numpy()[np.maximum(o_local, 0)], -1)
    pos = {int(r): i for i, r in enumerate(sub_rows.tolist())}
    max_norm = float(np.linalg.norm(xs.astype(np.float64), axis=1).max())
    counts = Counts()
    for n, i in enumerate(sel):
        scale = max_norm * float(np.linalg.norm(qn[n].astype(np.float64)))
        counts += check_lists(gi[i].numpy(), gs[i], o_ids[n], o_scores[n],
                              lambda j, n=n: oracle.pair_score(xs[pos[j]], qn[n], metric), metric,
                              scale=scale, n_valid=N)
    # swaps that fp32 rounding does not explain are accepted by the 2e-3 rule but not expected
    assert counts.wide == 0, str(counts)
    return counts, sub_rows.numel()


@pytest.fixture(scope="module")
def c3_corpus():
    c = workloads.CONFIGS["C3"]
    x, assign = workloads.mixture_corpus(c.N, c.d, c.n_centres, workloads.seed_for(3), device=DEV)
    yield x, assign
    del x, assign
    torch.cuda.empty_cache()


@pytest.mark.parametrize("k", [1, 20])
def test_c3_full_size_s8(c3_corpus, k):
    """The headline configuration: 21 M x 768, inner product, s = 8."""
    ralm = _ralm()
    x, _ = c3_corpus
    q, src = workloads.noisy_copy_queries(x, 8, workloads.seed_for(3, "queries"))
    idx = ralm.Index(x, oracle.IP, max_s=8, max_k=k)
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src.tolist()
    counts, n_sub = _sampled_parity(x, q, ids, scores, oracle.IP, k, 30, 16_384, seed=3300 + k)
    print("C3 k=%d: %s over a %d-row sub-corpus" % (k, counts, n_sub))
    # every s in 1..8 returns the same rows for the queries it shares with the full batch
    for s in (1, 3, 5):
        ids_s, _ = ralm.search(idx, q[:s].contiguous(), k)
        assert torch.equal(ids_s, ids[:s])
    idx.close()


def test_c3_full_corpus_oracle_pass_s8_k20(c3_corpus):
    """The headline corpus against the oracle over EVERY row, not a sample: the corpus comes back
    in 1 Mi-row pieces, the oracle scores each piece for each of the 8 queries into one [N] array
    per query and ranks it, and all 8 x 20 ids and scores are compared. A row the GPU wrongly
    dropped anywhere in the 21 M shows here. (About 21 M x 8 fp64 dot products: minutes of CPU.)"""
    ralm = _ralm()
    x, _ = c3_corpus
    N, k = x.shape[0], 20
    q, src = workloads.noisy_copy_queries(x, 8, workloads.seed_for(3, "queries"))
    idx = ralm.Index(x, oracle.IP, max_s=8, max_k=k)
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    idx.close()
    qn = q.cpu().numpy()
    all_scores = np.empty((8, N), dtype=np.float64)
    piece = 1 << 20
    for lo in range(0, N, piece):
        hi = min(N, lo + piece)
        rows = x[lo:hi].cpu().numpy()
        for i in range(8):
            oracle.scores(rows, qn[i], oracle.IP, out=all_scores[i, lo:hi])
    gi, gs = ids.cpu().numpy(), scores.cpu().numpy()
    counts = Counts()
    for i in range(8):
        o_ids, o_scores = oracle.rank(all_scores[i], oracle.IP, k)
        assert o_ids[0] == int(src[i])
        counts += check_lists(gi[i], gs[i], o_ids, o_scores, lambda j, i=i: all_scores[i, j], oracle.IP,
                              scale=float(np.linalg.norm(qn[i].astype(np.float64))), n_valid=N)
    print("C3 s=8 k=20, full-corpus oracle pass: %s" % counts)
    assert counts.wide == 0, str(counts)


def _cache_step_against_oracle(ralm, x, assign, cfg, metric):
    """R requests x C-entry caches x q queries on the full corpus: the cache lookup against the
    oracle on the gathered rows (it only needs the cached rows), then verify on both sides."""
    R, stride, C = cfg.requests, cfg.stride, cfg.cache_entries
    q, src = workloads.noisy_copy_queries(x, R * stride, workloads.seed_for(cfg.index, "queries"))
    cache = workloads.speculation_cache_ids(assign, cfg.N, src.reshape(R, stride), C,
                                            workloads.seed_for(cfg.index, "caches"), n_centres=cfg.n_centres)
    idx = ralm.Index(x, metric, max_s=R * stride, max_k=20)
    qr = q.reshape(R, stride, cfg.d).contiguous()
    spec, spec_scores = ralm.cache_search(idx, cache, qr, 1)
    retr, _ = ralm.search(idx, q, 20 if R * stride > 64 else 1)
    ld = retr.shape[1]
    m = ralm.verify(spec.reshape(R, stride).contiguous(), retr.reshape(R, stride, ld).contiguous())
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert retr[:, 0].tolist() == src.tolist()
    cache_h = cache.cpu()
    uniq = torch.unique(cache_h[cache_h >= 0])
    xs = x[uniq.to(DEV)].cpu().numpy()
    local = torch.searchsorted(uniq, cache_h.clamp_min(0))
    local = torch.where(cache_h >= 0, local, torch.full_like(local, -1)).numpy()
    o_local, o_scores = oracle.cache_search(xs, local, qr.cpu().numpy(), metric, 1)
    o_spec = np.where(o_local >= 0, uniq.numpy()[np.maximum(o_local, 0)], -1)
    assert np.array_equal(spec.cpu().numpy(), o_spec)
    np.testing.assert_allclose(spec_scores.cpu().numpy(), o_scores, rtol=2e-3, atol=1e-5)
    o_m = oracle.verify(o_spec.reshape(R, stride), retr.cpu().numpy().reshape(R, stride, ld))
    assert np.array_equal(m.cpu().numpy(), o_m)
    idx.close()
    return m.cpu().tolist()


def test_c5_serving_step_cache_and_verify(c3_corpus):
    """The high-concurrency configuration's speculation step: 64 requests x 512-entry caches x
    stride 8 (512 cache queries, 32 768 cached rows gathered) against the oracle, and the
    first-mismatch positions of all 64 requests after the 512-query search."""
    ralm = _ralm()
    x, assign = c3_corpus
    m = _cache_step_against_oracle(ralm, x, assign, workloads.CONFIGS["C5"], oracle.IP)
    print("C5 first-mismatch positions:", m)
    assert len(m) == 64 and min(m) < 8 and max(m) > 0     # neither all hits nor all misses


def test_c3_serving_step_cache_and_verify(c3_corpus):
    """8 concurrent requests x 512-entry caches x stride 8 on the full corpus: cache lookup and
    first-mismatch positions against the oracle (which only needs the cached rows)."""
    ralm = _ralm()
    x, assign = c3_corpus
    c = workloads.CONFIGS["C3"]
    R, stride, C = c.requests, c.stride, c.cache_entries
    q, src = workloads.noisy_copy_queries(x, R * stride, workloads.seed_for(3, "queries"))
    cache = workloads.speculation_cache_ids(assign, c.N, src.reshape(R, stride), C,
                                            workloads.seed_for(3, "caches"), n_centres=c.n_centres)
    idx = ralm.Index(x, oracle.IP, max_s=R * stride, max_k=1)
    qr = q.reshape(R, stride, c.d).contiguous()
    spec, spec_scores = ralm.cache_search(idx, cache, qr, 1)
    retr, _ = ralm.search(idx, q, 1)
    m = ralm.verify(spec.reshape(R, stride).contiguous(), retr.reshape(R, stride, 1).contiguous())
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert retr[:, 0].tolist() == src.tolist()
    # oracle on the cached rows only: gather them, rank locally, map back
    cache_h = cache.cpu()
    uniq = torch.unique(cache_h[cache_h >= 0])
    xs = x[uniq.to(DEV)].cpu().numpy()
    local = torch.searchsorted(uniq, cache_h.clamp_min(0))
    local = torch.where(cache_h >= 0, local, torch.full_like(local, -1)).numpy()
    o_local, o_scores = oracle.cache_search(xs, local, qr.cpu().numpy(), oracle.IP, 1)
    o_spec = np.where(o_local >= 0, uniq.numpy()[np.maximum(o_local, 0)], -1)
    assert np.array_equal(spec.cpu().numpy(), o_spec)
    np.testing.assert_allclose(spec_scores.cpu().numpy(), o_scores, rtol=2e-3, atol=1e-5)
    o_m = oracle.verify(o_spec.reshape(R, stride), retr.cpu().numpy().reshape(R, stride, 1))
    assert np.array_equal(m.cpu().numpy(), o_m)
    print("C3 first-mismatch positions:", m.cpu().tolist())
    idx.close()


@pytest.mark.parametrize("k", [1, 20])
def test_c3_full_size_s8_with_8bit_filter_copy(c3_corpus, k):
    """The headline configuration through the 8-bit scan (ralm_index_enable_q8: the one-byte copy
    filters, every pair it lets through is scored again from the fp16 row): the same sampled
    check against the oracle, and the same lists as the fp16 scan of the same index shape."""
    ralm = _ralm()
    x, _ = c3_corpus
    q, src = workloads.noisy_copy_queries(x, 8, workloads.seed_for(3, "queries"))
    idx = ralm.Index(x, oracle.IP, max_s=8, max_k=k)
    ids16, scores16 = ralm.search(idx, q, k)
    idx.enable_q8()
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src.tolist()
    counts, n_sub = _sampled_parity(x, q, ids, scores, oracle.IP, k, 30, 16_384, seed=3700 + k)
    print("C3 8-bit scan k=%d: %s over a %d-row sub-corpus" % (k, counts, n_sub))
    assert torch.equal(ids[:, 0], ids16[:, 0])
    torch.testing.assert_close(scores, scores16, rtol=1e-5, atol=1e-6)
    for s in (1, 5):
        ids_s, _ = ralm.search(idx, q[:s].contiguous(), k)
        assert torch.equal(ids_s, ids[:s])
    idx.close()


@pytest.mark.parametrize("s,k", [(16, 1), (16, 20), (32, 20), (64, 20)])
def test_c3_full_size_mid_batches(c3_corpus, s, k):
    """Between the two headline cases: 16 and 32 queries run as one pass of the small-batch scan
    (two and four query groups per staged tile), 64 on the tcgen05 scan."""
    ralm = _ralm()
    x, _ = c3_corpus
    q, src = workloads.noisy_copy_queries(x, s, workloads.seed_for(3, "queries") + s)
    idx = ralm.Index(x, oracle.IP, max_s=s, max_k=k)
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src.tolist()
    counts, n_sub = _sampled_parity(x, q, ids, scores, oracle.IP, k, 8, 16_384, seed=3600 + s + k,
                                          query_sel=range(0, s, max(1, s // 16)))
    print("C3 s=%d k=%d: %s over a %d-row sub-corpus" % (s, k, counts, n_sub))
    idx.close()


def test_c5_full_size_512_queries(c3_corpus):
    """The high-concurrency configuration: 512 queries, k = 20, on the tcgen05 scan."""
    ralm = _ralm()
    x, _ = c3_corpus
    q, src = workloads.noisy_copy_queries(x, 512, workloads.seed_for(3, "queries"))
    idx = ralm.Index(x, oracle.IP, max_s=512, max_k=20)
    ids, scores = ralm.search(idx, q, 20)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src.tolist()
    counts, n_sub = _sampled_parity(x, q, ids, scores, oracle.IP, 20, 6, 16_384, seed=3500,
                                          query_sel=range(0, 512, 8))
    print("C5: %s over a %d-row sub-corpus, 64 of 512 queries" % (counts, n_sub))
    # the first 8 queries through the small-batch scan give the same rows
    ids8, scores8 = ralm.search(idx, q[:8].contiguous(), 20)
    assert torch.equal(ids8[:, 0], ids[:8, 0])
    torch.testing.assert_close(scores8, scores[:8], rtol=1e-4, atol=1e-5)
    idx.close()


def test_c4_full_size_l2_k1024():
    """The KNN-LM datastore: 50 M x 1024 (102.4 GB), L2, s = 4, k = 1024."""
    ralm = _ralm()
    c = workloads.CONFIGS["C4"]
    free, _ = torch.cuda.mem_get_info()
    if free < c.N * c.d * 2 + (8 << 30):
        pytest.skip("needs %.0f GB of free device memory" % ((c.N * c.d * 2 + (8 << 30)) / 1e9))
    x, _ = workloads.mixture_corpus(c.N, c.d, c.n_centres, workloads.seed_for(4), device=DEV,
                                    normalise=False, lognormal_sigma=c.lognormal_sigma)
    q, src = workloads.noisy_copy_queries(x, 4, workloads.seed_for(4, "queries"))
    idx = ralm.Index(x, oracle.L2, max_s=4, max_k=1024)
    ids, scores = ralm.search(idx, q, 1024)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src.tolist()
    counts, n_sub = _sampled_parity(x, q, ids, scores, oracle.L2, 1024, 14, 16_384, seed=3400)
    print("C4: %s over a %d-row sub-corpus" % (counts, n_sub))
    # the same search through the 8-bit filter copy (51 GB more): identical neighbours, distances
    # from the same direct form
    free, _ = torch.cuda.mem_get_info()
    if free > c.N * c.d + (6 << 30):
        idx.enable_q8()
        ids8, scores8 = ralm.search(idx, q, 1024)
        torch.cuda.synchronize()
        assert idx.device_status() == 0
        assert idx.last_dispatch()["kernel_name"] == "scan_q8_kernel"
        counts8, n_sub = _sampled_parity(x, q, ids8, scores8, oracle.L2, 1024, 14, 16_384, seed=3401)
        print("C4 8-bit scan: %s over a %d-row sub-corpus" % (counts8, n_sub))
        assert torch.equal(ids8[:, 0], ids[:, 0])
        torch.testing.assert_close(scores8, scores, rtol=1e-5, atol=1e-4)
    else:
        print("C4 8-bit scan: skipped, %.0f GB free" % (free / 1e9))
    idx.close()
    # 64 concurrent queries, k = 20: L2 on the large-batch scan (lower-bound sample, filter, rescoring)
    q64, src64 = workloads.noisy_copy_queries(x, 64, workloads.seed_for(4, "queries") + 5)
    idx = ralm.Index(x, oracle.L2, max_s=64, max_k=20)
    ids, scores = ralm.search(idx, q64, 20)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src64.tolist()
    counts, n_sub = _sampled_parity(x, q64, ids, scores, oracle.L2, 20, 6, 16_384, seed=3450,
                                          query_sel=range(0, 64, 4))
    print("C4, 64 queries: %s over a %d-row sub-corpus, 16 of 64 queries" % (counts, n_sub))
    idx.close()
    # 16 concurrent queries, k = 20: one pass of the small-batch scan with two query groups
    q16, src16 = workloads.noisy_copy_queries(x, 16, workloads.seed_for(4, "queries") + 9)
    idx = ralm.Index(x, oracle.L2, max_s=16, max_k=20)
    ids, scores = ralm.search(idx, q16, 20)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    assert ids[:, 0].tolist() == src16.tolist()
    counts, n_sub = _sampled_parity(x, q16, ids, scores, oracle.L2, 20, 6, 16_384, seed=3460)
    print("C4, 16 queries: %s over a %d-row sub-corpus" % (counts, n_sub))
    idx.close()
    del x
    torch.cuda.empty_cache()
