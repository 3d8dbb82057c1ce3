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
from parity import Counts, check_lists, sampled_parity as _sampled_parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ralm():
    import paper_2401_14021_b200 as ralm
    return ralm


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
