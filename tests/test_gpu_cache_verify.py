"""GPU parity: ralm_cache_search and ralm_verify against the oracle, plus the chained step."""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import Counts, check_lists

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _ralm():
    import paper_2401_14021_b200 as ralm
    return ralm


def _check_cache(ralm, idx, x, cache, q, metric, k):
    ids, scores = ralm.cache_search(idx, cache, q, k)
    torch.cuda.synchronize()
    xn, qn = x.cpu().numpy(), q.cpu().numpy()
    oi, osc = oracle.cache_search(xn, cache.cpu().numpy(), qn, metric, k)
    gi, gs = ids.cpu().numpy(), scores.cpu().numpy()
    counts = Counts()
    for r in range(cache.shape[0]):
        for u in range(q.shape[1]):
            counts += check_lists(gi[r, u], gs[r, u], oi[r, u], osc[r, u],
                                  lambda j: oracle.pair_score(xn[j], qn[r, u], metric), metric,
                                  scale=float(np.abs(osc[r, u][np.isfinite(osc[r, u])]).max(initial=1.0)),
                                  n_valid=xn.shape[0])
    return ids, counts


@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
@pytest.mark.parametrize("R,C,q,k,d", [(1, 64, 4, 5, 768), (8, 512, 8, 20, 768), (3, 100, 9, 1, 64),
                                       (2, 4096, 2, 1024, 1024), (5, 1, 1, 3, 8)])
def test_cache_search_parity(metric, R, C, q, k, d):
    ralm = _ralm()
    N = 60_000
    x, assign = workloads.mixture_corpus(N, d, 64, seed=61, device=DEV)
    qs, src = workloads.noisy_copy_queries(x, R * q, seed=62)
    cache = workloads.speculation_cache_ids(assign, N, src.reshape(R, q), C, seed=63, n_centres=64,
                                            empty_slots=C // 7)
    idx = ralm.Index(x, metric, 8, max(k, 1))
    _check_cache(ralm, idx, x, cache, qs.reshape(R, q, d).contiguous(), metric, k)
    assert idx.device_status() == 0


def test_cache_integer_inputs_bit_exact_with_duplicates_and_empty():
    ralm = _ralm()
    x = workloads.integer_valued((500, 64), seed=64, lo=-3, hi=3, device=DEV)
    q = workloads.integer_valued((2, 3, 64), seed=65, lo=-3, hi=3, device=DEV)
    cache = torch.randint(0, 500, (2, 40), device=DEV, generator=torch.Generator(DEV).manual_seed(1))
    cache[0, 5] = cache[0, 6]                       # repeated id counts once
    cache[0, 10:14] = -1
    cache[1, :] = -1                                # an entirely empty cache
    for metric in (oracle.IP, oracle.L2):
        idx = ralm.Index(x, metric, 8, 40)
        ids, scores = ralm.cache_search(idx, cache, q, 40)
        oi, osc = oracle.cache_search(x.cpu().numpy(), cache.cpu().numpy(), q.cpu().numpy(), metric, 40)
        assert np.array_equal(ids.cpu().numpy(), oi)
        assert np.array_equal(scores.cpu().numpy().astype(np.float64), osc)
        assert (ids[1] == -1).all()


def test_cache_search_with_more_requests_than_a_grid_dimension_holds():
    """100 000 requests of 8 slots (the key buffer's limit is R * q * C <= 2^20): the request index
    must not sit in a grid dimension that stops at 65 535."""
    ralm = _ralm()
    R, C, d = 100_000, 8, 64
    x = workloads.integer_valued((500, d), seed=66, lo=-3, hi=3, device=DEV)
    q = workloads.integer_valued((R, 1, d), seed=67, lo=-3, hi=3, device=DEV)
    cache = torch.randint(0, 500, (R, C), device=DEV, generator=torch.Generator(DEV).manual_seed(2))
    idx = ralm.Index(x, oracle.IP, 8, 2)
    ids, scores = ralm.cache_search(idx, cache, q, 2)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    oi, osc = oracle.cache_search(x.cpu().numpy(), cache.cpu().numpy(), q.cpu().numpy(), oracle.IP, 2)
    assert np.array_equal(ids.cpu().numpy(), oi)
    assert np.array_equal(scores.cpu().numpy().astype(np.float64), osc)


def test_cache_over_all_ids_equals_search():
    """Rank preservation: a cache holding every row ranks exactly like the corpus search."""
    ralm = _ralm()
    x, _ = workloads.mixture_corpus(2048, 128, 8, seed=66, device=DEV)
    q, _ = workloads.noisy_copy_queries(x, 6, seed=67)
    idx = ralm.Index(x, oracle.IP, 8, 30)
    ids, scores = ralm.search(idx, q, 30)
    cache = torch.randperm(2048, device=DEV).reshape(1, 2048).repeat(2, 1).contiguous()
    cids, cscores = ralm.cache_search(idx, cache, q.reshape(2, 3, 128).contiguous(), 30)
    assert torch.equal(cids.reshape(6, 30), ids)
    torch.testing.assert_close(cscores.reshape(6, 30), scores, rtol=1e-5, atol=1e-6)


def test_bad_cache_id_sets_status_and_is_skipped():
    ralm = _ralm()
    x = workloads.integer_valued((100, 8), seed=68, device=DEV)
    q = workloads.integer_valued((1, 1, 8), seed=69, device=DEV)
    cache = torch.tensor([[3, 100, 7, -5]], dtype=torch.int64, device=DEV)
    idx = ralm.Index(x, oracle.IP, 1, 4)
    ids, _ = ralm.cache_search(idx, cache, q, 4)
    assert idx.device_status() == 6          # RALM_ERR_BAD_CACHE_ID, then cleared
    assert idx.device_status() == 0
    assert sorted(ids[0, 0, :2].tolist()) == [3, 7] and ids[0, 0, 2:].tolist() == [-1, -1]


# ------------------------------------------------------------------ verify
def test_verify_paper_toy_example():
    ralm = _ralm()
    for line in open(os.path.join(GOLDEN, "verify_toy_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        stride, spec, retr, want = [f.strip() for f in line.split("|")]
        sp = torch.tensor([[int(v) for v in spec.split()]], dtype=torch.int64, device=DEV)
        rt = torch.tensor([[int(v) for v in retr.split()]], dtype=torch.int64, device=DEV)
        assert ralm.verify(sp, rt).tolist() == [int(want)]


@pytest.mark.parametrize("R,stride,ld,cmp_k", [(1, 3, 1, 1), (8, 8, 20, 1), (64, 8, 20, 1), (5, 100, 4, 3),
                                               (1000, 33, 2, 2), (7, 1, 1, 1)])
def test_verify_bit_exact(R, stride, ld, cmp_k):
    ralm = _ralm()
    g = torch.Generator(DEV).manual_seed(R * 131 + stride)
    retr = torch.randint(0, 1 << 40, (R, stride, ld), device=DEV, generator=g)
    spec = retr[:, :, :cmp_k].clone()
    flip = torch.rand((R, stride, cmp_k), device=DEV, generator=g) < 0.15
    spec = torch.where(flip, spec + 1, spec).contiguous()
    spec[0] = retr[0, :, :cmp_k]                 # at least one full match
    got = ralm.verify(spec, retr, cmp_k=cmp_k)
    want = oracle.verify(spec.cpu().numpy(), retr.cpu().numpy(), cmp_k=cmp_k)
    assert np.array_equal(got.cpu().numpy(), want)
    assert got[0].item() == stride


def test_verify_zero_stride_and_zero_requests():
    ralm = _ralm()
    spec = torch.empty((3, 0), dtype=torch.int64, device=DEV)
    retr = torch.empty((3, 0, 1), dtype=torch.int64, device=DEV)
    assert ralm.verify(spec, retr).tolist() == [0, 0, 0]
    assert ralm.verify(spec[:0], retr[:0]).shape == (0,)


def test_verify_expected_verified_documents_closed_form():
    """Bernoulli(gamma) speculation: E[min(m + 1, s)] = (1 - gamma^s) / (1 - gamma)."""
    ralm = _ralm()
    gamma, stride, R = 0.6, 8, 100_000
    retr = torch.arange(R * stride, dtype=torch.int64, device=DEV).reshape(R, stride)
    spec = workloads.bernoulli_speculation(retr, gamma, seed=71)
    m = ralm.verify(spec, retr).double()
    verified = torch.clamp(m + 1, max=stride)
    closed = (1 - gamma ** stride) / (1 - gamma)
    assert abs(verified.mean().item() - closed) < 4 * verified.std().item() / R ** 0.5


# ------------------------------------------------------------------ the chained step
def test_speculate_search_verify_chain():
    """One verification step as the serving loop runs it, all on one stream: cache lookup
    (speculation), batched search (verification retrieval), first-mismatch."""
    ralm = _ralm()
    R, stride, C, k, d, N = 8, 8, 512, 20, 768, 300_000
    x, assign = workloads.mixture_corpus(N, d, 256, seed=72, device=DEV)
    q, src = workloads.noisy_copy_queries(x, R * stride, seed=73)
    cache = workloads.speculation_cache_ids(assign, N, src.reshape(R, stride), C, seed=74, n_centres=256)
    idx = ralm.Index(x, oracle.IP, R * stride, k)
    spec_ids, _ = ralm.cache_search(idx, cache, q.reshape(R, stride, d).contiguous(), 1)
    retr_ids, retr_scores = ralm.search(idx, q, k)
    m = ralm.verify(spec_ids.reshape(R, stride).contiguous(), retr_ids.reshape(R, stride, k).contiguous())
    torch.cuda.synchronize()
    # verify is integer-only: bit-exact given the GPU's own ids
    want = oracle.verify(spec_ids.reshape(R, stride).cpu().numpy(), retr_ids.reshape(R, stride, k).cpu().numpy())
    assert np.array_equal(m.cpu().numpy(), want)
    # and the whole chain equals the all-oracle pipeline (noisy copies: rank 0 is never a near tie)
    xn, qn = x.cpu().numpy(), q.cpu().numpy()
    o_spec, _ = oracle.cache_search(xn, cache.cpu().numpy(), qn.reshape(R, stride, d), oracle.IP, 1)
    o_retr, _ = oracle.search(xn, qn, oracle.IP, k)
    o_m = oracle.verify(o_spec.reshape(R, stride), o_retr.reshape(R, stride, k))
    assert np.array_equal(m.cpu().numpy(), o_m)
    assert 0 < (o_m < stride).sum() and o_m.max() >= 1     # mismatches and matches both occur
    assert idx.device_status() == 0


# ------------------------------------------------------------------ cache update
@pytest.mark.parametrize("R,C,stride,ld,top,next_n", [(1, 4, 4, 2, 1, 0), (8, 512, 8, 20, 1, 0), (8, 512, 8, 20, 20, 0),
                                                      (3, 37, 5, 6, 4, 0), (4, 64, 8, 4, 2, 10), (2, 4096, 3, 64, 64, 0),
                                                      (5, 1, 2, 3, 3, 0), (2, 16, 4, 1024, 1024, 0)])
def test_cache_update_is_bit_exact(R, C, stride, ld, top, next_n):
    from oracle.cache_update import cache_update as oracle_update
    ralm = _ralm()
    g = torch.Generator().manual_seed(1000 * R + C + stride)
    N = 3 * C + 50
    cache = torch.stack([torch.randperm(N, generator=g)[:C] for _ in range(R)]).to(torch.int64)
    cache[torch.rand(cache.shape, generator=g) < 0.3] = -1
    cursor = torch.randint(0, C, (R,), generator=g, dtype=torch.int32)
    retrieved = torch.randint(-1, N, (R, stride, ld), generator=g, dtype=torch.int64)
    steps = torch.randint(0, stride + 2, (R,), generator=g, dtype=torch.int32)      # also beyond stride: clamped
    for use_steps in (True, False):
        want_cache, want_cur = oracle_update(cache.numpy(), cursor.numpy(), retrieved.numpy(), top,
                                             steps.numpy() if use_steps else None, next_n, N)
        d_cache, d_cur = cache.to(DEV), cursor.to(DEV)
        ralm.cache_update(d_cache, d_cur, retrieved.to(DEV), top, N, steps.to(DEV) if use_steps else None, next_n)
        torch.cuda.synchronize()
        assert np.array_equal(d_cache.cpu().numpy(), want_cache)
        assert np.array_equal(d_cur.cpu().numpy(), want_cur)


def test_cache_update_closes_the_speculation_loop():
    """After the retrieved documents enter the caches, speculating the same queries again finds
    them: every step matches and first_mismatch equals the stride."""
    ralm = _ralm()
    N, d, R, stride, C = 80_000, 256, 4, 8, 128
    x, assign = workloads.mixture_corpus(N, d, 64, seed=81, device=DEV)
    q, src = workloads.noisy_copy_queries(x, R * stride, seed=82)
    idx = ralm.Index(x, oracle.IP, R * stride, 5)
    cache = torch.full((R, C), -1, dtype=torch.int64, device=DEV)
    cursor = torch.zeros((R,), dtype=torch.int32, device=DEV)
    qr = q.reshape(R, stride, d).contiguous()
    spec, _ = ralm.cache_search(idx, cache, qr, 1)
    retr, _ = ralm.search(idx, q, 5)
    retr = retr.reshape(R, stride, 5).contiguous()
    m = ralm.verify(spec.reshape(R, stride).contiguous(), retr)
    assert m.tolist() == [0] * R                                    # empty caches: nothing matches
    ralm.cache_update(cache, cursor, retr, 5, N)                    # top-k update with all steps
    spec, _ = ralm.cache_search(idx, cache, qr, 1)
    m = ralm.verify(spec.reshape(R, stride).contiguous(), retr)
    torch.cuda.synchronize()
    assert m.tolist() == [stride] * R
    assert cursor.tolist() == [int((cache[r] >= 0).sum()) % C for r in range(R)]
    # argument errors
    with pytest.raises(ralm.RalmError):
        ralm.cache_update(cache, cursor, retr, 6, N)                # top > ld
