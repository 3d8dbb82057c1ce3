"""Pins for the CPU oracle: each test ties it to something other than itself.

P1  exhaustive pairwise definition of top-k with exact integer arithmetic
P2  planted duplicates (L2 distance exactly 0; lower id first on exact ties)
P3  output invariants (sorted, unique, in range, padding at the tail)
P4  exact rational recomputation of returned scores
P5  numpy float64 matmul + lexsort (library routine) on up to 1e4 rows
P6  rank preservation between cache and corpus (Section 3, "Speculative retrieval")
P7  the paper's worked verification example (tests/golden/verify_toy_example.txt)
P8  expected verified documents = (1 - g^s) / (1 - g) (Appendix A.2)
P9  batched retrieval == the sequential retrievals (Section 1; Algorithm 1)
plus the fp16 decoder against numpy's conversion on every finite bit pattern.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _np16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy()


# ---------------------------------------------------------------- fp16 decode
def test_half_decode_all_finite_patterns_match_numpy():
    bits = np.arange(1 << 16, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    finite = np.isfinite(ref)
    got = np.array([oracle.half_to_double(int(b)) for b in bits[finite]])
    assert np.array_equal(got, ref[finite])
    # sign of zero survives
    assert np.signbit(oracle.half_to_double(0x8000)) and oracle.half_to_double(0x8000) == 0.0


def test_half_decode_closed_forms():
    assert oracle.half_to_double(0x3C00) == 1.0
    assert oracle.half_to_double(0x0001) == 2.0 ** -24          # smallest subnormal
    assert oracle.half_to_double(0x03FF) == 1023 * 2.0 ** -24   # largest subnormal
    assert oracle.half_to_double(0x0400) == 2.0 ** -14          # smallest normal
    assert oracle.half_to_double(0x7BFF) == 65504.0             # largest finite
    assert oracle.half_to_double(0xBC00) == -1.0
    assert oracle.half_to_double(0x3555) == 1365 * 2.0 ** -12   # 0.333251953125


# ---------------------------------------------------------------- P1 exhaustive pairwise
def _exact_int_scores(x: np.ndarray, q: np.ndarray, metric: int):
    """Python-int scores of integer-valued rows; no floating point involved."""
    xi = [[int(v) for v in row] for row in x.astype(np.float64)]
    qi = [int(v) for v in q.astype(np.float64)]
    out = []
    for row in xi:
        if metric == oracle.IP:
            out.append(sum(a * b for a, b in zip(qi, row)))
        else:
            out.append(sum((a - b) * (a - b) for a, b in zip(qi, row)))
    return out


def _beats(sa, ia, sb, ib, metric):
    if sa != sb:
        return sa > sb if metric == oracle.IP else sa < sb
    return ia < ib


@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
@pytest.mark.parametrize("N,d,k", [(1, 8, 1), (7, 8, 3), (33, 16, 5), (64, 16, 64), (40, 8, 50)])
def test_p1_exhaustive_pairwise(metric, N, d, k):
    # small integers in [-2, 2] make many exact ties, so the id tie-break is exercised
    x = _np16(workloads.integer_valued((N, d), seed=11 + N, lo=-2, hi=2))
    q = _np16(workloads.integer_valued((3, d), seed=12 + N, lo=-2, hi=2))
    ids, sc = oracle.search(x, q, metric, k)
    for i in range(3):
        exact = _exact_int_scores(x, q[i], metric)
        # j is at rank p iff exactly p rows beat it under the total order
        n_beating = [sum(_beats(exact[o], o, exact[j], j, metric) for o in range(N) if o != j)
                     for j in range(N)]
        for p in range(k):
            if p < N:
                j = int(ids[i, p])
                assert n_beating[j] == p
                assert sc[i, p] == float(exact[j])
            else:
                assert ids[i, p] == -1
                assert sc[i, p] == (-np.inf if metric == oracle.IP else np.inf)


# ---------------------------------------------------------------- P2 planted duplicates
def test_p2_l2_duplicate_is_first_with_zero_distance():
    x, _ = workloads.mixture_corpus(2000, 64, 16, seed=5, normalise=False, lognormal_sigma=0.3)
    x = _np16(x)
    rows = [3, 777, 1999]
    ids, sc = oracle.search(x, x[rows], oracle.L2, 4)
    assert list(ids[:, 0]) == rows
    assert np.all(sc[:, 0] == 0.0)
    assert np.all(sc[:, 1] > 0.0)


def test_p2_ip_duplicate_first_on_normalised_rows_and_tie_order():
    x = _np16(workloads.unit_gaussian_corpus(3000, 64, seed=6)).copy()
    x[2500] = x[17]          # exact duplicate rows 17 < 2500
    ids, sc = oracle.search(x, x[[17, 123]], oracle.IP, 3)
    assert list(ids[0, :2]) == [17, 2500] and sc[0, 0] == sc[0, 1]
    assert ids[1, 0] == 123


# ---------------------------------------------------------------- P3 invariants
@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p3_invariants(metric):
    x, _ = workloads.mixture_corpus(5000, 64, 32, seed=7)
    q, _ = workloads.noisy_copy_queries(x, 5, seed=8)
    ids, sc = oracle.search(_np16(x), _np16(q), metric, 5003)
    for i in range(5):
        valid = ids[i] >= 0
        assert valid[:5000].all() and not valid[5000:].any()
        assert len(set(ids[i, :5000].tolist())) == 5000
        d = np.diff(sc[i, :5000])
        assert (d <= 0).all() if metric == oracle.IP else (d >= 0).all()
        assert np.all(np.isinf(sc[i, 5000:]))


# ---------------------------------------------------------------- P4 exact recomputation
def _fraction_of_half(bits: int) -> Fraction:
    sign = -1 if bits >> 15 else 1
    e, m = (bits >> 10) & 31, bits & 1023
    if e == 0:
        return sign * Fraction(m, 1 << 24)
    return sign * Fraction(1024 + m) * Fraction(2) ** (e - 25)


@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p4_scores_equal_exact_rational_sums(metric):
    x, _ = workloads.mixture_corpus(300, 96, 8, seed=9, normalise=False, lognormal_sigma=0.3)
    q, _ = workloads.noisy_copy_queries(x, 2, seed=10)
    xb, qb = _np16(x).view(np.uint16), _np16(q).view(np.uint16)
    ids, sc = oracle.search(xb, qb, metric, 10)
    for i in range(2):
        qf = [_fraction_of_half(int(b)) for b in qb[i]]
        for p in range(10):
            xf = [_fraction_of_half(int(b)) for b in xb[ids[i, p]]]
            if metric == oracle.IP:
                exact = sum(a * b for a, b in zip(qf, xf))
            else:
                exact = sum((a - b) ** 2 for a, b in zip(qf, xf))
            assert abs(Fraction(float(sc[i, p])) - exact) <= abs(exact) * Fraction(1, 10 ** 12)
            assert oracle.pair_score(xb[ids[i, p]], qb[i], metric) == sc[i, p]


# ---------------------------------------------------------------- P5 numpy matmul + lexsort
@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p5_matches_numpy_matmul_and_lexsort(metric):
    x, _ = workloads.mixture_corpus(10_000, 128, 64, seed=13)
    q, _ = workloads.noisy_copy_queries(x, 4, seed=14)
    xn, qn = _np16(x).astype(np.float64), _np16(q).astype(np.float64)
    if metric == oracle.IP:
        S = qn @ xn.T
        key = -S
    else:
        S = ((qn[:, None, :] - xn[None, :, :]) ** 2).sum(-1)
        key = S
    k = 50
    ids, sc = oracle.search(_np16(x), _np16(q), metric, k)
    for i in range(4):
        order = np.lexsort((np.arange(xn.shape[0]), key[i]))[:k]
        ref_s = S[i, order]
        # summation order differs (BLAS vs left-to-right): compare ids where the library's
        # own scores separate neighbours by more than its rounding, scores to 1e-12
        np.testing.assert_allclose(sc[i], ref_s, rtol=1e-12, atol=1e-12)
        gaps = np.abs(np.diff(np.concatenate([ref_s, S[i, np.lexsort((np.arange(xn.shape[0]), key[i]))[k:k + 1]]])))
        clear = gaps > 1e-10
        assert np.array_equal(ids[i][clear], order[clear])
        assert set(ids[i].tolist()) == set(order.tolist()) or not clear.all()


# ---------------------------------------------------------------- P6 rank preservation
@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p6_cache_over_all_ids_equals_search(metric):
    x, _ = workloads.mixture_corpus(257, 32, 4, seed=15)
    q, _ = workloads.noisy_copy_queries(x, 6, seed=16)
    ids, sc = oracle.search(_np16(x), _np16(q), metric, 9)
    perm = np.random.default_rng(0).permutation(257)
    cache = np.stack([perm, perm[::-1]])                      # R = 2, both hold every id
    qs = _np16(q).reshape(2, 3, 32)
    cids, csc = oracle.cache_search(_np16(x), cache, qs, metric, 9)
    assert np.array_equal(cids.reshape(6, 9), ids)
    assert np.array_equal(csc.reshape(6, 9), sc)


@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p6_cache_ranking_is_corpus_ranking_restricted(metric):
    x, assign = workloads.mixture_corpus(4000, 64, 16, seed=17)
    q, src = workloads.noisy_copy_queries(x, 8, seed=18)
    cache = workloads.speculation_cache_ids(assign, 4000, src.reshape(2, 4), 48, seed=19,
                                            n_centres=16, empty_slots=5)
    full_ids, _ = oracle.search(_np16(x), _np16(q), metric, 4000)
    cids, _ = oracle.cache_search(_np16(x), _np16(cache), _np16(q).reshape(2, 4, 64), metric, 48)
    for r in range(2):
        members = set(int(v) for v in _np16(cache)[r] if v >= 0)
        assert len(members) == 43
        for u in range(4):
            restricted = [j for j in full_ids[r * 4 + u].tolist() if j in members]
            got = cids[r, u].tolist()
            assert got[:len(restricted)] == restricted
            assert all(v == -1 for v in got[len(restricted):])
            # top-ranked corpus entry in the cache => it tops the cache ranking too
            if int(full_ids[r * 4 + u, 0]) in members:
                assert got[0] == int(full_ids[r * 4 + u, 0])


def test_cache_set_semantics_and_out_of_range_ids():
    x = _np16(workloads.integer_valued((10, 8), seed=20))
    q = _np16(workloads.integer_valued((1, 1, 8), seed=21))
    cache = np.array([[3, 3, -1, 7, 10, 99, -5, 7]], dtype=np.int64)   # set {3, 7}
    ids, sc = oracle.cache_search(x, cache, q, oracle.IP, 4)
    assert sorted(ids[0, 0, :2].tolist()) == [3, 7] and list(ids[0, 0, 2:]) == [-1, -1]
    empty, esc = oracle.cache_search(x, np.full((1, 4), -1), q, oracle.L2, 2)
    assert list(empty[0, 0]) == [-1, -1] and np.all(esc == np.inf)


# ---------------------------------------------------------------- P7 worked example
def test_p7_paper_toy_example():
    rows = []
    with open(os.path.join(GOLDEN, "verify_toy_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            stride, spec, retr, want = [f.strip() for f in line.split("|")]
            rows.append((int(stride), [int(v) for v in spec.split()],
                         [int(v) for v in retr.split()], int(want)))
    assert len(rows) == 2
    for stride, spec, retr, want in rows:
        got = oracle.verify(np.array([spec]), np.array([retr]))
        assert got.tolist() == [want]


def test_verify_positions_pitch_and_cmp_k():
    retr = np.arange(2 * 4 * 5).reshape(2, 4, 5)            # R=2, stride=4, ld=5
    spec = retr[:, :, 0].copy()
    assert oracle.verify(spec, retr).tolist() == [4, 4]
    spec[0, 0] = -1
    spec[1, 3] = -1
    assert oracle.verify(spec, retr).tolist() == [0, 3]
    spec2 = retr[:, :, :2].copy()                            # cmp_k = 2
    spec2[1, 1, 1] += 1                                      # only the second id differs
    assert oracle.verify(spec2, retr, cmp_k=2).tolist() == [4, 1]
    assert oracle.verify(spec2[:, :, :1], retr, cmp_k=1).tolist() == [4, 4]
    assert oracle.verify(np.zeros((3, 0), dtype=np.int64), np.zeros((3, 0, 1), dtype=np.int64)).tolist() == [0, 0, 0]


# ---------------------------------------------------------------- P8 closed form
@pytest.mark.parametrize("gamma,stride", [(0.6, 3), (0.3, 8), (0.9, 4)])
def test_p8_expected_verified_documents(gamma, stride):
    R = 200_000
    retrieved = torch.arange(R * stride, dtype=torch.int64).reshape(R, stride)
    spec = workloads.bernoulli_speculation(retrieved, gamma, seed=31)
    m = oracle.verify(_np16(spec), _np16(retrieved)).astype(np.float64)
    # documents verified per step: the matched prefix plus the corrected one, at most s
    verified = np.minimum(m + 1, stride)
    closed = (1 - gamma ** stride) / (1 - gamma)
    assert abs(verified.mean() - closed) < 4 * verified.std() / np.sqrt(R) + 1e-9
    # P(first mismatch at i) = gamma^i (1 - gamma)
    for i in range(stride):
        assert abs((m == i).mean() - gamma ** i * (1 - gamma)) < 0.01
    assert abs((m == stride).mean() - gamma ** stride) < 0.01


# ---------------------------------------------------------------- P9 batch independence
@pytest.mark.parametrize("metric", [oracle.IP, oracle.L2])
def test_p9_batched_equals_sequential(metric):
    x, _ = workloads.mixture_corpus(3000, 64, 16, seed=23)
    q, _ = workloads.noisy_copy_queries(x, 8, seed=24)
    ids, sc = oracle.search(_np16(x), _np16(q), metric, 20)
    for i in range(8):
        one_ids, one_sc = oracle.search(_np16(x), _np16(q)[i:i + 1], metric, 20)
        assert np.array_equal(one_ids[0], ids[i]) and np.array_equal(one_sc[0], sc[i])
    # thread count never changes the result
    ids1, sc1 = oracle.search(_np16(x), _np16(q), metric, 20, threads=1)
    assert np.array_equal(ids1, ids) and np.array_equal(sc1, sc)


def test_scores_then_rank_equals_search_in_chunks():
    x, _ = workloads.mixture_corpus(2500, 64, 16, seed=25)
    q, _ = workloads.noisy_copy_queries(x, 2, seed=26)
    xn, qn = _np16(x), _np16(q)
    ids, sc = oracle.search(xn, qn, oracle.IP, 7)
    for i in range(2):
        allsc = np.empty(2500)
        for lo in range(0, 2500, 1000):
            oracle.scores(xn[lo:lo + 1000], qn[i], oracle.IP, out=allsc[lo:lo + 1000])
        rid, rsc = oracle.rank(allsc, oracle.IP, 7)
        assert np.array_equal(rid, ids[i]) and np.array_equal(rsc, sc[i])


def test_empty_inputs():
    x = np.zeros((0, 8), dtype=np.uint16)
    q = np.zeros((2, 8), dtype=np.uint16)
    ids, sc = oracle.search(x, q, oracle.IP, 3)
    assert np.all(ids == -1) and np.all(sc == -np.inf)
    ids, sc = oracle.search(np.zeros((4, 8), dtype=np.uint16), np.zeros((0, 8), dtype=np.uint16), oracle.L2, 3)
    assert ids.shape == (0, 3)
