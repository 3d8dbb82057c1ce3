"""GPU parity of the 8-bit (E5M2) corpus scan: ralm_search on an index with ralm_index_enable_q8
against the fp64 oracle, through the C ABI. The 8-bit copy only filters; every (row, query) pair
it lets through is scored again from the fp16 row, so the results must be those of the plain
definition: the oracle is the same exact top-k as for every other path (Section 5.1: the exact
dense retriever), with no tolerance of its own."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import check_search

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _search(x, q, k, q8, metric=oracle.IP):
    import paper_2401_14021_b200 as ralm
    idx = ralm.Index(x, metric, max_s=max(1, q.shape[0]), max_k=k)
    if q8:
        # (forced: most of these corpora are too small for the sample phase, without which the
        # library would keep the fp16 scan)
        idx.enable_q8(force=True)
        idx.enable_q8(force=True)            # a second call builds nothing
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    launches = idx.launch_count()
    idx.close()
    return ids, scores, launches


# Integers up to 20 in magnitude: 9, 11, 13, 15, 17, 18, 19 have no E5M2 value, so the stored
# bound is non-zero and the filter really decides; every score is still an exact fp32 integer
# and ties abound, so ids (tie-break included) and scores must equal the oracle's bit for bit.
@pytest.mark.parametrize("N,d,s,k", [(1, 16, 1, 1), (15, 16, 3, 4), (17, 64, 8, 1), (33, 48, 2, 40),
                                     (1000, 80, 8, 7), (5000, 768, 4, 5), (3001, 1024, 5, 256),
                                     (40_000, 208, 8, 20), (9000, 128, 7, 1), (100_003, 768, 8, 1),
                                     (2_500_000, 64, 8, 1), (2_500_000, 64, 8, 20), (2_450_001, 32, 3, 100),
                                     (700, 48, 9, 1), (5000, 768, 16, 5), (40_000, 208, 12, 64), (33, 64, 16, 40),
                                     (2_450_000, 32, 16, 1), (2_450_000, 32, 13, 20)])
def test_q8_integer_inputs_are_bit_exact(N, d, s, k):
    x = workloads.integer_valued((N, d), seed=1100 + N % 1000 + d, lo=-20, hi=20, device=DEV)
    q = workloads.integer_valued((s, d), seed=1200 + N % 1000 + d, lo=-20, hi=20, device=DEV)
    ids, scores, _ = _search(x, q, k, q8=True)
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, k, exact=True)


@pytest.mark.parametrize("N,d,s,k", [(120_001, 768, 8, 20), (2_450_000, 128, 8, 1), (2_450_000, 128, 5, 20),
                                     (2_450_000, 128, 16, 20), (60_000, 768, 11, 1)])
def test_q8_mixture_rows_match_the_oracle_and_the_fp16_scan(N, d, s, k):
    """Real-valued mixture rows (near-ties inside a cluster): the band rule against the oracle,
    the planted source at rank 0, and the same ranking as the fp16 scan."""
    x, _ = workloads.mixture_corpus(N, d, 64, seed=1300 + d, device=DEV)
    q, src = workloads.noisy_copy_queries(x, s, seed=1301 + d)
    ids, scores, _ = _search(x, q, k, q8=True)
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, k)
    assert ids[:, 0].tolist() == src.tolist()
    ids16, scores16, _ = _search(x, q, k, q8=False)
    assert torch.equal(ids[:, 0], ids16[:, 0])
    torch.testing.assert_close(scores, scores16, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("N,d", [(3000, 64), (2_450_000, 32)])
def test_q8_bound_is_tight_where_the_rounding_error_is_parallel_to_the_query(N, d):
    """The worst case of the Cauchy-Schwarz bound. One row is all 9s: E5M2 stores 8 (9 is the
    midpoint of 8 and 10), so with an all-ones query its 8-bit score is 8 d while its true score
    is 9 d, and the difference equals |q| |x - x8| exactly. Every other row is made of 8s and 10s,
    which E5M2 holds exactly, with scores up to 9 d - 2: above the planted row's 8-bit score, below
    its true one. A bound that is the least bit too small drops the planted row."""
    g = torch.Generator(device=DEV).manual_seed(1700 + d)
    tens = torch.rand((N, d), generator=g, device=DEV) < 0.3
    x = torch.where(tens, 10.0, 8.0).to(torch.float16)
    # cap every decoy at d/2 - 1 tens: score <= 8 d + 2 (d/2 - 1) = 9 d - 2
    over = tens.sum(dim=1) > d // 2 - 1
    x[over] = 8.0
    planted = N - 7                                      # in the part the 8-bit launch covers
    x[planted] = 9.0
    x[5, : d // 2 - 1] = 10.0                            # the best decoy, in the sample part
    x[5, d // 2 - 1:] = 8.0
    q = torch.ones((3, d), dtype=torch.float16, device=DEV)
    q[1] = 2.0
    q[2, ::2] = 0.0                                      # half of the coordinates
    for k in (1, 5):
        ids, scores, _ = _search(x, q, k, q8=True)
        check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, k, exact=True)
        assert ids[0, 0].item() == planted and scores[0, 0].item() == 9.0 * d


def test_q8_large_values_saturate_without_losing_rows():
    """fp16 values beyond the largest finite E5M2 value (57344) are stored saturated; the bound
    covers the difference, so the row that holds them is still found."""
    N, d = 4000, 64
    x = workloads.integer_valued((N, d), seed=1400, lo=-4, hi=4, device=DEV)
    x[1234, 5] = 65504.0
    x[77, 9] = -65504.0
    q = torch.zeros((2, d), dtype=torch.float16, device=DEV)
    q[0, 5] = 1.0
    q[1, 9] = -1.0
    ids, scores, _ = _search(x, q, 3, q8=True)
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, 3, exact=True)
    assert ids[0, 0].item() == 1234 and ids[1, 0].item() == 77


def test_q8_unforced_small_corpus_keeps_the_fp16_scan_and_large_one_uses_the_copy():
    import paper_2401_14021_b200 as ralm
    for N, uses in ((200_000, False), (2_450_000, True)):
        x = workloads.integer_valued((N, 32), seed=1600, lo=-20, hi=20, device=DEV)
        q = workloads.integer_valued((8, 32), seed=1601, lo=-20, hi=20, device=DEV)
        idx = ralm.Index(x, oracle.IP, max_s=8, max_k=1)
        idx.enable_q8()
        before = idx.launch_count()
        ids, scores = ralm.search(idx, q, 1)
        torch.cuda.synchronize()
        # the 8-bit path is sample scan + merge + 8-bit scan + merge; the plain top-1 scan is 2 launches
        assert (idx.launch_count() - before == 4) == uses
        idx.close()
        check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, 1, exact=True)


def test_q8_is_refused_where_it_does_not_apply_and_falls_back_where_it_cannot_serve():
    import paper_2401_14021_b200 as ralm
    x = workloads.integer_valued((500, 24), seed=1500, lo=-3, hi=3, device=DEV)
    idx = ralm.Index(x, oracle.IP, max_s=4, max_k=4)      # d % 16 != 0
    with pytest.raises(ralm.RalmError):
        idx.enable_q8()
    idx.close()
    x = workloads.integer_valued((500, 32), seed=1501, lo=-3, hi=3, device=DEV)
    # k beyond the 8-bit scan's limits (up to 8 queries: 256, more where the index keeps its lists in
    # global memory; 9..16 queries: 64) and batches of more than 16 queries take the fp16 scans
    q = workloads.integer_valued((20, 32), seed=1502, lo=-3, hi=3, device=DEV)
    for s, k in ((4, 300), (12, 65), (20, 5)):
        ids, scores, _ = _search(x, q[:s].contiguous(), k, q8=True)
        check_search(ids, scores, x.cpu().numpy(), q[:s].cpu().numpy(), oracle.IP, k, exact=True)


# ---- L2 (the KNN-LM datastore's metric): the same filter on x.q bounds the squared distance from
# below; what passes is scored again in the direct form. Integer rows: distances are exact
# integers, ties abound, ids and distances must equal the oracle's bit for bit, also with lists
# that live in global memory (k > 256) and with planted zero-distance copies.
@pytest.mark.parametrize("N,d,s,k", [(1, 16, 1, 1), (17, 64, 8, 1), (33, 48, 2, 40), (5000, 768, 4, 5),
                                     (3001, 1024, 4, 1024), (40_000, 208, 8, 300), (100_003, 768, 8, 1),
                                     (2_500_000, 64, 8, 20), (2_450_001, 32, 3, 600), (5000, 768, 16, 5),
                                     (2_450_000, 32, 13, 20)])
def test_q8_l2_integer_inputs_are_bit_exact(N, d, s, k):
    x = workloads.integer_valued((N, d), seed=1500 + N % 1000 + d, lo=-20, hi=20, device=DEV)
    q = workloads.integer_valued((s, d), seed=1600 + N % 1000 + d, lo=-20, hi=20, device=DEV)
    if N > s:
        q[0] = x[N // 2]                       # an exact copy: distance 0, ranked first
    ids, scores, _ = _search(x, q, k, q8=True, metric=oracle.L2)
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.L2, k, exact=True)


@pytest.mark.parametrize("N,d,s,k", [(120_001, 1024, 4, 1024), (2_450_000, 128, 8, 1), (2_450_000, 128, 4, 20),
                                     (2_450_000, 128, 16, 20)])
def test_q8_l2_unnormalised_rows_match_the_oracle_and_the_fp16_scan(N, d, s, k):
    """Rows shaped like the KNN-LM keys (mixture, unnormalised, log-normal norms): the band rule
    against the oracle, the planted source first, and the fp16 L2 scan's ranking and distances."""
    x, _ = workloads.mixture_corpus(N, d, 256, seed=1700 + d, device=DEV, normalise=False, lognormal_sigma=0.3)
    q, src = workloads.noisy_copy_queries(x, s, seed=1701 + d)
    ids, scores, launches = _search(x, q, k, q8=True, metric=oracle.L2)
    counts = check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), oracle.L2, k)
    assert counts.wide == 0, str(counts)
    assert ids[:, 0].tolist() == src.tolist()
    ids16, scores16, _ = _search(x, q, k, q8=False, metric=oracle.L2)
    assert torch.equal(ids[:, 0], ids16[:, 0])
    torch.testing.assert_close(scores, scores16, rtol=1e-5, atol=1e-5)


def test_q8_l2_dispatch_is_the_8bit_scan():
    import paper_2401_14021_b200 as ralm
    x, _ = workloads.mixture_corpus(50_000, 128, 64, seed=1800, device=DEV, normalise=False, lognormal_sigma=0.3)
    q, _ = workloads.noisy_copy_queries(x, 4, seed=1801)
    idx = ralm.Index(x, oracle.L2, max_s=4, max_k=8)
    ralm.search(idx, q, 8)
    assert idx.last_dispatch()["kernel"] == 2          # the fp16 warp-MMA scan
    idx.enable_q8(force=True)
    ralm.search(idx, q, 8)
    assert idx.last_dispatch()["kernel_name"] == "scan_q8_kernel"
    idx.close()
