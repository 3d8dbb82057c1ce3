"""GPU parity at full size for the KNN-LM datastore configuration (50 M x 1024 fp16, L2, k = 1024):
a file of its own, so that the 32 GB corpus of the other full-size tests is released before this
one allocates 102 GB and, for the 8-bit filter copy, 52 GB more. The check is the sampled one of
tests/parity.py (sampled_parity)."""
import pytest
import torch

import oracle
import workloads
from parity import sampled_parity as _sampled_parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ralm():
    import paper_2401_14021_b200 as ralm
    return ralm


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
    torch.cuda.empty_cache()
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
