"""GPU parity on seeded random shapes: ralm_search (automatic variant choice) against the fp64
oracle, through the C ABI. The fixed parametrisations elsewhere sit on the boundaries somebody
thought of; this sweep draws N, d, s, k and the metric at random so that the dispatch between
the small-batch scan (1, 2 or 4 query groups per pass), the tcgen05 scan, one- and two-phase
scanning, shared- and global-memory candidate lists and the padding rules is crossed at
arbitrary points. Integer-valued rows make every score exact in fp32, so ids (tie-break
included) and scores must match the oracle bit for bit; a few real-valued cases use the
near-tie band rule."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import check_search

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
MAC_BUDGET = 1.2e9   # multiply-adds the oracle may spend on one case (about a second)


def _cases(n_cases: int, seed: int):
    rng = np.random.RandomState(seed)
    out = []
    while len(out) < n_cases:
        metric = oracle.IP if rng.rand() < 0.5 else oracle.L2
        d = 8 * int(rng.choice([1, 2, 3, 8, 9, 16, 33, 64, 96, 128, 160, 192]))
        s = int(rng.choice([1, 2, 3, 5, 8, 9, 12, 16, 17, 24, 32, 33, 47, 64, 100, 257, 300, 513]))
        k_hi = 1024 if s <= 8 else 64 if s > 32 else 300
        k = int(min(k_hi, rng.choice([1, 2, 5, 20, 31, 32, 33, 64, 65, 100, 256, 257, 1024])))
        n_hi = int(min(900_000, MAC_BUDGET / (d * s)))
        if n_hi < 1:
            continue
        # log-uniform N, with a share of very small corpora (N < k: padded outputs)
        N = int(np.exp(rng.uniform(0.0, np.log(n_hi)))) if rng.rand() < 0.8 else n_hi
        out.append((metric, max(1, N), d, s, k))
    return out


CASES = _cases(48, seed=20240114)


@pytest.mark.parametrize("case", range(len(CASES)))
def test_random_shape_integer_inputs_are_bit_exact(case):
    import paper_2401_14021_b200 as ralm
    metric, N, d, s, k = CASES[case]
    x = workloads.integer_valued((N, d), seed=9000 + case, lo=-2, hi=2, device=DEV)
    q = workloads.integer_valued((s, d), seed=9500 + case, lo=-2, hi=2, device=DEV)
    idx = ralm.Index(x, metric, max_s=s, max_k=k)
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    # a second call on the same index (workspace reused, thresholds reset) gives the same lists
    ids2, scores2 = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    idx.close()
    assert torch.equal(ids, ids2) and torch.equal(scores, scores2), (metric, N, d, s, k)
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), metric, k, exact=True)


REAL_CASES = [(oracle.IP, 70_001, 768, 8, 20), (oracle.IP, 300_017, 264, 24, 7), (oracle.L2, 50_003, 1024, 5, 300),
              (oracle.L2, 640_000, 64, 20, 9), (oracle.IP, 640_000, 64, 40, 33), (oracle.L2, 90_000, 200, 16, 64)]


@pytest.mark.parametrize("metric,N,d,s,k", REAL_CASES)
def test_random_shape_mixture_rows(metric, N, d, s, k):
    import paper_2401_14021_b200 as ralm
    l2 = metric == oracle.L2
    x, _ = workloads.mixture_corpus(N, d, 32, seed=700 + d, device=DEV, normalise=not l2,
                                    lognormal_sigma=0.3 if l2 else 0.0)
    q, src = workloads.noisy_copy_queries(x, s, seed=701 + d)
    idx = ralm.Index(x, metric, max_s=s, max_k=k)
    ids, scores = ralm.search(idx, q, k)
    torch.cuda.synchronize()
    assert idx.device_status() == 0
    idx.close()
    check_search(ids, scores, x.cpu().numpy(), q.cpu().numpy(), metric, k)
    assert ids[:, 0].tolist() == src.tolist()
