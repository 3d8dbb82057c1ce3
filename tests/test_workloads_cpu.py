"""The input generators: same seed, same bytes; chunks can be regenerated on their own; the
recipe's structure (unit norms, distinct sources, cache contents) holds."""
import torch

import workloads


def test_same_seed_same_bytes_and_chunks_regenerate_alone():
    a, asg = workloads.mixture_corpus(5000, 64, 16, seed=7, chunk_rows=2048)
    b, bsg = workloads.mixture_corpus(5000, 64, 16, seed=7, chunk_rows=2048)
    assert torch.equal(a, b) and torch.equal(asg, bsg)
    c, _ = workloads.mixture_corpus(5000, 64, 16, seed=8, chunk_rows=2048)
    assert not torch.equal(a, c)
    # the first chunk of a longer corpus is the same bytes (chunk b depends on seed and b only)
    d, _ = workloads.mixture_corpus(2048, 64, 16, seed=7, chunk_rows=2048)
    assert torch.equal(a[:2048], d)


def test_recipe_structure():
    x = workloads.unit_gaussian_corpus(3000, 96, seed=3)
    assert x.dtype == torch.float16
    assert torch.allclose(x.float().norm(dim=1), torch.ones(3000), atol=2e-3)
    m, assign = workloads.mixture_corpus(4000, 96, 8, seed=4)
    assert assign.min() >= 0 and assign.max() < 8 and torch.isfinite(m.float()).all()
    raw, _ = workloads.mixture_corpus(4000, 96, 8, seed=4, normalise=False, lognormal_sigma=0.3)
    norms = raw.float().norm(dim=1)
    assert norms.std() / norms.mean() > 0.15                   # log-normal spread of the row norms
    q, src = workloads.noisy_copy_queries(m, 16, seed=5)
    assert src.unique().numel() == 16                          # distinct source rows
    cos = torch.nn.functional.cosine_similarity(q.float(), m[src].float(), dim=1)
    assert (cos > 0.98).all()                                  # noise of relative norm 0.1
    cache = workloads.speculation_cache_ids(assign, 4000, src.reshape(2, 8), 128, seed=6, n_centres=8, empty_slots=5)
    for r in range(2):
        held = cache[r][cache[r] >= 0]
        assert held.numel() == 123 and held.unique().numel() == 123 and held.max() < 4000
    vals = workloads.integer_valued((50, 8), seed=9, lo=-3, hi=3)
    assert vals.dtype == torch.float16 and set(vals.flatten().tolist()) <= set(range(-3, 4))
    hits = workloads.bernoulli_speculation(torch.arange(1000).reshape(10, 100), 0.6, seed=10)
    frac = (hits >= 0).float().mean().item()
    assert 0.5 < frac < 0.7
