"""Input generators (no retrieval arithmetic here; see the package docstring)."""
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

CHUNK_ROWS = 1 << 20
_SEED_BASE = 240114000


def seed_for(config_index: int, what: str = "corpus") -> int:
    """Seeds: corpus = base + 10*c, queries = corpus + 1, caches = corpus + 2."""
    off = {"corpus": 0, "queries": 1, "caches": 2, "speculation": 3}[what]
    return _SEED_BASE + 10 * config_index + off


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    index: int
    N: int
    d: int
    metric: str            # "ip" | "l2"
    corpus: str            # "unit_gaussian" | "mixture"
    n_centres: int = 0
    sigma_within: float = 0.2
    normalise: bool = True
    lognormal_sigma: float = 0.0
    s_values: Tuple[int, ...] = (4,)
    k_values: Tuple[int, ...] = (1,)
    requests: int = 0
    cache_entries: int = 0
    stride: int = 0


CONFIGS = {
    "C1": WorkloadConfig("C1", 1, 100_000, 768, "ip", "unit_gaussian", s_values=(4,),
                         k_values=(1, 5), requests=1, cache_entries=64, stride=4),
    "C2": WorkloadConfig("C2", 2, 1_000_000, 768, "ip", "mixture", n_centres=1024,
                         s_values=(1, 2, 4, 8), k_values=(1, 20)),
    "C3": WorkloadConfig("C3", 3, 21_000_000, 768, "ip", "mixture", n_centres=1024,
                         s_values=(1, 2, 3, 4, 5, 6, 7, 8), k_values=(1, 20), requests=8,
                         cache_entries=512, stride=8),
    "C4": WorkloadConfig("C4", 4, 50_000_000, 1024, "l2", "mixture", n_centres=4096,
                         normalise=False, lognormal_sigma=0.3, s_values=(4,),
                         k_values=(1024,)),
    "C5": WorkloadConfig("C5", 3, 21_000_000, 768, "ip", "mixture", n_centres=1024,
                         s_values=(512,), k_values=(20,), requests=64, cache_entries=512,
                         stride=8),
}


def _gen(seed: int, chunk: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + chunk) % (2 ** 63 - 1))
    return g


def _range(N: int, row_range) -> Tuple[int, int]:
    lo, hi = (0, N) if row_range is None else row_range
    if not 0 <= lo <= hi <= N:
        raise ValueError("row_range outside the corpus")
    return lo, hi


def unit_gaussian_corpus(N: int, d: int, seed: int, device="cpu",
                         chunk_rows: int = CHUNK_ROWS, row_range=None) -> torch.Tensor:
    """Rows i.i.d. N(0, I_d), scaled to unit length in fp32, rounded to fp16.
    row_range = (lo, hi): only those rows of the N-row corpus (the same bytes the whole corpus
    holds there: every chunk is generated from its own seed)."""
    r_lo, r_hi = _range(N, row_range)
    out = torch.empty((r_hi - r_lo, d), dtype=torch.float16, device=device)
    for b, lo in enumerate(range(0, N, chunk_rows)):
        hi = min(N, lo + chunk_rows)
        if hi <= r_lo or lo >= r_hi:
            continue
        u = torch.randn((hi - lo, d), generator=_gen(seed, b, device), device=device,
                        dtype=torch.float32)
        u /= u.norm(dim=1, keepdim=True).clamp_min(1e-20)
        a, z = max(lo, r_lo), min(hi, r_hi)
        out[a - r_lo:z - r_lo] = u[a - lo:z - lo].to(torch.float16)
    return out


def mixture_corpus(N: int, d: int, n_centres: int, seed: int, device="cpu",
                   sigma_within: float = 0.2, normalise: bool = True,
                   lognormal_sigma: float = 0.0, clustered_order: bool = False,
                   chunk_rows: int = CHUNK_ROWS, row_range=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Gaussian-mixture corpus.

    Centres c_m ~ N(0, I_d). Row j picks a centre a_j uniformly and independently (so row
    order is NOT clustered unless `clustered_order`, which sorts the assignment to build
    the adversarial ordering), u_j = c_{a_j} + sigma_within * eps_j. Then either
    x_j = fp16(u_j / |u_j|) or, unnormalised, x_j = fp16(u_j * exp(lognormal_sigma * z_j)).
    Returns (corpus [N][d] fp16, assignment [N] int32). With row_range = (lo, hi) the corpus
    holds only those rows of the N-row corpus (the same bytes: every chunk is generated from its
    own seed); the assignment is still that of all N rows.
    """
    r_lo, r_hi = _range(N, row_range)
    centres = torch.randn((n_centres, d), generator=_gen(seed, 1_000_000, device),
                          device=device, dtype=torch.float32)
    out = torch.empty((r_hi - r_lo, d), dtype=torch.float16, device=device)
    assign = torch.empty((N,), dtype=torch.int32, device=device)
    for b, lo in enumerate(range(0, N, chunk_rows)):
        hi = min(N, lo + chunk_rows)
        g = _gen(seed, b, device)
        a = torch.randint(0, n_centres, (hi - lo,), generator=g, device=device)
        if clustered_order:
            a = (torch.arange(lo, hi, device=device) * n_centres) // max(N, 1)
        assign[lo:hi] = a.to(torch.int32)
        if hi <= r_lo or lo >= r_hi:
            continue
        u = torch.randn((hi - lo, d), generator=g, device=device, dtype=torch.float32)
        u.mul_(sigma_within).add_(centres[a])
        if normalise:
            u /= u.norm(dim=1, keepdim=True).clamp_min(1e-20)
        if lognormal_sigma > 0.0:
            z = torch.randn((hi - lo, 1), generator=g, device=device, dtype=torch.float32)
            u *= torch.exp(lognormal_sigma * z)
        first, last = max(lo, r_lo), min(hi, r_hi)
        out[first - r_lo:last - r_lo] = u[first - lo:last - lo].to(torch.float16)
        del u, a
    return out, assign


def noisy_copy_queries(corpus: torch.Tensor, s: int, seed: int, sigma: float = 0.1,
                       relative: bool = True, n_rows: Optional[int] = None,
                       fetch=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """s queries, each a noisy copy of a distinct random corpus row.

    When the corpus is spread over several holders, `corpus` is any tensor on the right device
    with d columns, `n_rows` the row count of the whole corpus and `fetch(ids)` returns its rows
    `ids` (fp16 [len(ids)][d]); the queries are then the same as for the corpus in one piece.

    relative=True: noise std per coordinate = sigma * |x_src| / sqrt(d) (noise of expected
    norm sigma * |x_src|). relative=False: noise std = sigma per coordinate.
    Returns (queries [s][d] fp16, source ids [s] int64).
    """
    N, d = corpus.shape
    if n_rows is not None:
        N = n_rows
    device = corpus.device
    g = _gen(seed, 0, device)
    if s <= N:
        src = torch.randperm(N, generator=g, device=device)[:s] if N <= (1 << 24) else \
            _distinct_randint(N, s, g, device)
    else:
        src = torch.randint(0, N, (s,), generator=g, device=device)
    x = (corpus[src] if fetch is None else fetch(src)).to(torch.float32)
    eps = torch.randn((s, d), generator=g, device=device, dtype=torch.float32)
    if relative:
        scale = sigma * x.norm(dim=1, keepdim=True) / (d ** 0.5)
    else:
        scale = sigma
    q = (x + scale * eps).to(torch.float16)
    return q, src.to(torch.int64)


def _distinct_randint(N: int, s: int, g: torch.Generator, device) -> torch.Tensor:
    """s distinct integers in [0, N) without materialising a permutation of N."""
    picked = torch.empty((0,), dtype=torch.int64, device=device)
    while picked.numel() < s:
        extra = torch.randint(0, N, (2 * s + 16,), generator=g, device=device)
        merged = torch.cat([picked, extra])
        uniq, first = _unique_stable(merged)
        picked = uniq
    return picked[:s]


def _unique_stable(x: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Unique values of x in order of first appearance."""
    vals, inverse = torch.unique(x, return_inverse=True)
    first = torch.full((vals.numel(),), x.numel(), dtype=torch.int64, device=x.device)
    first.scatter_reduce_(0, inverse, torch.arange(x.numel(), device=x.device), reduce="amin")
    order = torch.argsort(first)
    return vals[order], first[order]


def speculation_cache_ids(assign: Optional[torch.Tensor], N: int, sources: torch.Tensor,
                          C: int, seed: int, p_source: float = 0.6,
                          empty_slots: int = 0, n_centres: int = 1) -> torch.Tensor:
    """Per-request speculation cache: C corpus ids per request (int64, -1 = empty).

    sources [R][q] are the rows the request's queries were copied from. Each source id
    enters the cache independently with probability p_source; the rest is filled to C
    unique ids, half with rows of the sources' clusters (when `assign` is given), half
    uniform at random; the slots are then shuffled. `empty_slots` of them are set to -1.
    """
    R, q = sources.shape
    device = sources.device
    out = torch.full((R, C), -1, dtype=torch.int64, device=device)
    for r in range(R):
        g = _gen(seed, r, device)
        keep = torch.rand((q,), generator=g, device=device) < p_source
        chosen = sources[r][keep]
        pool = [chosen]
        if assign is not None:
            want = max(0, (C - chosen.numel()) // 2)
            clusters = assign[sources[r]].unique()
            # sample candidate rows and keep those that fall in the sources' clusters
            n_try = 4 * max(want, 1) * max(1, n_centres // max(1, clusters.numel()))
            cand = torch.randint(0, N, (min(n_try, 1 << 22),), generator=g, device=device)
            mask = torch.isin(assign[cand], clusters)
            pool.append(cand[mask][:want])
        pool.append(torch.randint(0, N, (4 * C + 16,), generator=g, device=device))
        merged = torch.cat(pool)
        # never let a source that lost its coin toss slip back in through the filler
        dropped = sources[r][~keep]
        uniq, _ = _unique_stable(merged)
        uniq = uniq[~torch.isin(uniq, dropped)]
        ids = uniq[:C]
        if ids.numel() < C:  # tiny N: fewer than C distinct rows exist
            ids = torch.cat([ids, torch.full((C - ids.numel(),), -1, dtype=torch.int64, device=device)])
        perm = torch.randperm(C, generator=g, device=device)
        ids = ids[perm]
        if empty_slots > 0:
            ids[:empty_slots] = -1
            ids = ids[torch.randperm(C, generator=g, device=device)]
        out[r] = ids
    return out


def bernoulli_speculation(retrieved_top1: torch.Tensor, gamma: float, seed: int,
                          wrong_id: int = -2) -> torch.Tensor:
    """Speculated ids that equal the retrieved id with probability gamma per step,
    independently, else `wrong_id` (never a valid row). retrieved_top1 is [R][stride]."""
    g = _gen(seed, 0, retrieved_top1.device)
    hit = torch.rand(retrieved_top1.shape, generator=g, device=retrieved_top1.device) < gamma
    return torch.where(hit, retrieved_top1, torch.full_like(retrieved_top1, wrong_id))


def integer_valued(shape, seed: int, lo: int = -8, hi: int = 8, device="cpu") -> torch.Tensor:
    """fp16 tensor of small integers: every inner product / squared distance of such rows
    is an integer that fp16 products, fp32 sums and fp64 sums all represent exactly."""
    g = _gen(seed, 0, device)
    return torch.randint(lo, hi + 1, tuple(shape), generator=g, device=device).to(torch.float16)
