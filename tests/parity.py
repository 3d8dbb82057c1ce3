"""Acceptance rule shared by the GPU parity tests.

For rank p of a query (oracle = fp64 CPU reference on the same fp16 bytes):
  strict-OK  gpu_id[p] == oracle_id[p]
  band-OK    gpu_id[p] is a valid row, appears once in the GPU list, and its ORACLE score
             is within 2e-3 relative of the oracle's score at rank p (the two rows sit in
             one near-tie band). Counted in two classes:
               tight  the two oracle scores differ by at most 1e-5 relative: a swap that the
                      rounding of an fp32 accumulation can explain
               wide   anything up to 2e-3: accepted by the rule, but not explained by
                      rounding -- the configuration tests assert that there is none
  FAIL       anything else
Scores: |gpu_score - oracle_score(gpu_id)| <= 2e-3 * |oracle_score| + 1e-5 * scale, where
`scale` bounds |q||x| (only matters for inner products near zero).
"""
from dataclasses import dataclass

import numpy as np
import torch

import oracle

REL = 2e-3
TIGHT_REL = 1e-5


@dataclass
class Counts:
    """Ranks by class; `band` = tight + wide."""
    strict: int = 0
    tight: int = 0
    wide: int = 0

    @property
    def band(self) -> int:
        return self.tight + self.wide

    def __iadd__(self, other):
        self.strict += other.strict
        self.tight += other.tight
        self.wide += other.wide
        return self

    def __str__(self):
        return "strict=%d tight=%d wide=%d" % (self.strict, self.tight, self.wide)


def check_lists(gpu_ids, gpu_scores, ora_ids, ora_scores, score_of, metric, scale=1.0, n_valid=None):
    """One query. score_of(id) -> oracle fp64 score of that row for this query.
    Returns Counts; raises AssertionError on FAIL."""
    k = len(ora_ids)
    n = Counts()
    seen = set()
    for p in range(k):
        gid, oid = int(gpu_ids[p]), int(ora_ids[p])
        if oid < 0:
            assert gid == -1, "rank %d: expected padding, got id %d" % (p, gid)
            assert np.isinf(gpu_scores[p]) and (gpu_scores[p] < 0) == (metric == oracle.IP)
            n.strict += 1
            continue
        assert gid >= 0 and (n_valid is None or gid < n_valid), "rank %d: invalid id %d" % (p, gid)
        assert gid not in seen, "rank %d: id %d repeated" % (p, gid)
        seen.add(gid)
        s_true = ora_scores[p] if gid == oid else score_of(gid)
        if gid == oid:
            n.strict += 1
        else:
            gap = abs(s_true - ora_scores[p])
            assert gap < REL * abs(ora_scores[p]) + 1e-30, \
                "rank %d: id %d (score %r) is outside the near-tie band of oracle id %d (score %r)" % (
                    p, gid, s_true, oid, ora_scores[p])
            if gap <= TIGHT_REL * abs(ora_scores[p]):
                n.tight += 1
            else:
                n.wide += 1
        assert abs(float(gpu_scores[p]) - s_true) <= REL * abs(s_true) + 1e-5 * scale, \
            "rank %d: score %r vs oracle %r" % (p, float(gpu_scores[p]), s_true)
    return n


def check_search(gpu_ids, gpu_scores, corpus_np, queries_np, metric, k, exact=False):
    """Whole-batch comparison against oracle.search. Returns the Counts totals."""
    ora_ids, ora_scores = oracle.search(corpus_np, queries_np, metric, k)
    gi, gs = gpu_ids.cpu().numpy(), gpu_scores.cpu().numpy()
    if exact:
        assert np.array_equal(gi, ora_ids)
        assert np.array_equal(gs.astype(np.float64), ora_scores)
        return Counts(strict=gi.size)
    total = Counts()
    norms = np.linalg.norm(corpus_np.astype(np.float64), axis=1).max() if corpus_np.shape[0] else 1.0
    for i in range(queries_np.shape[0]):
        scale = norms * np.linalg.norm(queries_np[i].astype(np.float64))
        total += check_lists(gi[i], gs[i], ora_ids[i], ora_scores[i],
                             lambda j, i=i: oracle.pair_score(corpus_np[j], queries_np[i], metric),
                             metric, scale=scale, n_valid=corpus_np.shape[0])
    return total


def sampled_parity(x, q, ids, scores, metric, k, n_chunks, chunk_rows, seed, query_sel=None):
    """Full-size check on a sub-corpus: seeded random chunks of rows, the first rows, the ragged tail
    and every row the GPU returned, ranked by the oracle. If the GPU's lists are the top-k of the
    whole corpus they are the top-k of that sub-corpus too. Returns (Counts, rows in the sub-corpus)
    and asserts that no swap needed the wide band."""
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
