"""CPU oracle for the speculation-cache update (test infrastructure only; shares nothing with
the CUDA library).

Section 3 of the paper ("Speculative retrieval", Fig. 3): after a verification step the local
cache is populated with the documents retrieved for it, either the top-ranked one per query
(top-1 update) or the first `top` of them (top-k update / prefetching). For KNN-LM (Section 5.3)
the cache receives, instead of the retrieved entries themselves, the next n entries after each
of them. The cache is a set of corpus ids held in a fixed number of slots; the paper does not
say what leaves a full cache: the reading taken here is first-in first-out, a ring with one
write cursor per request.

The update is defined by this sequence, in plain loops (a step is one query of the batch):

    for step i = 0 .. steps-1, rank j = 0 .. top-1:
        id = retrieved[i][j]                      (negative = padding, skipped)
        candidates = [id]            if next_n == 0
                     [id+1 .. id+n]  if next_n == n > 0, cut at the end of the corpus
        for c in candidates:
            if c is not in the cache: cache[cursor] = c; cursor = (cursor + 1) mod C
"""
import numpy as np


def cache_update(cache_ids, cursor, retrieved_ids, top, steps=None, next_n=0, N=None):
    """cache_ids int64 [R][C] and cursor int [R] are updated IN COPIES that are returned.
    retrieved_ids int64 [R][stride][ld]; steps int [R] or None (= every step)."""
    cache = np.array(cache_ids, dtype=np.int64, copy=True)
    cur = np.array(cursor, dtype=np.int32, copy=True)
    retrieved = np.asarray(retrieved_ids, dtype=np.int64)
    R, C = cache.shape
    stride, ld = retrieved.shape[1], retrieved.shape[2]
    assert 1 <= top <= ld
    for r in range(R):
        n_steps = stride if steps is None else max(0, min(int(steps[r]), stride))
        for i in range(n_steps):
            for j in range(top):
                doc = int(retrieved[r, i, j])
                if doc < 0:
                    continue
                cands = [doc] if next_n == 0 else [doc + o for o in range(1, next_n + 1)]
                for c in cands:
                    if N is not None and c >= N:
                        break
                    present = False
                    for slot in range(C):
                        if int(cache[r, slot]) == c:
                            present = True
                            break
                    if not present:
                        cache[r, int(cur[r])] = c
                        cur[r] = (int(cur[r]) + 1) % C
    return cache, cur
