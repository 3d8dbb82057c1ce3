"""Pins of the cache-update oracle: a worked example, the first-in first-out set model written
independently with a deque, and invariants."""
import collections
import random

import numpy as np

from oracle.cache_update import cache_update

EMPTY = -1


def test_worked_example_top1():
    # cache of 4 slots holding {7, 9}, cursor at slot 2; verification retrieved 9, 5, 5, 3
    cache = np.array([[7, 9, EMPTY, EMPTY]])
    retrieved = np.array([[[9, 1], [5, 2], [5, 8], [3, 6]]])
    out, cur = cache_update(cache, [2], retrieved, top=1)
    assert out.tolist() == [[7, 9, 5, 3]] and cur.tolist() == [0]       # 9 and the second 5 are already there
    # one more new id wraps around and evicts the oldest entry
    out2, cur2 = cache_update(out, cur, np.array([[[11, 0]]]), top=1)
    assert out2.tolist() == [[11, 9, 5, 3]] and cur2.tolist() == [1]


def test_worked_example_topk_steps_and_next_n():
    cache = np.full((1, 6), EMPTY)
    retrieved = np.array([[[4, 2], [4, 8], [1, 0]]])
    out, cur = cache_update(cache, [0], retrieved, top=2, steps=[2])      # third step is not inserted
    assert out.tolist() == [[4, 2, 8, EMPTY, EMPTY, EMPTY]] and cur.tolist() == [3]
    # KNN-LM rule: the n entries AFTER each retrieved item, cut at the end of the corpus (N = 10)
    out, cur = cache_update(cache, [0], np.array([[[7], [3]]]), top=1, next_n=3, N=10)
    assert out.tolist() == [[8, 9, 4, 5, 6, EMPTY]] and cur.tolist() == [5]
    # padding ids are skipped
    out, cur = cache_update(cache, [0], np.array([[[-1, 5]]]), top=2)
    assert out.tolist() == [[5, EMPTY, EMPTY, EMPTY, EMPTY, EMPTY]]


def test_equals_a_fifo_set_when_started_empty():
    """A ring that starts empty with its cursor at 0 is a first-in first-out set of capacity C:
    model it with a deque and compare contents and order."""
    rng = random.Random(3)
    for _ in range(200):
        C = rng.randint(1, 12)
        stride, ld = rng.randint(1, 5), rng.randint(1, 4)
        top = rng.randint(1, ld)
        cache, cur = np.full((1, C), EMPTY), np.array([0])
        fifo = collections.deque(maxlen=C)
        for _ in range(rng.randint(1, 6)):
            retrieved = np.array([[[rng.randint(-1, 14) for _ in range(ld)] for _ in range(stride)]])
            cache, cur = cache_update(cache, cur, retrieved, top=top)
            for i in range(stride):
                for j in range(top):
                    doc = int(retrieved[0, i, j])
                    if doc >= 0 and doc not in fifo:
                        fifo.append(doc)
        held = [int(x) for x in cache[0] if x != EMPTY]
        assert sorted(held) == sorted(fifo)
        assert len(set(held)) == len(held)
        # order: starting at the cursor and walking the ring visits the entries oldest first
        ring = [int(cache[0, (int(cur[0]) + t) % C]) for t in range(C)]
        assert [x for x in ring if x != EMPTY] == list(fifo)


def test_invariants_random():
    rng = random.Random(5)
    for _ in range(100):
        R, C = rng.randint(1, 4), rng.randint(2, 16)
        stride, ld = rng.randint(1, 6), rng.randint(1, 5)
        cache = np.array([rng.sample(range(40), C) for _ in range(R)])
        for r in range(R):
            for slot in rng.sample(range(C), rng.randint(0, C // 2)):
                cache[r, slot] = EMPTY
        cursor = np.array([rng.randrange(C) for _ in range(R)])
        retrieved = np.array([[[rng.randint(-1, 39) for _ in range(ld)] for _ in range(stride)] for _ in range(R)])
        steps = [rng.randint(0, stride) for _ in range(R)]
        out, cur = cache_update(cache, cursor, retrieved, top=ld, steps=steps)
        only_empty_overwritten = True
        for r in range(R):
            held = [int(x) for x in out[r] if x != EMPTY]
            assert len(set(held)) == len(held)                                   # still a set
            n_new = (int(cur[r]) - int(cursor[r])) % C
            wanted = {int(x) for x in retrieved[r, :steps[r]].flatten() if x >= 0}
            if len(wanted) >= C:              # the ring may have wrapped: the cursors do not say how often
                only_empty_overwritten = False
                continue
            written = [(int(cursor[r]) + t) % C for t in range(n_new)]
            # slots outside the written range are untouched; written slots hold wanted ids
            for slot in range(C):
                if slot in written:
                    assert int(out[r, slot]) in wanted
                else:
                    assert out[r, slot] == cache[r, slot]
            only_empty_overwritten &= all(cache[r, slot] == EMPTY for slot in written)
            if steps[r] == 0:
                assert np.array_equal(out[r], cache[r]) and cur[r] == cursor[r]
        # with no eviction (only empty slots were overwritten, fewer than C of them) every wanted id
        # is now held, and applying the same update again inserts nothing
        if only_empty_overwritten:
            for r in range(R):
                wanted = {int(x) for x in retrieved[r, :steps[r]].flatten() if x >= 0}
                assert wanted <= {int(x) for x in out[r]}
            again, cur2 = cache_update(out, cur, retrieved, top=ld, steps=steps)
            assert np.array_equal(again, out) and np.array_equal(cur2, cur)
