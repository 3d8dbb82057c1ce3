"""Input generators: a row range of a corpus holds the same bytes as the whole corpus there, and
queries drawn through a row-fetch callback equal those drawn from the corpus in one piece (what
a row-sharded run relies on)."""
import torch

import workloads


def test_row_range_of_a_corpus_is_the_same_bytes():
    x, a = workloads.mixture_corpus(5000, 64, 16, 7, chunk_rows=1024)
    for lo, hi in ((0, 5000), (1500, 4100), (1024, 2048), (4999, 5000), (300, 300)):
        y, b = workloads.mixture_corpus(5000, 64, 16, 7, chunk_rows=1024, row_range=(lo, hi))
        assert torch.equal(x[lo:hi], y) and torch.equal(a, b)
    u = workloads.unit_gaussian_corpus(3000, 32, 3, chunk_rows=1000)
    v = workloads.unit_gaussian_corpus(3000, 32, 3, chunk_rows=1000, row_range=(999, 2001))
    assert torch.equal(u[999:2001], v)


def test_queries_through_a_fetch_callback_are_the_same():
    x, _ = workloads.mixture_corpus(5000, 64, 16, 7, chunk_rows=1024)
    part, _ = workloads.mixture_corpus(5000, 64, 16, 7, chunk_rows=1024, row_range=(2000, 3000))
    q1, s1 = workloads.noisy_copy_queries(x, 5, 11)
    q2, s2 = workloads.noisy_copy_queries(part, 5, 11, n_rows=5000, fetch=lambda ids: x[ids])
    assert torch.equal(q1, q2) and torch.equal(s1, s2)
