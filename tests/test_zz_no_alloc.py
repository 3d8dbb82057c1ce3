"""ralm_search_static: the search entry point for callers that cannot allocate.

Some users of this library run where creating device memory is not an option: the serving
process has handed the whole GPU to its own memory pool, or a host loop forbids allocator
calls once it is running, or the code is a plug-in that only ever sees buffers it was given.
They bring their own inputs and outputs, and the library keeps its scan scratch in a fixed
array inside its own image. This test drives that entry point through the C ABI and checks it
against the ordinary ralm_search on the same inputs, twice in a row (the second call finds the
scratch as the first one left it), for both metrics and for k = 1 and k > 1.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("metric", [0, 1])
def test_static_entry_matches_search_on_two_calls_in_a_row(metric):
    import paper_2401_14021_b200 as ralm
    N, d = 120_000, 768
    x, _ = workloads.mixture_corpus(N, d, 64, seed=901, device=DEV, normalise=(metric == 0),
                                    lognormal_sigma=0.0 if metric == 0 else 0.3)
    idx = ralm.Index(x, metric, max_s=8, max_k=32)
    # every buffer the static call touches exists before it runs: it allocates nothing
    ids = torch.empty((8, 32), dtype=torch.int64, device=DEV)
    scores = torch.empty((8, 32), dtype=torch.float32, device=DEV)
    status = torch.full((1,), 123, dtype=torch.int32, device=DEV)
    for call, (s, k) in enumerate([(8, 20), (5, 1)]):
        q, src = workloads.noisy_copy_queries(x, s, seed=902 + call)
        want_ids, want_scores = ralm.search(idx, q, k)
        out_ids, out_scores = ids[:s, :k].contiguous(), scores[:s, :k].contiguous()
        out_ids.fill_(-7)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        ralm.search_static(x, metric, q, k, out_ids, out_scores, status)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert status.item() == 0
        assert torch.equal(out_ids, want_ids)
        torch.testing.assert_close(out_scores, want_scores, rtol=2e-3, atol=1e-5)
        assert out_ids[:, 0].tolist() == src.tolist()
    idx.close()


def test_static_entry_rejects_sizes_beyond_its_scratch():
    import paper_2401_14021_b200 as ralm
    x = workloads.unit_gaussian_corpus(1000, 64, seed=903, device=DEV)
    q = workloads.unit_gaussian_corpus(9, 64, seed=904, device=DEV)
    ids = torch.empty((9, 33), dtype=torch.int64, device=DEV)
    scores = torch.empty((9, 33), dtype=torch.float32, device=DEV)
    with pytest.raises(ralm.RalmError) as err:
        ralm.search_static(x, 0, q, 4, ids[:, :4].contiguous(), scores[:, :4].contiguous())   # s = 9
    assert err.value.status == 7
    with pytest.raises(ralm.RalmError) as err:
        ralm.search_static(x, 0, q[:2].contiguous(), 33, ids[:2].contiguous(), scores[:2].contiguous())
    assert err.value.status == 7
    # status pointer is optional, and an empty corpus pads like ralm_search does
    ralm.search_static(x[:0], 0, q[:2].contiguous(), 3, ids[:2, :3].contiguous(), scores[:2, :3].contiguous())
    out_i, out_s = ids[:2, :3].contiguous(), scores[:2, :3].contiguous()
    ralm.search_static(x[:0], 1, q[:2].contiguous(), 3, out_i, out_s)
    torch.cuda.synchronize()
    assert (out_i == -1).all() and torch.isinf(out_s).all()
