"""ralm_search_static: the search entry point for callers that cannot allocate.

Some users of this library run where creating device memory is not an option: the serving
process has handed the whole GPU to its own memory pool, or a host loop forbids allocator
calls once it is running, or the code is a plug-in that only ever sees buffers it was given.
They bring their own inputs and outputs, and the library keeps its scan scratch in a fixed
array inside its own image. This test drives that entry point through the C ABI and checks it
against the ordinary ralm_search on the same inputs and against the CPU oracle, twice in a row
(the second call finds the scratch as the first one left it), for both metrics and for k = 1
and k > 1. "Allocates nothing" is checked where an allocation would show: the driver's count of
free device bytes does not move across the call, and an allocation failure armed inside the
library before the call is still armed after it (the next index creation trips over it).

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import pytest
import torch

import oracle
import workloads
from parity import check_search

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
    lib = ralm.load_library()
    xn = x.cpu().numpy()
    for call, (s, k) in enumerate([(8, 20), (5, 1)]):
        q, src = workloads.noisy_copy_queries(x, s, seed=902 + call)
        want_ids, want_scores = ralm.search(idx, q, k)
        out_ids, out_scores = ids[:s, :k].contiguous(), scores[:s, :k].contiguous()
        out_ids.fill_(-7)
        torch.cuda.synchronize()
        # once without the checks below: the first call on a device looks up the scratch's address,
        # and the driver loads a kernel's code when it is first launched, which moves the free-byte
        # count without being an allocation of the library's
        ralm.search_static(x, metric, q, k, out_ids, out_scores, status)
        out_ids.fill_(-7)
        status.fill_(123)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        assert lib.ralm_debug_fail_allocation(1) == 0       # the library's next device allocation fails
        try:
            ralm.search_static(x, metric, q, k, out_ids, out_scores, status)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            # the injected failure was not consumed by the call: it made no device allocation
            with pytest.raises(ralm.RalmError) as err:
                ralm.Index(x, metric, max_s=8, max_k=32)
            assert err.value.status == 2                    # RALM_ERR_OOM
        finally:
            lib.ralm_debug_fail_allocation(0)
        assert free_after == free_before
        assert status.item() == 0
        assert torch.equal(out_ids, want_ids)
        torch.testing.assert_close(out_scores, want_scores, rtol=2e-3, atol=1e-5)
        assert out_ids[:, 0].tolist() == src.tolist()
        counts = check_search(out_ids, out_scores, xn, q.cpu().numpy(), metric, k)
        assert counts.wide == 0, str(counts)
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
    # no queries: nothing is searched, but a status word that was passed is still zeroed
    status = torch.full((1,), 55, dtype=torch.int32, device=DEV)
    ralm.search_static(x, 0, q[:0].contiguous(), 3, ids[:0, :3].contiguous(), scores[:0, :3].contiguous(), status)
    torch.cuda.synchronize()
    assert status.item() == 0
    # rows too long for the scratch-free scan (two 16-row tiles must fit in shared memory)
    wide = workloads.unit_gaussian_corpus(64, 4096, seed=905, device=DEV)
    with pytest.raises(ralm.RalmError) as err:
        ralm.search_static(wide, 0, wide[:1].contiguous(), 1, ids[:1, :1].contiguous(), scores[:1, :1].contiguous())
    assert err.value.status == 5                            # RALM_ERR_UNSUPPORTED
