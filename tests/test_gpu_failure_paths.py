"""Failure paths, exercised without faulting the GPU: a device-side wait that runs out, and a
device allocation that fails during index creation."""
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TIMEOUT, OOM = 4, 2


def test_a_wait_that_nothing_completes_gives_up_and_reports_it():
    import paper_2401_14021_b200 as ralm
    lib = ralm.load_library()
    status = torch.zeros((1,), dtype=torch.int32, device=DEV)
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.ralm_selftest_wait_timeout(2_000_000, status.data_ptr(), stream) == 0    # about a millisecond
    torch.cuda.synchronize()
    assert status.item() == TIMEOUT
    assert lib.ralm_selftest_wait_timeout(0, status.data_ptr(), stream) == 1           # limit out of range
    assert lib.ralm_selftest_wait_timeout(10, None, stream) == 1
    # the context is intact: an ordinary search still runs and reports no device-side anomaly
    x = workloads.unit_gaussian_corpus(20_000, 64, seed=11, device=DEV)
    q, src = workloads.noisy_copy_queries(x, 4, seed=12)
    idx = ralm.Index(x, ralm.IP, 4, 3)
    ids, _ = ralm.search(idx, q, 3)
    assert ids[:, 0].tolist() == src.tolist()
    assert idx.device_status() == 0


@pytest.mark.parametrize("metric,max_s,max_k", [(0, 16, 20), (1, 4, 1024)])
def test_index_creation_survives_a_failing_allocation(metric, max_s, max_k):
    import paper_2401_14021_b200 as ralm
    lib = ralm.load_library()
    x = workloads.unit_gaussian_corpus(10_000, 64, seed=13, device=DEV)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    failures = 0
    try:
        for nth in range(1, 12):
            assert lib.ralm_debug_fail_allocation(nth) == 0
            try:
                idx = ralm.Index(x, metric, max_s, max_k)
            except ralm.RalmError as err:
                assert err.status == OOM
                failures += 1
            else:
                idx.close()         # nth is beyond the allocations a creation makes
                break
    finally:
        lib.ralm_debug_fail_allocation(0)
    assert failures >= 7            # every allocation of a creation was made to fail in turn
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert abs(free_after - free_before) < (64 << 20)       # nothing of the failed creations is left
    idx = ralm.Index(x, metric, max_s, max_k)                # and creation works again
    q, src = workloads.noisy_copy_queries(x, 2, seed=14)
    ids, _ = ralm.search(idx, q, 1)
    assert ids[:, 0].tolist() == src.tolist()
    assert lib.ralm_debug_fail_allocation(-1) == 1
