"""Row-sharded search: partition arithmetic and the gather on CPU (two gloo ranks); the merge
kernel on one GPU, where several shards of one corpus must reproduce the unsharded search."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEV = "cuda:0"


def test_shard_rows_partition():
    from paper_2401_14021_b200.sharded import shard_rows
    for N in (0, 1, 255, 256, 257, 1000, 21_000_000, 50_000_001):
        for world in (1, 2, 3, 8):
            spans = [shard_rows(N, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == N
            for (lo, hi), (lo2, _) in zip(spans, spans[1:]):
                assert lo <= hi == lo2                      # contiguous, disjoint, in order
            assert all(lo % 256 == 0 or lo == N for lo, _ in spans)
    with pytest.raises(ValueError):
        shard_rows(10, 2, 2)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _gather_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2401_14021_b200.sharded import gather_lists, shard_rows
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = shard_rows(1000, world, rank)
        ids = torch.arange(6, dtype=torch.int64).reshape(2, 3) + 100 * rank      # this rank's [s][k] answer
        scores = ids.to(torch.float32) / 7
        all_ids, all_scores, offsets = gather_lists(ids, scores, lo)
        out.put((rank, all_ids.tolist(), all_scores.tolist(), offsets.tolist()))
        dist.barrier()
    except Exception as err:          # surface the reason instead of a silent time-out
        out.put((rank, repr(err), None, None))
        raise
    finally:
        dist.destroy_process_group()


def test_gather_lists_two_gloo_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=120) for _ in range(world)), key=lambda r: r[0])
    assert all(r[2] is not None for r in results), results
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want_ids = [[[0, 1, 2], [3, 4, 5]], [[100, 101, 102], [103, 104, 105]]]
    for rank, ids, scores, offsets in results:
        assert ids == want_ids                               # [G][s][k], rank-major, same on every rank
        assert offsets == [0, 512]
        assert scores[1][1][2] == pytest.approx(105 / 7)


@pytest.mark.gpu
@pytest.mark.parametrize("metric,k,G", [(0, 20, 2), (0, 1, 8), (1, 5, 3), (1, 1024, 5), (0, 600, 8)])
def test_shards_on_one_gpu_reproduce_the_unsharded_search(metric, k, G):
    import paper_2401_14021_b200 as ralm
    from paper_2401_14021_b200.sharded import shard_rows
    N, d, s = 40_003, 128, 6
    x = workloads.integer_valued((N, d), seed=31, lo=-2, hi=2, device=DEV)          # ties across shards abound
    q = workloads.integer_valued((s, d), seed=32, lo=-2, hi=2, device=DEV)
    full = ralm.Index(x, metric, s, k)
    want_ids, want_scores = ralm.search(full, q, k)
    ids, scores, offsets = [], [], []
    for g in range(G):
        lo, hi = shard_rows(N, G, g)
        shard = ralm.Index(x[lo:hi], metric, s, k)
        i, sc = ralm.search(shard, q, k)
        ids.append(i)
        scores.append(sc)
        offsets.append(lo)
        torch.cuda.synchronize()
        shard.close()
    got_ids, got_scores = ralm.merge_lists(torch.stack(ids), torch.stack(scores),
                                           torch.tensor(offsets, dtype=torch.int64, device=DEV), metric)
    torch.cuda.synchronize()
    # the reference is the oracle over the WHOLE corpus (integer data: ids and scores bit for bit,
    # ties across shard boundaries included); the library's own unsharded search must agree too
    import oracle
    from parity import check_search
    check_search(got_ids, got_scores, x.cpu().numpy(), q.cpu().numpy(), metric, k, exact=True)
    assert torch.equal(got_ids, want_ids) and torch.equal(got_scores, want_scores)


@pytest.mark.gpu
def test_shards_of_real_valued_rows_against_the_oracle():
    """Mixture rows (near ties, fp32 rounding): the merged answer of 4 shards against the oracle's
    ranking of the whole corpus, by the near-tie rule."""
    import paper_2401_14021_b200 as ralm
    import oracle
    from parity import check_search
    from paper_2401_14021_b200.sharded import shard_rows
    N, d, s, k, G = 120_000, 256, 8, 20, 4
    x, _ = workloads.mixture_corpus(N, d, 64, seed=35, device=DEV)
    q, src = workloads.noisy_copy_queries(x, s, seed=36)
    ids, scores, offsets = [], [], []
    for g in range(G):
        lo, hi = shard_rows(N, G, g)
        shard = ralm.Index(x[lo:hi], ralm.IP, s, k)
        i, sc = ralm.search(shard, q, k)
        torch.cuda.synchronize()
        ids.append(i)
        scores.append(sc)
        offsets.append(lo)
        shard.close()
    got_ids, got_scores = ralm.merge_lists(torch.stack(ids), torch.stack(scores),
                                           torch.tensor(offsets, dtype=torch.int64, device=DEV), ralm.IP)
    torch.cuda.synchronize()
    counts = check_search(got_ids, got_scores, x.cpu().numpy(), q.cpu().numpy(), oracle.IP, k)
    assert got_ids[:, 0].tolist() == src.tolist()
    assert counts.wide == 0, str(counts)


@pytest.mark.gpu
def test_sharded_index_single_rank_and_padding():
    import paper_2401_14021_b200 as ralm
    from paper_2401_14021_b200.sharded import ShardedIndex
    x, _ = workloads.mixture_corpus(30_000, 256, 32, seed=33, device=DEV)
    q, src = workloads.noisy_copy_queries(x, 4, seed=34)
    sh = ShardedIndex(x, 0, ralm.IP, 4, 10)
    ids, scores = sh.search(q, 10)
    ref = ralm.Index(x, ralm.IP, 4, 10)
    want_ids, want_scores = ralm.search(ref, q, 10)
    assert torch.equal(ids, want_ids) and torch.equal(scores, want_scores)
    sh.close()
    # shards smaller than k: padding (-1) in a shard's list must not reach the merged answer
    tiny = x[:25].contiguous()
    a, b = ralm.Index(tiny[:5], ralm.L2, 4, 10), ralm.Index(tiny[5:], ralm.L2, 4, 10)
    ia, sa = ralm.search(a, q, 10)
    ib, sb = ralm.search(b, q, 10)
    got_ids, got_scores = ralm.merge_lists(torch.stack([ia, ib]), torch.stack([sa, sb]),
                                           torch.tensor([0, 5], dtype=torch.int64, device=DEV), ralm.L2)
    want = ralm.Index(tiny, ralm.L2, 4, 10)
    wi, ws = ralm.search(want, q, 10)
    assert torch.equal(got_ids, wi) and torch.equal(got_scores, ws)
    with pytest.raises(ralm.RalmError):
        ralm.merge_lists(torch.stack([ia, ib]), torch.stack([sa, sb]),
                         torch.tensor([0, 5], dtype=torch.int64, device=DEV), 7)
