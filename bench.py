#!/usr/bin/env python
"""Benchmark of the exact-retrieval verification step on synthetic corpora.

One step = one verification step of the serving loop, all kernels on one stream:
  ralm_cache_search  speculation: R concurrent requests x q queries over their local caches
  ralm_search        verification retrieval: s queries against the whole N x d corpus
  ralm_verify        first mis-speculated position of the verified request
Throughput is verified queries per second = s * steps / time. Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                  [--workload C1|C2|C3|C4|C5] [--s S] [--k K] [--variant V] [--rows N]

With --gpus N > 1 (launched under torch.distributed.run) every rank runs an independent
replica on its own GPU (the path does not shard); the value is the sum over replicas and the
time is the maximum over ranks. --impl reference times the fp64 CPU oracle on a bounded
sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "verified queries/s at 21Mx768 fp16 top-1, s=8; % of HBM roofline"
UNIT = "queries/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=["C1", "C2", "C3", "C4", "C5"])
    ap.add_argument("--s", type=int, default=None)
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--q8", action="store_true",
                    help="stream the index's one-byte copy of the corpus (exact results; inner product, s <= 8)")
    ap.add_argument("--rows", type=int, default=None, help="override the corpus size (profiling)")
    ap.add_argument("--tune", default=None, help="consumer_warps,ring_depth,tile_rows (0 = default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="capture one step (cache lookup, search, verify) in a CUDA graph and replay it in the "
                         "timed region, as a launch-bound serving loop would (small corpora); the scan's own "
                         "events are then taken from plain steps after the timed region")
    ap.add_argument("--flush-l2", action="store_true",
                    help="write a buffer larger than L2 before every timed step (for corpora near L2 size); "
                         "the step time is then the sum of per-step event intervals, flushes excluded")
    ap.add_argument("--sharded", action="store_true",
                    help="row-sharded search: every rank holds N / world rows, the answers are all-gathered "
                         "and merged on every rank (strong scaling); without it ranks are replicas")
    return ap.parse_args()


def build_inputs(cfg, s, device, rows=None):
    """Corpus, verification queries, speculation caches and cache queries of one replica."""
    N = rows or cfg.N
    seed = workloads.seed_for(cfg.index)
    if cfg.corpus == "unit_gaussian":
        corpus, assign = workloads.unit_gaussian_corpus(N, cfg.d, seed, device=device), None
    else:
        corpus, assign = workloads.mixture_corpus(N, cfg.d, cfg.n_centres, seed, device=device,
                                                  sigma_within=cfg.sigma_within,
                                                  normalise=cfg.normalise,
                                                  lognormal_sigma=cfg.lognormal_sigma)
    R = max(cfg.requests, 1)
    stride = cfg.stride or s
    C = cfg.cache_entries or 64
    # request 0 is the one being verified; its first s queries form the verification batch
    nq = max(R * stride, s)
    queries, src = workloads.noisy_copy_queries(corpus, nq, workloads.seed_for(cfg.index, "queries"))
    cache_q = queries[:R * stride].reshape(R, stride, cfg.d).contiguous()
    cache = workloads.speculation_cache_ids(assign, N, src[:R * stride].reshape(R, stride), C,
                                            workloads.seed_for(cfg.index, "caches"),
                                            n_centres=max(cfg.n_centres, 1))
    return corpus, queries[:s].contiguous(), src[:s], cache, cache_q


def build_inputs_sharded(cfg, s, device, rank, world, dist, rows=None):
    """This rank's rows of the corpus (the same bytes the whole corpus holds there), and the same
    queries and speculation caches on every rank as the unsharded run builds. Rows that live on
    another rank (query sources, cached rows) arrive by one all-reduce of zero-filled buffers."""
    from paper_2401_14021_b200.sharded import shard_rows
    N = rows or cfg.N
    lo, hi = shard_rows(N, world, rank)
    seed = workloads.seed_for(cfg.index)
    if cfg.corpus == "unit_gaussian":
        local, assign = workloads.unit_gaussian_corpus(N, cfg.d, seed, device=device, row_range=(lo, hi)), None
    else:
        local, assign = workloads.mixture_corpus(N, cfg.d, cfg.n_centres, seed, device=device,
                                                 sigma_within=cfg.sigma_within, normalise=cfg.normalise,
                                                 lognormal_sigma=cfg.lognormal_sigma, row_range=(lo, hi))

    def fetch(ids):
        out = torch.zeros((ids.numel(), cfg.d), dtype=torch.float16, device=device)
        mine = (ids >= lo) & (ids < hi)
        out[mine] = local[ids[mine] - lo]
        if dist is not None:
            bits = out.view(torch.int32)      # integer sums of one owner's bits and zeros: exact
            dist.all_reduce(bits)
        return out

    R = max(cfg.requests, 1)
    stride = cfg.stride or s
    C = cfg.cache_entries or 64
    nq = max(R * stride, s)
    queries, src = workloads.noisy_copy_queries(local, nq, workloads.seed_for(cfg.index, "queries"),
                                                n_rows=N, fetch=fetch)
    cache_q = queries[:R * stride].reshape(R, stride, cfg.d).contiguous()
    cache = workloads.speculation_cache_ids(assign, N, src[:R * stride].reshape(R, stride), C,
                                            workloads.seed_for(cfg.index, "caches"),
                                            n_centres=max(cfg.n_centres, 1))
    # the cached vectors live with the requests (on every rank here): rows [R * C][d]
    cache_rows = fetch(cache.flatten())
    return local, lo, N, queries[:s].contiguous(), src[:s], cache, cache_q, cache_rows


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.proc = None
        self.path = None
        try:
            uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100", "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, smax, power = [], set(), None, []
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    smax = float(f[1])
                    power.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=smax, reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power) if power else None)
        return out


def cpu_baseline(corpus, queries, metric_id, k, N_full, s, budget_s=15.0):
    """The oracle, as it stands, on a bounded sample: the first rows of the same corpus."""
    import oracle
    probe = min(corpus.shape[0], 20_000)
    xq = queries.cpu().numpy()
    xs = corpus[:probe].cpu().numpy()
    t0 = time.perf_counter()
    _, _, cores = oracle.search(xs, xq, metric_id, k, return_threads=True)
    tp = time.perf_counter() - t0
    rows = int(min(corpus.shape[0], max(probe, probe * budget_s / max(tp, 1e-6)), 2_000_000))
    xs = corpus[:rows].cpu().numpy()
    t0 = time.perf_counter()
    _, _, cores = oracle.search(xs, xq, metric_id, k, return_threads=True)
    t = time.perf_counter() - t0
    value = s / (t * N_full / rows)
    return {"value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": "first %d of %d rows, all %d queries, k=%d, %.1f s; scaled linearly in N"
                      % (rows, N_full, s, k, t)}


def run_reference(args, cfg, s, k, metric_id):
    """The CPU oracle as the reference arm: every step runs the same three calls (cache lookup,
    search, verify) on a bounded row sample of the workload; the search time is scaled to N."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = min(cfg.N, args.rows or 60_000)
    seed = workloads.seed_for(cfg.index)
    if cfg.corpus == "unit_gaussian":
        corpus, assign = workloads.unit_gaussian_corpus(rows, cfg.d, seed), None
    else:
        corpus, assign = workloads.mixture_corpus(rows, cfg.d, cfg.n_centres, seed, normalise=cfg.normalise,
                                                  lognormal_sigma=cfg.lognormal_sigma)
    R = max(cfg.requests, 1)
    stride = cfg.stride or s
    C = cfg.cache_entries or 64
    nq = max(R * stride, s)
    q, src = workloads.noisy_copy_queries(corpus, nq, workloads.seed_for(cfg.index, "queries"))
    cache = workloads.speculation_cache_ids(assign, rows, src[:R * stride].reshape(R, stride), C,
                                            workloads.seed_for(cfg.index, "caches"),
                                            n_centres=max(cfg.n_centres, 1)).numpy()
    xn, qn = corpus.numpy(), q[:s].numpy()
    cache_q = q[:R * stride].reshape(R, stride, cfg.d).numpy()
    vstride = min(stride, s)
    nv = max(1, min(R, s // stride))
    steps, warmup = min(args.steps, 8), min(args.warmup, 1)
    cores = 1
    for _ in range(warmup):
        oracle.search(xn, qn, metric_id, k)
    t_search = t_rest = 0.0
    for _ in range(steps):
        t0 = time.perf_counter()
        spec, _ = oracle.cache_search(xn, cache, cache_q, metric_id, 1)
        t1 = time.perf_counter()
        ids, _, cores = oracle.search(xn, qn, metric_id, k, return_threads=True)
        t2 = time.perf_counter()
        oracle.verify(spec[:nv, :vstride, 0], ids[:nv * vstride].reshape(nv, vstride, k))
        t3 = time.perf_counter()
        t_search += t2 - t1
        t_rest += (t1 - t0) + (t3 - t2)
    # the search scans the corpus (scaled to the full N); cache lookup and verify do not depend on N
    t = (t_search * cfg.N / rows + t_rest) / steps
    value = s / t
    sample = "%d of %d rows per step (search time scaled linearly in N), %d queries, k=%d" % (rows, cfg.N, s, k)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": t * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": "%s %dx%d %s s=%d k=%d; cache lookup R=%d C=%d q=%d; verify stride %d"
                               % (cfg.name, cfg.N, cfg.d, cfg.metric, s, k, R, C, stride, vstride)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    args = parse_args()
    cfg = workloads.CONFIGS[args.workload]
    s = args.s or (8 if args.workload == "C3" else cfg.s_values[-1])
    k = args.k or cfg.k_values[0]
    metric_id = 0 if cfg.metric == "ip" else 1
    if args.impl == "reference":
        run_reference(args, cfg, s, k, metric_id)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    import paper_2401_14021_b200 as ralm

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sharded = None
    if args.sharded:
        # row-sharded search: this rank holds rows [row_lo, row_lo + local rows) of the N-row corpus
        from paper_2401_14021_b200.sharded import ShardedIndex
        corpus, row_lo, N, queries, src, cache, cache_q, cache_rows = build_inputs_sharded(
            cfg, s, device, rank, world, dist, args.rows)
        d = corpus.shape[1]
        sharded = ShardedIndex(corpus, row_lo, metric_id, max_s=max(s, 1), max_k=max(k, 1))
        idx = sharded.index
        # speculation runs over the cached vectors kept with the requests; its answers are positions
        # in cache_rows, translated back to corpus ids through the cache's own id list
        cache_index = ralm.Index(cache_rows, metric_id, max_s=8, max_k=1)
        cache_flat = cache.flatten()
        cache_local = torch.arange(cache_flat.numel(), dtype=torch.int64, device=device).reshape(cache.shape)
    else:
        corpus, queries, src, cache, cache_q = build_inputs(cfg, s, device, args.rows)
        N, d = corpus.shape
        idx = ralm.Index(corpus, metric_id, max_s=max(s, 1), max_k=max(k, 1))
    local_rows = corpus.shape[0]
    R, stride = cache_q.shape[0], cache_q.shape[1]
    if args.variant:
        idx.set_variant(args.variant)
    if args.q8:
        idx.enable_q8()
    if args.tune:
        idx.set_tuning(*[int(v) for v in args.tune.split(",")])
    stream = torch.cuda.current_stream()

    ids = torch.empty((s, k), dtype=torch.int64, device=device)
    scores = torch.empty((s, k), dtype=torch.float32, device=device)
    spec_ids = torch.empty((R, stride, 1), dtype=torch.int64, device=device)
    spec_scores = torch.empty((R, stride, 1), dtype=torch.float32, device=device)
    # the batch holds the strides of the first `nv` requests (one request at s <= stride)
    vstride = min(stride, s)
    nv = max(1, min(R, s // stride))
    first_mismatch = torch.empty((nv,), dtype=torch.int32, device=device)
    spec_view = spec_ids[:nv, :vstride, 0] if vstride < stride else spec_ids[:nv].reshape(nv, stride)
    retr_view = ids[:nv * vstride].reshape(nv, vstride, k)

    if sharded is None:
        def step(st=stream):
            ralm.cache_search(idx, cache, cache_q, 1, spec_ids, spec_scores, st)
            ralm.search(idx, queries, k, ids, scores, st)
            ralm.verify(spec_view, retr_view, 1, first_mismatch, st)
    else:
        spec_local = torch.empty((R, stride, 1), dtype=torch.int64, device=device)

        def step():
            ralm.cache_search(cache_index, cache_local, cache_q, 1, spec_local, spec_scores, stream)
            torch.take(cache_flat, spec_local, out=spec_ids)
            got_ids, got_scores = sharded.search(queries, k, stream)    # scan, all-gather, merge
            ids.copy_(got_ids)
            scores.copy_(got_scores)
            ralm.verify(spec_view, retr_view, 1, first_mismatch, stream)

    flush = torch.empty((512 << 20,), dtype=torch.uint8, device=device) if args.flush_l2 else None

    # ---- device-resident timing
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    idx.read_timing()
    use_graph = args.graph and sharded is None and flush is None
    graph = None
    if use_graph:
        # (the library's calls only enqueue work on the stream they are given, so a step can be captured)
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
            step(torch.cuda.current_stream())
        stream.wait_stream(side)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
    idx.set_timing(not use_graph)
    launches0 = idx.launch_count()
    sampler = ClockSampler(local_rank)
    time.sleep(0.25)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if flush is None:
        e0.record(stream)
        for _ in range(args.steps):
            if graph is not None:
                graph.replay()
            else:
                step()
        e1.record(stream)
        barrier()
        total_ms = e0.elapsed_time(e1)
    else:
        # L2 flushed before every step; the step time is the sum of the per-step intervals
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                 for _ in range(args.steps)]
        for a, b in pairs:
            flush.zero_()
            a.record(stream)
            step()
            b.record(stream)
        barrier()
        total_ms = sum(a.elapsed_time(b) for a, b in pairs)
    clocks = sampler.stop()
    if graph is not None:
        # events cannot be read back from a captured step: the scan's own times come from plain steps
        idx.set_timing(True)
        launches0 = idx.launch_count()
        for _ in range(args.steps):
            step()
        torch.cuda.synchronize()
    pass_ms = idx.read_timing_list(max(4096, 8 * args.steps))
    scan_ms, scan_launches = sum(pass_ms), len(pass_ms)
    dispatch = idx.last_dispatch()
    idx.set_timing(False)
    gpu_launches = idx.launch_count() - launches0 + args.steps   # + one verify launch per step
    # the whole search call by itself (scan launches, threshold kernel and merges), a few times
    n_search = max(3, min(20, args.steps))
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for _ in range(n_search):
        if sharded is None:
            ralm.search(idx, queries, k, ids, scores, stream)
        else:
            sharded.search(queries, k, stream)
    s1.record(stream)
    torch.cuda.synchronize()
    search_ms = s0.elapsed_time(s1) / n_search
    if sharded is not None:
        gpu_launches += 3 * args.steps                           # cache score + rank on the cached vectors, merge_lists
    assert idx.device_status() == 0, "device status word set during the timed region"
    assert ids[:, 0].tolist() == src.tolist(), "rank-0 ids are not the planted sources"

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    h_q = queries.cpu().pin_memory()
    h_cache = cache.cpu().pin_memory()
    h_cache_q = cache_q.cpu().pin_memory()
    h_ids = torch.empty((s, k), dtype=torch.int64).pin_memory()
    h_scores = torch.empty((s, k), dtype=torch.float32).pin_memory()
    h_spec = torch.empty((R, stride, 1), dtype=torch.int64).pin_memory()
    h_fm = torch.empty((nv,), dtype=torch.int32).pin_memory()
    d_cache, d_cache_q = torch.empty_like(cache), torch.empty_like(cache_q)
    retr1 = torch.empty((nv, vstride, 1), dtype=torch.int64, device=device)
    h_top1 = h_ids[:nv * vstride, :1].reshape(nv, vstride, 1)
    h2d = h_q.numel() * 2 + h_cache.numel() * 8 + h_cache_q.numel() * 2 + h_top1.numel() * 8
    d2h = h_ids.numel() * 8 + h_scores.numel() * 4 + h_spec.numel() * 8 + 4 * nv

    if sharded is None:
        def step_e2e():
            d_cache.copy_(h_cache, non_blocking=True)
            d_cache_q.copy_(h_cache_q, non_blocking=True)
            ralm.cache_search(idx, d_cache, d_cache_q, 1, spec_ids, spec_scores, stream)
            ralm.search_host(idx, h_q, k, h_ids, h_scores, stream)          # H2D, scan, D2H, sync
            retr1.copy_(h_top1, non_blocking=True)
            ralm.verify(spec_view, retr1, 1, first_mismatch, stream)
            h_spec.copy_(spec_ids, non_blocking=True)
            h_fm.copy_(first_mismatch, non_blocking=True)
            stream.synchronize()
    else:
        d_q = torch.empty_like(queries)
        h2d = h_q.numel() * 2 + h_cache_q.numel() * 2

        def step_e2e():
            d_cache_q.copy_(h_cache_q, non_blocking=True)
            d_q.copy_(h_q, non_blocking=True)
            ralm.cache_search(cache_index, cache_local, d_cache_q, 1, spec_local, spec_scores, stream)
            torch.take(cache_flat, spec_local, out=spec_ids)
            got_ids, got_scores = sharded.search(d_q, k, stream)
            ids.copy_(got_ids)
            h_ids.copy_(got_ids, non_blocking=True)
            h_scores.copy_(got_scores, non_blocking=True)
            ralm.verify(spec_view, retr_view, 1, first_mismatch, stream)
            h_spec.copy_(spec_ids, non_blocking=True)
            h_fm.copy_(first_mismatch, non_blocking=True)
            stream.synchronize()

    for _ in range(3):
        step_e2e()
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step_e2e()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    # ---- aggregate over ranks: time = max, work = sum
    from paper_2401_14021_b200 import replicas
    (total_ms, e2e_ms), job_queries = replicas.aggregate(
        [total_ms, e2e_ms], s * args.steps if (sharded is None or rank == 0) else 0, device)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        value = job_queries / (total_ms * 1e-3)
        e2e_value = job_queries / (e2e_ms * 1e-3)
        corpus_bytes = local_rows * d * 2            # what this GPU streams per pass
        passes = scan_launches / max(args.steps, 1)
        scan_avg_ms = scan_ms / max(scan_launches, 1)
        ordered = sorted(pass_ms)
        scan_median_ms = ordered[len(ordered) // 2] if ordered else None
        kernel = dispatch["kernel_name"]
        sample = dispatch["sample_rows"]
        # algorithmic bytes of one pass, from what the library says it ran: one read of the fp16
        # rows; the tcgen05 scan reads its sample's rows twice (sample launch, then the scan proper);
        # the 8-bit scan reads the sample in fp16 and the rest as one byte per element + one bound
        again = sample if dispatch["phases"] == 3 else 0     # sample rows the main launch scans again
        if dispatch["kernel"] == 5:
            pass_bytes = sample * d * 2 + (local_rows - sample + again) * (d + 4)
        else:
            pass_bytes = (local_rows + again) * d * 2
        achieved = pass_bytes / (scan_avg_ms * 1e-3) / 1e9 if scan_launches else None
        traffic = None
        if dispatch["kernel"] == 2 and cfg.metric == "ip" and s <= 8 and not args.tune and \
                TRAFFIC["sources_sha256_16"] == sources_hash(TRAFFIC["sources"]):
            traffic = corpus_bytes * TRAFFIC["ratio"]
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"] if achieved else None,
                    "peak_kind": peak_kind + " (copy bandwidth: read + write; a pure-read stream may exceed it)",
                    "frac_of_nominal_8000": achieved / 8000.0 if achieved else None,
                    "kernel": kernel, "bytes_per_launch": pass_bytes, "traffic": traffic,
                    "traffic_note": TRAFFIC["note"],
                    "median_frac": (pass_bytes / (scan_median_ms * 1e-3) / 1e9 / peaks["hbm_gbs"])
                    if scan_median_ms else None}
        if dispatch["kernel"] == 5:
            roofline["fp16_equivalent_gbs"] = corpus_bytes / (scan_avg_ms * 1e-3) / 1e9 if scan_launches else None
        per_pass_queries = s / max(dispatch["passes"], 1)
        if dispatch["kernel"] in (3, 4) and per_pass_queries > 255:
            # large batch: s flop per corpus byte is beyond the ridge, the tensor pipe bounds it.
            # fp16 runs at the bf16 rate; the kernel is timed inside a long step: sustained peak
            flops = 2.0 * per_pass_queries * (local_rows + again) * d
            tf = flops / (scan_avg_ms * 1e-3) / 1e12 if scan_launches else None
            peak_tf = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
            roofline = {"bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s",
                        "frac": tf / peak_tf if tf else None, "peak_kind": peak_kind + " (bf16 sustained)",
                        "frac_of_burst": tf / peaks["bf16_tflops"] if tf else None,
                        "kernel": kernel, "flops_per_launch": flops, "traffic": None,
                        "useful_tflops": 2.0 * per_pass_queries * local_rows * d / (scan_avg_ms * 1e-3) / 1e12
                        if scan_launches else None,
                        "hbm_gbs": achieved}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "strong" if sharded is not None else "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "%s %dx%d %s s=%d k=%d; cache lookup R=%d C=%d q=%d; verify stride %d"
                                   % (cfg.name, N, d, cfg.metric, s, k, R, cache.shape[1], stride, vstride),
                       "arithmetic": "fp16 corpus and queries, exact fp16 x fp16 products, fp32 accumulation",
                       "variant": args.variant, "tune": args.tune, "q8": bool(args.q8), "cuda_graph": bool(use_graph),
                       "replicas": 1 if sharded is not None else world,
                       "row_shards": world if sharded is not None else 1,
                       "dispatch": dispatch, "l2_flushed_every_step": bool(args.flush_l2),
                       "l2": "inputs larger than L2 (%.1f GB corpus streamed every step)"
                             % (corpus_bytes / 1e9) if corpus_bytes > 2.5e8 else
                             "corpus near L2 size: L2-warm figure, not an HBM number"},
            "scan_gbs": corpus_bytes / (scan_avg_ms * 1e-3) / 1e9 if scan_launches else None,
            "scan_ms": scan_avg_ms, "scan_median_ms": scan_median_ms, "scan_passes_per_step": passes,
            "search_ms": search_ms,
            "roofline": roofline,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(corpus, queries, metric_id, k, N, s)
        elif world > 1:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    idx.close()
    if sharded is not None:
        cache_index.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def sources_hash(names):
    """First 16 hex digits of the SHA-256 of the kernel sources a capture depends on."""
    import hashlib
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(ROOT, "paper_2401_14021_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


# DRAM traffic of the headline kernel (warp-MMA scan, inner product, up to 8 queries):
# (dram__bytes_read.sum + dram__bytes_write.sum) / corpus bytes of one scan launch, from an ncu
# capture of a 2 M-row case (traffic grows in proportion to the rows). Reported only while the
# sources the kernel is built from are the ones that were captured.
TRAFFIC = {"ratio": 1.0012, "sources": ("scan.cuh", "common.cuh"), "sources_sha256_16": "8f93b5697f0531e0",
           "note": "2M-row ncu capture scaled by rows; null when the kernel's sources changed since"}

if __name__ == "__main__":
    main()
