"""ctypes marshalling for libralm.so; names follow include/ralm.h."""
import ctypes
import os

import torch

IP = 0
L2 = 1

STATUS_NAMES = {0: "RALM_OK", 1: "RALM_ERR_INVALID_ARG", 2: "RALM_ERR_OOM", 3: "RALM_ERR_CUDA",
                4: "RALM_ERR_TIMEOUT", 5: "RALM_ERR_UNSUPPORTED", 6: "RALM_ERR_BAD_CACHE_ID",
                7: "RALM_ERR_STATIC_LIMIT", 8: "RALM_ERR_INTERNAL"}

_HERE = os.path.dirname(os.path.abspath(__file__))
_lib = None


class RalmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, STATUS_NAMES.get(status, str(status))))


def lib_path() -> str:
    """The compiled library; RALM_LIBRARY names another build of it (the bounds-checking one)."""
    return os.environ.get("RALM_LIBRARY") or os.path.join(_HERE, "libralm.so")


def load_library() -> ctypes.CDLL:
    """Load the compiled CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError("%s is missing: build it with `python -m paper_2401_14021_b200.build` "
                           "(there is no CPU fallback)" % path)
    lib = ctypes.CDLL(path)
    i32, i64, p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
    lib.ralm_index_create.restype = i32
    lib.ralm_index_create.argtypes = [p, i64, i32, i32, i32, i32, ctypes.POINTER(p)]
    lib.ralm_index_destroy.restype = i32
    lib.ralm_index_destroy.argtypes = [p]
    lib.ralm_search.restype = i32
    lib.ralm_search.argtypes = [p, p, i32, i32, p, p, p]
    lib.ralm_search_host.restype = i32
    lib.ralm_search_host.argtypes = [p, p, i32, i32, p, p, p]
    lib.ralm_search_static.restype = i32
    lib.ralm_search_static.argtypes = [p, i64, i32, i32, p, i32, i32, p, p, p, p]
    lib.ralm_cache_search.restype = i32
    lib.ralm_cache_search.argtypes = [p, p, i32, i32, p, i32, i32, p, p, p]
    lib.ralm_verify.restype = i32
    lib.ralm_verify.argtypes = [p, p, i32, i32, i32, i32, p, p]
    lib.ralm_cache_update.restype = i32
    lib.ralm_cache_update.argtypes = [p, p, i32, i32, p, i32, i32, i32, p, i32, i64, p]
    lib.ralm_merge_lists.restype = i32
    lib.ralm_merge_lists.argtypes = [p, p, p, i32, i32, i32, i32, p, p, p]
    lib.ralm_debug_fail_allocation.restype = i32
    lib.ralm_debug_fail_allocation.argtypes = [i32]
    lib.ralm_selftest_wait_timeout.restype = i32
    lib.ralm_selftest_wait_timeout.argtypes = [i64, p, p]
    lib.ralm_device_status.restype = i32
    lib.ralm_device_status.argtypes = [p, p]
    lib.ralm_index_enable_q8.restype = i32
    lib.ralm_index_enable_q8.argtypes = [p, i32]
    lib.ralm_index_set_variant.restype = i32
    lib.ralm_index_set_variant.argtypes = [p, i32]
    lib.ralm_index_set_tuning.restype = i32
    lib.ralm_index_set_tuning.argtypes = [p, i32, i32, i32]
    lib.ralm_index_launch_count.restype = i64
    lib.ralm_index_launch_count.argtypes = [p]
    lib.ralm_index_set_timing.restype = i32
    lib.ralm_index_set_timing.argtypes = [p, i32]
    lib.ralm_index_read_timing.restype = i32
    lib.ralm_index_read_timing.argtypes = [p, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    lib.ralm_index_read_timing_list.restype = i32
    lib.ralm_index_read_timing_list.argtypes = [p, ctypes.POINTER(ctypes.c_double), i64, ctypes.POINTER(i64)]
    lib.ralm_index_last_dispatch.restype = i32
    lib.ralm_index_last_dispatch.argtypes = [p, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                             ctypes.POINTER(i64)]
    f64 = ctypes.c_double
    lib.ralm_os3_expected_verified.restype = f64
    lib.ralm_os3_expected_verified.argtypes = [f64, i32]
    lib.ralm_os3_objective.restype = f64
    lib.ralm_os3_objective.argtypes = [f64, f64, f64, i32, i32]
    lib.ralm_os3_gamma.restype = i32
    lib.ralm_os3_gamma.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32), i32, f64, ctypes.POINTER(f64)]
    lib.ralm_os3_stride.restype = i32
    lib.ralm_os3_stride.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32), i32, f64, f64, f64, i32, i32,
                                    ctypes.POINTER(i32)]
    lib.ralm_status_string.restype = ctypes.c_char_p
    lib.ralm_status_string.argtypes = [i32]
    _lib = lib
    return lib


def _check(status: int, where: str):
    if status != 0:
        raise RalmError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("%s must be a contiguous CUDA tensor of %s" % (name, dtype))
    return t.data_ptr()


class Index:
    """ralm_index_create / ralm_index_destroy. Keeps a reference to the corpus tensor."""

    def __init__(self, corpus: torch.Tensor, metric: int, max_s: int = 8, max_k: int = 32):
        self._lib = load_library()
        self._handle = ctypes.c_void_p()
        if corpus.dim() != 2:
            raise TypeError("corpus must be [N][d]")
        ptr = _dev(corpus, torch.float16, "corpus") if corpus.numel() else 0
        self.corpus = corpus
        self.N, self.d = corpus.shape
        self.metric = metric
        self.max_s, self.max_k = max_s, max_k
        with torch.cuda.device(corpus.device):
            _check(self._lib.ralm_index_create(ptr, self.N, self.d, metric, max_s, max_k,
                                               ctypes.byref(self._handle)), "ralm_index_create")

    def close(self):
        if self._handle:
            self._lib.ralm_index_destroy(self._handle)
            self._handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._handle

    def enable_q8(self, force: bool = False):
        _check(self._lib.ralm_index_enable_q8(self._handle, int(force)), "ralm_index_enable_q8")

    def set_variant(self, variant: int):
        _check(self._lib.ralm_index_set_variant(self._handle, variant), "ralm_index_set_variant")

    def set_tuning(self, consumer_warps: int = 0, ring_depth: int = 0, tile_rows: int = 0):
        _check(self._lib.ralm_index_set_tuning(self._handle, consumer_warps, ring_depth, tile_rows),
               "ralm_index_set_tuning")

    def launch_count(self) -> int:
        return self._lib.ralm_index_launch_count(self._handle)

    def set_timing(self, enabled: bool):
        _check(self._lib.ralm_index_set_timing(self._handle, int(enabled)), "ralm_index_set_timing")

    def read_timing(self):
        """(sum of scan-kernel durations in ms, number of launches) since the last read."""
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(self._lib.ralm_index_read_timing(self._handle, ctypes.byref(ms), ctypes.byref(n)),
               "ralm_index_read_timing")
        return ms.value, n.value

    def read_timing_list(self, capacity: int = 4096):
        """Durations in ms of the scan passes timed since the last read, one by one."""
        buf = (ctypes.c_double * max(capacity, 1))()
        n = ctypes.c_int64()
        _check(self._lib.ralm_index_read_timing_list(self._handle, buf, capacity, ctypes.byref(n)),
               "ralm_index_read_timing_list")
        return [buf[i] for i in range(n.value)]

    KERNEL_NAMES = {0: None, 1: "scan_kernel<fma>", 2: "scan_kernel<mma>", 3: "scan_tc_kernel<pair>",
                    4: "scan_tc_kernel<single>", 5: "scan_q8_kernel"}

    def last_dispatch(self):
        """ralm_index_last_dispatch as a dict: kernel (number), kernel_name, passes, phases, sample_rows."""
        k, ps, ph = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        rows = ctypes.c_int64()
        _check(self._lib.ralm_index_last_dispatch(self._handle, ctypes.byref(k), ctypes.byref(ps), ctypes.byref(ph),
                                                  ctypes.byref(rows)), "ralm_index_last_dispatch")
        return {"kernel": k.value, "kernel_name": self.KERNEL_NAMES.get(k.value), "passes": ps.value,
                "phases": ph.value, "sample_rows": rows.value}

    def device_status(self, stream=None) -> int:
        return self._lib.ralm_device_status(self._handle, _stream_ptr(stream))


def search(index: Index, queries: torch.Tensor, k: int, ids: torch.Tensor = None,
           scores: torch.Tensor = None, stream=None):
    """ralm_search: queries fp16 [s][d] on the device -> (ids int64 [s][k], scores fp32 [s][k])."""
    s = queries.shape[0]
    if ids is None:
        ids = torch.empty((s, k), dtype=torch.int64, device=queries.device)
    if scores is None:
        scores = torch.empty((s, k), dtype=torch.float32, device=queries.device)
    qp = _dev(queries, torch.float16, "queries") if s else 0
    _check(index._lib.ralm_search(index.handle, qp, s, k, _dev(ids, torch.int64, "ids") if s else 0,
                                  _dev(scores, torch.float32, "scores") if s else 0,
                                  _stream_ptr(stream)), "ralm_search")
    return ids, scores


def search_host(index: Index, queries: torch.Tensor, k: int, ids: torch.Tensor, scores: torch.Tensor,
                stream=None):
    """ralm_search_host: all three tensors live in (preferably pinned) host memory."""
    s = queries.shape[0]
    for t, dt in ((queries, torch.float16), (ids, torch.int64), (scores, torch.float32)):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise TypeError("host tensors must be contiguous CPU tensors of the right dtype")
    _check(index._lib.ralm_search_host(index.handle, queries.data_ptr(), s, k, ids.data_ptr(),
                                       scores.data_ptr(), _stream_ptr(stream)), "ralm_search_host")
    return ids, scores


def search_static(corpus: torch.Tensor, metric: int, queries: torch.Tensor, k: int,
                  ids: torch.Tensor, scores: torch.Tensor, device_status: torch.Tensor = None,
                  stream=None):
    """ralm_search_static: the search for callers that cannot allocate device memory. No
    index; the caller brings every buffer (ids int64 [s][k], scores fp32 [s][k], optionally a
    one-element int32 status tensor) and the library uses its built-in scratch. This wrapper
    allocates nothing either."""
    lib = load_library()
    s = queries.shape[0]
    N, d = corpus.shape
    _check(lib.ralm_search_static(_dev(corpus, torch.float16, "corpus") if N else 0, N, d, metric,
                                  _dev(queries, torch.float16, "queries") if s else 0, s, k,
                                  _dev(ids, torch.int64, "ids") if s else 0,
                                  _dev(scores, torch.float32, "scores") if s else 0,
                                  _dev(device_status, torch.int32, "device_status")
                                  if device_status is not None else 0,
                                  _stream_ptr(stream)), "ralm_search_static")
    return ids, scores


def cache_search(index: Index, cache_ids: torch.Tensor, queries: torch.Tensor, k: int,
                 ids: torch.Tensor = None, scores: torch.Tensor = None, stream=None):
    """ralm_cache_search: cache_ids int64 [R][C], queries fp16 [R][q][d]."""
    R, C = cache_ids.shape
    q = queries.shape[1]
    if ids is None:
        ids = torch.empty((R, q, k), dtype=torch.int64, device=queries.device)
    if scores is None:
        scores = torch.empty((R, q, k), dtype=torch.float32, device=queries.device)
    _check(index._lib.ralm_cache_search(index.handle, _dev(cache_ids, torch.int64, "cache_ids") if R else 0,
                                        R, C, _dev(queries, torch.float16, "queries") if R else 0, q, k,
                                        _dev(ids, torch.int64, "ids") if R else 0,
                                        _dev(scores, torch.float32, "scores") if R else 0,
                                        _stream_ptr(stream)), "ralm_cache_search")
    return ids, scores


def verify(speculated_ids: torch.Tensor, retrieved_ids: torch.Tensor, cmp_k: int = 1,
           first_mismatch: torch.Tensor = None, stream=None):
    """ralm_verify: speculated int64 [R][stride] (or [R][stride][cmp_k]); retrieved int64
    [R][stride][ld] (or [R][stride], ld = 1) -> first_mismatch int32 [R]."""
    load_library()
    R, stride = speculated_ids.shape[0], speculated_ids.shape[1]
    ld = retrieved_ids.shape[2] if retrieved_ids.dim() == 3 else 1
    if first_mismatch is None:
        first_mismatch = torch.empty((R,), dtype=torch.int32, device=speculated_ids.device)
    sp = _dev(speculated_ids, torch.int64, "speculated_ids") if speculated_ids.numel() else 0
    rp = _dev(retrieved_ids, torch.int64, "retrieved_ids") if retrieved_ids.numel() else 0
    fp = _dev(first_mismatch, torch.int32, "first_mismatch") if R else 0
    _check(_lib.ralm_verify(sp, rp, R, stride, ld, cmp_k, fp, _stream_ptr(stream)), "ralm_verify")
    return first_mismatch


def cache_update(cache_ids: torch.Tensor, cursor: torch.Tensor, retrieved_ids: torch.Tensor, top: int,
                 N: int, steps: torch.Tensor = None, next_n: int = 0, stream=None):
    """ralm_cache_update: insert the ids retrieved by a verification step into the requests' caches
    (in place). cache_ids int64 [R][C], cursor int32 [R], retrieved_ids int64 [R][stride][ld],
    steps int32 [R] or None."""
    lib = load_library()
    R, C = cache_ids.shape
    stride, ld = retrieved_ids.shape[1], retrieved_ids.shape[2]
    _check(lib.ralm_cache_update(_dev(cache_ids, torch.int64, "cache_ids") if R else 0,
                                 _dev(cursor, torch.int32, "cursor") if R else 0, R, C,
                                 _dev(retrieved_ids, torch.int64, "retrieved_ids") if retrieved_ids.numel() else 0,
                                 stride, ld, top, _dev(steps, torch.int32, "steps") if steps is not None else 0,
                                 next_n, N, _stream_ptr(stream)), "ralm_cache_update")
    return cache_ids, cursor


def merge_lists(ids: torch.Tensor, scores: torch.Tensor, row_offset: torch.Tensor, metric: int,
                out_ids: torch.Tensor = None, out_scores: torch.Tensor = None, stream=None):
    """ralm_merge_lists: ids int64 [G][s][k] (shard-local), scores fp32 [G][s][k], row_offset int64 [G]
    -> (ids int64 [s][k] global, scores fp32 [s][k])."""
    lib = load_library()
    G, s, k = ids.shape
    if out_ids is None:
        out_ids = torch.empty((s, k), dtype=torch.int64, device=ids.device)
    if out_scores is None:
        out_scores = torch.empty((s, k), dtype=torch.float32, device=ids.device)
    _check(lib.ralm_merge_lists(_dev(ids, torch.int64, "ids") if s else 0,
                                _dev(scores, torch.float32, "scores") if s else 0,
                                _dev(row_offset, torch.int64, "row_offset"), G, s, k, metric,
                                _dev(out_ids, torch.int64, "out_ids") if s else 0,
                                _dev(out_scores, torch.float32, "out_scores") if s else 0,
                                _stream_ptr(stream)), "ralm_merge_lists")
    return out_ids, out_scores


def _i32_array(values):
    values = [int(v) for v in values]
    return (ctypes.c_int32 * max(len(values), 1))(*values), len(values)


def os3_gamma(matched, strides, gamma_max: float = 0.6) -> float:
    """ralm_os3_gamma: windowed estimate of the speculation accuracy from the first_mismatch values
    (`matched`) and strides of the most recent verification steps."""
    lib = load_library()
    m, w = _i32_array(matched)
    s, _ = _i32_array(strides)
    out = ctypes.c_double()
    _check(lib.ralm_os3_gamma(m, s, w, gamma_max, ctypes.byref(out)), "ralm_os3_gamma")
    return out.value


def os3_stride(matched, strides, a: float, b: float, s_max: int = 16, async_verify: bool = False,
               gamma_max: float = 0.6) -> int:
    """ralm_os3_stride: the speculation stride in 1..s_max that maximises the expected number of
    verified documents per unit time, given speculation-step latency a and verification latency b."""
    lib = load_library()
    m, w = _i32_array(matched)
    s, _ = _i32_array(strides)
    out = ctypes.c_int32()
    _check(lib.ralm_os3_stride(m, s, w, gamma_max, a, b, s_max, int(async_verify), ctypes.byref(out)),
           "ralm_os3_stride")
    return out.value
