"""fp64 CPU oracle for the exact-retrieval path (test infrastructure only).

Thin numpy/ctypes marshalling around oracle/ralm_oracle.cpp. Nothing here may be
imported by the CUDA package; only tests, the smoke check and the benchmark's
CPU-baseline leg use it.

Functions (all take fp16 data as numpy uint16 or float16 arrays):
  search        -- C.retrieve(q_1..q_s), Algorithm 1 batched verification step
  scores, rank  -- the two halves of `search`, so a corpus too large for host memory can
                   be scored chunk by chunk into one [N] array and then ranked
  cache_search  -- Q.retrieve(q_i), Algorithm 1 speculative retrieval step
  verify        -- m = argmin_i (speculated_i != retrieved_i), Algorithm 1
  pair_score    -- one (row, query) score
"""
import ctypes
import numpy as np

from .build import build as _build

IP = 0
L2 = 1

_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(_build())
    c_i32, c_i64, c_p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
    lib.ralm_oracle_half_to_double.restype = ctypes.c_double
    lib.ralm_oracle_half_to_double.argtypes = [ctypes.c_uint16]
    lib.ralm_oracle_pair_score.restype = ctypes.c_double
    lib.ralm_oracle_pair_score.argtypes = [c_p, c_p, c_i32, c_i32]
    lib.ralm_oracle_scores.restype = c_i32
    lib.ralm_oracle_scores.argtypes = [c_p, c_i64, c_i32, c_p, c_i32, c_p, c_i32]
    lib.ralm_oracle_rank.restype = None
    lib.ralm_oracle_rank.argtypes = [c_p, c_i64, c_i32, c_i32, c_p, c_p]
    lib.ralm_oracle_search.restype = c_i32
    lib.ralm_oracle_search.argtypes = [c_p, c_i64, c_i32, c_p, c_i32, c_i32, c_i32, c_p, c_p, c_i32]
    lib.ralm_oracle_cache_search.restype = None
    lib.ralm_oracle_cache_search.argtypes = [c_p, c_i64, c_i32, c_i32, c_p, c_i32, c_i32, c_p,
                                             c_i32, c_i32, c_p, c_p]
    lib.ralm_oracle_verify.restype = None
    lib.ralm_oracle_verify.argtypes = [c_p, c_p, c_i32, c_i32, c_i32, c_i32, c_p]
    _lib = lib
    return lib


def _as_u16(a):
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("fp16 data must be float16 or uint16, got %s" % a.dtype)
    return np.ascontiguousarray(a)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def half_to_double(bits: int) -> float:
    return _load().ralm_oracle_half_to_double(int(bits) & 0xFFFF)


def pair_score(row, query, metric: int) -> float:
    row, query = _as_u16(row), _as_u16(query)
    assert row.ndim == 1 and row.shape == query.shape
    return _load().ralm_oracle_pair_score(_ptr(row), _ptr(query), row.shape[0], metric)


def scores(rows, query, metric: int, out=None, threads: int = 0):
    """out[j] = score(query, rows[j]); returns (out, threads_used)."""
    rows, query = _as_u16(rows), _as_u16(query)
    n, d = rows.shape
    assert query.shape == (d,)
    if out is None:
        out = np.empty(n, dtype=np.float64)
    assert out.dtype == np.float64 and out.shape == (n,) and out.flags.c_contiguous
    used = _load().ralm_oracle_scores(_ptr(rows), n, d, _ptr(query), metric, _ptr(out), threads)
    return out, used


def rank(all_scores, metric: int, k: int):
    all_scores = np.ascontiguousarray(all_scores, dtype=np.float64)
    ids = np.empty(k, dtype=np.int64)
    sc = np.empty(k, dtype=np.float64)
    _load().ralm_oracle_rank(_ptr(all_scores), all_scores.shape[0], metric, k, _ptr(ids), _ptr(sc))
    return ids, sc


def search(corpus, queries, metric: int, k: int, threads: int = 0, return_threads: bool = False):
    corpus, queries = _as_u16(corpus), _as_u16(queries)
    n, d = corpus.shape
    s = queries.shape[0]
    assert queries.ndim == 2 and (s == 0 or queries.shape[1] == d)
    ids = np.empty((s, k), dtype=np.int64)
    sc = np.empty((s, k), dtype=np.float64)
    used = _load().ralm_oracle_search(_ptr(corpus), n, d, _ptr(queries), s, metric, k,
                                      _ptr(ids), _ptr(sc), threads)
    return (ids, sc, used) if return_threads else (ids, sc)


def cache_search(corpus, cache_ids, queries, metric: int, k: int):
    corpus, queries = _as_u16(corpus), _as_u16(queries)
    cache_ids = np.ascontiguousarray(cache_ids, dtype=np.int64)
    n, d = corpus.shape
    R, C = cache_ids.shape
    assert queries.ndim == 3 and queries.shape[0] == R and queries.shape[2] == d
    q = queries.shape[1]
    ids = np.empty((R, q, k), dtype=np.int64)
    sc = np.empty((R, q, k), dtype=np.float64)
    _load().ralm_oracle_cache_search(_ptr(corpus), n, d, metric, _ptr(cache_ids), R, C,
                                     _ptr(queries), q, k, _ptr(ids), _ptr(sc))
    return ids, sc


def verify(speculated, retrieved, cmp_k: int = 1):
    """speculated [R][stride][cmp_k] (or [R][stride]); retrieved [R][stride][ld]."""
    speculated = np.ascontiguousarray(speculated, dtype=np.int64)
    retrieved = np.ascontiguousarray(retrieved, dtype=np.int64)
    if speculated.ndim == 2:
        speculated = speculated[:, :, None]
    if retrieved.ndim == 2:
        retrieved = retrieved[:, :, None]
    R, stride, ck = speculated.shape
    assert ck == cmp_k and retrieved.shape[:2] == (R, stride) and retrieved.shape[2] >= cmp_k
    ld = retrieved.shape[2]
    out = np.empty(R, dtype=np.int32)
    _load().ralm_oracle_verify(_ptr(speculated), _ptr(retrieved), R, stride, ld, cmp_k, _ptr(out))
    return out
