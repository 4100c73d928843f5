"""ctypes access to the CPU oracle (oracle/deepsqueeze_oracle.c).

TEST INFRASTRUCTURE.  Imported only by the tests, by the smoke check and by
the benchmark's CPU-baseline leg.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_u32p = C.POINTER(C.c_uint32)
_i32p = C.POINTER(C.c_int32)
_f32p = C.POINTER(C.c_float)

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_log_u24.argtypes = [C.c_uint32]
        L.oracle_log_u24.restype = C.c_float
        L.oracle_log_u24_array.argtypes = [C.c_uint32, C.c_int64, _f32p]
        L.oracle_log_u24_array.restype = None
        L.oracle_t3_radius_u24_array.argtypes = [C.c_uint32, C.c_int64, _f32p]
        L.oracle_t3_radius_u24_array.restype = None
        L.oracle_sincos_u24_array.argtypes = [C.c_uint32, C.c_int64, _f32p, _f32p]
        L.oracle_sincos_u24_array.restype = None
        L.oracle_noise_row.argtypes = [C.c_int, C.c_uint64, C.c_uint32, C.c_uint64,
                                       C.c_int64, C.c_int64, _f32p]
        L.oracle_noise_row.restype = None
        L.oracle_rnd24_row.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64,
                                       C.c_int64, C.c_int64, _f32p]
        L.oracle_rnd24_row.restype = None
        L.oracle_level.argtypes = [C.c_int, C.c_int]
        L.oracle_level.restype = C.c_float
        L.oracle_compress_chunk.argtypes = [C.c_int, C.c_int, _f32p, C.c_int64, _f32p,
                                            _f32p, _u32p, _f32p]
        L.oracle_compress_chunk.restype = None
        L.oracle_pack_codes.argtypes = [C.c_int, _u32p, C.c_int64, C.c_int64, _u32p]
        L.oracle_pack_codes.restype = None
        L.oracle_step.argtypes = [
            C.c_int32, C.c_int64, C.c_int64, _i32p, _i32p, _f32p,
            C.c_int, C.c_int, C.c_int64,
            _f32p, _f32p, _f32p, _f32p,
            C.c_float, C.c_int, C.c_float, C.c_float,
            C.c_uint64, C.c_uint64,
            _u32p, C.c_int64, _f32p, C.c_int64, _f32p, _f32p, C.c_int64, _f32p]
        L.oracle_step.restype = C.c_int
        L.oracle_ecsgd_step.argtypes = [
            C.c_int32, C.c_int64, C.c_int64, _i32p, _i32p, _f32p,
            C.c_int, C.c_int, C.c_int64,
            _f32p, _f32p, _f32p, _f32p,
            C.c_float, C.c_int, C.c_float,
            C.c_uint64, C.c_uint64,
            _u32p, C.c_int64, _f32p, C.c_int64, _f32p]
        L.oracle_ecsgd_step.restype = C.c_int
        L.oracle_num_threads.argtypes = []
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_num_threads.argtypes = [C.c_int]
        L.oracle_set_num_threads.restype = None
        _lib = L
    return _lib


def _p(arr, typ):
    return arr.ctypes.data_as(typ)


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c, _u32p), _p(k, _u32p), _p(out, _u32p))
    return out


def log_u24_array(j0: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    lib().oracle_log_u24_array(j0, count, _p(out, _f32p))
    return out


def t3_radius_u24_array(j0: int, count: int) -> np.ndarray:
    """sqrt(3 ((j 2^-24)^(-2/3) - 1)) for j = j0 .. j0 + count - 1."""
    out = np.empty(count, dtype=np.float32)
    lib().oracle_t3_radius_u24_array(j0, count, _p(out, _f32p))
    return out


def sincos_u24_array(k0: int, count: int):
    c = np.empty(count, dtype=np.float32)
    s = np.empty(count, dtype=np.float32)
    lib().oracle_sincos_u24_array(k0, count, _p(c, _f32p), _p(s, _f32p))
    return c, s


def noise_row(kind: int, seed: int, node: int, step: int, k0: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    lib().oracle_noise_row(kind, seed, node, step, k0, count, _p(out, _f32p))
    return out


def rnd24_row(seed: int, node: int, step: int, k0: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    lib().oracle_rnd24_row(seed, node, step, k0, count, _p(out, _f32p))
    return out


def level(bits: int, q: int) -> float:
    return float(lib().oracle_level(bits, q))


def compress_chunk(kind: int, bits: int, v: np.ndarray, r: np.ndarray | None = None):
    v = np.ascontiguousarray(v, dtype=np.float32)
    m = v.shape[0]
    r = np.zeros(m, dtype=np.float32) if r is None else np.ascontiguousarray(r, dtype=np.float32)
    q = np.zeros(m, dtype=np.uint32)
    Cv = np.zeros(m, dtype=np.float32)
    s = C.c_float(0)
    lib().oracle_compress_chunk(kind, bits, _p(v, _f32p), m, _p(r, _f32p), C.byref(s),
                                _p(q, _u32p), _p(Cv, _f32p))
    return float(s.value), q, Cv


def pack_codes(bits: int, q: np.ndarray, first_elem: int = 0) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint32)
    words = np.zeros(((first_elem + q.shape[0]) * bits + 31) // 32, dtype=np.uint32)
    lib().oracle_pack_codes(bits, _p(q, _u32p), first_elem, q.shape[0], _p(words, _u32p))
    return words


def code_bits(comp_kind: int, bits: int) -> int:
    return 32 if comp_kind == 0 else (1 if comp_kind == 1 else bits)


def step(graph, comp_kind: int, bits: int, chunk: int, x: np.ndarray, delta: np.ndarray,
         a: np.ndarray, c: np.ndarray, N: int, sigma: float, noise_kind: int,
         gamma: float, eta: float, seed: int, step_index: int, want_vC: bool = False,
         k_first: int = 0, g_given: np.ndarray | None = None):
    """One iteration in place on x, delta ([n][ld] float32, C-contiguous).

    Returns (codes [n][words] uint32, scales [n][M] float32, v, C) with v, C
    [n][N] float32 when want_vC, else None.  k_first > 0: the arrays hold the
    columns [k_first, k_first + N) of a longer problem (k_first a multiple of
    the chunk length); the random streams are indexed by the global column.
    g_given: the stochastic gradient itself ([n][ld]); a, c, sigma, noise unused.
    """
    n, ld = x.shape
    for arr in (x, delta, a, c) + (() if g_given is None else (g_given,)):
        assert arr.dtype == np.float32 and arr.flags.c_contiguous and arr.shape == (n, ld)
    assert graph.n == n and N <= ld
    cb = code_bits(comp_kind, bits)
    words = (N * cb + 31) // 32
    ch = chunk if chunk > 0 else N
    M = (N + ch - 1) // ch
    codes = np.zeros((n, words), dtype=np.uint32)
    scales = np.zeros((n, M), dtype=np.float32)
    v = np.zeros((n, N), dtype=np.float32) if want_vC else None
    Cv = np.zeros((n, N), dtype=np.float32) if want_vC else None
    rp = np.ascontiguousarray(graph.row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(graph.col_idx, dtype=np.int32)
    w = np.ascontiguousarray(graph.w, dtype=np.float32)
    rc = lib().oracle_step(
        n, N, ld, _p(rp, _i32p), _p(ci, _i32p), _p(w, _f32p),
        comp_kind, bits, chunk,
        _p(x, _f32p), _p(delta, _f32p), _p(a, _f32p), _p(c, _f32p),
        sigma, noise_kind, gamma, eta, seed, step_index,
        _p(codes, _u32p), words, _p(scales, _f32p), M,
        _p(v, _f32p) if want_vC else None, _p(Cv, _f32p) if want_vC else None, k_first,
        None if g_given is None else _p(g_given, _f32p))
    if rc != 0:
        raise MemoryError("oracle_step could not allocate")
    return codes, scales, v, Cv


def ecsgd_step(graph, comp_kind: int, bits: int, chunk: int, x: np.ndarray, delta: np.ndarray,
               a: np.ndarray, c: np.ndarray, N: int, sigma: float, noise_kind: int,
               gamma: float, seed: int, step_index: int, g_given: np.ndarray | None = None):
    """One iteration of centralized error-compensated SGD (Section 1) in place
    on x, delta ([n][ld] float32): row i is worker i's copy of the model, the
    server's average uses row i of W.  Returns (codes, scales)."""
    n, ld = x.shape
    for arr in (x, delta, a, c) + (() if g_given is None else (g_given,)):
        assert arr.dtype == np.float32 and arr.flags.c_contiguous and arr.shape == (n, ld)
    assert graph.n == n and N <= ld
    cb = code_bits(comp_kind, bits)
    words = (N * cb + 31) // 32
    ch = chunk if chunk > 0 else N
    M = (N + ch - 1) // ch
    codes = np.zeros((n, words), dtype=np.uint32)
    scales = np.zeros((n, M), dtype=np.float32)
    rp = np.ascontiguousarray(graph.row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(graph.col_idx, dtype=np.int32)
    w = np.ascontiguousarray(graph.w, dtype=np.float32)
    rc = lib().oracle_ecsgd_step(
        n, N, ld, _p(rp, _i32p), _p(ci, _i32p), _p(w, _f32p), comp_kind, bits, chunk,
        _p(x, _f32p), _p(delta, _f32p), _p(a, _f32p), _p(c, _f32p),
        sigma, noise_kind, gamma, seed, step_index,
        _p(codes, _u32p), words, _p(scales, _f32p), M,
        None if g_given is None else _p(g_given, _f32p))
    if rc != 0:
        raise MemoryError("oracle_ecsgd_step could not allocate")
    return codes, scales


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(t: int) -> None:
    """Spread the (node, chunk) work items over t host threads from now on."""
    lib().oracle_set_num_threads(int(t))
