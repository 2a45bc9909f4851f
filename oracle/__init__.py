"""numpy front end of the CPU oracle (ctypes over oracle/libslowmo_oracle.so).

TEST INFRASTRUCTURE. The oracle restates the paper's Algorithm 1 and Table C.1 in plain
scalar C; it exists to check the CUDA library and shares nothing with it. Only the tests,
the smoke check and the benchmark's CPU-baseline leg import this package.
"""
import ctypes as C

import numpy as np

from . import build as _build

BASE = {"nesterov": 0, "adam": 1, "sgp_nesterov": 2, "sgp_adam": 3}
POLICY = {"reset": 0, "maintain": 1, "average": 2}
GRAD = {"generated": 0, "supplied_hash": 1, "supplied": 1, "supplied_array": 2}
TAG_CURVATURE, TAG_CENTRE, TAG_GRADNOISE, TAG_SUPPLIED = 1, 2, 3, 5


class _Cfg(C.Structure):
    _fields_ = [
        ("m", C.c_uint32), ("tau", C.c_uint32), ("T", C.c_uint32),
        ("alpha", C.c_float), ("beta", C.c_float), ("gamma", C.c_float),
        ("base", C.c_int32), ("mu", C.c_float), ("weight_decay", C.c_float),
        ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float),
        ("buffer_policy", C.c_int32), ("grad_mode", C.c_int32),
        ("seed", C.c_uint64),
        ("a_lo", C.c_float), ("a_hi", C.c_float), ("c_std", C.c_float), ("sigma", C.c_float),
        ("x_init", C.c_float), ("no_average", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        import os
        # tests that plant mistakes in a copy of the oracle point this at the copy's library
        L = C.CDLL(os.environ.get("SLOWMO_ORACLE_LIB") or _build.build())
        L.oracle_mix64.restype = C.c_uint64
        L.oracle_mix64.argtypes = [C.c_uint64]
        L.oracle_stream_word.restype = C.c_uint64
        L.oracle_stream_word.argtypes = [C.c_uint64, C.c_uint64]
        L.oracle_stream_key.restype = C.c_uint64
        L.oracle_stream_key.argtypes = [C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32]
        L.oracle_word_to_unit.restype = C.c_float
        L.oracle_word_to_unit.argtypes = [C.c_uint64]
        L.oracle_word_to_normal_pair.restype = None
        L.oracle_word_to_normal_pair.argtypes = [C.c_uint64, C.POINTER(C.c_float * 2)]
        L.oracle_words_to_normals.restype = None
        L.oracle_words_to_normals.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_stream_normal.restype = C.c_float
        L.oracle_stream_normal.argtypes = [C.c_uint64, C.c_uint64]
        L.oracle_stream_export.restype = None
        L.oracle_stream_export.argtypes = [C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32,
                                           C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        for name in ("slowmo_oracle_run_f32", "slowmo_oracle_run_f64"):
            f = getattr(L, name)
            f.restype = C.c_int
            f.argtypes = [C.POINTER(_Cfg), C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64] + [C.c_void_p] * 7
        for name in ("oracle_curvature", "oracle_centre", "oracle_supplied_gradient"):
            getattr(L, name).restype = C.c_float
        L.oracle_curvature.argtypes = [C.POINTER(_Cfg), C.c_uint64]
        L.oracle_centre.argtypes = [C.POINTER(_Cfg), C.c_uint32, C.c_uint64]
        L.oracle_supplied_gradient.argtypes = [C.POINTER(_Cfg), C.c_uint32, C.c_uint64]
        L.slowmo_oracle_threads.restype = C.c_int
        L.omp_set_num_threads.restype = None       # OpenMP runtime the library is linked with
        L.omp_set_num_threads.argtypes = [C.c_int]
        L.oracle_sgp_hops.restype = C.c_uint32
        L.oracle_sgp_hops.argtypes = [C.c_uint32, C.c_uint64]
        _lib = L
    return _lib


def make_config(*, m, tau, T, alpha=1.0, beta=0.0, gamma=0.1, base="nesterov", mu=0.0,
                weight_decay=0.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8,
                buffer_policy="reset", grad_mode="generated", seed=0, a_lo=0.5, a_hi=2.0,
                c_std=1.0, sigma=0.0, x_init=0.0, no_average=False, **_ignored):
    """Build the C config. Names follow Algorithm 1 / Table C.1 of the paper."""
    return _Cfg(m, tau, T, alpha, beta, gamma, BASE[base], mu, weight_decay, adam_b1, adam_b2,
                adam_eps, POLICY[buffer_policy], GRAD[grad_mode], seed, a_lo, a_hi, c_std, sigma,
                x_init, 1 if no_average else 0)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def run(cfg, *, j=None, j0=0, n=None, precision="f32", gamma_t=None, G=None, want_dbar=False, threads=None):
    """Run Algorithm 1 on coordinates `j` (uint64 array) or j0..j0+n-1.

    Returns dict with x,h,v [m,n], anchor,u [n] (and dbar [T,tau,n] if asked), in float32
    (precision="f32") or float64 (precision="f64"). `threads` limits the OpenMP threads of this
    one call (the coordinates are shared out among them; results do not depend on it).
    """
    if not isinstance(cfg, _Cfg):
        cfg = make_config(**cfg)
    if j is not None:
        j = np.ascontiguousarray(j, dtype=np.uint64)
        n = j.size
    assert n is not None
    dt = np.float32 if precision == "f32" else np.float64
    m = cfg.m
    out = {
        "x": np.empty((m, n), dt), "h": np.empty((m, n), dt), "v": np.empty((m, n), dt),
        "anchor": np.empty((m, n) if cfg.no_average else n, dt),
        "u": np.empty((m, n) if cfg.no_average else n, dt),
    }
    dbar = np.empty((cfg.T, cfg.tau, n), np.float64) if want_dbar else None
    if gamma_t is not None:
        gamma_t = np.ascontiguousarray(gamma_t, dtype=np.float32)
        assert gamma_t.size == cfg.T
    if G is not None:
        G = np.ascontiguousarray(G, dtype=np.float32)
        assert G.shape == (cfg.T * cfg.tau, m, n), G.shape
    fn = lib().slowmo_oracle_run_f32 if precision == "f32" else lib().slowmo_oracle_run_f64
    before = threads_in_use = lib().slowmo_oracle_threads()
    if threads is not None:
        lib().omp_set_num_threads(int(threads))
        threads_in_use = int(threads)
    try:
        rc = fn(C.byref(cfg), _ptr(gamma_t), _ptr(j), j0, n, _ptr(G), _ptr(out["x"]),
                _ptr(out["anchor"]), _ptr(out["u"]), _ptr(out["h"]), _ptr(out["v"]), _ptr(dbar))
    finally:
        if threads_in_use != before:
            lib().omp_set_num_threads(before)
    if rc != 0:
        raise ValueError("oracle rejected the configuration")
    if want_dbar:
        out["dbar"] = dbar
    return out


def normal_pair(word):
    """The two Box-Muller normals (cosine, sine) made from one 64-bit word."""
    z = (C.c_float * 2)()
    lib().oracle_word_to_normal_pair(word, C.byref(z))
    return float(z[0]), float(z[1])


def words_to_normals(words):
    """Both Box-Muller normals of every word: float32 array [n, 2]."""
    words = np.ascontiguousarray(words, dtype=np.uint64)
    out = np.empty((words.size, 2), np.float32)
    lib().oracle_words_to_normals(_ptr(words), words.size, _ptr(out))
    return out


def stream(tag, seed, t, k, w, j0, n, words=True, normals=True):
    """For j0 <= j < j0+n: words j of the stream (uint64) and/or the binary32 normals of
    coordinates j (coordinate j uses output j & 1 of the pair made from word j >> 1)."""
    wd = np.empty(n, np.uint64) if words else None
    z = np.empty(n, np.float32) if normals else None
    lib().oracle_stream_export(tag, seed, t, k, w, j0, n, _ptr(wd), _ptr(z))
    return wd, z


def curvature(cfg, j):
    return np.array([lib().oracle_curvature(C.byref(cfg), int(q)) for q in j], np.float32)


def centre(cfg, w, j):
    return np.array([lib().oracle_centre(C.byref(cfg), w, int(q)) for q in j], np.float32)


def supplied_gradient(cfg, w, j):
    return np.array([lib().oracle_supplied_gradient(C.byref(cfg), w, int(q)) for q in j], np.float32)


def sgp_hops(m, s):
    """Hop distance of the directed exponential graph at global step s."""
    return lib().oracle_sgp_hops(m, s)


def threads():
    return lib().slowmo_oracle_threads()
