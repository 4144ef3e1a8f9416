"""ctypes face of the fp64 CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It never imports the CUDA package and shares no code with it.  The C source
next to this file is the oracle; this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dynakv_oracle.c")
_LIB = os.path.join(_HERE, "libdynakv_oracle.so")

INIT_KMEANSPP = 0
INIT_RANDOM = 1
MODE_ADAPTIVE, MODE_STATIC, MODE_LOCAL, MODE_DELAYED = 0, 1, 2, 3
ST_BUDGET_EXCEEDED = 1
ST_MAX_CLUSTERS = 2
ST_MAX_TOKENS = 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        dp, ip, bp, lp = C.POINTER(C.c_double), C.POINTER(C.c_int), C.POINTER(C.c_ubyte), C.POINTER(C.c_long)
        L.ork_uniform.restype = C.c_double
        L.ork_uniform.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int64]
        L.ork_init_kmeanspp.restype = None
        L.ork_init_kmeanspp.argtypes = [dp, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_int, ip, C.c_double, ip, lp, lp]
        L.ork_init_random.restype = None
        L.ork_init_random.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_int, ip]
        L.ork_assign.restype = None
        L.ork_assign.argtypes = [dp, C.c_int, C.c_int, dp, C.c_int, bp, ip, C.c_double, ip, lp, lp]
        L.ork_update.restype = None
        L.ork_update.argtypes = [dp, C.c_int, C.c_int, ip, C.c_int, dp, ip]
        L.ork_inertia.restype = C.c_double
        L.ork_inertia.argtypes = [dp, C.c_int, C.c_int, dp, ip]
        L.ork_create.restype = C.c_void_p
        L.ork_create.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, C.c_double, C.c_int, C.c_int, C.c_double]
        L.ork_destroy.restype = None
        L.ork_destroy.argtypes = [C.c_void_p]
        L.ork_build.restype = C.c_int
        L.ork_build.argtypes = [C.c_void_p, dp, dp, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_int, C.c_int, ip, ip]
        L.ork_install.restype = C.c_int
        L.ork_install.argtypes = [C.c_void_p, dp, dp, C.c_int, ip, C.c_int]
        L.ork_score.restype = None
        L.ork_score.argtypes = [C.c_void_p, dp, dp]
        L.ork_select.restype = C.c_int
        L.ork_select.argtypes = [C.c_void_p, dp, C.c_int, ip, C.c_int, ip, ip]
        L.ork_attend.restype = None
        L.ork_attend.argtypes = [C.c_void_p, dp, ip, C.c_int, dp]
        L.ork_decode_step.restype = C.c_int
        L.ork_decode_step.argtypes = [C.c_void_p, dp, C.c_int, ip, C.c_int, dp, ip, ip]
        L.ork_append.restype = C.c_int
        L.ork_append.argtypes = [C.c_void_p, dp, dp, C.c_int]
        L.ork_split_check.restype = C.c_int
        L.ork_split_check.argtypes = [C.c_void_p, ip]
        for name, rt in [("ork_n", C.c_int), ("ork_M", C.c_int), ("ork_tau", C.c_double), ("ork_ties", C.c_long),
                         ("ork_violations", C.c_long), ("ork_status", C.c_uint), ("ork_n_splits", C.c_long)]:
            getattr(L, name).restype = rt
            getattr(L, name).argtypes = [C.c_void_p]
        L.ork_get_assign.argtypes = [C.c_void_p, ip]
        L.ork_get_centroids.argtypes = [C.c_void_p, dp]
        L.ork_get_counts.argtypes = [C.c_void_p, ip]
        L.ork_get_M2.argtypes = [C.c_void_p, dp]
        L.ork_get_live.argtypes = [C.c_void_p, bp]
        L.ork_set_tau.argtypes = [C.c_void_p, C.c_double]
        L.ork_set_mode.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.ork_set_buf_max.argtypes = [C.c_void_p, C.c_int]
        L.ork_get_flags.argtypes = [C.c_void_p, bp, ip]
    return _lib


def _d(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _dp(a: Optional[np.ndarray]):
    return a.ctypes.data_as(C.POINTER(C.c_double)) if a is not None else None


def _ip(a: Optional[np.ndarray]):
    return a.ctypes.data_as(C.POINTER(C.c_int)) if a is not None else None


def _bp(a: Optional[np.ndarray]):
    return a.ctypes.data_as(C.POINTER(C.c_ubyte)) if a is not None else None


def uniform(seed: int, unit: int, rnd: int, i: int) -> float:
    return lib().ork_uniform(seed, unit, rnd, i)


def init_kmeanspp(K, M: int, seed: int, unit: int = 0, hint=None, tol: float = 1e-5):
    K = _d(K); n, d = K.shape
    picks = np.zeros(M, np.int32)
    ties, viol = C.c_long(0), C.c_long(0)
    h = _i(hint) if hint is not None else None
    lib().ork_init_kmeanspp(_dp(K), n, d, M, seed, unit, _ip(h), tol, _ip(picks), C.byref(ties), C.byref(viol))
    return picks, ties.value, viol.value


def init_random(n: int, M: int, seed: int, unit: int = 0):
    picks = np.zeros(M, np.int32)
    lib().ork_init_random(n, M, seed, unit, _ip(picks))
    return picks


def assign(K, Cn, live=None, hint=None, tol: float = 1e-5):
    K = _d(K); Cn = _d(Cn); n, d = K.shape; M = Cn.shape[0]
    out = np.zeros(n, np.int32)
    ties, viol = C.c_long(0), C.c_long(0)
    lv = np.ascontiguousarray(live, dtype=np.uint8) if live is not None else None
    h = _i(hint) if hint is not None else None
    lib().ork_assign(_dp(K), n, d, _dp(Cn), M, _bp(lv), _ip(h), tol, _ip(out), C.byref(ties), C.byref(viol))
    return out, ties.value, viol.value


def update(K, a, Cprev):
    K = _d(K); a = _i(a); Cn = _d(Cprev).copy(); n, d = K.shape; M = Cn.shape[0]
    cnt = np.zeros(M, np.int32)
    lib().ork_update(_dp(K), n, d, _ip(a), M, _dp(Cn), _ip(cnt))
    return Cn, cnt


def inertia(K, Cn, a) -> float:
    K = _d(K); Cn = _d(Cn); a = _i(a)
    return lib().ork_inertia(_dp(K), K.shape[0], K.shape[1], _dp(Cn), _ip(a))


class OracleUnit:
    """One unit (one KV head) of the oracle: the four verbs of the library plus getters."""

    def __init__(self, d: int, G: int, max_tokens: int, max_clusters: int, gamma: float = 2.0,
                 alpha: float = 2.0, split_min_size: int = 8, split_iters: int = 8, tol: float = 1e-5,
                 mode: int = MODE_ADAPTIVE, local_max: int = 64, buf_max: int = 64):
        self.d, self.G, self.max_tokens, self.max_clusters = d, G, max_tokens, max_clusters
        self._h = C.c_void_p(lib().ork_create(d, G, max_tokens, max_clusters, gamma, alpha,
                                               split_min_size, split_iters, tol))
        lib().ork_set_mode(self._h, mode, local_max)
        lib().ork_set_buf_max(self._h, buf_max)

    def __del__(self):
        try:
            if self._h:
                lib().ork_destroy(self._h)
                self._h = None
        except Exception:
            pass

    def build(self, K, V, n_clusters: int, T: int, seed: int, unit_index: int = 0,
              init_mode: int = INIT_KMEANSPP, hint_picks=None, hint_assign=None) -> None:
        K = _d(K); V = _d(V)
        hp = _i(hint_picks) if hint_picks is not None else None
        ha = _i(hint_assign) if hint_assign is not None else None
        rc = lib().ork_build(self._h, _dp(K), _dp(V), K.shape[0], n_clusters, T, seed, unit_index,
                             init_mode, _ip(hp), _ip(ha))
        if rc != 0:
            raise ValueError("oracle build: bad sizes")

    def install(self, K, V, assign, n_ids: int) -> None:
        """Continue from a given partition: token -> cluster id map with `n_ids` ids in use; statistics are
        recomputed from the members (Eq. 4)."""
        K = _d(K); V = _d(V); a = _i(assign)
        if lib().ork_install(self._h, _dp(K), _dp(V), K.shape[0], _ip(a), n_ids) != 0:
            raise ValueError("oracle install: bad sizes or ids")

    def scores(self, q) -> np.ndarray:
        q = _d(q); s = np.zeros(self.M, np.float64)
        lib().ork_score(self._h, _dp(q), _dp(s))
        return s

    def select(self, scores, budget: int, hint_ids=None):
        scores = _d(scores)
        ids = np.full(max(self.M, 1), -1, np.int32)
        tok = C.c_int(0)
        h = _i(hint_ids) if hint_ids is not None else None
        n = lib().ork_select(self._h, _dp(scores), budget, _ip(h), (len(h) if h is not None else -1),
                             _ip(ids), C.byref(tok))
        return ids[:n].copy(), tok.value

    def attend(self, q, ids) -> np.ndarray:
        q = _d(q); ids = _i(ids)
        out = np.zeros((self.G, self.d), np.float64)
        lib().ork_attend(self._h, _dp(q), _ip(ids), len(ids), _dp(out))
        return out

    def decode_step(self, q, budget: int, hint_ids=None):
        q = _d(q)
        ids = np.full(max(self.M, 1), -1, np.int32)
        out = np.zeros((self.G, self.d), np.float64)
        tok = C.c_int(0)
        h = _i(hint_ids) if hint_ids is not None else None
        n = lib().ork_decode_step(self._h, _dp(q), budget, _ip(h), (len(h) if h is not None else -1),
                                  _dp(out), _ip(ids), C.byref(tok))
        return out, ids[:n].copy(), tok.value

    def append(self, k, v, hint_cluster: int = -1) -> int:
        k = _d(k); v = _d(v)
        return lib().ork_append(self._h, _dp(k), _dp(v), hint_cluster)

    def split_check(self, hint_assign_after=None) -> int:
        h = _i(hint_assign_after) if hint_assign_after is not None else None
        return lib().ork_split_check(self._h, _ip(h))

    # ---- state
    @property
    def n(self) -> int: return lib().ork_n(self._h)
    @property
    def M(self) -> int: return lib().ork_M(self._h)
    @property
    def tau(self) -> float: return lib().ork_tau(self._h)
    @tau.setter
    def tau(self, v: float) -> None: lib().ork_set_tau(self._h, v)
    @property
    def ties(self) -> int: return lib().ork_ties(self._h)
    @property
    def violations(self) -> int: return lib().ork_violations(self._h)
    @property
    def status(self) -> int: return lib().ork_status(self._h)
    @property
    def n_splits(self) -> int: return lib().ork_n_splits(self._h)

    def assign(self) -> np.ndarray:
        a = np.zeros(max(self.n, 1), np.int32); lib().ork_get_assign(self._h, _ip(a)); return a[: self.n]

    def centroids(self) -> np.ndarray:
        c = np.zeros((max(self.M, 1), self.d), np.float64); lib().ork_get_centroids(self._h, _dp(c)); return c[: self.M]

    def counts(self) -> np.ndarray:
        c = np.zeros(max(self.M, 1), np.int32); lib().ork_get_counts(self._h, _ip(c)); return c[: self.M]

    def M2(self) -> np.ndarray:
        c = np.zeros(max(self.M, 1), np.float64); lib().ork_get_M2(self._h, _dp(c)); return c[: self.M]

    def flags(self):
        """DELAYED mode: (flag [M] bool: a split is owed, buf [M]: entries buffered for the cluster)."""
        f = np.zeros(max(self.M, 1), np.uint8); b = np.zeros(max(self.M, 1), np.int32)
        lib().ork_get_flags(self._h, _bp(f), _ip(b))
        return f[: self.M].astype(bool), b[: self.M]

    def live(self) -> np.ndarray:
        c = np.zeros(max(self.M, 1), np.uint8); lib().ork_get_live(self._h, _bp(c)); return c[: self.M].astype(bool)
