"""ctypes loader for the BUZZ CPU oracle (TEST INFRASTRUCTURE, not the product).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module. It
compiles ``buzz_oracle.cpp`` with g++ on first use and exposes one Python class per
(layer, sequence, KV-head) instance. All numbers cross the boundary as float64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "buzz_oracle.cpp")
_LIB = os.path.join(_HERE, "libbuzz_oracle.so")
_lock = threading.Lock()
_lib = None

BO_OK, BO_BAD_ARG, BO_OVERFLOW, BO_NO_PROGRESS = 0, -1, -2, -3


def build(force: bool = False) -> str:
    """Compile the oracle's shared library if it is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        c_int = ctypes.c_int
        lib.bo_create.restype = ctypes.c_void_p
        lib.bo_create.argtypes = [c_int] * 8
        lib.bo_destroy.argtypes = [ctypes.c_void_p]
        lib.bo_prefill.restype = c_int
        lib.bo_prefill.argtypes = [ctypes.c_void_p, c_int, dp, dp, dp, dp, dp]
        lib.bo_decode.restype = c_int
        lib.bo_decode.argtypes = [ctypes.c_void_p, dp, dp, dp, dp]
        lib.bo_evict.restype = c_int
        lib.bo_evict.argtypes = [ctypes.c_void_p]
        lib.bo_get_counts.argtypes = [ctypes.c_void_p, ip, ip, ip]
        lib.bo_get_state.argtypes = [ctypes.c_void_p, ip, dp, dp, dp]
        lib.bo_set_scores.argtypes = [ctypes.c_void_p, dp]
        lib.bo_set_sampling.restype = c_int
        lib.bo_set_sampling.argtypes = [ctypes.c_void_p, c_int, c_int, c_int]
        lib.bo_set_policy.restype = c_int
        lib.bo_set_policy.argtypes = [ctypes.c_void_p, c_int]
        lib.bo_set_state.restype = c_int
        lib.bo_set_state.argtypes = [ctypes.c_void_p, c_int, c_int, c_int, ip, dp, dp, dp]
        _lib = lib
        return lib


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


class OracleHead:
    """One BUZZ cache instance: g query heads sharing one K/V head of dimension d."""

    def __init__(self, g, d, sink, window, segment, hitters, budget, logn=False):
        self._lib = _load()
        self.g, self.d = int(g), int(d)
        self.sink, self.window, self.segment = int(sink), int(window), int(segment)
        self.hitters, self.budget = int(hitters), int(budget)
        self._h = self._lib.bo_create(self.g, self.d, self.sink, self.window, self.segment,
                                      self.hitters, self.budget, int(bool(logn)))
        if not self._h:
            raise ValueError("oracle rejected the BUZZ parameters")

    def __del__(self):
        h = getattr(self, "_h", None)
        if h:
            self._lib.bo_destroy(h)
            self._h = None

    def set_sampling(self, interval_new, new_stride, old_stride):
        """Ablation variants (Section 4.3): interval sampling for new tokens, free strides."""
        rc = self._lib.bo_set_sampling(self._h, int(bool(interval_new)), int(new_stride), int(old_stride))
        if rc < 0:
            raise ValueError("oracle rejected the sampling parameters")
        self.segment = int(new_stride)

    def set_policy(self, global_topk):
        """False: BUZZ's sampling module; True: global top-k of the accumulated scores (Sections 3.2, 4.3)."""
        if self._lib.bo_set_policy(self._h, int(bool(global_topk))) < 0:
            raise ValueError("oracle rejected the policy")

    # -- the three steps -------------------------------------------------------------------
    def prefill(self, Q, K, V):
        """Q [g,N,d], K [N,d], V [N,d] -> (O [g,N,d], full column-sum scores [N], rounds)."""
        Q, K, V = _f64(Q), _f64(K), _f64(V)
        N = K.shape[0]
        assert Q.shape == (self.g, N, self.d) and K.shape == (N, self.d) and V.shape == (N, self.d)
        O = np.empty_like(Q)
        full = np.empty(N, dtype=np.float64)
        rc = self._lib.bo_prefill(self._h, N, _dp(Q), _dp(K), _dp(V), _dp(O), _dp(full))
        if rc < 0:
            raise RuntimeError(f"oracle prefill failed: {rc}")
        return O, full, rc

    def decode(self, q, k, v):
        """q [g,d], k [d], v [d] -> o [g,d]; appends the token and updates the scores."""
        q, k, v = _f64(q), _f64(k), _f64(v)
        assert q.shape == (self.g, self.d) and k.shape == (self.d,) and v.shape == (self.d,)
        o = np.empty_like(q)
        rc = self._lib.bo_decode(self._h, _dp(q), _dp(k), _dp(v), _dp(o))
        if rc < 0:
            raise RuntimeError(f"oracle decode failed: {rc}")
        return o

    def evict(self):
        """Returns 1 if the cache was compacted, 0 if the trigger did not fire, <0 on error."""
        return self._lib.bo_evict(self._h)

    # -- state -----------------------------------------------------------------------------
    def counts(self):
        n, n_old, tot = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        self._lib.bo_get_counts(self._h, ctypes.byref(n), ctypes.byref(n_old), ctypes.byref(tot))
        return n.value, n_old.value, tot.value

    def state(self, with_kv=True):
        n, _, _ = self.counts()
        pos = np.empty(n, dtype=np.int32)
        score = np.empty(n, dtype=np.float64)
        ip = ctypes.POINTER(ctypes.c_int32)
        if with_kv:
            K = np.empty((n, self.d), dtype=np.float64)
            V = np.empty((n, self.d), dtype=np.float64)
            self._lib.bo_get_state(self._h, pos.ctypes.data_as(ip), _dp(score), _dp(K), _dp(V))
            return pos, score, K, V
        self._lib.bo_get_state(self._h, pos.ctypes.data_as(ip), _dp(score), None, None)
        return pos, score

    def set_scores(self, score):
        score = _f64(score)
        assert score.shape == (self.counts()[0],)
        self._lib.bo_set_scores(self._h, _dp(score))

    def set_state(self, n_old, total_len, pos, score, K, V):
        pos = np.ascontiguousarray(np.asarray(pos, dtype=np.int32))
        score, K, V = _f64(score), _f64(K), _f64(V)
        n = pos.shape[0]
        assert score.shape == (n,) and K.shape == (n, self.d) and V.shape == (n, self.d)
        rc = self._lib.bo_set_state(self._h, n, int(n_old), int(total_len),
                                    pos.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                    _dp(score), _dp(K), _dp(V))
        if rc < 0:
            raise ValueError(f"oracle set_state failed: {rc}")
