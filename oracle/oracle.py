"""ctypes wrapper around ``kvs_oracle.c`` (test infrastructure, fp64, CPU).

Every function here only marshals numpy float64 arrays; the arithmetic is in
the C file, whose comments cite the passages of the KVSharer paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvs_oracle.c")
_SO = os.path.join(_HERE, "libkvs_oracle.so")
_lock = threading.Lock()
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp) if the .so is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_attend_unit.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_double, _dp]
    lib.oracle_attend_unit.restype = None
    lib.oracle_attend_units.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_double, _dp]
    lib.oracle_attend_units.restype = None
    lib.oracle_partial_unit.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_double, _dp, _dp, _dp]
    lib.oracle_partial_unit.restype = None
    lib.oracle_combine_partials.argtypes = [ctypes.c_int, ctypes.c_int, _dp, _dp, _dp, _dp]
    lib.oracle_combine_partials.restype = None
    lib.oracle_slot_table.argtypes = [_ip, ctypes.c_int, _ip, _ip]
    lib.oracle_slot_table.restype = ctypes.c_int
    lib.oracle_create.argtypes = [ctypes.c_int] * 5 + [_ip, ctypes.c_double]
    lib.oracle_create.restype = ctypes.c_void_p
    lib.oracle_destroy.argtypes = [ctypes.c_void_p]
    lib.oracle_destroy.restype = None
    lib.oracle_layer_forward.argtypes = [ctypes.c_void_p, ctypes.c_int, _dp, _dp, _dp, ctypes.c_int, _dp]
    lib.oracle_layer_forward.restype = ctypes.c_int
    lib.oracle_layer_prefill.argtypes = [ctypes.c_void_p, ctypes.c_int, _dp, ctypes.c_int, _dp, _dp, ctypes.c_int, _dp]
    lib.oracle_layer_prefill.restype = ctypes.c_int
    lib.oracle_len.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.oracle_len.restype = ctypes.c_int
    lib.oracle_unit_len.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    lib.oracle_unit_len.restype = ctypes.c_int
    lib.oracle_evict.argtypes = [ctypes.c_void_p, ctypes.c_int, _ip, _ip, ctypes.c_int]
    lib.oracle_evict.restype = ctypes.c_int
    lib.oracle_layer_distances.argtypes = [ctypes.c_void_p, _dp]
    lib.oracle_layer_distances.restype = ctypes.c_int
    lib.oracle_mean_cosine.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_longlong]
    lib.oracle_mean_cosine.restype = ctypes.c_double
    lib.oracle_get_cache.argtypes = [ctypes.c_void_p, ctypes.c_int, _dp, _dp]
    lib.oracle_get_cache.restype = ctypes.c_int
    _lib = lib
    return lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def attend_unit(q, K, V, scale: float | None = None) -> np.ndarray:
    """softmax(scale * q K^T) V for one query ``q[D]`` over ``K[n][D]``, ``V[n][D]``."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    n, D = K.shape
    assert q.shape == (D,) and V.shape == (n, D) and n >= 1
    out = np.empty(D, dtype=np.float64)
    s = (1.0 / np.sqrt(float(D))) if scale is None else float(scale)
    _load().oracle_attend_unit(_p(q), _p(K), _p(V), n, D, s, _p(out))
    return out


def attend_units(q, K, V, scale: float | None = None) -> np.ndarray:
    """Independent units: ``q[U][D]``, ``K[U][n][D]``, ``V[U][n][D]`` -> ``out[U][D]``."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    U, n, D = K.shape
    assert q.shape == (U, D) and V.shape == (U, n, D) and n >= 1
    out = np.empty((U, D), dtype=np.float64)
    s = (1.0 / np.sqrt(float(D))) if scale is None else float(scale)
    _load().oracle_attend_units(_p(q), _p(K), _p(V), U, n, D, s, _p(out))
    return out


def partial_unit(q, K, V, j0: int, j1: int, scale: float | None = None):
    """Un-normalised (o[D], m, l) of rows [j0, j1) of one unit."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    n, D = K.shape
    assert 0 <= j0 < j1 <= n
    o = np.empty(D, dtype=np.float64)
    m = ctypes.c_double()
    l = ctypes.c_double()
    s = (1.0 / np.sqrt(float(D))) if scale is None else float(scale)
    _load().oracle_partial_unit(_p(q), _p(K), _p(V), j0, j1, D, s, _p(o),
                                ctypes.byref(m), ctypes.byref(l))
    return o, m.value, l.value


def combine_partials(o, m, l) -> np.ndarray:
    o, m, l = _f64(o), _f64(m), _f64(l)
    S, D = o.shape
    assert m.shape == (S,) and l.shape == (S,)
    out = np.empty(D, dtype=np.float64)
    _load().oracle_combine_partials(S, D, _p(o), _p(m), _p(l), _p(out))
    return out


def mean_cosine(a, b) -> float:
    """Cosine similarity of the sentence-means of ``a[S][dim]`` and ``b[S][dim]``."""
    a, b = _f64(a), _f64(b)
    assert a.ndim == 2 and a.shape == b.shape
    return float(_load().oracle_mean_cosine(_p(a), _p(b), a.shape[0], a.shape[1]))


def slot_table(share_map):
    """(n_caches, root_of_layer, slot_of_layer) for a strategy, or None if it is illegal."""
    sm = np.ascontiguousarray(np.asarray(share_map, dtype=np.int32))
    L = sm.shape[0]
    root = np.empty(L, dtype=np.int32)
    slot = np.empty(L, dtype=np.int32)
    n = _load().oracle_slot_table(sm.ctypes.data_as(_ip), L, root.ctypes.data_as(_ip),
                                  slot.ctypes.data_as(_ip))
    if n < 0:
        return None
    return int(n), root, slot


class Oracle:
    """L literal per-layer caches; sharing is a deep copy made at the layer's turn."""

    def __init__(self, L, Hq, Hkv, D, B, share_map, scale: float | None = None):
        self.L, self.Hq, self.Hkv, self.D, self.B = L, Hq, Hkv, D, B
        sm = np.ascontiguousarray(np.asarray(share_map, dtype=np.int32))
        assert sm.shape == (L,)
        self._lib = _load()
        self._h = self._lib.oracle_create(L, Hq, Hkv, D, B, sm.ctypes.data_as(_ip),
                                          0.0 if scale is None else float(scale))
        if not self._h:
            raise ValueError("illegal configuration or share map")

    def close(self):
        if getattr(self, "_h", None):
            self._lib.oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def layer_forward(self, l, q=None, k_new=None, v_new=None):
        """One layer of one forward pass.

        ``k_new``/``v_new``: ``[B][n_new][Hkv][D]`` (ignored for a sharing layer, may be None);
        ``q``: ``[B][Hq][D]`` or None (cache update only).  Returns ``out[B][Hq][D]`` or None.
        """
        n_new = 0
        kp = vp = None
        if k_new is not None:
            k_new, v_new = _f64(k_new), _f64(v_new)
            assert k_new.shape == v_new.shape and k_new.ndim == 4
            assert k_new.shape[0] == self.B and k_new.shape[2:] == (self.Hkv, self.D)
            n_new = k_new.shape[1]
            kp, vp = _p(k_new), _p(v_new)
        qp = op = None
        out = None
        if q is not None:
            q = _f64(q)
            assert q.shape == (self.B, self.Hq, self.D)
            out = np.empty_like(q)
            qp, op = _p(q), _p(out)
        rc = self._lib.oracle_layer_forward(self._h, l, qp, kp, vp, n_new, op)
        if rc != 0:
            raise RuntimeError("oracle_layer_forward rejected its arguments")
        return out

    def layer_prefill(self, l, q, k_new=None, v_new=None):
        """One layer of the prefill pass: ``q[B][n_q][Hq][D]`` are the newest n_q positions (causal).

        ``k_new``/``v_new``: ``[B][n_new][Hkv][D]`` (ignored on a sharing layer).  Returns ``out[B][n_q][Hq][D]``.
        """
        n_new = 0
        kp = vp = None
        if k_new is not None:
            k_new, v_new = _f64(k_new), _f64(v_new)
            assert k_new.shape == v_new.shape and k_new.shape[0] == self.B and k_new.shape[2:] == (self.Hkv, self.D)
            n_new = k_new.shape[1]
            kp, vp = _p(k_new), _p(v_new)
        q = _f64(q)
        assert q.ndim == 4 and q.shape[0] == self.B and q.shape[2:] == (self.Hq, self.D)
        out = np.empty_like(q)
        rc = self._lib.oracle_layer_prefill(self._h, l, _p(q), q.shape[1], kp, vp, n_new, _p(out))
        if rc != 0:
            raise RuntimeError("oracle_layer_prefill rejected its arguments")
        return out

    def step(self, q, k_new, v_new):
        """One forward pass over all layers in order: ``q[L][B][Hq][D]``, ``k_new[L][B][n][Hkv][D]``."""
        return np.stack([self.layer_forward(l, q[l], k_new[l], v_new[l]) for l in range(self.L)])

    def length(self, l) -> int:
        return int(self._lib.oracle_len(self._h, l))

    def unit_len(self, l, b, h) -> int:
        return int(self._lib.oracle_unit_len(self._h, l, b, h))

    def evict(self, l, keep, n_keep):
        """Keep only rows ``keep[b][h][:n_keep[b][h]]`` (strictly ascending) of every unit of layer l."""
        keep = np.ascontiguousarray(np.asarray(keep, dtype=np.int32))
        n_keep = np.ascontiguousarray(np.asarray(n_keep, dtype=np.int32))
        assert keep.ndim == 3 and keep.shape[:2] == (self.B, self.Hkv) and n_keep.shape == (self.B, self.Hkv)
        rc = self._lib.oracle_evict(self._h, l, keep.ctypes.data_as(_ip), n_keep.ctypes.data_as(_ip), keep.shape[2])
        if rc != 0:
            raise RuntimeError("oracle_evict rejected its arguments")

    def layer_distances(self) -> np.ndarray:
        """``[L][L]`` Euclidean distances between the sample-mean K/V representations of the layers."""
        d = np.empty((self.L, self.L), dtype=np.float64)
        if self._lib.oracle_layer_distances(self._h, _p(d)) != 0:
            raise RuntimeError("oracle_layer_distances needs equally long, un-evicted caches")
        return d

    def cache(self, l):
        """Layer l's cache as (K, V), each ``[B][Hkv][len][D]`` float64."""
        n = self.length(l)
        K = np.empty((self.B, self.Hkv, n, self.D), dtype=np.float64)
        V = np.empty_like(K)
        self._lib.oracle_get_cache(self._h, l, _p(K), _p(V))
        return K, V
