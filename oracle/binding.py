"""ctypes access to the C++ oracle (``balancekv_oracle.cpp``) -- test infrastructure.

Argument marshalling only: every number the oracle reports is computed by the C++ file
beside this one, in double precision.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "balancekv_oracle.cpp")
_LIB = os.path.join(_HERE, "libbalancekv_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2 -fopenmp) if the shared object is stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", _SRC, "-o", tmp]
            )
            os.replace(tmp, _LIB)
    return _LIB


class OracleParams(C.Structure):
    """Mirror of ``okv_params``."""

    _fields_ = [
        ("d", C.c_int32),
        ("t", C.c_int32),
        ("T", C.c_int32),
        ("W", C.c_int32),
        ("center_keys", C.c_int32),
        ("layer", C.c_int32),
        ("head", C.c_int32),
        ("max_tokens", C.c_int32),
        ("seed", C.c_uint64),
        ("delta", C.c_double),
        ("c_override", C.c_double),
        ("r_key", C.c_double),
        ("r_value", C.c_double),
    ]

    def __init__(self, d, t, T=1, W=0, center_keys=0, layer=0, head=0, max_tokens=None, seed=0,
                 delta=0.0, c_override=0.0, r_key=0.0, r_value=0.0):
        super().__init__(d, t, T, W, center_keys, layer, head,
                         max_tokens if max_tokens is not None else t, seed, delta, c_override,
                         r_key, r_value)


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = C.CDLL(_LIB)
    dp = C.POINTER(C.c_double)
    lib.okv_walk_uniform.restype = C.c_double
    lib.okv_walk_uniform.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]
    lib.okv_walk_constant.restype = C.c_double
    lib.okv_walk_constant.argtypes = [C.POINTER(OracleParams), C.c_int]
    lib.okv_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.okv_softmax_balance.restype = C.c_int
    lib.okv_softmax_balance.argtypes = [C.POINTER(OracleParams), C.c_void_p, C.c_void_p, C.c_int,
                                        C.c_int, C.c_int] + [C.c_void_p] * 7
    lib.okv_stream_new.restype = C.c_void_p
    lib.okv_stream_new.argtypes = [C.POINTER(OracleParams)]
    lib.okv_stream_free.argtypes = [C.c_void_p]
    lib.okv_stream_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
    lib.okv_stream_force_eta.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int]
    lib.okv_stream_compress.argtypes = [C.c_void_p]
    lib.okv_stream_compress.restype = C.c_int
    lib.okv_streams_compress.argtypes = [C.c_void_p, C.c_int]
    lib.okv_streams_compress.restype = C.c_int
    lib.okv_stream_len.restype = C.c_int64
    lib.okv_stream_len.argtypes = [C.c_void_p]
    lib.okv_stream_level_sizes.argtypes = [C.c_void_p, C.c_void_p]
    lib.okv_stream_view.argtypes = [C.c_void_p] * 5
    lib.okv_stream_num_calls.argtypes = [C.c_void_p]
    lib.okv_stream_num_calls.restype = C.c_int
    lib.okv_stream_call_info.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
    lib.okv_stream_call_data.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 6
    lib.okv_stream_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
    lib.okv_stream_exact.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
    lib.okv_weighted_attn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int,
                                      C.c_void_p, C.c_int, C.c_void_p]
    lib.okv_weighted_sums.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_void_p]
    lib.okv_num_threads.restype = C.c_int
    _ = dp
    _lib = lib
    return lib


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def num_threads() -> int:
    return int(_load().okv_num_threads())


def philox4x32_10(key, ctr):
    k = np.asarray(key, dtype=np.uint32).copy()
    c = np.asarray(ctr, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().okv_philox4x32_10(_ptr(k), _ptr(c), _ptr(out))
    return out


def walk_uniform(seed, layer, head, ordinal, level, j) -> float:
    return float(_load().okv_walk_uniform(seed, layer, head, ordinal, level, j))


def walk_constant(params: OracleParams, m: int) -> float:
    return float(_load().okv_walk_constant(C.byref(params), m))


def softmax_balance(params: OracleParams, K, V, ordinal=0, level=0, forced=None):
    """One SoftmaxBalance call plus strict-half selection.  Returns a dict of arrays."""
    K = _f64(K)
    V = _f64(V)
    m = K.shape[0]
    eta = np.zeros(m, np.int8)
    S = np.zeros(m)
    p = np.zeros(m)
    u = np.zeros(m)
    kept = np.zeros(m, np.int32)
    stats = np.zeros(4)
    f = None if forced is None else np.ascontiguousarray(np.asarray(forced, dtype=np.int8))
    nk = _load().okv_softmax_balance(C.byref(params), _ptr(K), _ptr(V), m, ordinal, level, _ptr(f),
                                     _ptr(eta), _ptr(S), _ptr(p), _ptr(u), _ptr(kept), _ptr(stats))
    return dict(eta=eta, S=S, p=p, u=u, kept=kept[:nk].copy(), rk2=stats[0], rv2=stats[1],
                c=stats[2], fails=int(stats[3]))


def weighted_attention(K, V, w, q):
    """z = sum w_i e^{<k_i,q>/sqrt d} v_i / sum w_i e^{<k_i,q>/sqrt d}; q: [nq,d]."""
    K = _f64(K)
    V = _f64(V)
    q = _f64(q).reshape(-1, K.shape[1])
    wv = None if w is None else _f64(w)
    out = np.zeros_like(q)
    _load().okv_weighted_attn(_ptr(K), _ptr(V), _ptr(wv), K.shape[0], K.shape[1], _ptr(q),
                              q.shape[0], _ptr(out))
    return out


def weighted_sums(K, V, w, q):
    """(num [nq,d], den [nq], logmax [nq]): sum w e^{<k,q>/sqrt d - m} v, sum w e^{... - m}, m (natural log)."""
    K = _f64(K)
    V = _f64(V)
    q = _f64(q).reshape(-1, K.shape[1])
    wv = None if w is None else _f64(w)
    num = np.zeros_like(q)
    den = np.zeros(q.shape[0])
    mx = np.zeros(q.shape[0])
    _load().okv_weighted_sums(_ptr(K), _ptr(V), _ptr(wv), K.shape[0], K.shape[1], _ptr(q), q.shape[0],
                              _ptr(num), _ptr(den), _ptr(mx))
    return num, den, mx


def two_instance_estimate(numerator_view, denominator_view, q):
    """Algorithm 1's output ratio from the (K, V, w) view of the numerator instance and the
    (K, ., w) view of the denominator instance."""
    Kn, Vn, wn = numerator_view[:3]
    Kd, Vd, wd = denominator_view[:3]
    num, _, mn = weighted_sums(Kn, Vn, wn, q)
    _, den, md = weighted_sums(Kd, Vd, wd, q)
    return num * np.exp(mn - md)[:, None] / den[:, None]


def merged_estimate(numerator_views, denominator_views, q):
    """Value sums of several (K, V, w) views over weight sums of several views: the estimator over the
    union of caches (same views on both sides) or Algorithm 1's ratio (numerator instances above,
    the denominator instance below)."""
    q = _f64(q).reshape(-1, numerator_views[0][0].shape[1])
    nums = [weighted_sums(v[0], v[1], v[2], q) for v in numerator_views if len(v[2])]
    dens = [weighted_sums(v[0], v[1], v[2], q) for v in denominator_views if len(v[2])]
    m = np.max(np.stack([x[2] for x in nums + dens]), axis=0)
    num = sum(x[0] * np.exp(x[2] - m)[:, None] for x in nums)
    den = sum(x[1] * np.exp(x[2] - m) for x in dens)
    return num / den[:, None]


class OracleStream:
    """One (sequence, layer, KV head) stream driven by MergeAndReduce."""

    def __init__(self, params: OracleParams):
        self.params = params
        self.d = params.d
        self._lib = _load()
        self._h = C.c_void_p(self._lib.okv_stream_new(C.byref(params)))

    def __del__(self):
        try:
            if self._h:
                self._lib.okv_stream_free(self._h)
                self._h = None
        except Exception:
            pass

    def append(self, K, V):
        K = _f64(K).reshape(-1, self.d)
        V = _f64(V).reshape(-1, self.d)
        assert K.shape == V.shape
        self._lib.okv_stream_append(self._h, _ptr(K), _ptr(V), K.shape[0])

    def force_eta(self, level, ordinal, eta):
        e = np.ascontiguousarray(np.asarray(eta, dtype=np.int8))
        self._lib.okv_stream_force_eta(self._h, level, ordinal, _ptr(e), e.shape[0])

    def compress(self) -> int:
        return int(self._lib.okv_stream_compress(self._h))

    def __len__(self):
        return int(self._lib.okv_stream_len(self._h))

    def level_sizes(self):
        s = np.zeros(self.params.T + 1, np.int64)
        self._lib.okv_stream_level_sizes(self._h, _ptr(s))
        return s

    def view(self):
        n = len(self)
        K = np.zeros((n, self.d))
        V = np.zeros((n, self.d))
        w = np.zeros(n)
        idx = np.zeros(n, np.int32)
        self._lib.okv_stream_view(self._h, _ptr(K), _ptr(V), _ptr(w), _ptr(idx))
        return K, V, w, idx

    def calls(self):
        out = []
        for c in range(int(self._lib.okv_stream_num_calls(self._h))):
            info = np.zeros(4, np.int32)
            st = np.zeros(3)
            self._lib.okv_stream_call_info(self._h, c, _ptr(info), _ptr(st))
            m = int(info[2])
            idx = np.zeros(m, np.int32)
            eta = np.zeros(m, np.int8)
            S = np.zeros(m)
            p = np.zeros(m)
            u = np.zeros(m)
            kept = np.zeros(m // 2, np.int32)
            self._lib.okv_stream_call_data(self._h, c, _ptr(idx), _ptr(eta), _ptr(S), _ptr(p),
                                           _ptr(u), _ptr(kept))
            out.append(dict(level=int(info[0]), ordinal=int(info[1]), m=m, fails=int(info[3]),
                            rk2=st[0], rv2=st[1], c=st[2], idx=idx, eta=eta, S=S, p=p, u=u,
                            kept=kept))
        return out

    def decode(self, q):
        q = _f64(q).reshape(-1, self.d)
        out = np.zeros_like(q)
        self._lib.okv_stream_decode(self._h, _ptr(q), q.shape[0], _ptr(out))
        return out

    def exact(self, q):
        q = _f64(q).reshape(-1, self.d)
        out = np.zeros_like(q)
        self._lib.okv_stream_exact(self._h, _ptr(q), q.shape[0], _ptr(out))
        return out


def compress_streams(streams) -> int:
    """Run every ready call of every stream; OpenMP over the independent streams."""
    arr = (C.c_void_p * len(streams))(*[s._h for s in streams])
    return int(_load().okv_streams_compress(arr, len(streams)))
