"""ctypes binding of libbalancekv.so: argument marshalling only.

Every step of the hot path runs inside the CUDA library; this module converts torch tensors
to device pointers and error codes to exceptions.  There is no CPU fallback: a missing
library or a failing CUDA call raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbalancekv.so")
_lib = None

OK, E_INVAL, E_NOMEM, E_STATE, E_CUDA, E_TIMEOUT = 0, -1, -2, -3, -4, -5

EXPORTS = [
    "balancekv_create", "balancekv_destroy", "balancekv_stream_append", "balancekv_stream_append_layer",
    "balancekv_stream_append_layer_host", "balancekv_compress", "balancekv_compress_layer",
    "balancekv_decode_attn", "balancekv_decode_attn_host", "balancekv_cache_load_level",
    "balancekv_cache_view", "balancekv_level_sizes", "balancekv_debug_enable", "balancekv_debug_call",
    "balancekv_stats", "balancekv_strerror", "balancekv_plan_calls", "balancekv_reset",
    "balancekv_profile_enable", "balancekv_profile_sample", "balancekv_profile_read", "balancekv_decode_attn_static",
    "balancekv_stream_step", "balancekv_stream_step_host", "balancekv_stream_append_layer_keys",
    "balancekv_decode_attn_two", "balancekv_decode_attn_merged", "balancekv_stream_append_bucketed",
    "balancekv_stream_append_layer_bucketed", "balancekv_stream_append_layer_preserving", "balancekv_debug_set_status", "balancekv_decode_attn_static_status", "balancekv_debug_scratch_used",
]
PROFILE_CLASSES = ("append", "radii", "gram_walk", "compact", "decode", "bookkeeping")


class BalanceKVError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = load().balancekv_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{what}: {msg} ({code})")


class Config(C.Structure):
    """Mirror of ``balancekv_config``."""

    _fields_ = [
        ("n_seqs", C.c_int32), ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("n_q_heads", C.c_int32),
        ("head_dim", C.c_int32), ("dtype", C.c_int32), ("block", C.c_int32), ("levels", C.c_int32),
        ("max_tokens", C.c_int32), ("max_pending", C.c_int32), ("recent_window", C.c_int32),
        ("center_keys", C.c_int32), ("gram_path", C.c_int32), ("decode_splits", C.c_int32),
        ("seed", C.c_uint64), ("delta", C.c_float), ("c_override", C.c_float), ("r_key", C.c_float),
        ("r_value", C.c_float),
    ]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("tokens_appended", "tokens_stored", "calls_run", "walk_fails",
                                         "device_status", "bytes_resident", "kernels_launched", "walk_kernel",
                                         "decode_kernel")]


def load():
    """Load the shared library (building it with nvcc if it is absent); raises on failure."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        from . import build as _build

        _build.build()
    lib = C.CDLL(LIB_PATH)
    vp, ci = C.c_void_p, C.c_int
    lib.balancekv_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    lib.balancekv_destroy.argtypes = [vp]
    lib.balancekv_stream_append.argtypes = [vp, ci, ci, ci, vp, vp, ci, vp]
    lib.balancekv_stream_append_layer.argtypes = [vp, ci, vp, vp, ci, vp]
    lib.balancekv_stream_append_layer_host.argtypes = [vp, ci, vp, vp, ci, vp]
    lib.balancekv_compress.argtypes = [vp, ci, vp]
    lib.balancekv_compress_layer.argtypes = [vp, ci, ci, vp]
    lib.balancekv_decode_attn.argtypes = [vp, ci, vp, vp, vp]
    lib.balancekv_decode_attn_host.argtypes = [vp, ci, vp, vp, vp]
    lib.balancekv_cache_load_level.argtypes = [vp, ci, ci, vp, vp, vp, ci, vp]
    lib.balancekv_cache_view.argtypes = [vp, ci, ci, ci] + [C.POINTER(vp)] * 4 + [C.POINTER(ci)]
    lib.balancekv_level_sizes.argtypes = [vp, ci, ci, ci, vp]
    lib.balancekv_debug_enable.argtypes = [vp, ci]
    lib.balancekv_debug_call.argtypes = [vp, ci, ci, ci, ci, ci] + [C.POINTER(vp)] * 3 + [C.POINTER(ci)]
    lib.balancekv_stats.argtypes = [vp, C.POINTER(Stats)]
    lib.balancekv_strerror.argtypes = [ci]
    lib.balancekv_strerror.restype = C.c_char_p
    lib.balancekv_plan_calls.argtypes = [ci, ci, ci, vp, ci, vp, ci]
    lib.balancekv_reset.argtypes = [vp, vp]
    lib.balancekv_stream_step.argtypes = [vp, ci, vp, vp, vp, vp, vp]
    lib.balancekv_stream_step_host.argtypes = [vp, ci, vp, vp, vp, vp, vp]
    lib.balancekv_profile_enable.argtypes = [vp, ci]
    lib.balancekv_profile_sample.argtypes = [vp, ci, ci]
    lib.balancekv_stream_append_layer_keys.argtypes = [vp, ci, vp, ci, vp]
    lib.balancekv_decode_attn_two.argtypes = [vp, ci, ci, vp, vp, vp]
    lib.balancekv_decode_attn_merged.argtypes = [vp, vp, ci, vp, ci, vp, vp, vp]
    lib.balancekv_profile_read.argtypes = [vp, vp]
    lib.balancekv_stream_append_bucketed.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, ci, C.c_float, vp, vp, vp]
    lib.balancekv_stream_append_layer_bucketed.argtypes = [vp, ci, ci, ci, vp, vp, ci, C.c_float, vp, vp, vp]
    lib.balancekv_stream_append_layer_preserving.argtypes = [vp, ci, vp, vp, ci, C.c_float, vp, vp, vp]
    lib.balancekv_decode_attn_static.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, ci, ci, ci, vp]
    lib.balancekv_decode_attn_static_status.argtypes = [vp, vp]
    lib.balancekv_debug_set_status.argtypes = [vp, ci]
    lib.balancekv_debug_scratch_used.argtypes = [vp, C.POINTER(C.c_int64)]
    for name in EXPORTS:
        if name != "balancekv_strerror":
            getattr(lib, name).restype = ci
    _lib = lib
    return lib


def _check(code: int, what: str):
    if code != OK:
        raise BalanceKVError(code, what)


def _stream_ptr(stream):
    import torch

    if isinstance(stream, int):          # a raw cudaStream_t
        return C.c_void_p(stream)
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _torch_dtype(dtype_code: int):
    import torch

    return torch.bfloat16 if dtype_code == 1 else torch.float32


def plan_calls(block: int, levels: int, recent_window: int, appended_after_event):
    """Host-only bookkeeping of Algorithm 3: list of (event, level, ordinal) per call."""
    import numpy as np

    ev = np.ascontiguousarray(appended_after_event, dtype=np.int32)
    cap = 4 * (int(ev[-1]) // block + 1) + 8 if len(ev) else 8
    out = np.zeros((cap, 3), np.int32)
    n = load().balancekv_plan_calls(block, levels, recent_window, ev.ctypes.data_as(C.c_void_p), len(ev),
                                    out.ctypes.data_as(C.c_void_p), cap)
    _check(min(n, 0), "balancekv_plan_calls")
    assert n <= cap
    return [tuple(int(x) for x in r) for r in out[:n]]


class Context:
    """Owns one ``balancekv_ctx``.  Tensor arguments are CUDA torch tensors of the context's dtype."""

    def __init__(self, n_seqs=1, n_layers=1, n_kv_heads=1, n_q_heads=None, head_dim=128, dtype="bf16", block=1024,
                 levels=2, max_tokens=32768, max_pending=0, recent_window=0, center_keys=0, gram_path=0, seed=0,
                 decode_splits=0, delta=0.0, c_override=0.0, r_key=0.0, r_value=0.0):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("balancekv needs a CUDA device; there is no CPU fallback")
        self.lib = load()
        self.cfg = Config(n_seqs, n_layers, n_kv_heads, n_q_heads if n_q_heads else n_kv_heads, head_dim,
                          1 if dtype == "bf16" else 0, block, levels, max_tokens, max_pending, recent_window,
                          center_keys, gram_path, decode_splits, seed, delta, c_override, r_key, r_value)
        self.dtype = _torch_dtype(self.cfg.dtype)
        self._h = C.c_void_p()
        _check(self.lib.balancekv_create(C.byref(self.cfg), C.byref(self._h)), "balancekv_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            self.lib.balancekv_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dev(self, t, name):
        if not t.is_cuda or t.dtype != self.dtype or not t.is_contiguous():
            raise ValueError(f"{name}: expected a contiguous CUDA tensor of dtype {self.dtype}")
        return C.c_void_p(t.data_ptr())

    def stream_append(self, seq, layer, kv_head, K_blk, V_blk, stream=None):
        assert K_blk.shape == V_blk.shape and K_blk.shape[-1] == self.cfg.head_dim
        _check(self.lib.balancekv_stream_append(self._h, seq, layer, kv_head, self._dev(K_blk, "K_blk"),
                                                self._dev(V_blk, "V_blk"), K_blk.shape[0], _stream_ptr(stream)),
               "balancekv_stream_append")

    def stream_append_layer(self, layer, K, V, stream=None):
        c = self.cfg
        assert tuple(K.shape) == tuple(V.shape) and K.shape[0] == c.n_seqs and K.shape[1] == c.n_kv_heads
        assert K.shape[3] == c.head_dim
        _check(self.lib.balancekv_stream_append_layer(self._h, layer, self._dev(K, "K"), self._dev(V, "V"),
                                                      K.shape[2], _stream_ptr(stream)),
               "balancekv_stream_append_layer")

    def stream_append_layer_host(self, layer, K_host, V_host, stream=None):
        c = self.cfg
        assert not K_host.is_cuda and K_host.dtype == self.dtype and K_host.is_contiguous() and V_host.is_contiguous()
        assert tuple(K_host.shape) == tuple(V_host.shape) and K_host.shape[:2] == (c.n_seqs, c.n_kv_heads)
        _check(self.lib.balancekv_stream_append_layer_host(self._h, layer, C.c_void_p(K_host.data_ptr()),
                                                           C.c_void_p(V_host.data_ptr()), K_host.shape[2],
                                                           _stream_ptr(stream)),
               "balancekv_stream_append_layer_host")

    def compress(self, T=None, stream=None):
        _check(self.lib.balancekv_compress(self._h, self.cfg.levels if T is None else T, _stream_ptr(stream)),
               "balancekv_compress")

    def compress_layer(self, layer, T=None, stream=None):
        _check(self.lib.balancekv_compress_layer(self._h, layer, self.cfg.levels if T is None else T,
                                                 _stream_ptr(stream)), "balancekv_compress_layer")

    def decode_attn(self, layer, q, out=None, stream=None):
        import torch

        c = self.cfg
        assert tuple(q.shape) == (c.n_seqs, c.n_q_heads, c.head_dim)
        if out is None:
            out = torch.empty_like(q)
        _check(self.lib.balancekv_decode_attn(self._h, layer, self._dev(q, "q"), self._dev(out, "out"),
                                              _stream_ptr(stream)), "balancekv_decode_attn")
        return out

    def stream_step(self, layer, q, k_new, v_new, out, stream=None):
        """Append one token per stream of the layer and decode: q, out [B, Hq, d]; k_new, v_new [B, H, d]."""
        _check(self.lib.balancekv_stream_step(self._h, layer, self._dev(q, "q"), self._dev(k_new, "k_new"),
                                              self._dev(v_new, "v_new"), self._dev(out, "out"), _stream_ptr(stream)),
               "balancekv_stream_step")
        return out

    def stream_append_layer_keys(self, layer, K, stream=None):
        """Denominator instance of Algorithm 1: append (k_j, 1); K [B, H, n, d] on the device."""
        _check(self.lib.balancekv_stream_append_layer_keys(self._h, layer, self._dev(K, "K"), K.shape[2],
                                                           _stream_ptr(stream)), "balancekv_stream_append_layer_keys")

    def stream_append_layer_bucketed(self, layer0, n_buckets, i_top, K, V, erase_ratio=0.0, want_slots=False,
                                     stream=None):
        """Algorithm 1's bucketing step for every stream of a layer: K, V [B, H, n, d] on the device;
        slot layer0 + b receives the rows with 2^(i_top-b-1) < ||v|| <= 2^(i_top-b).  Returns the
        per-stream counts [B*H, n_buckets + 1] (last column: dropped rows) and, if asked, the int8
        slot of every row [B, H, n]."""
        import numpy as np
        import torch

        assert K.shape == V.shape and K.dim() == 4
        counts = np.zeros((K.shape[0] * K.shape[1], n_buckets + 1), np.int32)
        slots = torch.empty(K.shape[:3], dtype=torch.int8, device=K.device) if want_slots else None
        _check(self.lib.balancekv_stream_append_layer_bucketed(
            self._h, layer0, n_buckets, i_top, self._dev(K, "K"), self._dev(V, "V"), K.shape[2], float(erase_ratio),
            slots.data_ptr() if want_slots else None, counts.ctypes.data, _stream_ptr(stream)),
            "balancekv_stream_append_layer_bucketed")
        return (counts, slots) if want_slots else counts

    def stream_append_layer_preserving(self, layer0, K, V, tau, want_slots=False, stream=None):
        """Section 4.3's augmented variant: rows whose key has cosine <= tau with the block's mean key go to slot
        layer0 (kept exactly), the rest to slot layer0 + 1.  Returns counts [B*H, 3] (preserved, rest, dropped)
        and, if asked, the int8 slot of every row [B, H, n]."""
        import numpy as np
        import torch

        assert K.shape == V.shape and K.dim() == 4
        counts = np.zeros((K.shape[0] * K.shape[1], 3), np.int32)
        slots = torch.empty(K.shape[:3], dtype=torch.int8, device=K.device) if want_slots else None
        _check(self.lib.balancekv_stream_append_layer_preserving(
            self._h, layer0, self._dev(K, "K"), self._dev(V, "V"), K.shape[2], float(tau),
            slots.data_ptr() if want_slots else None, counts.ctypes.data, _stream_ptr(stream)),
            "balancekv_stream_append_layer_preserving")
        return (counts, slots) if want_slots else counts

    def stream_append_bucketed(self, seq, layer0, n_buckets, i_top, kv_head, K, V, erase_ratio=0.0, want_slots=False,
                               stream=None):
        """Same for one stream: K, V [n, d] on the device."""
        import numpy as np
        import torch

        assert K.shape == V.shape and K.dim() == 2
        counts = np.zeros((1, n_buckets + 1), np.int32)
        slots = torch.empty(K.shape[0], dtype=torch.int8, device=K.device) if want_slots else None
        _check(self.lib.balancekv_stream_append_bucketed(
            self._h, seq, layer0, n_buckets, i_top, kv_head, self._dev(K, "K"), self._dev(V, "V"), K.shape[0],
            float(erase_ratio), slots.data_ptr() if want_slots else None, counts.ctypes.data, _stream_ptr(stream)),
            "balancekv_stream_append_bucketed")
        return (counts[0], slots) if want_slots else counts[0]

    def decode_attn_two(self, layer_num, layer_den, q, out=None, stream=None):
        """Algorithm 1's output ratio: numerator from slot layer_num, denominator from slot layer_den."""
        import torch

        if out is None:
            out = torch.empty_like(q)
        _check(self.lib.balancekv_decode_attn_two(self._h, layer_num, layer_den, self._dev(q, "q"), self._dev(out, "out"),
                                                  _stream_ptr(stream)), "balancekv_decode_attn_two")
        return out

    def decode_attn_merged(self, layers_num, layers_den, q, out=None, stream=None):
        """Value sums of the slots layers_num over weight sums of the slots layers_den (see balancekv.h)."""
        import torch

        if out is None:
            out = torch.empty_like(q)
        ln = (C.c_int32 * len(layers_num))(*layers_num)
        ld = (C.c_int32 * len(layers_den))(*layers_den)
        _check(self.lib.balancekv_decode_attn_merged(self._h, ln, len(layers_num), ld, len(layers_den), self._dev(q, "q"),
                                                     self._dev(out, "out"), _stream_ptr(stream)), "balancekv_decode_attn_merged")
        return out

    def stream_step_host(self, layer, q_host, k_host, v_host, out_host, stream=None):
        _check(self.lib.balancekv_stream_step_host(self._h, layer, C.c_void_p(q_host.data_ptr()),
                                                   C.c_void_p(k_host.data_ptr()), C.c_void_p(v_host.data_ptr()),
                                                   C.c_void_p(out_host.data_ptr()), _stream_ptr(stream)),
               "balancekv_stream_step_host")
        return out_host

    def decode_attn_host(self, layer, q_host, out_host, stream=None):
        assert not q_host.is_cuda and not out_host.is_cuda and q_host.dtype == self.dtype
        _check(self.lib.balancekv_decode_attn_host(self._h, layer, C.c_void_p(q_host.data_ptr()),
                                                   C.c_void_p(out_host.data_ptr()), _stream_ptr(stream)),
               "balancekv_decode_attn_host")
        return out_host

    def cache_load_level(self, layer, level, K, V, orig_idx=None, stream=None):
        import torch

        idx_p = None
        if orig_idx is not None:
            assert orig_idx.is_cuda and orig_idx.dtype == torch.int32 and orig_idx.is_contiguous()
            idx_p = C.c_void_p(orig_idx.data_ptr())
        _check(self.lib.balancekv_cache_load_level(self._h, layer, level, self._dev(K, "K"), self._dev(V, "V"),
                                                   idx_p, K.shape[2], _stream_ptr(stream)),
               "balancekv_cache_load_level")

    def level_sizes(self, seq, layer, kv_head):
        import numpy as np

        s = np.zeros(self.cfg.levels + 1, np.int32)
        _check(self.lib.balancekv_level_sizes(self._h, seq, layer, kv_head, s.ctypes.data_as(C.c_void_p)),
               "balancekv_level_sizes")
        return s

    def cache_view(self, seq, layer, kv_head):
        """Copies of the stream's weighted set as torch tensors: K, V [len,d], w [len], idx [len]."""
        import torch

        pk, pv, pw, pi = C.c_void_p(), C.c_void_p(), C.c_void_p(), C.c_void_p()
        n = C.c_int()
        _check(self.lib.balancekv_cache_view(self._h, seq, layer, kv_head, C.byref(pk), C.byref(pv), C.byref(pw),
                                             C.byref(pi), C.byref(n)), "balancekv_cache_view")
        n = n.value
        d = self.cfg.head_dim
        K = _from_ptr(pk.value, (n, d), self.dtype)
        V = _from_ptr(pv.value, (n, d), self.dtype)
        w = _from_ptr(pw.value, (n,), torch.float32)
        idx = _from_ptr(pi.value, (n,), torch.int32)
        return K, V, w, idx

    def debug_enable(self, on=True):
        _check(self.lib.balancekv_debug_enable(self._h, 1 if on else 0), "balancekv_debug_enable")

    def debug_call(self, seq, layer, kv_head, level, ordinal):
        import torch

        pe, ps, pp = C.c_void_p(), C.c_void_p(), C.c_void_p()
        m = C.c_int()
        _check(self.lib.balancekv_debug_call(self._h, seq, layer, kv_head, level, ordinal, C.byref(pe), C.byref(ps),
                                             C.byref(pp), C.byref(m)), "balancekv_debug_call")
        torch.cuda.synchronize()
        return (_from_ptr(pe.value, (m.value,), torch.int8), _from_ptr(ps.value, (m.value,), torch.float32),
                _from_ptr(pp.value, (m.value,), torch.float32))

    def debug_scratch_used(self) -> int:
        """Words of the split-K decode scratch that are not empty (0 between launches)."""
        n = C.c_int64(0)
        _check(self.lib.balancekv_debug_scratch_used(self._h, C.byref(n)), "balancekv_debug_scratch_used")
        return int(n.value)

    def debug_set_status(self, value):
        """Testing aid: overwrite the device status word (1 = a bounded wait gave up)."""
        _check(self.lib.balancekv_debug_set_status(self._h, int(value)), "balancekv_debug_set_status")

    def reset(self, stream=None):
        _check(self.lib.balancekv_reset(self._h, _stream_ptr(stream)), "balancekv_reset")

    def profile_enable(self, on=True, classes=None):
        """Time every kernel class, or only the named ones (see PROFILE_CLASSES)."""
        flag = 1 if on else 0
        if on and classes is not None:
            flag = sum(2 << PROFILE_CLASSES.index(n) for n in classes)
        _check(self.lib.balancekv_profile_enable(self._h, flag), "balancekv_profile_enable")

    def profile_sample(self, kernel_class, every):
        """Time only every `every`-th launch of one class (name from PROFILE_CLASSES)."""
        _check(self.lib.balancekv_profile_sample(self._h, PROFILE_CLASSES.index(kernel_class), int(every)),
               "balancekv_profile_sample")

    def profile_read(self):
        """{class name: (launches, total ms)} since the last read."""
        buf = (C.c_double * (2 * len(PROFILE_CLASSES)))()
        _check(self.lib.balancekv_profile_read(self._h, buf), "balancekv_profile_read")
        return {n: (int(buf[2 * i]), float(buf[2 * i + 1])) for i, n in enumerate(PROFILE_CLASSES)}

    def stats(self):
        s = Stats()
        code = self.lib.balancekv_stats(self._h, C.byref(s))
        if code != E_TIMEOUT:               # a timed-out wait is reported through device_status; the record is filled
            _check(code, "balancekv_stats")
        return {n: getattr(s, n) for n, _ in Stats._fields_}


def decode_attn_static(K, V, n_heavy, level, q, out=None, stream=None):
    """Allocation-free decode attention over caller-owned caches (see balancekv.h).

    K, V: CUDA tensors [n_streams, cache_len, d]; q: [n_streams, group, d]; the first
    ``n_heavy`` rows of every stream weigh 2**level, the rest 1.  ``out`` must be supplied by
    callers that may not allocate; when it is None a tensor is created for convenience."""
    import torch

    assert K.is_cuda and V.is_cuda and q.is_cuda and K.is_contiguous() and V.is_contiguous() and q.is_contiguous()
    assert K.shape == V.shape and K.dtype == V.dtype == q.dtype and q.shape[0] == K.shape[0] and q.shape[2] == K.shape[2]
    if out is None:
        out = torch.empty_like(q)
    dtype_code = {torch.float32: 0, torch.bfloat16: 1}[K.dtype]
    _check(load().balancekv_decode_attn_static(C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()), K.shape[0],
                                               K.shape[1], n_heavy, level, C.c_void_p(q.data_ptr()),
                                               C.c_void_p(out.data_ptr()), q.shape[1], K.shape[2], dtype_code,
                                               _stream_ptr(stream)), "balancekv_decode_attn_static")
    return out


def decode_attn_static_status(stream=None):
    """Status word of the allocation-free entry point on the current device: 0, or 1 if a bounded
    wait of one of its launches gave up since the last read (reading clears it).  Synchronises the stream."""
    v = C.c_int(0)
    _check(load().balancekv_decode_attn_static_status(C.byref(v), _stream_ptr(stream)), "balancekv_decode_attn_static_status")
    return v.value


class _RawDevice:
    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"data": (ptr, False), "shape": tuple(shape), "typestr": typestr,
                                         "version": 2}


def _from_ptr(ptr, shape, dtype):
    """Copy ``shape`` elements of ``dtype`` from a raw device pointer into a new torch tensor."""
    import torch

    n = 1
    for s in shape:
        n *= s
    if n == 0 or not ptr:
        return torch.empty(shape, dtype=dtype, device="cuda")
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.int8: "|i1", torch.bfloat16: "<i2"}[dtype]
    raw = torch.as_tensor(_RawDevice(ptr, shape, typestr), device="cuda")
    if dtype == torch.bfloat16:
        raw = raw.view(torch.bfloat16)
    out = raw.clone()
    torch.cuda.synchronize()
    return out
