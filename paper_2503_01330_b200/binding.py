"""Thin ctypes binding of the C ABI in include/wkv.h: argument marshalling only.

Every step of the decode path runs inside libwkv.so's CUDA kernels.  There is no fallback: if the shared
library has not been built, loading raises.  torch tensors are used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwkv.so")

WKV_F32, WKV_BF16 = 0, 1
WKV_SCHEDULE_AUTO, WKV_SCHEDULE_SPLIT, WKV_SCHEDULE_CLUSTER, WKV_SCHEDULE_FLAT = 0, 1, 2, 3
WKV_OK, WKV_ERR_INVALID, WKV_ERR_ALLOC, WKV_ERR_CUDA, WKV_ERR_STATE, WKV_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5

ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
RELEASE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class wkv_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("budget", C.c_int32), ("window", C.c_int32), ("sink", C.c_int32),
                ("dtype", C.c_int32), ("scale", C.c_float), ("merge", C.c_int32), ("n_splits", C.c_int32), ("schedule", C.c_int32),
                ("stream", C.c_void_p), ("alloc", ALLOC_FN), ("release", RELEASE_FN), ("user", C.c_void_p)]


EXPORTS = ["wkv_config_error", "wkv_create", "wkv_destroy", "wkv_reset", "wkv_set_stream", "wkv_decode_step",
           "wkv_decode_step_layers", "wkv_decode_step_static", "wkv_decode_step_host", "wkv_decode_step_layers_host", "wkv_prefill", "wkv_prefill_bulk", "wkv_prefill_bulk_layers", "wkv_export_state", "wkv_export_slots", "wkv_import_state",
           "wkv_status", "wkv_selftest_wait_timeout", "wkv_launch_count", "wkv_device_bytes", "wkv_splits", "wkv_strerror", "wkv_last_error"]

_lib = None


def lib():
    """Loads libwkv.so (once).  Raises if it is missing: the CUDA library is the only implementation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2503_01330_b200.build.build_library()")
        L = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        L.wkv_config_error.restype = C.c_char_p
        L.wkv_config_error.argtypes = [C.POINTER(wkv_config)]
        L.wkv_create.argtypes = [C.POINTER(wkv_config), C.POINTER(vp)]
        L.wkv_destroy.restype = None
        L.wkv_destroy.argtypes = [vp]
        L.wkv_reset.argtypes = [vp]
        L.wkv_set_stream.argtypes = [vp, vp]
        L.wkv_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
        L.wkv_decode_step_layers.argtypes = [vp, vp, vp, vp, vp, vp]
        L.wkv_decode_step_static.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.wkv_decode_step_host.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.wkv_decode_step_layers_host.argtypes = [vp, vp, vp, vp, vp, vp]
        L.wkv_prefill.argtypes = [vp, i32, vp, vp, vp, vp, i32, vp, vp]
        L.wkv_prefill_bulk.argtypes = [vp, i32, vp, vp, vp, vp, i32, vp, vp]
        L.wkv_prefill_bulk_layers.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp]
        L.wkv_export_state.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.wkv_export_slots.argtypes = [vp, i32, i32, i32, vp]
        L.wkv_import_state.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.wkv_status.argtypes = [vp]
        L.wkv_selftest_wait_timeout.argtypes = [vp]
        L.wkv_launch_count.restype = C.c_int64
        L.wkv_launch_count.argtypes = [vp]
        L.wkv_device_bytes.restype = C.c_int64
        L.wkv_device_bytes.argtypes = [vp]
        L.wkv_splits.restype = i32
        L.wkv_splits.argtypes = [vp]
        L.wkv_strerror.restype = C.c_char_p
        L.wkv_strerror.argtypes = [C.c_int]
        L.wkv_last_error.restype = C.c_char_p
        L.wkv_last_error.argtypes = [vp]
        _lib = L
    return _lib


class WkvError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"wkv error {code}: {text}")
        self.code = code


def _dp(t):
    """Device (or host) address of a tensor, None -> NULL."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("wkv: tensors crossing the C ABI must be contiguous")
    return C.c_void_p(t.data_ptr())


def make_config(n_layers, batch, n_q_heads, n_kv_heads, head_dim, budget, window, sink=0, dtype=WKV_BF16, scale=0.0,
                merge=1, n_splits=0, stream=None, schedule=0):
    cfg = wkv_config()
    cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_layers, batch, n_q_heads, n_kv_heads, head_dim
    cfg.budget, cfg.window, cfg.sink, cfg.dtype, cfg.scale, cfg.merge, cfg.n_splits = (budget, window, sink, dtype, scale,
                                                                                     merge, n_splits)
    cfg.stream = stream
    cfg.schedule = schedule
    return cfg


def wkv_config_error(cfg):
    msg = lib().wkv_config_error(C.byref(cfg))
    return None if msg is None else msg.decode()


class Context:
    """One wkv_ctx.  Device memory comes from torch's caching allocator through the provider callbacks."""

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, head_dim, budget, window, sink=0, dtype=WKV_BF16,
                 scale=0.0, merge=1, n_splits=0, device="cuda:0", torch_alloc=True, schedule=0):
        self.device = torch.device(device)
        self.dtype = dtype
        self.tdtype = torch.bfloat16 if dtype == WKV_BF16 else torch.float32
        self.shape = (n_layers, batch, n_q_heads, n_kv_heads, head_dim)
        self.budget = budget
        self._bufs = {}
        cfg = make_config(n_layers, batch, n_q_heads, n_kv_heads, head_dim, budget, window, sink, dtype, scale, merge,
                          n_splits, schedule=schedule)
        err = wkv_config_error(cfg)
        if err is not None:
            raise WkvError(WKV_ERR_INVALID, err)
        torch.cuda.set_device(self.device)
        cfg.stream = torch.cuda.current_stream(self.device).cuda_stream
        if torch_alloc:
            def _alloc(nbytes, _user):
                try:
                    buf = torch.empty(int(nbytes), dtype=torch.uint8, device=self.device)
                except Exception:
                    return None
                self._bufs[buf.data_ptr()] = buf
                return buf.data_ptr()

            def _release(ptr, _user):
                self._bufs.pop(ptr, None)

            self._alloc_cb, self._release_cb = ALLOC_FN(_alloc), RELEASE_FN(_release)
            cfg.alloc, cfg.release = self._alloc_cb, self._release_cb
        h = C.c_void_p()
        rc = lib().wkv_create(C.byref(cfg), C.byref(h))
        if rc != WKV_OK:
            raise WkvError(rc, lib().wkv_strerror(rc).decode())
        self._h = h

    # -- plumbing ---------------------------------------------------------------------------------
    def _check(self, rc):
        if rc != WKV_OK:
            raise WkvError(rc, (lib().wkv_last_error(self._h) or b"").decode() or lib().wkv_strerror(rc).decode())

    def close(self):
        if getattr(self, "_h", None):
            lib().wkv_destroy(self._h)
            self._h = None
            self._bufs.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, same names ----------------------------------------------------------------------
    def wkv_reset(self):
        self._check(lib().wkv_reset(self._h))

    def wkv_set_stream(self, stream):
        self._check(lib().wkv_set_stream(self._h, C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else stream)))

    def wkv_decode_step(self, layer, q, k, v, out, evicted_pos=None, probs=None):
        self._check(lib().wkv_decode_step(self._h, layer, _dp(q), _dp(k), _dp(v), _dp(out), _dp(evicted_pos), _dp(probs)))

    def wkv_decode_step_layers(self, q, k, v, out, evicted_pos=None):
        self._check(lib().wkv_decode_step_layers(self._h, _dp(q), _dp(k), _dp(v), _dp(out), _dp(evicted_pos)))

    def wkv_decode_step_static(self, layer, q, k, v, out, evicted_pos=None):
        """wkv_decode_step with its scratch in the library's built-in device array: for callers that may not
        allocate device memory.  Raises WkvError(WKV_ERR_INVALID) when the shape needs more than the array holds."""
        self._check(lib().wkv_decode_step_static(self._h, layer, _dp(q), _dp(k), _dp(v), _dp(out), _dp(evicted_pos)))

    def wkv_decode_step_host(self, layer, q, k, v, out, evicted_pos=None):
        self._check(lib().wkv_decode_step_host(self._h, layer, _dp(q), _dp(k), _dp(v), _dp(out), _dp(evicted_pos)))

    def wkv_decode_step_layers_host(self, q, k, v, out, evicted_pos=None):
        self._check(lib().wkv_decode_step_layers_host(self._h, _dp(q), _dp(k), _dp(v), _dp(out), _dp(evicted_pos)))

    def wkv_prefill(self, layer, Q, K, V, seq_lens=None, out=None, evicted_pos=None):
        T_max = Q.shape[1]
        self._check(lib().wkv_prefill(self._h, layer, _dp(Q), _dp(K), _dp(V), _dp(seq_lens), T_max, _dp(out),
                                      _dp(evicted_pos)))

    def wkv_prefill_bulk(self, layer, Q, K, V, seq_lens=None, out=None, evicted_pos=None):
        T_max = Q.shape[1]
        self._check(lib().wkv_prefill_bulk(self._h, layer, _dp(Q), _dp(K), _dp(V), _dp(seq_lens), T_max, _dp(out),
                                           _dp(evicted_pos)))

    def wkv_prefill_bulk_layers(self, Q, K, V, seq_lens=None, out=None, evicted_pos=None):
        T_max = Q.shape[2]
        self._check(lib().wkv_prefill_bulk_layers(self._h, _dp(Q), _dp(K), _dp(V), _dp(seq_lens), T_max, _dp(out),
                                                  _dp(evicted_pos)))

    def wkv_export_state(self, layer, b, kv_head):
        """Position-ordered host copy of one lane: dict(len, tokens, pos, a, K, V)."""
        d = self.shape[4]
        n, tok = C.c_int32(), C.c_int32()
        pos = torch.empty(self.budget, dtype=torch.int32)
        a = torch.empty(self.budget, dtype=torch.float32)
        K = torch.empty(self.budget, d, dtype=self.tdtype)
        V = torch.empty(self.budget, d, dtype=self.tdtype)
        self._check(lib().wkv_export_state(self._h, layer, b, kv_head, C.byref(n), C.byref(tok), _dp(pos), _dp(a), _dp(K),
                                           _dp(V)))
        L = n.value
        return {"len": L, "tokens": tok.value, "pos": pos[:L], "a": a[:L], "K": K[:L], "V": V[:L]}

    def wkv_export_slots(self, layer, b, kv_head):
        sp = torch.empty(self.budget + 1, dtype=torch.int32)
        self._check(lib().wkv_export_slots(self._h, layer, b, kv_head, _dp(sp)))
        return sp

    def wkv_import_state(self, layer, b, kv_head, tokens, pos, a, K, V):
        pos = pos.to(torch.int32).contiguous().cpu()
        a = a.to(torch.float32).contiguous().cpu()
        K = K.to(self.tdtype).contiguous().cpu()
        V = V.to(self.tdtype).contiguous().cpu()
        self._check(lib().wkv_import_state(self._h, layer, b, kv_head, int(pos.numel()), int(tokens), _dp(pos), _dp(a),
                                           _dp(K), _dp(V)))

    def wkv_status(self):
        return lib().wkv_status(self._h)

    def wkv_selftest_wait_timeout(self):
        self._check(lib().wkv_selftest_wait_timeout(self._h))

    def wkv_launch_count(self):
        return int(lib().wkv_launch_count(self._h))

    def wkv_device_bytes(self):
        return int(lib().wkv_device_bytes(self._h))

    def wkv_splits(self):
        return int(lib().wkv_splits(self._h))
