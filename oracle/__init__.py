"""ctypes front end of the WeightedKV CPU oracle (``wkv_oracle.cpp``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU-baseline leg load this
package; the CUDA library never does, and nothing here touches the CUDA library.

``build()`` compiles the C++ source next to this file with g++ (no CUDA, no intrinsics) and
``Oracle`` wraps one ``wkvo`` handle: ``step`` consumes one token for every lane, exactly one loop
iteration of the paper's Algorithm 1 per lane.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wkv_oracle.cpp")
_LIB = os.path.join(_HERE, "libwkv_oracle.so")

F32, BF16 = 0, 1
MODE_DOUBLE, MODE_PINNED = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-o", _LIB + ".tmp", _SRC]
    subprocess.run(cmd, check=True)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_lanes", "group", "head_dim", "budget", "window", "sink", "dtype", "mode",
                                         "merge", "track")] + [("scale", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.wkvo_create.restype = C.c_void_p
        L.wkvo_create.argtypes = [C.POINTER(_Config)]
        L.wkvo_destroy.argtypes = [C.c_void_p]
        L.wkvo_step.argtypes = [C.c_void_p] + [C.c_void_p] * 7
        L.wkvo_len.restype = C.c_int32
        L.wkvo_len.argtypes = [C.c_void_p, C.c_int32]
        L.wkvo_tokens.restype = C.c_int64
        L.wkvo_tokens.argtypes = [C.c_void_p, C.c_int32]
        L.wkvo_dropped_score.restype = C.c_double
        L.wkvo_dropped_score.argtypes = [C.c_void_p, C.c_int32]
        L.wkvo_last_step.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 4
        L.wkvo_impose_pick.argtypes = [C.c_void_p, C.c_void_p]
        L.wkvo_last_pick.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 4
        L.wkvo_export.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 7
        L.wkvo_import.restype = C.c_int32
        L.wkvo_import.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int64] + [C.c_void_p] * 4
        L.wkvo_pinned_exp.restype = C.c_float
        L.wkvo_pinned_exp.argtypes = [C.c_float]
        L.wkvo_pinned_dot.restype = C.c_float
        L.wkvo_pinned_dot.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_float]
        L.wkvo_pinned_softmax.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.wkvo_round_bf16.restype = C.c_float
        L.wkvo_round_bf16.argtypes = [C.c_float]
        L.wkvo_round_bf16_from_double.restype = C.c_float
        L.wkvo_round_bf16_from_double.argtypes = [C.c_double]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Oracle:
    """One oracle instance: ``n_lanes`` independent (layer, batch, kv-head) lanes of Algorithm 1."""

    def __init__(self, n_lanes, head_dim, budget, window=1, sink=0, group=1, dtype=F32, mode=MODE_DOUBLE, merge=1,
                 track=False, scale=0.0):
        self.n_lanes, self.d, self.m, self.G = n_lanes, head_dim, budget, group
        self.window, self.sink, self.dtype, self.mode = window, sink, dtype, mode
        cfg = _Config(n_lanes, group, head_dim, budget, window, sink, dtype, mode, merge, int(track), float(scale))
        self._h = lib().wkvo_create(C.byref(cfg))
        if not self._h:
            raise ValueError("invalid oracle configuration")

    def close(self):
        if self._h:
            lib().wkvo_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, q, k, v, active=None, want_out=True, want_probs=False):
        """q [n_lanes, G, d]; k, v [n_lanes, d] (any float array of T values).

        Returns (out [n_lanes, G, d] fp64 or None, evicted [n_lanes] int32, probs or None)."""
        q = np.ascontiguousarray(q, dtype=np.float32).reshape(self.n_lanes, self.G, self.d)
        k = np.ascontiguousarray(k, dtype=np.float32).reshape(self.n_lanes, self.d)
        v = np.ascontiguousarray(v, dtype=np.float32).reshape(self.n_lanes, self.d)
        act = None if active is None else np.ascontiguousarray(active, dtype=np.uint8)
        out = np.empty((self.n_lanes, self.G, self.d), dtype=np.float64) if want_out else None
        ev = np.empty(self.n_lanes, dtype=np.int32)
        pr = np.zeros((self.n_lanes, self.G, self.m + 1), dtype=np.float64) if want_probs else None
        lib().wkvo_step(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(act), _ptr(out), _ptr(ev), _ptr(pr))
        return out, ev, pr

    def length(self, lane=0):
        return int(lib().wkvo_len(self._h, lane))

    def tokens(self, lane=0):
        return int(lib().wkvo_tokens(self._h, lane))

    def dropped_score(self, lane=0):
        return float(lib().wkvo_dropped_score(self._h, lane))

    def last_step(self, lane=0):
        """(removed list index or -1, w_j, w_r, sum of the probabilities folded into a)."""
        idx = C.c_int32()
        wj, wr, ps = C.c_double(), C.c_double(), C.c_double()
        lib().wkvo_last_step(self._h, lane, C.byref(idx), C.byref(wj), C.byref(wr), C.byref(ps))
        return idx.value, wj.value, wr.value, ps.value

    def impose_pick(self, pos):
        """Every lane with pos[lane] >= 0 removes the entry at that original position on its next compressing step
        instead of its own argmin (one shot; used to keep two arithmetic modes on one trajectory across a near-tie)."""
        pos = np.ascontiguousarray(pos, np.int32).reshape(self.n_lanes)
        lib().wkvo_impose_pick(self._h, _ptr(pos))

    def last_pick(self, lane=0):
        """(position the lane's own argmin chose, its average score, the average score of the entry actually removed,
        1 if an imposed position was outside the evictable range) for the lane's last compressing step."""
        own = C.c_int32()
        bad = C.c_int32()
        oa, ta = C.c_double(), C.c_double()
        lib().wkvo_last_pick(self._h, lane, C.byref(own), C.byref(oa), C.byref(ta), C.byref(bad))
        return own.value, oa.value, ta.value, bad.value

    def import_state(self, lane, tokens, pos, a, K, V):
        """Replace one lane by a position-ordered state (pos int32 strictly increasing and < tokens; K, V as stored)."""
        pos = np.ascontiguousarray(pos, np.int32)
        a = np.ascontiguousarray(a, np.float64)
        K = np.ascontiguousarray(K, np.float32)
        V = np.ascontiguousarray(V, np.float32)
        rc = lib().wkvo_import(self._h, lane, len(pos), int(tokens), _ptr(pos), _ptr(a), _ptr(K), _ptr(V))
        if rc != 0:
            raise ValueError("wkvo_import rejected the state")

    def export(self, lane=0, coeff=False):
        """Position-ordered state of one lane as a dict of numpy arrays."""
        L, T = self.length(lane), self.tokens(lane)
        pos = np.empty(L, np.int32)
        n = np.empty(L, np.int64)
        a = np.empty(L, np.float64)
        K = np.empty((L, self.d), np.float32)
        V = np.empty((L, self.d), np.float32)
        cnt = np.empty(L, np.int32)
        Cm = np.zeros((L, T), np.float64) if coeff else None
        lib().wkvo_export(self._h, lane, _ptr(pos), _ptr(n), _ptr(a), _ptr(K), _ptr(V), _ptr(cnt), _ptr(Cm))
        return {"pos": pos, "n": n, "a": a, "K": K, "V": V, "cnt": cnt, "coeff": Cm}


def pinned_exp(x):
    return float(lib().wkvo_pinned_exp(C.c_float(float(x))))


def pinned_dot(q, k, scale32):
    q = np.ascontiguousarray(q, np.float32)
    k = np.ascontiguousarray(k, np.float32)
    return float(lib().wkvo_pinned_dot(_ptr(q), _ptr(k), q.size, C.c_float(float(scale32))))


def pinned_softmax(s):
    s = np.ascontiguousarray(s, np.float32)
    p = np.empty_like(s)
    lib().wkvo_pinned_softmax(_ptr(s), s.size, _ptr(p))
    return p


def round_bf16(x):
    return float(lib().wkvo_round_bf16(C.c_float(float(x))))


def round_bf16_from_double(x):
    return float(lib().wkvo_round_bf16_from_double(C.c_double(float(x))))
