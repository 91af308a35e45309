"""ctypes binding of the CPU oracle (`hivis_oracle.cpp`).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA product path never does.  The oracle is built twice from
the same source: `real = double` (default for parity) and `real = float` (the
plain fp32 program that is timed as the CPU baseline).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hivis_oracle.cpp")
_LIBS: Dict[str, C.CDLL] = {}

_WNAMES = ("embed", "lm_head", "fc", "norm1", "wq", "wk", "wv", "bq", "bk", "bv", "wo", "norm2",
           "w_gate", "w_up", "w_down")


class _Dims(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("d", "hq", "hkv", "dh", "ffn", "vocab")] + \
               [("eps", C.c_double), ("rope_base", C.c_double)]


class _Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WNAMES]


class _Taps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("u", "q", "k", "v", "attn", "y", "act", "g")]


def lib_path(real: str) -> str:
    return os.path.join(_HERE, f"libhvo_{real}.so")


def build(force: bool = False) -> None:
    """Compile the oracle for both arithmetic types (g++, OpenMP)."""
    for real, ctype in (("f64", "double"), ("f32", "float")):
        out = lib_path(real)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        cmd = ["g++", "-O3", "-mavx2", "-mfma", "-fopenmp", "-std=c++17", "-shared", "-fPIC",
               f"-DHVO_REAL={ctype}", _SRC, "-o", out]
        subprocess.run(cmd, check=True)


def _lib(real: str) -> C.CDLL:
    if real not in _LIBS:
        build()
        lib = C.CDLL(lib_path(real))
        lib.hvo_real_bytes.restype = C.c_int
        lib.hvo_num_threads.restype = C.c_int
        lib.hvo_argmax.restype = C.c_int
        lib.hvo_argmax_f32.restype = C.c_int
        assert lib.hvo_real_bytes() == (8 if real == "f64" else 4)
        _LIBS[real] = lib
    return _LIBS[real]


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


class Oracle:
    """The drafter, on the CPU.  `dims` is any object with d, n_q_heads, n_kv_heads, head_dim,
    ffn, vocab, rms_eps, rope_base; `weights` maps names to fp32 arrays ([out, in])."""

    def __init__(self, dims, weights: Dict[str, np.ndarray], real: str = "f64"):
        self.real = real
        self.rt = np.float64 if real == "f64" else np.float32
        self.lib = _lib(real)
        self.dims = dims
        self.D = _Dims(dims.d, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.ffn,
                       dims.vocab, float(dims.rms_eps), float(dims.rope_base))
        self._keep = {k: _f32(v) for k, v in weights.items() if v is not None}
        self.W = _Weights(*[_p(self._keep.get(n)) for n in _WNAMES])
        self.kvw = dims.n_kv_heads * dims.head_dim
        self.qw = dims.n_q_heads * dims.head_dim

    # ---- helpers
    def _r(self, a) -> np.ndarray:
        return np.ascontiguousarray(a, dtype=self.rt)

    def num_threads(self) -> int:
        return int(self.lib.hvo_num_threads())

    # ---- primitives (one call each into the C oracle)
    def fuse(self, f, tok: int, rho=None) -> np.ndarray:
        f = self._r(f)
        rho = None if rho is None else self._r(rho)
        u = np.empty(self.dims.d, self.rt)
        self.lib.hvo_fuse(C.byref(self.D), C.byref(self.W), _p(f), int(tok), _p(rho), _p(u))
        return u

    def fold_residuals(self, r, w=None) -> np.ndarray:
        r = _f32(r)
        R, d = r.shape
        w = None if w is None else _f32(w)
        rho = np.empty((R, d), self.rt)
        self.lib.hvo_fold_residuals(d, R, _p(r), _p(w), _p(rho))
        return rho

    def rmsnorm(self, x, gamma, eps: float) -> np.ndarray:
        x, gamma = self._r(x), _f32(gamma)
        out = np.empty_like(x)
        self.lib.hvo_rmsnorm(x.size, _p(x), _p(gamma), C.c_double(eps), _p(out))
        return out

    def rope(self, x, n_heads: int, dh: int, base: float, pos: int) -> np.ndarray:
        x = self._r(x).copy()
        self.lib.hvo_rope(n_heads, dh, C.c_double(base), int(pos), _p(x))
        return x

    def qkv(self, a):
        a = self._r(a)
        q, k, v = np.empty(self.qw, self.rt), np.empty(self.kvw, self.rt), np.empty(self.kvw, self.rt)
        self.lib.hvo_qkv(C.byref(self.D), C.byref(self.W), _p(a), _p(q), _p(k), _p(v))
        return q, k, v

    def attend(self, q, Kc, Vc, length: int) -> np.ndarray:
        q, Kc, Vc = self._r(q), self._r(Kc), self._r(Vc)
        out = np.empty(self.qw, self.rt)
        self.lib.hvo_attend(C.byref(self.D), _p(q), _p(Kc), _p(Vc), int(length), _p(out))
        return out

    def mlp(self, y):
        y = self._r(y)
        act, g = np.empty(self.dims.ffn, self.rt), np.empty(self.dims.d, self.rt)
        self.lib.hvo_mlp(C.byref(self.D), C.byref(self.W), _p(y), _p(act), _p(g))
        return g, act

    def argmax(self, x):
        x = self._r(x)
        gap = np.zeros(1, self.rt)
        i = self.lib.hvo_argmax(x.size, _p(x), _p(gap))
        return int(i), float(gap[0])

    # ---- the path
    def new_cache(self, max_len: int):
        return np.zeros((max_len, self.kvw), self.rt), np.zeros((max_len, self.kvw), self.rt)

    def position(self, f, tok, rho, pos, Kc, Vc, taps: bool = False):
        f, rho = self._r(f), self._r(rho)
        g = np.empty(self.dims.d, self.rt)
        tp, store = None, None
        if taps:
            store = {"u": np.empty(self.dims.d, self.rt), "q": np.empty(self.qw, self.rt),
                     "k": np.empty(self.kvw, self.rt), "v": np.empty(self.kvw, self.rt),
                     "attn": np.empty(self.qw, self.rt), "y": np.empty(self.dims.d, self.rt),
                     "act": np.empty(self.dims.ffn, self.rt), "g": np.empty(self.dims.d, self.rt)}
            tp = C.byref(_Taps(*[_p(store[n]) for n in ("u", "q", "k", "v", "attn", "y", "act", "g")]))
        self.lib.hvo_position(C.byref(self.D), C.byref(self.W), _p(f), int(tok), _p(rho), int(pos),
                              _p(Kc), _p(Vc), _p(g), tp)
        return (g, store) if taps else g

    def prefill(self, ids, hidden, rho0, Kc, Vc, start_pos: int = 0) -> None:
        """K/V of pairs 0..T-2 into rows start_pos.. ; pair T-1 stays pending for the draft."""
        ids, hidden, rho0 = _i32(ids), _f32(hidden), self._r(rho0)
        self.lib.hvo_prefill(C.byref(self.D), C.byref(self.W), int(ids.size), _p(ids), _p(hidden),
                             _p(rho0), int(start_pos), _p(Kc), _p(Vc))

    def draft(self, n_cached: int, pend_id: int, pend_hidden, k: int, rho, Kc, Vc,
              forced_ids=None, want_logits: bool = True):
        pend_hidden, rho = _f32(pend_hidden), self._r(rho)
        forced = None if forced_ids is None else _i32(forced_ids)
        ids = np.empty(k, np.int32)
        logits = np.empty((k, self.dims.vocab), self.rt) if want_logits else None
        gaps = np.empty(k, self.rt)
        g = np.empty((k, self.dims.d), self.rt)
        self.lib.hvo_draft(C.byref(self.D), C.byref(self.W), int(n_cached), int(pend_id),
                           _p(pend_hidden), int(k), _p(rho), int(rho.shape[0]), _p(Kc), _p(Vc),
                           _p(forced), _p(ids), _p(logits), _p(gaps), _p(g))
        return {"ids": ids, "logits": logits, "gaps": gaps, "g": g}

    def draft_bruteforce(self, ids, hidden, k: int, rho, forced_ids=None):
        ids, hidden, rho = _i32(ids), _f32(hidden), self._r(rho)
        forced = None if forced_ids is None else _i32(forced_ids)
        out_ids = np.empty(k, np.int32)
        logits = np.empty((k, self.dims.vocab), self.rt)
        g = np.empty((k, self.dims.d), self.rt)
        self.lib.hvo_draft_bruteforce(C.byref(self.D), C.byref(self.W), int(ids.size), _p(ids),
                                      _p(hidden), int(k), _p(rho), int(rho.shape[0]), _p(forced),
                                      _p(out_ids), _p(logits), _p(g))
        return {"ids": out_ids, "logits": logits, "g": g}

    def verify(self, draft_ids, logits, base_len: int):
        """draft_ids [k], logits [(k+1), V] fp32; base_len = true-feature pairs in the sequence."""
        draft_ids, logits = _i32(draft_ids), _f32(logits)
        k = draft_ids.size
        n, nxt, kv = C.c_int(), C.c_int(), C.c_int()
        self.lib.hvo_verify(k, logits.shape[-1], _p(draft_ids), _p(logits), int(base_len),
                            C.byref(n), C.byref(nxt), C.byref(kv))
        return n.value, nxt.value, kv.value

    # ---- whole-workload convenience: run prefill + draft for every sequence of a packed batch
    def run_batch(self, ids, hidden, cu_seqlens, k: int, resid, resid_proj=None, forced_ids=None,
                  want_logits: bool = True):
        rho = self.fold_residuals(resid, resid_proj)
        B = len(cu_seqlens) - 1
        outs = []
        for b in range(B):
            lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
            T = hi - lo
            Kc, Vc = self.new_cache(T + k)
            self.prefill(ids[lo:hi], hidden[lo:hi], rho[0], Kc, Vc)
            o = self.draft(T - 1, int(ids[hi - 1]), hidden[hi - 1], k, rho, Kc, Vc,
                           None if forced_ids is None else forced_ids[b], want_logits)
            o["K"], o["V"], o["T"] = Kc, Vc, T
            outs.append(o)
        return outs
