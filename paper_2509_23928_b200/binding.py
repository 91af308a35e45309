"""ctypes binding of include/hivis.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhivis.so")

HIVIS_F32, HIVIS_BF16 = 0, 1
HIVIS_MAX_BATCH, HIVIS_MAX_K = 64, 16
TAPS = {"u": 0, "attn": 1, "y": 2, "act": 3, "g": 4, "q": 5}
ERRORS = {0: "OK", -1: "ARG", -2: "SHAPE", -3: "DTYPE", -4: "STATE", -5: "CAPACITY", -6: "CUDA",
          -7: "TIMEOUT", -8: "NOMEM"}

EXPORTS = ("hivis_init", "hivis_destroy", "hivis_prefill", "hivis_draft", "hivis_verify", "hivis_reset",
           "hivis_get_kv_len", "hivis_set_kv_len", "hivis_read_kv", "hivis_debug_tap", "hivis_step_bytes",
           "hivis_launch_count", "hivis_last_error", "hivis_profile_begin", "hivis_profile_end", "hivis_set_option",
           "hivis_status", "hivis_verify_noalloc", "hivis_read_phase_times", "hivis_draft_tree", "hivis_verify_tree", "hivis_verify_sampled", "hivis_draft_sampled",
           "hivis_set_kv_len_batch")
HIVIS_OPT_CHAIN_KERNEL = 0
HIVIS_OPT_TC_KERNEL = 1
HIVIS_OPT_WAIT_LIMIT_US = 2
HIVIS_OPT_DEBUG_MISS_BARRIER = 3
HIVIS_OPT_PHASE_TIMES = 4
HIVIS_OPT_L2_KEEP = 5
HIVIS_OPT_TC_PREFILL = 6
HIVIS_PHASE_EVENTS = 24
PROFILE_CLASSES = ("fuse_fc", "qkv", "attention", "o_proj", "gate_up", "down", "lm_head_argmax", "setup_finish",
                   "draft_chain")


class HivisError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"HIVIS_ERR_{ERRORS.get(code, code)} ({code}): {msg}")
        self.code = code


class hivis_config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("dtype", C.c_int), ("d", C.c_int), ("n_q_heads", C.c_int),
                ("n_kv_heads", C.c_int), ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int),
                ("rms_eps", C.c_float), ("rope_base", C.c_float), ("max_batch", C.c_int),
                ("max_len", C.c_int), ("max_k", C.c_int)]


_WNAMES = ("embed", "lm_head", "fc", "norm1", "wq", "wk", "wv", "bq", "bk", "bv", "wo", "norm2", "w_gate",
           "w_up", "w_down", "resid_proj")


class hivis_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WNAMES]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        from . import build as _b          # nvcc is part of the toolchain image; build in-tree once
        _b.build()
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing and could not be built: the CUDA library is required")
    L = C.CDLL(LIB_PATH)
    vp, ip, i32 = C.c_void_p, C.POINTER(C.c_int), C.c_int
    L.hivis_init.argtypes = [C.POINTER(vp), C.POINTER(hivis_config), C.POINTER(hivis_weights), vp]
    L.hivis_destroy.argtypes = [vp]
    L.hivis_prefill.argtypes = [vp, i32, ip, vp, vp, ip, ip, vp, vp]
    L.hivis_draft.argtypes = [vp, i32, ip, i32, vp, i32, vp, vp, vp, vp]
    L.hivis_verify.argtypes = [vp, i32, ip, i32, vp, vp, i32, vp, vp, vp, vp]
    L.hivis_reset.argtypes = [vp, i32, vp]
    L.hivis_get_kv_len.argtypes = [vp, i32, ip, ip, vp]
    L.hivis_set_kv_len.argtypes = [vp, i32, i32, i32, vp]
    L.hivis_set_kv_len_batch.argtypes = [vp, i32, ip, ip, i32, vp]
    L.hivis_read_kv.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    L.hivis_debug_tap.argtypes = [vp, i32, vp, vp]
    L.hivis_step_bytes.argtypes = [vp, i32, ip]
    L.hivis_step_bytes.restype = C.c_int64
    L.hivis_launch_count.argtypes = [vp]
    L.hivis_launch_count.restype = C.c_int64
    L.hivis_set_option.argtypes = [vp, i32, i32]
    L.hivis_status.argtypes = [vp, vp]
    L.hivis_profile_begin.argtypes = [vp]
    L.hivis_profile_end.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
    L.hivis_verify_noalloc.argtypes = [i32, i32, i32, vp, vp, i32, vp, vp, vp, vp, vp]
    L.hivis_verify_sampled.argtypes = [vp, i32, ip, i32, vp, vp, vp, i32, C.c_float, vp, vp, vp, vp, vp, vp]
    L.hivis_draft_sampled.argtypes = [vp, i32, ip, i32, vp, i32, C.c_float, vp, vp, vp, vp]
    L.hivis_draft_tree.argtypes = [vp, i32, i32, i32, i32, vp, i32, vp, vp, vp, vp, vp]
    L.hivis_verify_tree.argtypes = [vp, i32, vp, i32, vp, vp, vp, vp, vp]
    L.hivis_read_phase_times.argtypes = [vp, vp, C.c_longlong, ip, ip, vp]
    L.hivis_last_error.argtypes = [vp]
    L.hivis_last_error.restype = C.c_char_p
    for n in EXPORTS:
        getattr(L, n)
    return L


lib = _load()


def _ints(seq: Optional[Sequence[int]]):
    if seq is None:
        return None
    seq = [int(x) for x in seq]
    return (C.c_int * len(seq))(*seq)


def _ptr(t) -> Optional[int]:
    """Device address of a torch tensor (None stays None); plain ints pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def hivis_last_error(ctx=None) -> str:
    return (lib.hivis_last_error(ctx) or b"").decode()


def _check(rc: int, ctx=None):
    if rc != 0:
        raise HivisError(rc, hivis_last_error(ctx))


# ------------------------------------------------------------------ functions named as in hivis.h
def hivis_init(cfg: hivis_config, weights: hivis_weights, stream=None) -> int:
    out = C.c_void_p()
    _check(lib.hivis_init(C.byref(out), C.byref(cfg), C.byref(weights), _stream(stream)))
    return out.value


def hivis_destroy(ctx) -> None:
    _check(lib.hivis_destroy(ctx))


def hivis_prefill(ctx, B, seq_slots, ids, hidden, cu_seqlens, start_pos=None, resid0=None, stream=None):
    _check(lib.hivis_prefill(ctx, int(B), _ints(seq_slots), _ptr(ids), _ptr(hidden), _ints(cu_seqlens),
                             _ints(start_pos), _ptr(resid0), _stream(stream)), ctx)


def hivis_draft(ctx, B, seq_slots, k, resid, n_resid, out_ids, forced_ids=None, out_logits=None, stream=None):
    _check(lib.hivis_draft(ctx, int(B), _ints(seq_slots), int(k), _ptr(resid), int(n_resid), _ptr(out_ids),
                           _ptr(forced_ids), _ptr(out_logits), _stream(stream)), ctx)


def hivis_draft_sampled(ctx, B, seq_slots, k, resid, n_resid, temperature, uniforms, out_ids, out_logits=None, stream=None):
    _check(lib.hivis_draft_sampled(ctx, int(B), _ints(seq_slots), int(k), _ptr(resid), int(n_resid), float(temperature),
                                   _ptr(uniforms), _ptr(out_ids), _ptr(out_logits), _stream(stream)), ctx)


def hivis_verify(ctx, B, seq_slots, k, draft_ids, target_logits, logits_dtype, out_accept, out_next,
                 out_kv_len=None, stream=None):
    _check(lib.hivis_verify(ctx, int(B), _ints(seq_slots), int(k), _ptr(draft_ids), _ptr(target_logits),
                            int(logits_dtype), _ptr(out_accept), _ptr(out_next), _ptr(out_kv_len),
                            _stream(stream)), ctx)


def hivis_verify_sampled(ctx, B, seq_slots, k, draft_ids, draft_logits, target_logits, logits_dtype, temperature, u_accept,
                         u_sample, out_accept, out_next, out_kv_len=None, stream=None):
    _check(lib.hivis_verify_sampled(ctx, int(B), _ints(seq_slots), int(k), _ptr(draft_ids), _ptr(draft_logits),
                                    _ptr(target_logits), int(logits_dtype), float(temperature), _ptr(u_accept), _ptr(u_sample),
                                    _ptr(out_accept), _ptr(out_next), _ptr(out_kv_len), _stream(stream)), ctx)


def hivis_draft_tree(ctx, slot, topk, depth, keep, resid, n_resid, out_tokens, out_parents, out_scores, out_count,
                     stream=None):
    _check(lib.hivis_draft_tree(ctx, int(slot), int(topk), int(depth), int(keep), _ptr(resid), int(n_resid),
                                _ptr(out_tokens), _ptr(out_parents), _ptr(out_scores), _ptr(out_count), _stream(stream)), ctx)


def hivis_verify_tree(ctx, slot, target_logits, logits_dtype, out_accept, out_path, out_next, out_kv_len=None, stream=None):
    _check(lib.hivis_verify_tree(ctx, int(slot), _ptr(target_logits), int(logits_dtype), _ptr(out_accept), _ptr(out_path),
                                 _ptr(out_next), _ptr(out_kv_len), _stream(stream)), ctx)


def hivis_verify_noalloc(B, k, vocab, draft_ids, target_logits, logits_dtype, rows_before, out_accept,
                         out_next, out_kv_len=None, stream=None):
    """Context-free greedy verification for callers that must not allocate device memory: the
    argmax keys sit in a fixed array inside the library (at most 64 sequences, k <= 16)."""
    _check(lib.hivis_verify_noalloc(int(B), int(k), int(vocab), _ptr(draft_ids), _ptr(target_logits),
                                    int(logits_dtype), _ptr(rows_before), _ptr(out_accept), _ptr(out_next),
                                    _ptr(out_kv_len), _stream(stream)))


def hivis_reset(ctx, slot, stream=None):
    _check(lib.hivis_reset(ctx, int(slot), _stream(stream)), ctx)


def hivis_get_kv_len(ctx, slot, stream=None):
    n, p = C.c_int(), C.c_int()
    _check(lib.hivis_get_kv_len(ctx, int(slot), C.byref(n), C.byref(p), _stream(stream)), ctx)
    return n.value, bool(p.value)


def hivis_set_kv_len(ctx, slot, n_rows, restore_pending=False, stream=None):
    _check(lib.hivis_set_kv_len(ctx, int(slot), int(n_rows), int(bool(restore_pending)), _stream(stream)), ctx)


def hivis_set_kv_len_batch(ctx, B, seq_slots, n_rows, restore_pending=False, stream=None):
    _check(lib.hivis_set_kv_len_batch(ctx, int(B), _ints(seq_slots), _ints(n_rows), 1 if restore_pending else 0,
                                      _stream(stream)), ctx)


def hivis_read_kv(ctx, slot, row0, n, out_k, out_v, stream=None):
    _check(lib.hivis_read_kv(ctx, int(slot), int(row0), int(n), _ptr(out_k), _ptr(out_v), _stream(stream)), ctx)


def hivis_debug_tap(ctx, which, out, stream=None):
    _check(lib.hivis_debug_tap(ctx, int(which), _ptr(out), _stream(stream)), ctx)


def hivis_step_bytes(ctx, kv_rows: Sequence[int]) -> int:
    return int(lib.hivis_step_bytes(ctx, len(kv_rows), _ints(kv_rows)))


def hivis_set_option(ctx, option: int, value: int) -> None:
    _check(lib.hivis_set_option(ctx, int(option), int(value)), ctx)


def hivis_status(ctx, stream=None) -> None:
    """Synchronise and raise HivisError(TIMEOUT) if a kernel gave up on a bounded wait."""
    _check(lib.hivis_status(ctx, _stream(stream)), ctx)


def hivis_profile_begin(ctx) -> None:
    _check(lib.hivis_profile_begin(ctx), ctx)


def hivis_profile_end(ctx):
    """-> {class name: (device ms, launches)} accumulated since hivis_profile_begin."""
    ms = (C.c_float * len(PROFILE_CLASSES))()
    n = (C.c_int64 * len(PROFILE_CLASSES))()
    _check(lib.hivis_profile_end(ctx, ms, n), ctx)
    return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(PROFILE_CLASSES)}


def hivis_read_phase_times(ctx, stream=None):
    """-> uint64 array [k, HIVIS_PHASE_EVENTS, grid] of the last recorded tensor-core chain launch (ns; 0 = no event)."""
    import numpy as np
    k, g = C.c_int(), C.c_int()
    rc = lib.hivis_read_phase_times(ctx, None, 0, C.byref(k), C.byref(g), _stream(stream))
    if rc != -5:
        _check(rc, ctx)
    out = np.zeros((k.value, HIVIS_PHASE_EVENTS, g.value), dtype=np.uint64)
    _check(lib.hivis_read_phase_times(ctx, out.ctypes.data_as(C.c_void_p), out.size, C.byref(k), C.byref(g),
                                      _stream(stream)), ctx)
    return out


def hivis_launch_count(ctx) -> int:
    return int(lib.hivis_launch_count(ctx))


# ------------------------------------------------------------------ convenience wrapper (torch tensors)
class Drafter:
    """Owns one hivis context.  `weights`: name -> CUDA tensor in the context dtype, [out, in]."""

    def __init__(self, dims, weights: Dict[str, "object"], max_batch: int, max_len: int, max_k: int = 8,
                 stream=None):
        import torch
        self.torch = torch
        self.dims = dims
        self.dtype = HIVIS_BF16 if dims.dtype == "bf16" else HIVIS_F32
        self.tdtype = torch.bfloat16 if self.dtype == HIVIS_BF16 else torch.float32
        cfg = hivis_config(C.sizeof(hivis_config), self.dtype, dims.d, dims.n_q_heads, dims.n_kv_heads,
                           dims.head_dim, dims.ffn, dims.vocab, float(dims.rms_eps), float(dims.rope_base),
                           int(max_batch), int(max_len), int(max_k))
        w = hivis_weights(*[_ptr(weights.get(n)) for n in _WNAMES])
        self.ctx = hivis_init(cfg, w, stream)
        torch.cuda.current_stream().synchronize()      # the caller may now drop its weight tensors
        self.max_batch, self.max_len, self.max_k = max_batch, max_len, max_k
        self.dev = torch.device("cuda", torch.cuda.current_device())

    def close(self):
        if getattr(self, "ctx", None):
            hivis_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, ids, hidden, cu_seqlens, slots=None, start_pos=None, resid0=None):
        B = len(cu_seqlens) - 1
        hivis_prefill(self.ctx, B, slots, ids, hidden, cu_seqlens, start_pos, resid0)

    def draft(self, B, k, resid=None, slots=None, forced_ids=None, want_logits=False, out_ids=None):
        t = self.torch
        if out_ids is None:
            out_ids = t.empty((B, k), dtype=t.int32, device=self.dev)
        logits = t.empty((B, k, self.dims.vocab), dtype=t.float32, device=self.dev) if want_logits else None
        n_resid = 0 if resid is None else int(resid.shape[0])
        hivis_draft(self.ctx, B, slots, k, resid, n_resid, out_ids, forced_ids, logits)
        return (out_ids, logits) if want_logits else out_ids

    def draft_sampled(self, B, k, temperature, uniforms, resid=None, slots=None, want_logits=True):
        """Chained drafting with every token drawn from softmax(logits / temperature); uniforms fp32 [B, k, vocab]."""
        t = self.torch
        out_ids = t.empty((B, k), dtype=t.int32, device=self.dev)
        logits = t.empty((B, k, self.dims.vocab), dtype=t.float32, device=self.dev) if want_logits else None
        hivis_draft_sampled(self.ctx, B, slots, k, resid, 0 if resid is None else int(resid.shape[0]), temperature, uniforms,
                            out_ids, logits)
        return (out_ids, logits) if want_logits else out_ids

    def verify(self, draft_ids, target_logits, slots=None):
        t = self.torch
        B, k = draft_ids.shape
        ldt = HIVIS_BF16 if target_logits.dtype == t.bfloat16 else HIVIS_F32
        acc = t.empty(B, dtype=t.int32, device=self.dev)
        nxt = t.empty(B, dtype=t.int32, device=self.dev)
        kv = t.empty(B, dtype=t.int32, device=self.dev)
        hivis_verify(self.ctx, B, slots, k, draft_ids, target_logits, ldt, acc, nxt, kv)
        return acc, nxt, kv

    def verify_sampled(self, draft_ids, draft_logits, target_logits, temperature, u_accept, u_sample, slots=None):
        t = self.torch
        B, k = draft_ids.shape
        ldt = HIVIS_BF16 if target_logits.dtype == t.bfloat16 else HIVIS_F32
        acc = t.empty((B + 3) // 4 * 4, dtype=t.int32, device=self.dev)
        nxt = t.empty_like(acc)
        kv = t.empty_like(acc)
        hivis_verify_sampled(self.ctx, B, slots, k, draft_ids, draft_logits, target_logits, ldt, temperature, u_accept,
                             u_sample, acc, nxt, kv)
        return acc[:B], nxt[:B], kv[:B]

    def draft_tree(self, slot, topk, depth, keep, resid=None):
        """-> (tokens, parents, scores, count) of the draft tree of one sequence; count is a 1-element tensor."""
        t = self.torch
        tokens = t.full((keep,), -1, dtype=t.int32, device=self.dev)
        parents = t.full((keep,), -2, dtype=t.int32, device=self.dev)
        scores = t.zeros((keep,), dtype=t.float32, device=self.dev)
        count = t.zeros((4,), dtype=t.int32, device=self.dev)
        hivis_draft_tree(self.ctx, slot, topk, depth, keep, resid, 0 if resid is None else int(resid.shape[0]), tokens,
                         parents, scores, count)
        return tokens, parents, scores, count

    def verify_tree(self, slot, depth, target_logits):
        """-> (n accepted, path [depth], next token, rows) tensors."""
        t = self.torch
        ldt = HIVIS_BF16 if target_logits.dtype == t.bfloat16 else HIVIS_F32
        acc = t.zeros((4,), dtype=t.int32, device=self.dev)
        path = t.full(((depth + 3) // 4 * 4,), -2, dtype=t.int32, device=self.dev)
        nxt = t.zeros((4,), dtype=t.int32, device=self.dev)
        kv = t.zeros((4,), dtype=t.int32, device=self.dev)
        hivis_verify_tree(self.ctx, slot, target_logits, ldt, acc, path, nxt, kv)
        return acc, path, nxt, kv

    def kv_len(self, slot):
        return hivis_get_kv_len(self.ctx, slot)

    def set_kv_len(self, slot, n_rows, restore_pending=False):
        hivis_set_kv_len(self.ctx, slot, n_rows, restore_pending)

    def set_kv_len_batch(self, n_rows, slots=None, restore_pending=False):
        hivis_set_kv_len_batch(self.ctx, len(n_rows), slots, [int(x) for x in n_rows], restore_pending)

    def reset(self, slot):
        hivis_reset(self.ctx, slot)

    def read_kv(self, slot, row0, n):
        t = self.torch
        kvw = self.dims.n_kv_heads * self.dims.head_dim
        k = t.empty((n, kvw), dtype=t.float32, device=self.dev)
        v = t.empty((n, kvw), dtype=t.float32, device=self.dev)
        hivis_read_kv(self.ctx, slot, row0, n, k, v)
        return k, v

    def tap(self, name, B):
        t = self.torch
        width = {"u": self.dims.d, "attn": self.dims.n_q_heads * self.dims.head_dim, "y": self.dims.d,
                 "act": self.dims.ffn, "g": self.dims.d, "q": self.dims.n_q_heads * self.dims.head_dim}[name]
        out = t.empty((B, width), dtype=t.float32, device=self.dev)
        hivis_debug_tap(self.ctx, TAPS[name], out)
        return out

    def set_chain_kernel(self, on: bool):
        hivis_set_option(self.ctx, HIVIS_OPT_CHAIN_KERNEL, 1 if on else 0)

    def set_tc_kernel(self, on):
        """False/0: never; True: for every batch size it supports (2 in the C API); "auto"/1: the default."""
        v = 1 if on == "auto" else (2 if on is True else int(on))
        hivis_set_option(self.ctx, HIVIS_OPT_TC_KERNEL, v)

    def set_wait_limit_us(self, us: int):
        hivis_set_option(self.ctx, HIVIS_OPT_WAIT_LIMIT_US, int(us))

    def miss_next_barrier(self):
        """Test aid: the grid barriers of the next draft cannot complete, so its waits run out."""
        hivis_set_option(self.ctx, HIVIS_OPT_DEBUG_MISS_BARRIER, 1)

    def set_tc_prefill(self, on):
        """False: hivis_prefill always uses the 16-pairs-per-pass kernels; True: the default threshold; an int n > 1:
        calls of n pairs or more take the tensor-core path."""
        hivis_set_option(self.ctx, HIVIS_OPT_TC_PREFILL, int(on))

    def set_l2_keep(self, mask: int):
        """Bit p set: the tensor-core chain kernel asks L2 to keep the weights of matrix p (0 FC .. 5 LM head)."""
        hivis_set_option(self.ctx, HIVIS_OPT_L2_KEEP, int(mask))

    def record_phase_times(self, on: bool = True):
        hivis_set_option(self.ctx, HIVIS_OPT_PHASE_TIMES, 1 if on else 0)

    def phase_times(self):
        return hivis_read_phase_times(self.ctx)

    def status(self):
        hivis_status(self.ctx)

    def step_bytes(self, kv_rows):
        return hivis_step_bytes(self.ctx, kv_rows)

    def launch_count(self):
        return hivis_launch_count(self.ctx)
