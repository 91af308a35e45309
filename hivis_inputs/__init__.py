"""Seeded synthetic inputs for the HiViS drafter step.

This module only draws random numbers and shapes them: weights, target hidden
states, token ids, step residuals, ragged text lengths and target logits with
a planted accept length.  It contains none of the method's arithmetic and is
the single piece of code that both the CPU oracle's tests and the CUDA path's
tests use, so that both sides receive identical bytes.

Every tensor is generated once on the host in fp32.  For a bf16 workload the
fp32 values are rounded to the nearest bf16 (ties to even) and kept as fp32
arrays holding bf16-representable values; `to_bf16_bits` gives the 16-bit
storage form of the same values for the device.

Recipe (one `numpy.random.Generator(PCG64(seed))` per workload, sub-streams
spawned in a fixed order: weights, hidden, ids, residuals, lengths, logits,
planted accept lengths):
  * matrices, embedding table, LM head: N(0, 0.02)
  * RMSNorm gains: 1 + N(0, 0.02)
  * target hidden states: N(0, 1); token ids: uniform in [0, vocab)
  * step residual rows: N(0, 0.02), n_resid = 4 rows
  * ragged text lengths: uniform integers in [lo, hi]
  * target logits: N(0, 1) with the argmax forced to follow the draft ids for
    a prefix of planted length, and forced to differ right after it.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

__all__ = [
    "DrafterDims", "Workload", "WORKLOADS", "workload",
    "to_bf16_bits", "round_to_bf16", "bf16_bits_to_f32",
    "make_weights", "make_prompt", "make_residuals", "make_target_logits",
    "WEIGHT_NAMES",
]

WEIGHT_NAMES = ("embed", "lm_head", "fc", "norm1", "wq", "wk", "wv", "wo",
                "norm2", "w_gate", "w_up", "w_down")


@dataclass(frozen=True)
class DrafterDims:
    d: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    dtype: str = "bf16"          # storage type of weights, hidden states, KV
    n_resid: int = 4

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def weight_shapes(self) -> Dict[str, Tuple[int, ...]]:
        d, f, v = self.d, self.ffn, self.vocab
        return {
            "embed": (v, d), "lm_head": (v, d), "fc": (d, 2 * d),
            "norm1": (d,), "wq": (self.q_dim, d), "wk": (self.kv_dim, d),
            "wv": (self.kv_dim, d), "wo": (d, self.q_dim), "norm2": (d,),
            "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
        }

    def step_params(self) -> int:
        """Weight elements streamed by one draft step (embedding row excluded)."""
        d, f, v = self.d, self.ffn, self.vocab
        return 2 * d * d + (self.q_dim + 2 * self.kv_dim) * d + d * self.q_dim + 3 * d * f + v * d


@dataclass(frozen=True)
class Workload:
    name: str
    dims: DrafterDims
    batch: int
    k: int
    seed: int
    text_len: Optional[int] = None            # fixed length per sequence
    text_len_range: Optional[Tuple[int, int]] = None   # ragged: uniform in [lo, hi]
    leading_positions: int = 0                # naive-drafter arm: extra leading (visual) positions
    logits_dtype: str = "f32"

    def lengths(self) -> np.ndarray:
        """Per-sequence number of (hidden, id) pairs, leading positions included."""
        if self.text_len_range is not None:
            rng = _stream(self.seed, "lengths")
            lo, hi = self.text_len_range
            t = rng.integers(lo, hi + 1, size=self.batch)
        else:
            t = np.full(self.batch, int(self.text_len))
        return (t + self.leading_positions).astype(np.int32)


TINY = DrafterDims(d=256, n_q_heads=4, n_kv_heads=4, head_dim=64, ffn=688, vocab=1024,
                   rms_eps=1e-5, dtype="f32")
LLAVA = DrafterDims(d=4096, n_q_heads=32, n_kv_heads=32, head_dim=128, ffn=11008, vocab=32000,
                    rms_eps=1e-5, dtype="bf16")
QWEN = DrafterDims(d=3584, n_q_heads=28, n_kv_heads=4, head_dim=128, ffn=18944, vocab=152064,
                   rms_eps=1e-6, dtype="bf16")
# Reduced shapes: same structure (ragged tails, GQA, odd vocab) at sizes the CPU oracle finishes in seconds.
MINI_MHA = DrafterDims(d=512, n_q_heads=4, n_kv_heads=4, head_dim=128, ffn=1376, vocab=4000,
                       rms_eps=1e-5, dtype="bf16")
MINI_GQA = DrafterDims(d=448, n_q_heads=7, n_kv_heads=1, head_dim=64, ffn=1184, vocab=5031,
                       rms_eps=1e-6, dtype="bf16")

# Head groups of 2, 4 and 8 query heads per KV head (the Qwen shape has 7).
GQA2 = DrafterDims(d=512, n_q_heads=8, n_kv_heads=4, head_dim=64, ffn=1024, vocab=3001,
                   rms_eps=1e-6, dtype="bf16")
GQA4 = DrafterDims(d=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1024, vocab=3001,
                   rms_eps=1e-6, dtype="bf16")
GQA8 = DrafterDims(d=512, n_q_heads=8, n_kv_heads=1, head_dim=64, ffn=1024, vocab=3001,
                   rms_eps=1e-6, dtype="bf16")

# Many heads at a small width: more (sequence, head group) pairs than a B200 has attention warps (740).
WIDE_GQA = DrafterDims(d=128, n_q_heads=336, n_kv_heads=48, head_dim=64, ffn=256, vocab=1000,
                       rms_eps=1e-6, dtype="bf16")
WIDE_MHA = DrafterDims(d=128, n_q_heads=48, n_kv_heads=48, head_dim=64, ffn=256, vocab=1000,
                       rms_eps=1e-5, dtype="bf16")

WORKLOADS: Dict[str, Workload] = {w.name: w for w in [
    Workload("c1_tiny_f32_b1", TINY, batch=1, k=4, seed=1001, text_len=32, logits_dtype="f32"),
    Workload("c2_llava_b1", LLAVA, batch=1, k=5, seed=1002, text_len=128, logits_dtype="bf16"),
    Workload("c3_llava_b16_ragged", LLAVA, batch=16, k=5, seed=1003, text_len_range=(64, 512),
             logits_dtype="bf16"),
    Workload("c4_qwen_b8", QWEN, batch=8, k=7, seed=1004, text_len=256, logits_dtype="bf16"),
    Workload("c5a_llava_b16_text_only", LLAVA, batch=16, k=5, seed=1005, text_len=128,
             logits_dtype="bf16"),
    Workload("c5b_llava_b16_naive_kv", LLAVA, batch=16, k=5, seed=1005, text_len=128,
             leading_positions=576, logits_dtype="bf16"),
    # reduced-size parity cases
    Workload("mini_mha_b1", MINI_MHA, batch=1, k=5, seed=2001, text_len=37, logits_dtype="bf16"),
    Workload("mini_mha_b5_ragged", MINI_MHA, batch=5, k=6, seed=2002, text_len_range=(1, 150),
             logits_dtype="bf16"),
    Workload("mini_gqa_b16_ragged", MINI_GQA, batch=16, k=7, seed=2003, text_len_range=(3, 300),
             logits_dtype="f32"),
    Workload("mini_gqa_b3", MINI_GQA, batch=3, k=2, seed=2004, text_len=65, logits_dtype="bf16"),
    Workload("tiny_f32_b4_ragged", TINY, batch=4, k=6, seed=2005, text_len_range=(1, 70),
             logits_dtype="f32"),
    Workload("wide_gqa_b16_ragged", WIDE_GQA, batch=16, k=3, seed=2006, text_len_range=(2, 70),
             logits_dtype="bf16"),
    Workload("wide_mha_b16_ragged", WIDE_MHA, batch=16, k=3, seed=2007, text_len_range=(2, 70),
             logits_dtype="bf16"),
    Workload("gqa2_b5_ragged", GQA2, batch=5, k=4, seed=2008, text_len_range=(1, 140), logits_dtype="bf16"),
    Workload("gqa4_b16_ragged", GQA4, batch=16, k=3, seed=2009, text_len_range=(2, 100), logits_dtype="bf16"),
    Workload("gqa8_b16_ragged", GQA8, batch=16, k=3, seed=2010, text_len_range=(2, 100), logits_dtype="f32"),
    Workload("gqa4_b5_ragged", GQA4, batch=5, k=4, seed=2011, text_len_range=(1, 140), logits_dtype="bf16"),
]}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


_STREAM_ORDER = ("weights", "hidden", "ids", "residuals", "lengths", "logits", "planted")


def _stream(seed: int, which: str) -> np.random.Generator:
    idx = _STREAM_ORDER.index(which)
    ss = np.random.SeedSequence(seed).spawn(len(_STREAM_ORDER))[idx]
    return np.random.Generator(np.random.PCG64(ss))


# ----------------------------------------------------------------------------- bf16 helpers
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(to_bf16_bits(x)).reshape(np.shape(x))


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_to_bf16(x) if dtype == "bf16" else x


def _normal(rng: np.random.Generator, shape, scale: float) -> np.ndarray:
    out = rng.standard_normal(size=shape, dtype=np.float32)
    out *= np.float32(scale)
    return out


# ----------------------------------------------------------------------------- generators
def make_weights(dims: DrafterDims, seed: int) -> Dict[str, np.ndarray]:
    """All drafter weights, row-major [out, in], fp32 arrays (bf16-valued for bf16 dims)."""
    rng = _stream(seed, "weights")
    out: Dict[str, np.ndarray] = {}
    for name, shape in dims.weight_shapes().items():      # dict order is the draw order
        if name in ("norm1", "norm2"):
            w = np.float32(1.0) + _normal(rng, shape, 0.02)
        else:
            w = _normal(rng, shape, 0.02)
        out[name] = _store(w, dims.dtype)
    return out


def make_prompt(wl: Workload):
    """Packed prompt: ids [sum T] int32, hidden [sum T, d] fp32, cu_seqlens [B+1] int32.

    ids[p] is the token that follows the one whose target hidden state is hidden[p].
    Leading (visual stand-in) positions, if any, are drawn the same way.
    """
    lens = wl.lengths()
    total = int(lens.sum())
    hid = _store(_normal(_stream(wl.seed, "hidden"), (total, wl.dims.d), 1.0), wl.dims.dtype)
    ids = _stream(wl.seed, "ids").integers(0, wl.dims.vocab, size=total).astype(np.int32)
    cu = np.zeros(wl.batch + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return ids, hid, cu


def make_residuals(wl: Workload) -> np.ndarray:
    """Step residual rows [n_resid, d], fp32 (bf16-valued for bf16 dims)."""
    r = _normal(_stream(wl.seed, "residuals"), (wl.dims.n_resid, wl.dims.d), 0.02)
    return _store(r, wl.dims.dtype)


def make_target_logits(wl: Workload, draft_ids: np.ndarray, planted: Optional[np.ndarray] = None):
    """Target logits [B, k+1, V] fp32 (bf16-valued if wl.logits_dtype == 'bf16') and planted n [B].

    Row j stands for the target's prediction after the root token and j draft tokens.
    Rows j < n get a large value at draft id j; row n (if n < k) is made to disagree with
    draft id n; rows after it stay random.
    """
    B, k, V = wl.batch, wl.k, wl.dims.vocab
    draft_ids = np.asarray(draft_ids).reshape(B, k)
    logits = _normal(_stream(wl.seed, "logits"), (B, k + 1, V), 1.0)
    if planted is None:
        planted = _stream(wl.seed, "planted").integers(0, k + 1, size=B)
    planted = np.asarray(planted, dtype=np.int32)
    for b in range(B):
        n = int(planted[b])
        for j in range(n):
            logits[b, j, draft_ids[b, j]] = 12.0
        if n < k:
            logits[b, n, draft_ids[b, n]] = -12.0
    return _store(logits, wl.logits_dtype), planted


def scaled(wl: Workload, **changes) -> Workload:
    """A copy of a workload with some fields replaced (tests use it for edge cases)."""
    return replace(wl, **changes)
