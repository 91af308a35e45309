"""Shared helpers of the GPU parity tests: put a seeded workload on the device, run the CUDA
library and the CPU oracle on the same bytes, compare with the stated tolerances."""
from __future__ import annotations

import numpy as np

import hivis_inputs as hi
import oracle
from hivis_inputs.device import dev_weights, to_dev  # noqa: F401  (re-exported for the tests)

LOGIT_RTOL = 2e-2          # max |gpu - ref| / max |ref| per logits row (bf16 storage, fp32 accumulation)
LOGIT_RTOL_F32 = 2e-4      # fp32 workloads
ID_GAP = 1e-2              # ids may differ only where the oracle's top-2 logit gap is below this


class Case:
    """One workload on both sides."""

    def __init__(self, wl: hi.Workload, max_len=None, max_k=None, W=None, real="f64", extra_weights=None):
        import torch
        from paper_2509_23928_b200 import Drafter
        self.torch = torch
        self.wl = wl
        self.dims = wl.dims
        self.W = dict(W) if W is not None else hi.make_weights(wl.dims, wl.seed)
        if extra_weights:
            self.W.update(extra_weights)
        self.ids, self.hidden, self.cu = hi.make_prompt(wl)
        self.resid = hi.make_residuals(wl)
        self.lens = np.diff(self.cu)
        self.max_len = int(max_len or (self.lens.max() + wl.k + 8))
        self.oracle = oracle.Oracle(wl.dims, self.W, real)
        dW = dev_weights(self.W, wl.dims.dtype)
        self.drafter = Drafter(wl.dims, dW, max_batch=wl.batch, max_len=self.max_len, max_k=max_k or max(wl.k, 8))
        del dW
        self.d_ids = torch.from_numpy(self.ids).cuda()
        self.d_hidden = to_dev(self.hidden, wl.dims.dtype)
        self.d_resid = to_dev(self.resid, wl.dims.dtype)

    def close(self):
        self.drafter.close()

    # ---- GPU side
    def gpu_prefill(self):
        self.drafter.prefill(self.d_ids, self.d_hidden, [int(x) for x in self.cu], resid0=self.d_resid[0])

    def gpu_restore(self):
        self.drafter.set_kv_len_batch([int(l) - 1 for l in self.lens], restore_pending=True)

    def gpu_draft(self, k=None, forced=None, want_logits=True):
        t = self.torch
        k = k or self.wl.k
        f = None if forced is None else t.from_numpy(np.ascontiguousarray(forced, np.int32)).cuda()
        out = self.drafter.draft(self.wl.batch, k, self.d_resid, forced_ids=f, want_logits=want_logits)
        t.cuda.synchronize()
        if want_logits:
            return out[0].cpu().numpy(), out[1].cpu().numpy()
        return out.cpu().numpy(), None

    # ---- oracle side
    def oracle_run(self, k=None, forced=None, want_logits=True):
        return self.oracle.run_batch(self.ids, self.hidden, self.cu, k or self.wl.k, self.resid,
                                     forced_ids=forced, want_logits=want_logits)


def row_rel_err(got, ref):
    """max_i |got_i - ref_i| / max_j |ref_j| for every row (last axis)."""
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    return np.abs(got - ref).max(-1) / np.maximum(np.abs(ref).max(-1), 1e-30)


def check_draft_parity(case: Case, k=None, rtol=None):
    """Free-running ids, then teacher-forced logits of every step, against the oracle."""
    wl = case.wl
    k = k or wl.k
    rtol = rtol or (LOGIT_RTOL if wl.dims.dtype == "bf16" else LOGIT_RTOL_F32)
    ref = case.oracle_run(k)
    ids_o = np.stack([r["ids"] for r in ref])                  # [B, k]
    gaps = np.stack([r["gaps"] for r in ref])
    logits_o = np.stack([r["logits"] for r in ref])            # [B, k, V]

    case.gpu_prefill()
    ids_g, logits_g = case.gpu_draft(k)
    excused = 0
    for b in range(wl.batch):
        for s in range(k):
            if ids_g[b, s] != ids_o[b, s]:
                assert gaps[b, s] < ID_GAP, f"seq {b} step {s}: id {ids_g[b, s]} != {ids_o[b, s]}, gap {gaps[b, s]}"
                excused += 1
                break                                          # later free-running steps legitimately diverge
            err = row_rel_err(logits_g[b, s], logits_o[b, s])
            assert err <= rtol, f"free run seq {b} step {s}: logits rel err {err}"
    # teacher forcing with the oracle's ids: every step's logits are comparable
    case.gpu_restore()
    ids_f, logits_f = case.gpu_draft(k, forced=ids_o)
    err = row_rel_err(logits_f, logits_o)
    assert err.max() <= rtol, f"teacher-forced logits rel err {err.max()} at {np.unravel_index(err.argmax(), err.shape)}"
    bad = (ids_f != ids_o) & (gaps >= ID_GAP)
    assert not bad.any(), f"teacher-forced ids differ outside the gap zone at {np.argwhere(bad)}"
    return {"ref": ref, "ids_o": ids_o, "ids_g": ids_g, "max_rel_err": float(err.max()), "excused": excused}


def check_kv_parity(case: Case, ref, seqs=None, rtol=1e-2):
    """Cached K/V rows written by prefill and by the draft steps against the oracle's cache."""
    t = case.torch
    for b in (seqs if seqs is not None else range(case.wl.batch)):
        T = int(case.lens[b])
        n = T - 1 + case.wl.k
        if n == 0:
            continue
        k_g, v_g = case.drafter.read_kv(b, 0, n)
        t.cuda.synchronize()
        for got, want, nm in ((k_g, ref[b]["K"][:n], "K"), (v_g, ref[b]["V"][:n], "V")):
            got = got.cpu().numpy()
            e = np.abs(got - want).max() / max(np.abs(want).max(), 1e-30)
            assert e <= rtol, f"{nm} cache of seq {b}: rel err {e}"


def check_verify_parity(case: Case, draft_ids, planted=None):
    t = case.torch
    wl = case.wl
    logits, planted = hi.make_target_logits(wl, draft_ids, planted)
    d_logits = to_dev(logits, wl.logits_dtype)
    d_draft = t.from_numpy(np.ascontiguousarray(draft_ids, np.int32)).cuda()
    acc, nxt, kv = case.drafter.verify(d_draft, d_logits)
    t.cuda.synchronize()
    acc, nxt, kv = acc.cpu().numpy(), nxt.cpu().numpy(), kv.cpu().numpy()
    for b in range(wl.batch):
        n, nx, kvl = case.oracle.verify(draft_ids[b], logits[b], int(case.lens[b]))
        assert (acc[b], nxt[b], kv[b]) == (n, nx, kvl), f"seq {b}: gpu {(acc[b], nxt[b], kv[b])} oracle {(n, nx, kvl)}"
        assert n == planted[b]
        assert case.drafter.kv_len(b)[0] == kvl
    return acc, nxt, kv
