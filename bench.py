#!/usr/bin/env python
"""Benchmark of the HiViS drafter step (draft steps/s, us/step, HBM roofline fraction).

One benchmark "step" = one pass of the hot path over one batch: k chained draft steps
(fuse+residual, RMSNorm, QKV, RoPE, attention over the text-only cache, O, SwiGLU, LM head,
argmax) followed by batched greedy verification with KV rollback.  `value` counts draft steps
(k per benchmark step).  Inputs are seeded and synthetic; weights are random-init in the shape of
the named backbone.

The metric is quoted at batch 1 and batch 16.  Without --workload the run times the batch-1
workload (the headline `value`, `roofline`, `e2e`) and then, in the same process, the batch-16
workload with the text-only cache (key `batch16`: its own value, roofline, e2e and clock sample) and
its naive-cache twin with 576 extra leading positions (key `batch16_naive_kv`: the ablation pair).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

--gpus N > 1 means N independent replicas, one process per GPU (no collective on the path).  Under
torchrun the ranks come from the environment; started plainly, the script launches its own N ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import hivis_inputs as hi  # noqa: E402

METRIC = "draft_steps_per_s"
UNIT = "draft steps/s"
HEADLINE = "c2_llava_b1"
BATCH16 = "c5a_llava_b16_text_only"
BATCH16_NAIVE = "c5b_llava_b16_naive_kv"
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


CHAIN_KERNEL_SOURCES = ("kernels_tc.cu", "kernels_chain.cu", "attn_body.cuh", "attn_warp.cuh", "attn_mma.cuh")


def kernel_source_hash() -> str:
    """Hash of the sources the two chain kernels are compiled from: ties a stored profiler figure to the kernels it
    was taken from."""
    csrc = os.path.join(ROOT, "paper_2509_23928_b200", "csrc")
    h = hashlib.sha256()
    for name in CHAIN_KERNEL_SOURCES:
        h.update(name.encode())
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def captured_traffic(workload: str):
    """DRAM bytes (read + written) of ONE launch of the chain kernel on `workload`, from the ncu capture recorded
    in profiles/ncu_traffic.json; None when there is no capture or the kernels have changed since it was taken."""
    try:
        rec = json.load(open(TRAFFIC_FILE))["captures"][workload]
    except Exception:
        return None
    if rec.get("source_hash") != kernel_source_hash():
        return None
    return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])


def max_over_ranks(value: float, dist, device: str) -> float:
    """Largest `value` over all ranks (the job's time is the slowest replica's); identity without a group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, steps: int, k: int, slowest_ms: float) -> float:
    """Whole-job draft steps/s of `world` independent replicas that each ran `steps` benchmark steps of k
    draft steps, timed by the slowest replica."""
    return world * steps * k / (slowest_ms * 1e-3)


def replica_workload(wl, rank: int, world: int):
    """Replica `rank` of `world`: same shapes, its own seed (no data is shared, no collective on the path)."""
    return wl if world == 1 else hi.scaled(wl, seed=wl.seed + 100 * rank)


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_replicas(n: int, argv) -> int:
    """Start n ranks of this script (one per GPU) with the rendezvous variables torchrun would set; rank 0 prints
    the job's line.  Returns the first non-zero exit code, else 0."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.proc = gpu_index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "25", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self, first_row: int = 0):
        """Summary of the samples from row `first_row` on (the rows before it were taken during the warm-up)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], None, set()
        for r in self.rows[first_row:]:
            try:
                sm.append(float(r[1])); mx = float(r[2])
            except Exception:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def run_oracle_sample(wl, steps: int, warmup: int):
    """The CPU oracle (fp32 build) as it stands, timed on the host cores on a bounded sample of
    the same workload: the k-step chain of the first sequence(s) after an untimed prefill."""
    import oracle
    W = hi.make_weights(wl.dims, wl.seed)
    ids, hidden, cu = hi.make_prompt(wl)
    resid = hi.make_residuals(wl)
    o = oracle.Oracle(wl.dims, W, "f32")
    rho = o.fold_residuals(resid)
    nseq = min(wl.batch, 2)
    caches = []
    for b in range(nseq):
        lo, hi_ = int(cu[b]), int(cu[b + 1])
        T = hi_ - lo
        Kc, Vc = o.new_cache(T + wl.k)
        o.prefill(ids[lo:hi_], hidden[lo:hi_], rho[0], Kc, Vc)
        caches.append((T, Kc, Vc, int(ids[hi_ - 1]), hidden[hi_ - 1]))
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        for (T, Kc, Vc, pid, ph) in caches:
            o.draft(T - 1, pid, ph, wl.k, rho, Kc, Vc, want_logits=False)
        times.append(time.perf_counter() - t0)
    t = float(np.mean(times[warmup:]))
    per_seq_step = t / (nseq * wl.k)
    # one batched draft step on the CPU = batch sequential single-sequence steps
    return {"value": 1.0 / (per_seq_step * wl.batch), "unit": UNIT, "cores": o.num_threads(), "kind": "oracle",
            "sample": f"{steps} timed repetitions (after {warmup} warm-up) of the {wl.k}-step chain for {nseq} of "
                      f"{wl.batch} sequence(s), prefill untimed; a batched step costed as batch x the "
                      f"single-sequence step", "us_per_step": per_seq_step * wl.batch * 1e6,
            "ms_per_bench_step": t / nseq * wl.batch * 1e3}


def workload_config(wl, world: int):
    return {"workload": wl.name, "batch": wl.batch, "k": wl.k, "draft_steps_per_bench_step": wl.k,
            "text_len": wl.text_len if wl.text_len else list(wl.text_len_range),
            "leading_positions": wl.leading_positions, "d": wl.dims.d, "ffn": wl.dims.ffn,
            "vocab": wl.dims.vocab, "heads": [wl.dims.n_q_heads, wl.dims.n_kv_heads, wl.dims.head_dim],
            "logits_dtype": wl.logits_dtype, "parallelism": f"replicas x{world} (no collective)",
            "l2": "weights streamed per step (>= 734 MB) exceed the 126 MB L2; no flush needed"}


class WeightCache:
    """Device weights per (dims, seed): the batch-16 workload and its naive-cache twin share one set."""

    def __init__(self):
        self.key, self.dW = None, None

    def get(self, wl):
        from hivis_inputs.device import dev_weights
        key = (wl.dims, wl.seed)
        if key != self.key:
            self.dW = None
            W = hi.make_weights(wl.dims, wl.seed)
            self.dW = dev_weights(W, wl.dims.dtype)
            self.key = key
        return self.dW


def time_workload(wl, steps: int, warmup: int, rank: int, local_rank: int, world: int, dist, weights: WeightCache,
                  want_e2e: bool, short: bool = False, l2_keep: int = 0):
    """Prefill (untimed), then `steps` timed benchmark steps of `wl` on this rank's GPU.  Returns the pieces of the
    JSON line that belong to one workload.  short=True: device timing of the chain only (no e2e, no clock sample)."""
    import torch
    from hivis_inputs.device import to_dev
    from paper_2509_23928_b200 import (Drafter, hivis_profile_begin, hivis_profile_end, hivis_verify, hivis_draft,
                                       HIVIS_BF16, HIVIS_F32)
    ids, hidden, cu = hi.make_prompt(wl)
    resid = hi.make_residuals(wl)
    lens = np.diff(cu)
    B, k = wl.batch, wl.k
    dr = Drafter(wl.dims, weights.get(wl), max_batch=B, max_len=int(lens.max()) + k + 8, max_k=max(k, 8))
    if l2_keep:
        dr.set_l2_keep(l2_keep)
    torch.cuda.empty_cache()
    d_ids = torch.from_numpy(ids).cuda()
    d_hidden = to_dev(hidden, wl.dims.dtype)
    d_resid = to_dev(resid, wl.dims.dtype)
    dr.prefill(d_ids, d_hidden, [int(x) for x in cu], resid0=d_resid[0])
    out_ids = torch.empty((B, k), dtype=torch.int32, device="cuda")
    # target logits with planted accept lengths, built from the ids of one untimed draft
    dr.draft(B, k, d_resid, out_ids=out_ids)
    torch.cuda.synchronize()
    logits_np, planted = hi.make_target_logits(wl, out_ids.cpu().numpy())
    d_logits = to_dev(logits_np, wl.logits_dtype)
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    nxt = torch.empty(B, dtype=torch.int32, device="cuda")
    kvl = torch.empty(B, dtype=torch.int32, device="cuda")
    ldt = HIVIS_BF16 if wl.logits_dtype == "bf16" else HIVIS_F32
    stream = torch.cuda.current_stream()

    rows_after_prefill = [int(l) - 1 for l in lens]

    def restore():
        dr.set_kv_len_batch(rows_after_prefill, restore_pending=True)

    def one_step():
        hivis_draft(dr.ctx, B, None, k, d_resid, d_resid.shape[0], out_ids, None, None, stream)
        hivis_verify(dr.ctx, B, None, k, out_ids, d_logits, ldt, acc, nxt, kvl, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- timed region: K steps, CUDA events on the launching stream
    sampler = ClockSampler(local_rank)
    if rank == 0 and not short:
        sampler.start()
    for _ in range(max(warmup, 3)):
        restore(); one_step()
    if sampler.proc is not None:
        # nvidia-smi takes a moment to deliver its first line: keep the same load running until it does
        t_wait = time.perf_counter()
        while not sampler.rows and time.perf_counter() - t_wait < 2.0:
            restore(); one_step(); torch.cuda.synchronize()
    barrier()
    first_sample = len(sampler.rows)
    n0 = dr.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    draft_ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        restore()
        ev[i][0].record(stream)
        hivis_draft(dr.ctx, B, None, k, d_resid, d_resid.shape[0], out_ids, None, None, stream)
        draft_ev[i].record(stream)
        hivis_verify(dr.ctx, B, None, k, out_ids, d_logits, ldt, acc, nxt, kvl, stream)
        ev[i][1].record(stream)
    barrier()
    launches = dr.launch_count() - n0 - steps                   # the restore kernel sits outside the events
    step_ms = np.array([a.elapsed_time(b) for a, b in ev])
    draft_ms = np.array([ev[i][0].elapsed_time(draft_ev[i]) for i in range(steps)])
    total_ms = float(step_ms.sum())
    clocks = None
    if rank == 0 and not short:
        extended = False
        if sampler.proc is not None and len(sampler.rows) - first_sample < 3:
            # a timed region shorter than three sampling periods: the same load goes on (untimed) until three samples exist
            extended = True
            t_wait = time.perf_counter()
            while len(sampler.rows) - first_sample < 3 and time.perf_counter() - t_wait < 2.0:
                restore(); one_step(); torch.cuda.synchronize()
        clocks = sampler.stop(first_sample)
        if extended:
            clocks["note"] = "timed region shorter than three sampling periods: sampling went on under the same load"
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ok_planted = bool((acc.cpu().numpy() == planted).all())
    dr.status()                                                  # no wait ran out, no id was out of range

    # ---------------- per-kernel device time (separate pass: events around every launch)
    restore()
    hivis_profile_begin(dr.ctx)
    reps = min(steps, 20)
    for _ in range(reps):
        hivis_draft(dr.ctx, B, None, k, d_resid, d_resid.shape[0], out_ids, None, None, stream)
        restore()
    prof = hivis_profile_end(dr.ctx)
    kv_rows = [int(l) - 1 + k // 2 for l in lens]               # mid-chain cache length
    step_bytes = dr.step_bytes(kv_rows)
    es = 2 if wl.dims.dtype == "bf16" else 4
    D = wl.dims
    class_bytes = {"fuse_fc": 2 * D.d * D.d * es, "qkv": (D.q_dim + 2 * D.kv_dim) * D.d * es,
                   "attention": sum(2 * (r + 1) * D.kv_dim * es for r in kv_rows), "o_proj": D.d * D.q_dim * es,
                   "gate_up": 2 * D.ffn * D.d * es, "down": D.d * D.ffn * es, "lm_head_argmax": D.vocab * D.d * es}
    peak, peak_kind = measured_peaks()
    kern = {}
    for name, (ms, n) in prof.items():
        if n and name in class_bytes:
            us = ms / n * 1e3
            kern[name] = {"us": round(us, 2), "launches_per_draft_step": n // (reps * k),
                          "GBps": round(class_bytes[name] / (us * 1e-6) / 1e9, 1)}
    chain_ms, chain_n = prof.get("draft_chain", (0.0, 0))
    if chain_n:                      # the whole k-step chain is a single persistent kernel
        us = chain_ms / chain_n * 1e3
        nbytes = k * step_bytes
        kern["draft_chain"] = {"us": round(us, 2), "launches_per_bench_step": 1,
                               "GBps": round(nbytes / (us * 1e-6) / 1e9, 1)}
        kern["draft_chain"]["kernel"] = ("draft_chain_kernel (one sequence, fp32 FMA, all k steps in one launch)" if B == 1 else
                                        "tc_chain_kernel (tcgen05, all k steps in one launch)")
        dom, dom_bytes = "draft_chain", nbytes
    else:
        dom = max((n for n in kern), key=lambda n: prof[n][0])
        dom_bytes = class_bytes[dom]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kern[dom]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": round(kern[dom]["GBps"] / peak, 4), "peak_kind": peak_kind,
                "traffic": captured_traffic(wl.name) if (dom == "draft_chain" and world == 1) else None,
                "algorithmic_bytes_per_launch": dom_bytes, "per_kernel": kern}

    draft_us_per_step = float(np.median(draft_ms)) / k * 1e3
    chain = {"us_per_draft_step_median": round(draft_us_per_step, 2),
             "us_per_draft_step_min": round(float(draft_ms.min()) / k * 1e3, 2),
             "verify_us_median": round(float(np.median(step_ms - draft_ms)) * 1e3, 2),
             "algorithmic_bytes_per_draft_step": step_bytes,
             "GBps": round(step_bytes / (draft_us_per_step * 1e-6) / 1e9, 1),
             "frac_of_peak": round(step_bytes / (draft_us_per_step * 1e-6) / 1e9 / peak, 4),
             "frac_of_8TBps": round(step_bytes / (draft_us_per_step * 1e-6) / 1e9 / 8000.0, 4),
             "tokens_per_s": round(B / (draft_us_per_step * 1e-6), 1)}

    # ---------------- end to end through the C ABI with HOST buffers
    e2e = None
    if want_e2e and not short:
        h_resid = d_resid.cpu().pin_memory()
        h_logits = d_logits.cpu().pin_memory()
        h_ids = torch.empty((B, k), dtype=torch.int32).pin_memory()
        Bp = (B + 3) // 4 * 4                                    # rows stay 16-byte aligned
        h_res = torch.empty((3, Bp), dtype=torch.int32).pin_memory()
        d_res = torch.empty((3, Bp), dtype=torch.int32, device="cuda")
        d_resid2 = torch.empty_like(d_resid)
        d_logits2 = torch.empty_like(d_logits)
        n_e2e = max(3, min(steps, 20))
        copy_stream = torch.cuda.Stream()                        # the logits cross PCIe while the draft kernel runs
        landed = torch.cuda.Event()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            restore()
            with torch.cuda.stream(copy_stream):
                d_logits2.copy_(h_logits, non_blocking=True)     # the target's logits arrive from the host
                landed.record(copy_stream)
            d_resid2.copy_(h_resid, non_blocking=True)
            hivis_draft(dr.ctx, B, None, k, d_resid2, d_resid2.shape[0], out_ids, None, None, stream)
            h_ids.copy_(out_ids, non_blocking=True)
            stream.wait_event(landed)
            hivis_verify(dr.ctx, B, None, k, out_ids, d_logits2, ldt, d_res[0], d_res[1], d_res[2], stream)
            h_res.copy_(d_res, non_blocking=True)
            torch.cuda.synchronize()                             # (also keeps the next step's copy off this step's logits)
        t_e2e = time.perf_counter() - t0
        t_e2e = max_over_ranks(t_e2e, dist, "cuda")
        e2e = {"value": job_throughput(world, n_e2e, k, t_e2e * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": int(h_resid.numel() * h_resid.element_size() + h_logits.numel() * h_logits.element_size()),
               "d2h_bytes_per_step": int(h_ids.numel() * 4 + 3 * B * 4), "steps": n_e2e,
               "ms_per_step": t_e2e / n_e2e * 1e3}
    dr.close()
    return {"value": job_throughput(world, steps, k, total_ms), "ms_per_step": total_ms / steps, "clocks": clocks,
            "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "draft_chain": chain,
            "verify_matches_planted": ok_planted}


PHASES = ("gather", "fc", "qkv", "attention", "o_proj", "gate_up", "down", "lm_head")


def phase_breakdown(wl, weights: WeightCache, reps: int = 20):
    """Where a draft step of the tensor-core chain kernel goes: the kernel's own time stamps (option
    HIVIS_OPT_PHASE_TIMES), `reps` recorded launches, medians over launches.  Per phase: its cost (last arrival on
    the previous grid barrier -> last arrival on its own), the spread of the arrivals, how long after the previous
    barrier completed the operand producers got going, and the tail after the last accumulator was complete."""
    import torch
    from hivis_inputs.device import to_dev
    from paper_2509_23928_b200 import Drafter
    ids, hidden, cu = hi.make_prompt(wl)
    resid = hi.make_residuals(wl)
    lens = np.diff(cu)
    B, k = wl.batch, wl.k
    dr = Drafter(wl.dims, weights.get(wl), max_batch=B, max_len=int(lens.max()) + k + 8, max_k=max(k, 8))
    d_resid = to_dev(resid, wl.dims.dtype)
    dr.prefill(torch.from_numpy(ids).cuda(), to_dev(hidden, wl.dims.dtype), [int(x) for x in cu], resid0=d_resid[0])
    out_ids = torch.empty((B, k), dtype=torch.int32, device="cuda")

    def restore():
        for b in range(B):
            dr.set_kv_len(b, int(lens[b]) - 1, restore_pending=True)

    for _ in range(5):
        dr.draft(B, k, d_resid, out_ids=out_ids); restore()
    dr.record_phase_times(True)
    cost, spread, start, tail, late = [], [], [], [], np.zeros(0)
    for _ in range(reps):
        dr.draft(B, k, d_resid, out_ids=out_ids)
        T = dr.phase_times().astype(np.float64) / 1e3        # [k, events, grid] in us; 0 = no event
        restore()
        T[T == 0] = np.nan
        arr = T[:, :8, :].reshape(k * 8, -1)                 # arrivals in barrier order
        done = np.nanmax(arr, axis=1)                        # completion of every barrier
        prev = np.concatenate([[np.nan], done[:-1]])
        cost.append((done - prev).reshape(k, 8))
        spread.append((done - np.nanmin(arr, axis=1)).reshape(k, 8))
        gemm_bar = np.array([1, 2, 4, 5, 6, 7])              # barrier index of the six GEMM phases
        st = np.full((k, 8), np.nan); tl = np.full((k, 8), np.nan)
        for s in range(k):
            for j, e in enumerate(gemm_bar):
                before = prev[s * 8 + e]
                st[s, e] = np.nanmedian(T[s, 8 + j]) - before          # operand producers under way
                tl[s, e] = np.nanmedian(T[s, e] - T[s, 14 + j])        # last accumulator -> arrival
            st[s, 3] = np.nanmedian(T[s, 20]) - prev[s * 8 + 3]
        start.append(st); tail.append(tl)
        lateness = arr - np.nanmin(arr, axis=1, keepdims=True)          # per barrier and CTA
        late = lateness if late.size == 0 else late + lateness
    dr.record_phase_times(False)
    dr.close()
    med = lambda xs: np.nanmedian(np.stack(xs), axis=0)
    cost, spread, start, tail = med(cost), med(spread), med(start), med(tail)
    steps = slice(1, None) if k > 1 else slice(0, None)      # step 0 has no previous barrier for its gather
    out = {"workload": wl.name, "launches": reps, "unit": "us", "per_phase": {}}
    for e, name in enumerate(PHASES):
        out["per_phase"][name] = {"cost": round(float(np.nanmean(cost[steps, e])), 2),
                                  "arrival_spread": round(float(np.nanmean(spread[steps, e])), 2),
                                  "input_wait_passed_after": None if np.isnan(start[steps, e]).all() else round(float(np.nanmean(start[steps, e])), 2),
                                  "tail_after_last_accumulator": None if np.isnan(tail[steps, e]).all() else round(float(np.nanmean(tail[steps, e])), 2)}
    out["step_us"] = round(float(sum(v["cost"] for v in out["per_phase"].values())), 2)
    # are the same CTAs late in every phase?  mean lateness per CTA over the GEMM barriers of all steps and launches
    gemm_rows = [s * 8 + e for s in range(k) for e in (1, 2, 4, 5, 6, 7)]
    per_cta = np.nanmean(late[gemm_rows], axis=0) / reps
    order = np.argsort(-per_cta)
    out["cta_lateness"] = {"mean": round(float(np.nanmean(per_cta)), 2), "max": round(float(np.nanmax(per_cta)), 2),
                           "latest_ctas": [int(c) for c in order[:12]],
                           "their_lateness": [round(float(per_cta[c]), 2) for c in order[:12]],
                           "earliest_ctas": [int(c) for c in order[-6:]]}
    return out


def prefill_ablation(reps: int = 5):
    """The visual-token-hiding ablation on the prefix build: time of hivis_prefill for the LLaVA-shaped drafter at batch 16
    with 128 text positions and 0 (text-only), 576 or 2048 leading positions standing in for visual tokens, on the
    tensor-core path and on the 16-pairs-per-pass path.  CUDA events around the call, median of `reps`."""
    import torch
    from hivis_inputs.device import to_dev
    from paper_2509_23928_b200 import Drafter
    base = hi.workload(BATCH16)
    weights = WeightCache()
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    tf_peak = float(peaks.get("bf16_tflops", 1590.0))
    out = {"workload": "LLaVA-shaped drafter, batch 16, 128 text positions + leading positions", "unit": "ms per hivis_prefill call",
           "tensor_peak_tflops": tf_peak, "tensor_peak_kind": "measured" if "bf16_tflops" in peaks else "fallback", "rows": []}
    for lead in (0, 576, 2048):
        wl = hi.scaled(base, leading_positions=lead, name=f"llava_b16_lead{lead}")
        ids, hidden, cu = hi.make_prompt(wl)
        resid = hi.make_residuals(wl)
        lens = np.diff(cu)
        B, k, D = wl.batch, wl.k, wl.dims
        dr = Drafter(D, weights.get(wl), max_batch=B, max_len=int(lens.max()) + k + 8, max_k=8)
        d_ids = torch.from_numpy(ids).cuda()
        d_hidden = to_dev(hidden, D.dtype)
        d_resid = to_dev(resid, D.dtype)
        pairs = int(cu[-1])
        flops = 2.0 * pairs * (2 * D.d * D.d + D.d * 2 * D.kv_dim)
        row = {"leading_positions": lead, "pairs": pairs}
        for label, on in (("tensor_core", True), ("per_pass", False)):
            dr.set_tc_prefill(on)
            ts = []
            for it in range(reps + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                dr.prefill(d_ids, d_hidden, [int(x) for x in cu], start_pos=[0] * B, resid0=d_resid[0])
                e1.record()
                torch.cuda.synchronize()
                if it >= 2:
                    ts.append(e0.elapsed_time(e1))
            ms = float(np.median(ts))
            row[label] = {"ms": round(ms, 3), "pairs_per_s": round(pairs / (ms * 1e-3)), "tflops": round(flops / (ms * 1e-3) / 1e12, 1),
                          "frac_of_tensor_peak": round(flops / (ms * 1e-3) / 1e12 / tf_peak, 4)}
        dr.status()
        dr.close()
        out["rows"].append(row)
    t0 = out["rows"][0]["tensor_core"]["ms"]
    for r in out["rows"]:
        r["tensor_core_over_text_only"] = round(r["tensor_core"]["ms"] / t0, 2)
    return out


def tree_and_sampling(weights: WeightCache, reps: int = 30):
    """The two widened rows, timed with CUDA events around the calls (medians of `reps`, caches warm as in a running
    decode loop; between tree drafts the target logits of the previous verification are rewritten, 23 MB):
    tree drafting and greedy tree verification of one sequence of the headline workload with the paper's tree shapes
    (top-10, depth 6, 60 kept; top-8, depth 4, 30 kept), and verification by speculative sampling at batch 16.
    Algorithmic bytes of a tree draft: every level streams the drafter's weights once and reads the prefix rows of the
    cache once per expanded node."""
    import torch
    from hivis_inputs.device import to_dev
    from paper_2509_23928_b200 import Drafter
    peak, peak_kind = measured_peaks()
    out = {"unit": "us", "peak_GBps": peak, "peak_kind": peak_kind, "trees": [], "launches": reps}
    ev = lambda: torch.cuda.Event(enable_timing=True)

    wl = hi.workload(HEADLINE)
    ids, hidden, cu = hi.make_prompt(wl)
    resid = hi.make_residuals(wl)
    T = int(cu[1])
    D = wl.dims
    es = 2 if D.dtype == "bf16" else 4
    dr = Drafter(D, weights.get(wl), max_batch=1, max_len=T + 80, max_k=8)
    d_resid = to_dev(resid, D.dtype)
    dr.prefill(torch.from_numpy(ids).cuda(), to_dev(hidden, D.dtype), [int(x) for x in cu], resid0=d_resid[0])
    weight_bytes = dr.step_bytes([0]) - 2 * D.kv_dim * es               # one position with an empty prefix: the weights
    rng = np.random.default_rng(7)
    for topk, depth, keep in ((10, 6, 60), (8, 4, 30)):
        logits = to_dev(rng.standard_normal((keep + 1, D.vocab)).astype(np.float32), wl.logits_dtype)
        d_ms, v_ms = [], []
        n0 = dr.launch_count()
        for i in range(reps + 3):
            dr.set_kv_len(0, T - 1, restore_pending=True)
            a, b, c = ev(), ev(), ev()
            a.record()
            tok, par, sc, cnt = dr.draft_tree(0, topk, depth, keep, d_resid)
            b.record()
            dr.verify_tree(0, depth, logits)
            c.record()
            torch.cuda.synchronize()
            if i >= 3:
                d_ms.append(a.elapsed_time(b)); v_ms.append(b.elapsed_time(c))
        launches = (dr.launch_count() - n0) / (reps + 3) - 1            # the restore kernel
        nodes = 1 + (depth - 1) * topk                                   # positions that run through the layer
        nbytes = depth * weight_bytes + nodes * 2 * (T - 1) * D.kv_dim * es
        us = float(np.median(d_ms)) * 1e3
        out["trees"].append({"workload": wl.name, "topk": topk, "depth": depth, "keep": keep, "kept": int(cnt[0].item()),
                             "draft_tree_us": round(us, 1), "verify_tree_us": round(float(np.median(v_ms)) * 1e3, 1),
                             "launches_per_tree": round(launches, 1), "layer_positions": nodes,
                             "algorithmic_bytes": int(nbytes), "GBps": round(nbytes / (us * 1e-6) / 1e9, 1),
                             "frac_of_peak": round(nbytes / (us * 1e-6) / 1e9 / peak, 4)})
    dr.status()
    dr.close()

    wl = hi.workload(BATCH16)
    B, k, V = wl.batch, wl.k, wl.dims.vocab
    ids, hidden, cu = hi.make_prompt(wl)
    lens = np.diff(cu)
    resid = hi.make_residuals(wl)
    dr = Drafter(wl.dims, weights.get(wl), max_batch=B, max_len=int(lens.max()) + k + 8, max_k=8)
    d_resid = to_dev(resid, wl.dims.dtype)
    dr.prefill(torch.from_numpy(ids).cuda(), to_dev(hidden, wl.dims.dtype), [int(x) for x in cu], resid0=d_resid[0])
    out_ids, d_logits = dr.draft(B, k, d_resid, want_logits=True)
    target = to_dev(rng.standard_normal((B, k + 1, V)).astype(np.float32), wl.logits_dtype)
    ua = torch.from_numpy(rng.random((B, k)).astype(np.float32)).cuda()
    us_ = torch.from_numpy(rng.random(B).astype(np.float32)).cuda()
    flush = torch.empty(160 << 20, dtype=torch.uint8, device="cuda")
    t_ms = []
    for i in range(reps + 3):
        for b in range(B):
            dr.set_kv_len(b, int(lens[b]) - 1, restore_pending=True)
        dr.draft(B, k, d_resid, out_ids=out_ids)
        flush.zero_()                                                    # the logits come from DRAM
        a, b_ = ev(), ev()
        a.record()
        dr.verify_sampled(out_ids, d_logits, target, 1.0, ua, us_)
        b_.record()
        torch.cuda.synchronize()
        if i >= 3:
            t_ms.append(a.elapsed_time(b_))
    tb = 2 if wl.logits_dtype == "bf16" else 4
    # every logit once for the row statistics, then per sequence the target and draft rows at the first rejection
    lbytes = B * k * V * 4 + B * (k + 1) * V * tb + B * V * (4 + tb)
    us = float(np.median(t_ms)) * 1e3
    out["sampled_verification"] = {"workload": wl.name, "batch": B, "k": k, "vocab": V, "temperature": 1.0,
                                   "us": round(us, 1), "launches": 2, "algorithmic_bytes": int(lbytes),
                                   "GBps": round(lbytes / (us * 1e-6) / 1e9, 1),
                                   "frac_of_peak": round(lbytes / (us * 1e-6) / 1e9 / peak, 4)}
    # chained drafting with drawn tokens (T = 1) against greedy drafting, same batch
    uni = torch.from_numpy((rng.random((B, k, V)) * (1 - 2e-6) + 1e-6).astype(np.float32)).cuda()
    g_ms, s_ms = [], []
    for i in range(reps + 3):
        for sampled in (False, True):
            for b in range(B):
                dr.set_kv_len(b, int(lens[b]) - 1, restore_pending=True)
            a, b_ = ev(), ev()
            a.record()
            if sampled:
                dr.draft_sampled(B, k, 1.0, uni, d_resid, want_logits=False)
            else:
                dr.draft(B, k, d_resid, out_ids=out_ids)
            b_.record()
            torch.cuda.synchronize()
            if i >= 3:
                (s_ms if sampled else g_ms).append(a.elapsed_time(b_))
    out["sampled_drafting"] = {"workload": wl.name, "batch": B, "k": k, "temperature": 1.0,
                               "us_per_draft_step": round(float(np.median(s_ms)) / k * 1e3, 2),
                               "greedy_us_per_draft_step": round(float(np.median(g_ms)) / k * 1e3, 2),
                               "uniform_bytes_per_step": int(B * V * 4)}
    dr.status()
    dr.close()
    return out


def draft_verify_refresh_loop(weights: WeightCache, rounds: int = 40, tc_prefill_min: int = 0):
    """Algorithm 1 as a loop on the drafter's side, batch 16 of the headline shape: draft k tokens, verify them against a
    toy target whose accept lengths are planted (a truncated geometric law with ratio 0.75, drawn per sequence and
    round), then rebuild the rows of the accepted tokens from the target's "true" features (seeded noise standing in for
    them) with hivis_prefill(start_pos) and go on with the next round.  The accept counts travel to the host every round,
    as they do to whoever runs the target.  Reported: tokens committed per round and sequence, the time of the three calls
    (CUDA events), and committed tokens per second of drafter-side time."""
    import torch
    from hivis_inputs.device import to_dev
    from paper_2509_23928_b200 import Drafter
    wl = hi.workload(BATCH16)
    B, k, V, d = wl.batch, wl.k, wl.dims.vocab, wl.dims.d
    ids, hidden, cu = hi.make_prompt(wl)
    lens = np.diff(cu).astype(np.int64)
    resid = hi.make_residuals(wl)
    dr = Drafter(wl.dims, weights.get(wl), max_batch=B, max_len=int(lens.max()) + rounds * (k + 1) + 8, max_k=8)
    if tc_prefill_min:
        dr.set_tc_prefill(tc_prefill_min)
    d_resid = to_dev(resid, wl.dims.dtype)
    dr.prefill(torch.from_numpy(ids).cuda(), to_dev(hidden, wl.dims.dtype), [int(x) for x in cu], resid0=d_resid[0])
    rng = np.random.default_rng(wl.seed + 99)
    base_logits = to_dev(rng.standard_normal((B, k + 1, V)).astype(np.float32), wl.logits_dtype)
    pool = to_dev(rng.standard_normal((B * (k + 1) * 4, d)).astype(np.float32), wl.dims.dtype)   # "true" features to draw from
    pw = 0.75 ** np.arange(k + 1); pw /= pw.sum()
    out_ids = torch.empty((B, k), dtype=torch.int32, device="cuda")
    rows_b = torch.arange(B, device="cuda")[:, None]
    cols_k = torch.arange(k + 1, device="cuda")[None, :]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_draft, t_verify, t_refresh, committed = [], [], [], 0
    T = lens.copy()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for r in range(rounds):
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record()
        dr.draft(B, k, d_resid, out_ids=out_ids)
        e1.record()
        # the toy target (not timed as drafter work, but inside the wall clock): its logits agree with the first n drafted
        # tokens of every sequence and disagree at position n
        n_plant = torch.from_numpy(rng.choice(k + 1, size=B, p=pw)).cuda()
        logits = base_logits.clone()
        idx = torch.cat([out_ids.long(), out_ids[:, -1:].long()], 1)                       # [B, k+1] (last column unused)
        bump = torch.where(cols_k < n_plant[:, None], 12.0, torch.where(cols_k == n_plant[:, None], -12.0, 0.0))
        bump[:, k] = 0.0
        logits[rows_b, cols_k, idx] = (logits[rows_b, cols_k, idx].float() + bump).to(logits.dtype)
        torch.cuda.current_stream().synchronize()
        e1b = ev(); e1b.record()
        acc, nxt, kv = dr.verify(out_ids, logits)
        e2.record()
        n = acc.cpu().numpy().astype(np.int64)                                             # the host learns the outcome
        nx = nxt.cpu().numpy()
        oi = out_ids.cpu().numpy()
        new_ids = np.concatenate([np.concatenate([oi[b, :n[b]], nx[b:b + 1]]) for b in range(B)]).astype(np.int32)
        cu_new = np.concatenate([[0], np.cumsum(n + 1)]).astype(np.int32)
        off = int(rng.integers(0, pool.shape[0] - int(cu_new[-1])))
        dr.prefill(torch.from_numpy(new_ids).cuda(), pool[off:off + int(cu_new[-1])], [int(x) for x in cu_new],
                   start_pos=[int(t) for t in T], resid0=d_resid[0])
        e3.record()
        torch.cuda.synchronize()
        T += n + 1
        committed += int((n + 1).sum())
        if r >= 3:
            t_draft.append(e0.elapsed_time(e1)); t_verify.append(e1b.elapsed_time(e2)); t_refresh.append(e2.elapsed_time(e3))
    wall = time.perf_counter() - t0
    dr.status()
    dr.close()
    us = lambda xs: round(float(np.median(xs)) * 1e3, 1)
    side = us(t_draft) + us(t_verify) + us(t_refresh)
    tau = committed / (rounds * B)
    return {"workload": wl.name, "batch": B, "k": k, "rounds": rounds, "planted_accept_law": "P(n) ~ 0.75^n, n = 0..k",
            "tokens_per_round_and_sequence": round(tau, 3), "draft_us": us(t_draft), "verify_us": us(t_verify),
            "refresh_us": us(t_refresh), "refresh_includes": "D2H of the outcome, host packing, H2D of the new ids",
            "drafter_side_us_per_round": round(side, 1),
            "committed_tokens_per_s_of_drafter_time": round(B * tau / (side * 1e-6), 1),
            "wall_ms_per_round_with_toy_target": round(wall / rounds * 1e3, 3),
            "tc_prefill_min_pairs": tc_prefill_min or "default"}


def stub_replica(rank: int) -> dict:
    """Stands in for the device work when HIVIS_BENCH_STUB=1 (CPU test of the launch path only): fixed fake
    times, rank 1 slower.  The line it leads to is marked as a stub and carries no measurement."""
    return {"total_ms": 10.0 + 5.0 * rank}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, help="time this workload only (default: batch 1, then batch 16)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--l2-keep", type=lambda x: int(x, 0), default=0,
                    help="mask of weight matrices the tensor-core chain kernel asks L2 to keep (HIVIS_OPT_L2_KEEP; study aid)")
    ap.add_argument("--prefill-ablation", action="store_true",
                    help="time the prefix build with 0 / 576 / 2048 leading (visual stand-in) positions and exit")
    ap.add_argument("--tree-and-sampling", action="store_true",
                    help="time tree drafting + tree verification (one sequence) and speculative-sampling verification (batch 16)")
    ap.add_argument("--loop", action="store_true",
                    help="draft -> verify -> refresh rounds at batch 16 against a toy target with planted accept lengths")
    ap.add_argument("--tc-prefill-min", type=int, default=0, help="with --loop: smallest prefill call (pairs) on the tensor-core path")
    ap.add_argument("--phase-times", action="store_true",
                    help="print where a draft step of the tensor-core chain kernel goes (its own time stamps) and exit")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "ours":
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))          # one process per GPU; rank 0 prints the line
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "ours" and world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but {world} rank(s) were started: refusing to report replicas that did not run")
    wl = hi.workload(args.workload or HEADLINE)
    config = workload_config(wl, world)

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        warm = max(1, min(args.warmup, 1))
        cb = run_oracle_sample(wl, steps, warm)
        line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": steps, "warmup": warm, "ms_per_step": cb["ms_per_bench_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
                "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    stub = os.environ.get("HIVIS_BENCH_STUB") == "1"
    if stub:
        import torch.distributed as dist
        if world > 1:
            dist.init_process_group("gloo", rank=rank, world_size=world)
        slowest = max_over_ranks(stub_replica(rank)["total_ms"], dist if world > 1 else None, "cpu")
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "data": "stub (no device work: launch-path test)", "config": config,
                              "stub_slowest_ms": slowest}))
        if world > 1:
            dist.destroy_process_group()
        return

    import torch
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    wl = replica_workload(wl, rank, world)                 # independent replicas, same shapes
    weights = WeightCache()
    if args.prefill_ablation:
        print(json.dumps(prefill_ablation()))
        return
    if args.tree_and_sampling:
        print(json.dumps(tree_and_sampling(weights)))
        return
    if args.loop:
        print(json.dumps(draft_verify_refresh_loop(weights, tc_prefill_min=args.tc_prefill_min)))
        return
    if args.phase_times:
        print(json.dumps(phase_breakdown(hi.workload(args.workload or BATCH16), weights)))
        return
    res = time_workload(wl, args.steps, args.warmup, rank, local_rank, world, dist, weights, not args.no_e2e,
                        l2_keep=args.l2_keep)
    if args.l2_keep:
        config["l2_keep_mask"] = args.l2_keep

    extra = {}
    if args.workload is None:
        # the batch-16 half of the metric, and the visual-token-hiding pair (text-only cache vs naive cache)
        w16 = replica_workload(hi.workload(BATCH16), rank, world)
        r16 = time_workload(w16, args.steps, args.warmup, rank, local_rank, world, dist, weights, not args.no_e2e)
        r16["config"] = workload_config(w16, world)
        wnv = replica_workload(hi.workload(BATCH16_NAIVE), rank, world)
        rnv = time_workload(wnv, min(args.steps, 100), args.warmup, rank, local_rank, world, dist, weights, False,
                            short=True)
        a, b = r16["draft_chain"], rnv["draft_chain"]
        extra["batch16"] = r16
        extra["batch16_naive_kv"] = {
            "workload": wnv.name, "leading_positions": wnv.leading_positions,
            "us_per_draft_step": b["us_per_draft_step_median"], "GBps": b["GBps"], "frac_of_peak": b["frac_of_peak"],
            "algorithmic_bytes_per_draft_step": b["algorithmic_bytes_per_draft_step"],
            "roofline_frac": rnv["roofline"]["frac"], "kernel_us_per_launch": rnv["roofline"]["per_kernel"].get("draft_chain", {}).get("us"),
            "text_only_us_per_draft_step": a["us_per_draft_step_median"],
            "naive_over_text_only": round(b["us_per_draft_step_median"] / a["us_per_draft_step_median"], 4),
            "verify_matches_planted": rnv["verify_matches_planted"]}
    weights = None

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        torch.cuda.empty_cache()
        cb = run_oracle_sample(wl, 3, 1)
        cpu_baseline = {k_: cb[k_] for k_ in ("value", "unit", "cores", "kind", "sample")}
        cpu_baseline["us_per_step"] = round(cb["us_per_step"], 1)

    if rank == 0:
        D = wl.dims
        line = {"metric": METRIC, "value": res["value"], "unit": UNIT,
                "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate" if D.dtype == "bf16" else "f32",
                "data": "synthetic", "config": config, "clocks": res["clocks"], "e2e": res["e2e"],
                "gpu_launches": res["gpu_launches"], "roofline": res["roofline"], "cpu_baseline": cpu_baseline,
                "draft_chain": res["draft_chain"], "verify_matches_planted": res["verify_matches_planted"]}
        line.update(extra)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
