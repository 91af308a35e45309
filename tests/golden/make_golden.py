"""Writes tests/golden/c1_tiny_oracle.json from the CPU oracle alone (never from the CUDA path).

The paper prints no worked numeric example, so this file is not a paper value: it freezes what
the pinned fp64 oracle gives on the tiny fp32 workload, so that a later edit of the oracle's
arithmetic shows up as a diff.  Run:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import hivis_inputs as hi  # noqa: E402
import oracle  # noqa: E402


def main():
    wl = hi.workload("c1_tiny_f32_b1")
    W = hi.make_weights(wl.dims, wl.seed)
    ids, hid, cu = hi.make_prompt(wl)
    r = hi.make_residuals(wl)
    o = oracle.Oracle(wl.dims, W, "f64")
    out = o.run_batch(ids, hid, cu, wl.k, r)[0]
    logits, planted = hi.make_target_logits(wl, out["ids"][None])
    n, nxt, kv = o.verify(out["ids"], logits[0], out["T"])
    doc = {
        "workload": wl.name,
        "draft_ids": [int(t) for t in out["ids"]],
        "top2_gap": [float(g) for g in out["gaps"]],
        "logits_head": [[float(x) for x in row[:8]] for row in out["logits"]],
        "logits_abs_sum": [float(np.abs(row).sum()) for row in out["logits"]],
        "planted_accept": int(planted[0]), "accept": n, "next": nxt, "kv_len": kv,
    }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_tiny_oracle.json")
    with open(path, "w") as fh:
        json.dump(doc, fh, indent=1)
        fh.write("\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
