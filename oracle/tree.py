"""Tree drafting and greedy tree verification on the CPU.  TEST INFRASTRUCTURE ONLY (see the package header).

The paper drafts with the dynamic draft tree of EAGLE-2 (Sec. 2.1, last paragraph) and states its shape
under "Inference Setup": a top-10 tree expanded to depth 6, of which the 60 paths with the highest
cumulative probability are kept (the variant of the supplementary material: 8 per expansion, depth 4,
30 kept).  The steps below are that procedure written out on top of the oracle's one-position layer
(`Oracle.position`, which is pinned on its own): nothing is blocked, fused or reordered.

  level 0      the pending pair (target feature, token) runs through the layer at the next cache row P;
               its output distribution gives the `topk` candidates of depth 1.
  level l>=1   the `topk` candidates of depth l with the highest cumulative log-probability (the frontier)
               each run through the layer at position P + l: input = (layer output of the forward that
               proposed the node, the node's token), residual row min(l, R-1) as in chained drafting
               ("Training Setup"), attention over the prefix, the node's ancestors and itself (tree
               attention).  Each yields `topk` candidates of depth l + 1 with
               score = score(parent) + log-softmax(logits)[token].
  after `depth` levels every candidate ever proposed is ranked by score and the best `keep` are the draft
  tree.  A child's score never exceeds its parent's, and equal scores are ordered by creation, so the kept
  set is closed under "parent of".

Order of equal values everywhere: the candidate created first wins (level by level, parents in frontier
order, children by rank); among equal logits the lower token id ranks first.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np


def log_softmax(x: np.ndarray) -> np.ndarray:
    """x - logsumexp(x) with the maximum taken out first."""
    x = np.asarray(x, np.float64)
    m = x.max()
    return x - m - np.log(np.exp(x - m).sum())


def top_k(x: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest values, largest first; among equal values the lower index first."""
    x = np.asarray(x)
    order = np.lexsort((np.arange(x.size), -x))
    return order[:k]


@dataclass
class DraftTree:
    """Kept nodes in creation order (parents before children)."""
    tokens: np.ndarray            # [n] int32
    parents: np.ndarray           # [n] int32 index into this list, -1 = child of the root
    depths: np.ndarray            # [n] int32, 1-based
    scores: np.ndarray            # [n] float64 cumulative log-probability
    expanded: np.ndarray          # [n] bool: the node ran through the layer (it has a K/V row)
    k_rows: List[np.ndarray] = field(default_factory=list)   # per kept node: its K row (None if not expanded)
    v_rows: List[np.ndarray] = field(default_factory=list)
    root_k: np.ndarray = None     # K/V row of the root position (row P of the cache)
    root_v: np.ndarray = None
    n_cached: int = 0
    margin: float = np.inf        # smallest gap between neighbours in any ranking that decided the tree's shape or order:
                                  # an implementation whose scores are off by less than half of it builds the same tree


def tree_draft(o, n_cached: int, pend_id: int, pend_hidden, rho, Kc, Vc, topk: int, depth: int, keep: int) -> DraftTree:
    """Kc, Vc hold rows [0, n_cached); they are not modified (row n_cached is returned as root_k / root_v)."""
    lm = o._keep["lm_head"].astype(o.rt)
    R = rho.shape[0]
    P = n_cached
    kvw = o.kvw

    def forward(feature, token, level, anc_k, anc_v):
        """One node through the layer at position P + level, attending to the prefix and the given ancestor rows."""
        kc = np.zeros((P + level + 1, kvw), o.rt)
        vc = np.zeros((P + level + 1, kvw), o.rt)
        kc[:P], vc[:P] = Kc[:P], Vc[:P]
        for j, (kr, vr) in enumerate(zip(anc_k, anc_v)):
            kc[P + j], vc[P + j] = kr, vr
        g = o.position(feature, int(token), rho[min(level, R - 1)], P + level, kc, vc)
        return g, kc[P + level].copy(), vc[P + level].copy(), log_softmax(lm @ g)

    margin = [np.inf]

    def note_gaps(values_sorted_desc):
        v = np.asarray(values_sorted_desc, np.float64)
        if v.size > 1:
            margin[0] = min(margin[0], float(np.min(v[:-1] - v[1:])))

    # candidate list (creation order)
    tok, par, dep, sc = [], [], [], []
    exp_k, exp_v = {}, {}                                   # candidate index -> its K/V row once expanded
    g_root, rk, rv, lp = forward(np.asarray(pend_hidden, o.rt), pend_id, 0, [], [])
    frontier = []                                           # (candidate index, feature to feed with it)
    note_gaps(lp[top_k(lp, topk + 1)])
    for t in top_k(lp, topk):
        tok.append(int(t)); par.append(-1); dep.append(1); sc.append(float(lp[t]))
        frontier.append((len(tok) - 1, g_root))
    for level in range(1, depth):
        children = []                                       # (score, creation order) of this level's new candidates
        for ci, feat in frontier:
            chain = []                                      # ancestors of ci, root side first
            a = ci
            while a >= 0:
                chain.append(a)
                a = par[a]
            chain = chain[::-1][:-1]
            anc_k = [rk] + [exp_k[a] for a in chain]
            anc_v = [rv] + [exp_v[a] for a in chain]
            g, kr, vr, lp = forward(feat, tok[ci], level, anc_k, anc_v)
            exp_k[ci], exp_v[ci] = kr, vr
            note_gaps(lp[top_k(lp, topk + 1)])
            for t in top_k(lp, topk):
                tok.append(int(t)); par.append(ci); dep.append(level + 1); sc.append(sc[ci] + float(lp[t]))
                children.append((len(tok) - 1, g))
        if level + 1 < depth:
            note_gaps(sorted((sc[c[0]] for c in children), reverse=True)[:topk + 1])
            order = sorted(range(len(children)), key=lambda i: (-sc[children[i][0]], children[i][0]))[:topk]
            frontier = [children[i] for i in sorted(order)]          # frontier kept in creation order
    n_all = len(tok)
    note_gaps(sorted(sc, reverse=True)[:keep + 1])
    ranked = sorted(range(n_all), key=lambda i: (-sc[i], i))[:min(keep, n_all)]
    kept = sorted(ranked)
    pos = {c: i for i, c in enumerate(kept)}
    for c in kept:
        assert par[c] < 0 or par[c] in pos, "a kept node lost its parent"
    return DraftTree(
        tokens=np.array([tok[c] for c in kept], np.int32),
        parents=np.array([pos[par[c]] if par[c] >= 0 else -1 for c in kept], np.int32),
        depths=np.array([dep[c] for c in kept], np.int32),
        scores=np.array([sc[c] for c in kept], np.float64),
        expanded=np.array([c in exp_k for c in kept], bool),
        k_rows=[exp_k.get(c) for c in kept], v_rows=[exp_v.get(c) for c in kept],
        root_k=rk, root_v=rv, n_cached=P, margin=margin[0])


def tree_verify(tree: DraftTree, target_logits: np.ndarray):
    """Greedy verification of a draft tree (Sec. 2.1: the target keeps the draft tokens it would have produced
    itself and replaces the first that differs).  target_logits [n + 1, V]: row 0 is the target's prediction after
    the root token, row 1 + i its prediction after the path that ends in kept node i.  Returns (n_accepted, path as
    kept-node indices, next token, cache rows to keep)."""
    logits = np.asarray(target_logits, np.float32)
    cur, path = -1, []
    while True:
        t = int(np.argmax(logits[cur + 1]))                 # first maximum
        nxt = [i for i in range(tree.tokens.size) if tree.parents[i] == cur and tree.tokens[i] == t]
        if not nxt:
            break
        cur = nxt[0]
        path.append(cur)
    with_rows = 0
    for i in path:                                          # expanded nodes form a prefix of any path
        if tree.expanded[i]:
            with_rows += 1
    return len(path), path, t, tree.n_cached + 1 + with_rows


def tree_commit(tree: DraftTree, path, Kc, Vc) -> int:
    """KV compaction: the root's row and the rows of the accepted nodes that have one, in path order, right after the
    prefix.  Returns the new row count."""
    P = tree.n_cached
    Kc[P], Vc[P] = tree.root_k, tree.root_v
    n = P + 1
    for i in path:
        if not tree.expanded[i]:
            break
        Kc[n], Vc[n] = tree.k_rows[i], tree.v_rows[i]
        n += 1
    return n
