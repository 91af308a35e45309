"""Pins for the oracle's tree drafting and tree verification (oracle/tree.py).  Nothing here touches the CUDA path.

The procedure follows the paper's statement of its draft tree (Sec. 2.1: the tree of EAGLE-2; "Inference Setup":
top-10, depth 6, 60 kept by cumulative probability).  Each test ties it to something else: library routines, the
pinned chain drafter run once per path, brute-force enumeration of every path of a small tree, the losslessness
of greedy verification."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import tree as ot
from tests.test_oracle_pins import rand_weights, small_dims


def setup(seed=0, T=5, room=12, **kw):
    dims = small_dims(d=24, n_q_heads=4, n_kv_heads=2, head_dim=6, ffn=20, vocab=31, **kw)
    W = rand_weights(dims, seed=60 + seed, scale=0.5, bias=True)
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(70 + seed)
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((3, dims.d)).astype(np.float32)
    rho = o.fold_residuals(resid)
    Kc, Vc = o.new_cache(T + room)
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    return dims, W, o, ids, hidden, rho, Kc, Vc


def chain(o, ids, hidden, rho, forced, k):
    """The pinned chain drafter on a fresh cache, teacher-forced along `forced`."""
    T = len(ids)
    Kc, Vc = o.new_cache(T + k + 1)
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    f = np.array(list(forced) + [0] * (k - len(forced)), np.int32) if len(forced) else None
    out = o.draft(T - 1, int(ids[-1]), hidden[-1], k, rho, Kc, Vc, forced_ids=f)
    return out, Kc, Vc


def test_log_softmax_and_top_k_against_library_routines():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(200) * 5
    np.testing.assert_allclose(ot.log_softmax(x), torch.log_softmax(torch.from_numpy(x), 0).numpy(), rtol=1e-13, atol=1e-13)
    big = np.array([1000.0, 999.0, -1000.0])
    assert np.isfinite(ot.log_softmax(big)).all() and abs(np.exp(ot.log_softmax(big)).sum() - 1) < 1e-12
    y = rng.integers(0, 6, 50).astype(np.float64)                       # many ties
    got = ot.top_k(y, 9)
    want = sorted(range(50), key=lambda i: (-y[i], i))[:9]
    assert list(got) == want
    assert list(ot.top_k(np.array([1.0, 3.0, 3.0, 2.0]), 3)) == [1, 2, 3]


def test_a_tree_with_one_branch_is_chained_drafting():
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(0)
    T, depth = len(ids), 5
    tr = ot.tree_draft(o, T - 1, int(ids[-1]), hidden[-1], rho, Kc, Vc, topk=1, depth=depth, keep=depth)
    ref, Kr, Vr = chain(o, ids, hidden, rho, [], depth)
    np.testing.assert_array_equal(tr.tokens, ref["ids"])
    assert list(tr.parents) == [-1, 0, 1, 2, 3] and list(tr.depths) == [1, 2, 3, 4, 5]
    lp = [ot.log_softmax(ref["logits"][s])[ref["ids"][s]] for s in range(depth)]
    np.testing.assert_allclose(tr.scores, np.cumsum(lp), rtol=1e-12, atol=1e-12)
    assert list(tr.expanded) == [True] * (depth - 1) + [False]            # the last token never ran through the layer
    np.testing.assert_allclose(tr.root_k, Kr[T - 1], rtol=1e-12, atol=1e-13)
    for j in range(depth - 1):
        np.testing.assert_allclose(tr.k_rows[j], Kr[T + j], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(tr.v_rows[j], Vr[T + j], rtol=1e-12, atol=1e-13)


def test_tree_attention_equals_running_every_path_as_its_own_chain():
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(1)
    T = len(ids)
    tr = ot.tree_draft(o, T - 1, int(ids[-1]), hidden[-1], rho, Kc, Vc, topk=3, depth=4, keep=25)
    assert tr.tokens.size == 25 and (tr.depths <= 4).all() and (np.diff(tr.depths) >= 0).all()
    for i in range(tr.tokens.size):
        path = []
        a = i
        while a >= 0:
            path.append(a)
            a = tr.parents[a]
        path = path[::-1]
        toks = [int(tr.tokens[a]) for a in path]
        ref, Kr, Vr = chain(o, ids, hidden, rho, toks, len(toks) + 1)      # one step more: the node's own forward
        lp = sum(ot.log_softmax(ref["logits"][s])[toks[s]] for s in range(len(toks)))
        assert abs(tr.scores[i] - lp) < 1e-10, f"node {i}"
        if tr.expanded[i]:                                              # its K/V row is the chain's row at that position
            np.testing.assert_allclose(tr.k_rows[i], Kr[T - 1 + len(toks)], rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(tr.v_rows[i], Vr[T - 1 + len(toks)], rtol=1e-11, atol=1e-12)
    # every kept node's parent is kept and precedes it; siblings carry different tokens
    for i in range(tr.tokens.size):
        assert tr.parents[i] < i
        assert tr.depths[i] == (1 if tr.parents[i] < 0 else tr.depths[tr.parents[i]] + 1)
    for p in set(tr.parents.tolist()):
        sib = tr.tokens[tr.parents == p]
        assert len(set(sib.tolist())) == sib.size


@pytest.mark.parametrize("seed,keep", [(2, 6), (3, 10), (4, 3)])
def test_small_tree_against_enumeration_of_every_path(seed, keep):
    """top-2, depth 3: all 2 + 4 + 8 paths are scored by brute force (one chain run each); the frontier of each level
    and the kept set follow from those scores by plain sorting."""
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(seed)
    T, K, depth = len(ids), 2, 3
    tr = ot.tree_draft(o, T - 1, int(ids[-1]), hidden[-1], rho, Kc, Vc, topk=K, depth=depth, keep=keep)

    def children(prefix):
        """top-K continuations of a path and their log-probabilities, from a chain run along the path"""
        ref, _, _ = chain(o, ids, hidden, rho, prefix, len(prefix) + 1)
        lp = ot.log_softmax(ref["logits"][len(prefix)])
        order = sorted(range(lp.size), key=lambda t: (-lp[t], t))[:K]
        return [(t, lp[t]) for t in order]

    cands = []                                       # (path tokens, score) in creation order
    level = [((t,), s) for t, s in children(())]
    cands += level
    frontier = level
    for d in range(2, depth + 1):
        new = []
        for path, s in frontier:
            new += [(path + (t,), s + l) for t, l in children(path)]
        cands += new
        best = sorted(range(len(new)), key=lambda i: (-new[i][1], i))[:K]
        frontier = [new[i] for i in sorted(best)]
    ranked = sorted(range(len(cands)), key=lambda i: (-cands[i][1], i))[:keep]
    want = [cands[i] for i in sorted(ranked)]
    assert tr.tokens.size == len(want) == min(keep, 2 + 4 + 4)
    for i, (path, s) in enumerate(want):
        got_path = []
        a = i
        while a >= 0:
            got_path.append(int(tr.tokens[a]))
            a = tr.parents[a]
        assert tuple(got_path[::-1]) == path
        assert abs(tr.scores[i] - s) < 1e-10


def toy_target(prefix_tokens, vocab):
    """A fixed function of the token prefix: what a deterministic greedy target would emit next."""
    h = 17
    for t in prefix_tokens:
        h = (h * 31 + int(t) + 7) % 1000003
    return h % vocab


def test_greedy_tree_verification_reproduces_the_target_stream():
    """Losslessness: whatever the drafter proposes, accepted tokens + the target's own token are the target's greedy
    stream.  The toy target is rigged to agree with the drafter's best child most of the time so that paths of
    several tokens get accepted."""
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(5, T=4, room=48)
    V = dims.vocab
    rng = np.random.default_rng(9)
    text = [int(t) for t in ids]                     # token history the toy target conditions on
    T = len(ids)
    pend_id, pend_h = int(ids[-1]), hidden[-1]
    lens = []
    for rnd in range(6):
        tr = ot.tree_draft(o, T - 1, pend_id, pend_h, rho, Kc, Vc, topk=3, depth=4, keep=12)
        n = tr.tokens.size

        def target_after(path_tokens):
            kids = [int(tr.tokens[i]) for i in range(n) if _path(tr, i)[:-1] == list(path_tokens)]
            t = toy_target(text + list(path_tokens), V)
            if kids and (t % 4) != 0:                # agree with the first proposed child three times out of four
                t = kids[0]
            return t
        logits = rng.standard_normal((n + 1, V)).astype(np.float32)
        want_stream, cur = [], []
        logits[0, target_after([])] = 20.0
        for i in range(n):
            logits[1 + i, target_after(_path(tr, i))] = 20.0
        while True:                                  # the target's own greedy walk
            t = target_after(cur)
            want_stream.append(t)
            if not any(_path(tr, i) == cur + [t] for i in range(n)):
                break
            cur = cur + [t]
        acc, path, nxt, rows = ot.tree_verify(tr, logits)
        got_stream = [int(tr.tokens[i]) for i in path] + [nxt]
        assert got_stream == want_stream and 0 <= acc <= 4 and acc == len(want_stream) - 1
        assert rows == T - 1 + 1 + sum(bool(tr.expanded[i]) for i in path)
        lens.append(acc)
        # commit: the compacted cache is what chained drafting along the accepted tokens leaves behind
        new_rows = ot.tree_commit(tr, path, Kc, Vc)
        assert new_rows == rows
        ref, Kr, Vr = chain_from(o, Kc, Vc, T, pend_id, pend_h, rho, [int(tr.tokens[i]) for i in path])
        np.testing.assert_allclose(Kc[T - 1:rows], Kr[T - 1:rows], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(Vc[T - 1:rows], Vr[T - 1:rows], rtol=1e-10, atol=1e-12)
        # next round: the target's features for the accepted tokens arrive and refresh the rows (Eq. 2)
        new_tokens = got_stream
        new_hidden = rng.standard_normal((len(new_tokens), dims.d)).astype(np.float32)
        o.prefill(np.array([pend_id] + new_tokens, np.int32), np.concatenate([pend_h[None], new_hidden]), rho[0], Kc, Vc,
                  start_pos=T - 1)
        text += new_tokens
        T += len(new_tokens)
        pend_id, pend_h = new_tokens[-1], new_hidden[-1]
    assert max(lens) >= 2, f"the rigged target never accepted a path of two tokens: {lens}"


def _path(tr, i):
    out = []
    while i >= 0:
        out.append(int(tr.tokens[i]))
        i = tr.parents[i]
    return out[::-1]


def chain_from(o, Kc, Vc, T, pend_id, pend_h, rho, forced):
    K2, V2 = Kc.copy(), Vc.copy()
    k = len(forced) + 1
    f = np.array(list(forced) + [0], np.int32)
    out = o.draft(T - 1, pend_id, pend_h, k, rho, K2, V2, forced_ids=f)
    return out, K2, V2


def test_verification_edge_cases():
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(6)
    T = len(ids)
    tr = ot.tree_draft(o, T - 1, int(ids[-1]), hidden[-1], rho, Kc, Vc, topk=2, depth=3, keep=8)
    n, V = tr.tokens.size, dims.vocab
    other = [t for t in range(V) if t not in set(tr.tokens.tolist())][0]
    logits = np.zeros((n + 1, V), np.float32)
    logits[:, other] = 5.0                                              # the target wants a token nobody drafted
    assert ot.tree_verify(tr, logits) == (0, [], other, T)
    # a planted full-depth path: the deepest kept node and its ancestors
    leaf = int(np.argmax(tr.depths))
    path = []
    a = leaf
    while a >= 0:
        path.append(a)
        a = int(tr.parents[a])
    path = path[::-1]
    logits = np.zeros((n + 1, V), np.float32)
    logits[:, other] = 1.0
    logits[0, tr.tokens[path[0]]] = 9.0
    for a, b in zip(path[:-1], path[1:]):
        logits[1 + a, tr.tokens[b]] = 9.0
    acc, got, nxt, rows = ot.tree_verify(tr, logits)
    assert acc == len(path) == tr.depths[leaf] and got == path and nxt == other
    assert rows == T + sum(bool(tr.expanded[i]) for i in path)
    # ties in the target's row go to the lowest token id, as in chained verification
    logits = np.zeros((n + 1, V), np.float32)
    t0 = int(min(tr.tokens[tr.parents == -1]))
    assert ot.tree_verify(tr, logits)[2] == 0 or t0 == 0
