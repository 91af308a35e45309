"""GPU parity of tree drafting and tree verification against the oracle (oracle/tree.py), through the C ABI."""
import numpy as np
import pytest

import hivis_inputs as hi
from oracle import tree as ot
from tests.harness import Case, to_dev

pytestmark = pytest.mark.gpu


def oracle_tree(case, b, topk, depth, keep):
    o = case.oracle
    lo, hi_ = int(case.cu[b]), int(case.cu[b + 1])
    T = hi_ - lo
    rho = o.fold_residuals(case.resid)
    Kc, Vc = o.new_cache(T + depth + 2)
    o.prefill(case.ids[lo:hi_], case.hidden[lo:hi_], rho[0], Kc, Vc)
    tr = ot.tree_draft(o, T - 1, int(case.ids[hi_ - 1]), case.hidden[hi_ - 1], rho, Kc, Vc, topk, depth, keep)
    return tr, Kc, Vc, rho, T


def gpu_tree(case, b, topk, depth, keep):
    t = case.torch
    tok, par, sc, cnt = case.drafter.draft_tree(b, topk, depth, keep, case.d_resid)
    t.cuda.synchronize()
    n = int(cnt[0])
    return tok.cpu().numpy()[:n], par.cpu().numpy()[:n], sc.cpu().numpy()[:n], n


def path_of(par, i):
    out = []
    while i >= 0:
        out.append(i)
        i = int(par[i])
    return out[::-1]


def check_tree_is_well_formed(tok, par, topk, depth, vocab):
    n = tok.size
    dep = np.zeros(n, int)
    for i in range(n):
        assert -1 <= par[i] < i, f"node {i}: parent {par[i]} does not precede it"
        dep[i] = 1 if par[i] < 0 else dep[par[i]] + 1
        assert 0 <= tok[i] < vocab
    assert (dep <= depth).all() and (np.diff(dep) >= 0).all()
    for p in set(par.tolist()):
        sib = tok[par == p]
        assert len(set(sib.tolist())) == sib.size and sib.size <= topk
    return dep


def check_scores_along_paths(case, b, tok, par, sc, depth, tol_per_level):
    """Every node's score against the oracle's chain run along the node's own token path (whatever tree the oracle
    itself would have built): the cumulative log-probability of those tokens."""
    o = case.oracle
    lo, hi_ = int(case.cu[b]), int(case.cu[b + 1])
    T = hi_ - lo
    rho = o.fold_residuals(case.resid)
    leaves = [i for i in range(tok.size) if not (par == i).any()]
    worst = 0.0
    for leaf in leaves:
        p = path_of(par, leaf)
        toks = [int(tok[i]) for i in p]
        Kc, Vc = o.new_cache(T + len(toks) + 1)
        o.prefill(case.ids[lo:hi_], case.hidden[lo:hi_], rho[0], Kc, Vc)
        ref = o.draft(T - 1, int(case.ids[hi_ - 1]), case.hidden[hi_ - 1], len(toks), rho, Kc, Vc,
                      forced_ids=np.array(toks, np.int32))
        cum = 0.0
        for s_, i in enumerate(p):
            cum += ot.log_softmax(ref["logits"][s_])[toks[s_]]
            err = abs(float(sc[i]) - cum)
            worst = max(worst, err)
            assert err <= tol_per_level * (s_ + 1), f"node {i} (depth {s_ + 1}): score {sc[i]} vs {cum}"
    return worst


CASES = [  # workload, sequence, topk, depth, keep
    ("c1_tiny_f32_b1", 0, 4, 4, 20),
    ("tiny_f32_b4_ragged", 2, 10, 6, 60),            # the paper's shape of tree: top-10, depth 6, 60 kept
    ("tiny_f32_b4_ragged", 0, 8, 4, 30),             # the variant of the supplementary material
    ("mini_mha_b1", 0, 10, 6, 60),
    ("mini_gqa_b3", 1, 8, 4, 30),
    ("gqa4_b5_ragged", 3, 5, 3, 12),
    ("mini_mha_b5_ragged", 4, 1, 6, 6),              # one branch: a chain
    ("mini_mha_b5_ragged", 2, 16, 2, 256),           # widest level, more room than candidates
    ("mini_mha_b1", 0, 3, 1, 3),                     # depth 1: the root's proposals only
    ("c2_llava_b1", 0, 10, 6, 60),                   # full size, the configuration bench.py --tree-and-sampling times
]


@pytest.mark.parametrize("name,b,topk,depth,keep", CASES)
def test_tree_draft_and_verify_parity(name, b, topk, depth, keep):
    run_tree_parity(name, b, topk, depth, keep, True)


@pytest.mark.parametrize("name,b,topk,depth,keep", [("mini_mha_b1", 0, 10, 6, 60), ("mini_gqa_b3", 1, 8, 4, 30)])
def test_tree_parity_with_the_per_phase_kernels(name, b, topk, depth, keep):
    """bf16 drafters run the levels in the tensor-core chain kernel by default; with that kernel switched off the
    per-phase kernels must build the tree to the same bar."""
    run_tree_parity(name, b, topk, depth, keep, False)


def run_tree_parity(name, b, topk, depth, keep, tc):
    import torch
    wl = hi.workload(name)
    case = Case(wl, max_len=int(np.diff(hi.make_prompt(wl)[2]).max()) + 1 + depth * topk + 8, max_k=16)
    try:
        f32 = wl.dims.dtype == "f32"
        if not tc:
            case.drafter.set_tc_kernel(False)
        case.gpu_prefill()
        tok, par, sc, n = gpu_tree(case, b, topk, depth, keep)
        case.drafter.status()
        tr, Kc, Vc, rho, T = oracle_tree(case, b, topk, depth, keep)
        assert n == tr.tokens.size == min(keep, topk + (depth - 1) * topk * topk)
        dep = check_tree_is_well_formed(tok, par, topk, depth, wl.dims.vocab)
        tol = 2e-4 if f32 else 3e-2                  # per level: fp32 accumulation / bf16 storage of weights and cache
        worst = check_scores_along_paths(case, b, tok, par, sc, depth, tol)
        same = tr.margin > 2 * max(worst, 1e-6)      # the oracle's rankings were decided by more than the observed error
        print(f"{name}[{b}] top{topk} depth{depth} keep{keep}: worst score error {worst:.2e}, oracle margin {tr.margin:.2e}, "
              f"{'identical tree required' if same else 'near-tie: own tree checked'}")
        if same:
            np.testing.assert_array_equal(tok, tr.tokens)
            np.testing.assert_array_equal(par, tr.parents)
            np.testing.assert_array_equal(dep, tr.depths)
            np.testing.assert_allclose(sc, tr.scores, atol=tol * depth)
        else:                                        # a near-tie somewhere: the GPU's own tree stands in (it is well formed and
            tr = None                                # its scores are the oracle's along its paths), shapes may differ
        # ---- verification: the target accepts the deepest kept path; then one where it rejects at once
        V = wl.dims.vocab
        leaf = int(np.argmax(dep))
        path = path_of(par, leaf)
        other = [t for t in range(V) if t not in set(tok.tolist())][0]
        rng = np.random.default_rng(5)
        logits = rng.standard_normal((n + 1, V)).astype(np.float32)
        logits[0, tok[path[0]]] = 15.0
        for a, c_ in zip(path[:-1], path[1:]):
            logits[1 + a, tok[c_]] = 15.0
        logits[1 + leaf, other] = 15.0
        logits = hi.round_to_bf16(logits) if wl.logits_dtype == "bf16" else logits
        acc, gpath, nxt, kv = case.drafter.verify_tree(b, depth, to_dev(logits, wl.logits_dtype))
        torch.cuda.synchronize()
        acc, nxt, kv = int(acc[0]), int(nxt[0]), int(kv[0])
        gpath = gpath.cpu().numpy()[:depth]
        assert acc == len(path) and list(gpath[:acc]) == path and (gpath[acc:] == -1).all() and nxt == other
        if tr is not None:
            o_acc, o_path, o_next, o_rows = ot.tree_verify(tr, logits)
            assert (acc, list(gpath[:acc]), nxt, kv) == (o_acc, o_path, o_next, o_rows)
            assert case.drafter.kv_len(b)[0] == o_rows
            rows = ot.tree_commit(tr, o_path, Kc, Vc)
            k_g, v_g = case.drafter.read_kv(b, 0, rows)
            torch.cuda.synchronize()
            for got, want in ((k_g, Kc[:rows]), (v_g, Vc[:rows])):
                e = np.abs(got.cpu().numpy() - want).max() / np.abs(want).max()
                assert e <= (1e-4 if f32 else 1e-2), f"compacted cache: rel err {e}"
        else:
            assert T <= kv <= T + acc
    finally:
        case.close()


def test_tree_verify_rejects_everything_and_state_errors():
    import torch
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload("mini_mha_b1")
    case = Case(wl, max_len=120, max_k=8)
    try:
        dr = case.drafter
        with pytest.raises(HivisError) as e:                     # no pending pair yet
            dr.draft_tree(0, 4, 3, 10, case.d_resid)
        assert e.value.code == -4
        case.gpu_prefill()
        for bad in ((17, 3, 10), (4, 9, 10), (4, 3, 257), (0, 3, 10)):
            with pytest.raises(HivisError) as e:
                dr.draft_tree(0, *bad, case.d_resid)
            assert e.value.code == -5
        logits0 = torch.zeros((11, wl.dims.vocab), device="cuda")
        with pytest.raises(HivisError) as e:                     # nothing to verify
            dr.verify_tree(0, 3, logits0)
        assert e.value.code == -4
        tok, par, sc, cnt = dr.draft_tree(0, 4, 3, 10, case.d_resid)
        torch.cuda.synchronize()
        T = int(case.lens[0])
        assert dr.kv_len(0)[0] == T - 1                          # the tree does not move the row count
        taken = set(tok.cpu().numpy().tolist())
        other = [t for t in range(wl.dims.vocab) if t not in taken][0]
        logits0[:, other] = 3.0
        acc, path, nxt, kv = dr.verify_tree(0, 3, logits0)
        torch.cuda.synchronize()
        assert (int(acc[0]), int(nxt[0]), int(kv[0])) == (0, other, T) and (path.cpu().numpy()[:3] == -1).all()
        with pytest.raises(HivisError) as e:                     # the tree was consumed
            dr.verify_tree(0, 3, logits0)
        assert e.value.code == -4
    finally:
        case.close()
