"""GPU parity of verification by speculative sampling (hivis_verify_sampled) against the oracle (oracle/sampled.py)."""
import numpy as np
import pytest

import hivis_inputs as hi
from oracle import sampled as osmp
from tests.harness import Case, to_dev

pytestmark = pytest.mark.gpu

# A uniform number closer than this to the threshold that decides its outcome is not compared: the acceptance ratio
# is a quotient of two fp32 softmax values, the draw a position in a cumulative sum of up to 150 000 fp32 masses.
MARGIN_ACCEPT = 1e-4
MARGIN_DRAW = 5e-6


@pytest.mark.parametrize("name,temperature,closeness", [
    ("mini_gqa_b16_ragged", 1.0, 0.3), ("mini_gqa_b16_ragged", 0.7, 1.5), ("mini_gqa_b3", 1.0, 0.0),
    ("mini_mha_b5_ragged", 1.3, 0.6), ("tiny_f32_b4_ragged", 1.0, 0.4),
])
def test_sampled_verification_parity(name, temperature, closeness):
    """closeness: the target's logits are the drafter's plus noise of that size (0: identical distributions, so
    every token is kept and the bonus token is drawn from p)."""
    import torch
    wl = hi.workload(name)
    case = Case(wl)
    try:
        B, k, V = wl.batch, wl.k, wl.dims.vocab
        rng = np.random.default_rng(31)
        compared = 0
        case.gpu_prefill()
        for trial in range(3):
            case.gpu_restore()
            _, dl = case.gpu_draft(k)                                   # the drafter's logits [B, k, V] fp32
            # drafted tokens: drawn from q for most positions, a uniformly random token now and then
            ids = np.zeros((B, k), np.int32)
            for b in range(B):
                for j in range(k):
                    q = osmp.softmax_t(dl[b, j], temperature)
                    ids[b, j] = rng.choice(V, p=q) if rng.random() < 0.8 else rng.integers(0, V)
            tl = np.concatenate([dl, rng.standard_normal((B, 1, V)).astype(np.float32)], 1)
            tl = tl + closeness * rng.standard_normal(tl.shape).astype(np.float32)
            tl = hi.round_to_bf16(tl) if wl.logits_dtype == "bf16" else tl.astype(np.float32)
            ua = rng.random((B, k)).astype(np.float32)
            us = rng.random(B).astype(np.float32)
            acc, nxt, kv = case.drafter.verify_sampled(torch.from_numpy(ids).cuda(), torch.from_numpy(dl).cuda(),
                                                       to_dev(tl, wl.logits_dtype), temperature,
                                                       torch.from_numpy(ua).cuda(), torch.from_numpy(us).cuda())
            torch.cuda.synchronize()
            acc, nxt, kv = acc.cpu().numpy(), nxt.cpu().numpy(), kv.cpu().numpy()
            for b in range(B):
                n, nx, kvl, margin = osmp.verify_sampled(ids[b], dl[b], tl[b], temperature, ua[b], float(us[b]), int(case.lens[b]))
                assert 0 <= acc[b] <= k and 0 <= nxt[b] < V
                assert kv[b] == int(case.lens[b]) + min(int(acc[b]), k - 1)
                assert case.drafter.kv_len(b)[0] == kv[b]
                if margin[0] > MARGIN_ACCEPT:
                    assert (int(acc[b]), int(kv[b])) == (n, kvl), f"trial {trial} seq {b} (margin {margin[0]:.1e})"
                    if margin[1] > MARGIN_DRAW:
                        assert int(nxt[b]) == nx, f"trial {trial} seq {b}: drawn token (margin {margin[1]:.1e})"
                        compared += 1
                if closeness == 0.0 and wl.logits_dtype == "f32":
                    assert acc[b] == k
        assert compared >= 0.8 * 3 * B, f"only {compared} of {3 * B} sequences were away from every threshold"
    finally:
        case.close()


def test_sampled_verification_errors():
    import torch
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload("mini_gqa_b3")
    case = Case(wl)
    try:
        B, k, V = wl.batch, wl.k, wl.dims.vocab
        ids = torch.zeros((B, k), dtype=torch.int32, device="cuda")
        dl = torch.zeros((B, k, V), device="cuda")
        tl = torch.zeros((B, k + 1, V), device="cuda")
        u = torch.zeros((B, k), device="cuda")
        with pytest.raises(HivisError) as e:                     # no draft to verify
            case.drafter.verify_sampled(ids, dl, tl, 1.0, u, u[:, 0].contiguous())
        assert e.value.code == -4
        case.gpu_prefill()
        case.gpu_draft(k, want_logits=False)
        with pytest.raises(HivisError) as e:                     # temperature must be positive
            case.drafter.verify_sampled(ids, dl, tl, 0.0, u, u[:, 0].contiguous())
        assert e.value.code == -1
        acc, nxt, kv = case.drafter.verify_sampled(ids, dl, tl, 1.0, u, u[:, 0].contiguous())
        torch.cuda.synchronize()
        assert (acc.cpu().numpy() == k).all() and (nxt.cpu().numpy() == 0).all()      # uniform vs uniform, u = 0
    finally:
        case.close()


# ------------------------------------------------------------------------------------------ drafting at T > 0
@pytest.mark.parametrize("name,temperature", [
    ("c1_tiny_f32_b1", 1.0), ("mini_mha_b1", 0.6), ("mini_mha_b5_ragged", 1.0), ("mini_gqa_b16_ragged", 0.8),
    ("gqa4_b5_ragged", 1.5), ("c2_llava_b1", 1.0),
])
def test_sampled_drafting_parity(name, temperature):
    """hivis_draft_sampled against the oracle's chain with the same uniform numbers: ids step by step (a drawn token
    may differ only where the two largest perturbed values lie closer than the logits' tolerance allows; the
    sequence is then left, later steps legitimately diverge), the unperturbed logits of every compared step, the
    appended cache rows of fully compared sequences, and on the GPU side alone: every id is the maximum of the GPU's own
    logits / T plus the noise (fp64)."""
    import torch
    from tests.harness import LOGIT_RTOL, LOGIT_RTOL_F32, row_rel_err
    wl = hi.workload(name)
    full = name.startswith("c2_")
    case = Case(wl)
    try:
        B, k, V = wl.batch, wl.k, wl.dims.vocab
        rtol = LOGIT_RTOL if wl.dims.dtype == "bf16" else LOGIT_RTOL_F32
        rng = np.random.default_rng(77)
        u = (rng.random((B, k, V)) * (1 - 2e-6) + 1e-6).astype(np.float32)
        case.gpu_prefill()
        ids_g, logits_g = case.drafter.draft_sampled(B, k, temperature, torch.from_numpy(u).cuda(), case.d_resid)
        torch.cuda.synchronize()
        case.drafter.status()
        ids_g, logits_g = ids_g.cpu().numpy(), logits_g.cpu().numpy()
        # the GPU's draw against its own logits
        z = logits_g.astype(np.float64) / temperature + osmp.gumbel(u.astype(np.float64))
        top2 = np.sort(z, axis=-1)[..., -2:]
        for b in range(B):
            for s in range(k):
                if top2[b, s, 1] - top2[b, s, 0] > 1e-4:
                    assert ids_g[b, s] == int(np.argmax(z[b, s])), f"seq {b} step {s}: not the maximum of its own perturbed logits"
        assert len(np.unique(ids_g)) > 1
        # against the oracle
        rho = case.oracle.fold_residuals(case.resid)
        compared, total = 0, 0
        for b in (range(B) if not full else [0]):
            lo, hi_ = int(case.cu[b]), int(case.cu[b + 1])
            T = hi_ - lo
            Kc, Vc = case.oracle.new_cache(T + k)
            case.oracle.prefill(case.ids[lo:hi_], case.hidden[lo:hi_], rho[0], Kc, Vc)
            ids_o, logits_o, gaps = osmp.draft_sampled(case.oracle, T - 1, int(case.ids[hi_ - 1]), case.hidden[hi_ - 1], k, rho,
                                                       Kc, Vc, temperature, u[b].astype(np.float64))
            total += k
            whole = True
            for s in range(k):
                err = row_rel_err(logits_g[b, s], logits_o[s])
                assert err <= rtol, f"seq {b} step {s}: logits rel err {err}"
                if ids_g[b, s] != ids_o[s]:
                    allowed = 2 * rtol * np.abs(logits_o[s]).max() / temperature + 1e-4
                    assert gaps[s] < allowed, f"seq {b} step {s}: drew {ids_g[b, s]}, oracle {ids_o[s]}, gap {gaps[s]:.2e}"
                    whole = False
                    break
                compared += 1
            if whole:
                gk, gv = case.drafter.read_kv(b, T - 1, k)
                np.testing.assert_allclose(gk.cpu().numpy(), Kc[T - 1:T - 1 + k], rtol=0, atol=3e-2 if wl.dims.dtype == "bf16" else 1e-4)
                np.testing.assert_allclose(gv.cpu().numpy(), Vc[T - 1:T - 1 + k], rtol=0, atol=3e-2 if wl.dims.dtype == "bf16" else 1e-4)
        print(f"{name}: {compared} of {total} steps compared with the oracle")
        assert compared >= 0.6 * total
    finally:
        case.close()


def test_sampled_drafting_refusals():
    import torch
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload("tiny_f32_b4_ragged")                     # fp32 and four sequences: no chain kernel takes it
    case = Case(wl)
    try:
        B, k, V = wl.batch, wl.k, wl.dims.vocab
        case.gpu_prefill()
        u = torch.full((B, k, V), 0.5, device="cuda")
        with pytest.raises(HivisError) as e:
            case.drafter.draft_sampled(B, k, 1.0, u, case.d_resid)
        assert e.value.code == -2
        with pytest.raises(HivisError) as e:
            case.drafter.draft_sampled(1, k, 0.0, u, case.d_resid)
        assert e.value.code == -1
        ids = case.drafter.draft_sampled(1, k, 1.0, u, case.d_resid, want_logits=False)     # one sequence works; equal noise = greedy
        case.drafter.set_kv_len(0, int(case.lens[0]) - 1, restore_pending=True)
        ref = case.drafter.draft(1, k, case.d_resid)
        torch.cuda.synchronize()
        assert (ids.cpu().numpy() == ref.cpu().numpy()).all()
    finally:
        case.close()


def test_drawn_draft_plus_sampled_verification_emit_the_target_distribution():
    """The point of the T > 0 path, end to end on the GPU: a token drawn by hivis_draft_sampled and then accepted or
    replaced by hivis_verify_sampled is distributed as the TARGET's softmax, whatever the drafter's distribution.
    16 sequences x 2500 rounds with fresh uniform numbers; the target's first row is the drafter's own step-0 logits
    with eight tokens raised by 6, so that both the acceptance and the replacement branch are taken often.  The
    frequencies of the eight raised tokens and of "any other token" are compared with the target's probabilities
    (computed in fp64 from the logits the GPU returned) at four standard deviations."""
    import torch
    wl = hi.scaled(hi.workload("mini_gqa_b16_ragged"), k=1)
    case = Case(wl)
    try:
        B, V, T = wl.batch, wl.dims.vocab, 1.0
        case.gpu_prefill()
        _, l0 = case.gpu_draft(1)                                    # step-0 logits [B, 1, V]: independent of any draw
        rng = np.random.default_rng(123)
        raised = np.stack([rng.choice(V, 8, replace=False) for _ in range(B)])          # [B, 8]
        tl = np.zeros((B, 2, V), np.float32)
        tl[:, 0] = l0[:, 0]
        for b in range(B):
            tl[b, 0, raised[b]] += 6.0
        tl[:, 1] = rng.standard_normal((B, V)).astype(np.float32)
        p = np.stack([osmp.softmax_t(tl[b, 0], T) for b in range(B)])                   # the target's distribution [B, V]
        q = np.stack([osmp.softmax_t(l0[b, 0], T) for b in range(B)])
        accept_rate = float(np.mean([np.minimum(p[b], q[b]).sum() for b in range(B)]))
        assert 0.2 < accept_rate < 0.95                              # both branches matter
        d_tl = torch.from_numpy(tl).cuda()
        d_raised = torch.from_numpy(raised).cuda()
        gen = torch.Generator(device="cuda"); gen.manual_seed(9)
        rounds = 2500
        hits = torch.zeros((B, 8), dtype=torch.int64, device="cuda")
        kept = torch.zeros((), dtype=torch.int64, device="cuda")
        for _ in range(rounds):
            case.gpu_restore()
            u = torch.rand((B, 1, V), generator=gen, device="cuda") * (1 - 2e-6) + 1e-6
            ids, dl = case.drafter.draft_sampled(B, 1, T, u, case.d_resid)
            ua = torch.rand((B, 1), generator=gen, device="cuda")
            us = torch.rand((B,), generator=gen, device="cuda")
            acc, nxt, _ = case.drafter.verify_sampled(ids, dl, d_tl, T, ua, us)
            first = torch.where(acc >= 1, ids[:, 0], nxt)            # the token that is emitted at the first position
            hits += (first[:, None] == d_raised).long()
            kept += (acc >= 1).sum()
        torch.cuda.synchronize()
        case.drafter.status()
        hits = hits.cpu().numpy()
        n = rounds
        for b in range(B):
            exp = p[b, raised[b]]
            sd = np.sqrt(exp * (1 - exp) / n)
            assert np.all(np.abs(hits[b] / n - exp) < 4 * sd + 2e-3), (b, hits[b] / n, exp)
            other = 1.0 - hits[b].sum() / n
            eo = 1.0 - exp.sum()
            assert abs(other - eo) < 4 * np.sqrt(eo * (1 - eo) / n) + 2e-3
        # over all sequences: tighter
        tot = hits.sum(0) / (n * B)
        np.testing.assert_allclose(tot, p[np.arange(B)[:, None], raised].mean(0), atol=4e-3)
        got_rate = int(kept.item()) / (n * B)
        assert abs(got_rate - accept_rate) < 0.02, (got_rate, accept_rate)
        print(f"acceptance rate {got_rate:.3f} (expected {accept_rate:.3f})")
    finally:
        case.close()
