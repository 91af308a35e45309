"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest

import hivis_inputs as hi
from tests.harness import Case, check_draft_parity, check_kv_parity, check_verify_parity, to_dev, row_rel_err

pytestmark = pytest.mark.gpu

SMALL = ["c1_tiny_f32_b1", "mini_mha_b1", "mini_mha_b5_ragged", "mini_gqa_b16_ragged", "mini_gqa_b3",
         "tiny_f32_b4_ragged"]


@pytest.mark.parametrize("tc", [True, False])
@pytest.mark.parametrize("name", SMALL)
def test_draft_kv_verify_parity_small(name, tc):
    """tc=True: the persistent tensor-core kernel (bf16 workloads); tc=False: the per-step kernels
    (and, for one sequence, the ALU chain kernel)."""
    case = Case(hi.workload(name))
    try:
        case.drafter.set_tc_kernel(tc)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])              # cache after the teacher-forced run = oracle's run
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


@pytest.mark.parametrize("name", ["wide_gqa_b16_ragged", "wide_mha_b16_ragged"])
def test_more_head_groups_than_attention_warps(name):
    """16 sequences x 48 KV heads = 768 (sequence, head group) pairs against the 740 attention warps of the
    tensor-core chain kernel: a warp takes several whole keys (head groups of 7), or a range of units that
    spans several keys (single heads)."""
    case = Case(hi.workload(name))
    try:
        case.drafter.set_tc_kernel(True)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


@pytest.mark.parametrize("name", ["mini_gqa_b16_ragged", "mini_mha_b5_ragged", "wide_mha_b16_ragged"])
def test_tensor_core_chain_kernel_repeats_bit_for_bit(name):
    """Tiles shared between CTAs and keys shared between warps are summed in a fixed order whoever arrives
    last, and the argmax is an integer maximum: two runs of the same draft give the same bits."""
    case = Case(hi.workload(name))
    try:
        case.drafter.set_tc_kernel(True)
        case.gpu_prefill()
        ids_a, logits_a = case.gpu_draft()
        for _ in range(3):
            case.gpu_restore()
            ids_b, logits_b = case.gpu_draft()
            np.testing.assert_array_equal(ids_a, ids_b)
            np.testing.assert_array_equal(logits_a.view(np.uint32), logits_b.view(np.uint32))
        case.drafter.status()
    finally:
        case.close()


EDGE = [  # (base workload, batch, k, shortest and longest text length)
    ("wide_mha_b16_ragged", 16, 2, 1, 1),            # no prefix at all: every key is its tail unit only
    ("mini_gqa_b16_ragged", 3, 16, 1, 1),            # ... and the longest chain (16 appended rows)
    ("mini_mha_b5_ragged", 5, 1, 32, 32),            # prefix of 31 rows: one block, not full
    ("mini_gqa_b16_ragged", 16, 5, 33, 33),          # prefix of exactly one block
    ("mini_mha_b5_ragged", 9, 8, 31, 34),            # lengths around the block boundary
    ("wide_gqa_b16_ragged", 16, 16, 127, 129),       # several whole keys per warp, long chain
    ("mini_gqa_b16_ragged", 2, 8, 1, 200),           # two sequences: keys cut into many parts
    ("mini_mha_b5_ragged", 3, 5, 300, 300),          # long uniform prefixes, few keys
    ("wide_mha_b16_ragged", 9, 16, 1, 90),
]


@pytest.mark.parametrize("base,batch,k,lo,hi_len", EDGE)
def test_tensor_core_chain_kernel_edge_lengths(base, batch, k, lo, hi_len):
    """Cache lengths at and around the 32-row block boundaries of the attention, an empty prefix, the
    longest chain: the tensor-core chain kernel against the oracle."""
    wl = hi.scaled(hi.workload(base), batch=batch, k=k, seed=9100 + batch + k + lo, text_len=None,
                   text_len_range=(lo, hi_len))
    case = Case(wl, max_k=16)
    try:
        case.drafter.set_tc_kernel(True)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


GROUPS = ["gqa2_b5_ragged", "gqa4_b16_ragged", "gqa8_b16_ragged", "gqa4_b5_ragged"]


@pytest.mark.parametrize("tc", [True, False])
@pytest.mark.parametrize("name", GROUPS)
def test_head_groups_of_2_4_8(name, tc):
    """2, 4 and 8 query heads per KV head, head dimensions 64 and 128, ragged batches of 5 and 16: in the
    tensor-core chain kernel these run the single-head attention body with several query heads mapped onto one
    KV head (the tensor-core attention body takes groups that are multiples of 7)."""
    case = Case(hi.workload(name))
    try:
        case.drafter.set_tc_kernel(tc)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


def test_smaller_batch_after_a_larger_one_on_the_same_context():
    """A draft of 16 sequences followed, on the same context, by a draft of 4 of them: nothing the larger call
    left in the operand buffers (embedding rows, rounding-remainder rows) may leak into the smaller one."""
    import torch
    wl = hi.workload("mini_gqa_b16_ragged")
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(True)
        ref = case.oracle_run()
        ids_o = np.stack([r["ids"] for r in ref])
        logits_o = np.stack([r["logits"] for r in ref])
        case.gpu_prefill()
        case.gpu_draft()                                   # all 16 sequences
        case.gpu_restore()
        sub = [9, 2, 14, 5]
        f = torch.from_numpy(np.ascontiguousarray(ids_o[sub], np.int32)).cuda()
        ids_g, logits_g = case.drafter.draft(len(sub), wl.k, case.d_resid, slots=sub, forced_ids=f, want_logits=True)
        torch.cuda.synchronize()
        case.drafter.status()
        err = row_rel_err(logits_g.cpu().numpy(), logits_o[sub])
        assert err.max() <= 2e-2, f"logits rel err {err.max()}"
        # and bit for bit what a fresh context computes for the same four sequences
        case2 = Case(wl)
        try:
            case2.drafter.set_tc_kernel(True)
            case2.gpu_prefill()
            ids_h, logits_h = case2.drafter.draft(len(sub), wl.k, case2.d_resid, slots=sub, forced_ids=f, want_logits=True)
            torch.cuda.synchronize()
            assert torch.equal(logits_g, logits_h) and torch.equal(ids_g, ids_h)
        finally:
            case2.close()
    finally:
        case.close()


@pytest.mark.parametrize("name,tc,chain", [("mini_mha_b1", False, True), ("mini_mha_b1", False, False),
                                           ("mini_mha_b5_ragged", True, True), ("mini_mha_b5_ragged", False, True)])
def test_out_of_range_token_id_is_reported_not_followed(name, tc, chain):
    """Token ids live in device memory, so only the kernels can check them.  A forced id beyond the vocabulary is
    read as token 0 (no lookup leaves the embedding table), hivis_status reports HIVIS_ERR_ARG once, and the
    logits are those of a chain fed token 0 at that step."""
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload(name)
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(tc)
        case.drafter.set_chain_kernel(chain)
        ref0 = case.oracle_run()
        forced = np.stack([r["ids"] for r in ref0]).copy()
        bad = forced.copy()
        bad[wl.batch - 1, 1] = wl.dims.vocab + 12345         # consumed by step 2
        if wl.batch > 1:
            bad[0, 0] = -7
        clean = bad.copy()
        clean[(bad < 0) | (bad >= wl.dims.vocab)] = 0
        ref = case.oracle_run(forced=clean)
        case.gpu_prefill()
        ids_g, logits_g = case.gpu_draft(forced=bad)
        with pytest.raises(HivisError) as e:
            case.drafter.status()
        assert e.value.code == -1
        case.drafter.status()                              # the record was cleared
        err = row_rel_err(logits_g, np.stack([r["logits"] for r in ref]))
        assert err.max() <= 2e-2
        case.gpu_restore()
        case.gpu_draft(forced=clean)
        case.drafter.status()                              # valid ids: nothing to report
    finally:
        case.close()


@pytest.mark.parametrize("name,tc", [("mini_mha_b1", False), ("mini_mha_b5_ragged", True), ("mini_mha_b5_ragged", False)])
def test_nan_hidden_state_gives_token_zero_on_both_sides(name, tc):
    """A NaN in the pending hidden state makes every logit of the chain NaN.  NaN never wins an argmax and an
    all-NaN row gives index 0, on both sides; nothing is looked up outside the embedding table."""
    import torch
    wl = hi.workload(name)
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(tc)
        b = wl.batch - 1
        last = int(case.cu[b + 1]) - 1
        case.hidden[last, 3] = np.nan
        case.d_hidden = to_dev(case.hidden, wl.dims.dtype)
        ref = case.oracle_run(k=3)
        assert (ref[b]["ids"] == 0).all() and np.isnan(ref[b]["logits"]).all()
        case.gpu_prefill()
        ids_g, logits_g = case.gpu_draft(3)
        case.drafter.status()
        assert (ids_g[b] == 0).all() and np.isnan(logits_g[b]).all()
        for o in range(wl.batch - 1):                      # the other sequences are untouched
            assert np.isfinite(logits_g[o]).all()
    finally:
        case.close()


@pytest.mark.parametrize("name", ["mini_gqa_b16_ragged", "mini_mha_b5_ragged", "gqa4_b16_ragged", "wide_gqa_b16_ragged"])
def test_tensor_core_prefill_against_oracle_and_per_pass_prefill(name):
    """The prefix build as two tcgen05 GEMMs over all pairs (calls of more than 16 pairs) and the 16-pairs-per-pass
    kernels: the cached K/V rows of both against the oracle's, and the draft that follows."""
    import torch
    wl = hi.workload(name)
    case = Case(wl)
    try:
        assert int(case.cu[-1]) >= 128
        ref = case.oracle_run()
        rows = {}
        for tc_prefill in (True, False):
            case.drafter.set_tc_prefill(tc_prefill)
            case.drafter.prefill(case.d_ids, case.d_hidden, [int(x) for x in case.cu], start_pos=[0] * wl.batch,
                                 resid0=case.d_resid[0])
            case.drafter.status()
            for b in range(wl.batch):
                n = int(case.lens[b]) - 1
                if n == 0:
                    continue
                k_g, v_g = case.drafter.read_kv(b, 0, n)
                torch.cuda.synchronize()
                for got, want, nm in ((k_g, ref[b]["K"][:n], "K"), (v_g, ref[b]["V"][:n], "V")):
                    e = np.abs(got.cpu().numpy() - want).max() / np.abs(want).max()
                    assert e <= 1e-2, f"tc_prefill={tc_prefill} {nm} cache of seq {b}: rel err {e}"
                rows[(tc_prefill, b)] = (k_g.cpu().numpy(), v_g.cpu().numpy())
        for b in range(wl.batch):
            if (True, b) in rows:
                for x, y in zip(rows[(True, b)], rows[(False, b)]):
                    assert np.abs(x - y).max() / np.abs(y).max() <= 1e-2
        case.drafter.set_tc_prefill(True)
        for b in range(wl.batch):
            case.drafter.reset(b)
        res = check_draft_parity(case)                 # prefill (tensor-core path) + draft against the oracle
        check_kv_parity(case, res["ref"])
    finally:
        case.close()


def test_more_sequences_than_the_chain_kernels_take():
    """20 sequences: beyond the 16 of the tensor-core chain kernel, so the per-phase kernels run in two passes."""
    wl = hi.scaled(hi.workload("mini_gqa_b16_ragged"), batch=20, k=3, seed=2103)
    case = Case(wl)
    try:
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


def test_c1_ids_exact_and_tight_logits():
    case = Case(hi.workload("c1_tiny_f32_b1"))
    try:
        res = check_draft_parity(case, rtol=1e-4)
        assert res["excused"] == 0
        np.testing.assert_array_equal(res["ids_g"], res["ids_o"])
    finally:
        case.close()


@pytest.mark.parametrize("name", ["c1_tiny_f32_b1", "mini_mha_b1"])
def test_chain_kernel_and_stepwise_kernels_agree(name):
    """One sequence: the persistent chain kernel and the per-step kernels compute the same thing."""
    wl = hi.workload(name)
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(False)
        case.drafter.set_chain_kernel(False)
        res_step = check_draft_parity(case)
        case.gpu_restore()
        ids_s, logits_s = case.gpu_draft(forced=res_step["ids_o"])
        case.drafter.set_chain_kernel(True)
        case.gpu_restore()
        ids_c, logits_c = case.gpu_draft(forced=res_step["ids_o"])
        case.drafter.status()
        assert row_rel_err(logits_c, logits_s).max() < 1e-4
        check_kv_parity(case, res_step["ref"])
    finally:
        case.close()


@pytest.mark.parametrize("tc", [True, False])
@pytest.mark.parametrize("T,k", [(300, 8), (1, 2), (64, 1)])
def test_chain_kernel_long_and_short(T, k, tc):
    wl = hi.scaled(hi.workload("mini_mha_b1"), text_len=T, k=k, seed=4000 + T)
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(tc)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
    finally:
        case.close()


@pytest.mark.parametrize("tc", [True, False])
def test_chain_kernel_gqa_b1(tc):
    wl = hi.scaled(hi.workload("mini_gqa_b3"), batch=1, k=4)
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(tc)
        res = check_draft_parity(case)
        case.drafter.status()
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


@pytest.mark.parametrize("tc", [True, False])
def test_intermediate_taps_match_oracle(tc):
    wl = hi.workload("mini_mha_b5_ragged")
    case = Case(wl)
    try:
        case.drafter.set_tc_kernel(tc)
        case.gpu_prefill()
        case.gpu_draft(1)
        rho = case.oracle.fold_residuals(case.resid)
        for b in range(wl.batch):
            lo, hi_ = int(case.cu[b]), int(case.cu[b + 1])
            T = hi_ - lo
            Kc, Vc = case.oracle.new_cache(T + 1)
            case.oracle.prefill(case.ids[lo:hi_], case.hidden[lo:hi_], rho[0], Kc, Vc)
            _, taps = case.oracle.position(case.hidden[hi_ - 1], int(case.ids[hi_ - 1]), rho[0], T - 1, Kc, Vc, taps=True)
            for name in ("u", "attn", "y", "act", "g"):
                got = case.drafter.tap(name, wl.batch)[b].cpu().numpy()
                e = np.abs(got - taps[name]).max() / np.abs(taps[name]).max()
                assert e < 2e-2, f"tap {name} seq {b}: rel err {e}"
            # q leaves the library before the rotary embedding; the oracle's tap is taken after it
            D = wl.dims
            q_g = case.drafter.tap("q", wl.batch)[b].cpu().numpy()
            q_rot = case.oracle.rope(q_g, D.n_q_heads, D.head_dim, D.rope_base, T - 1)
            e = np.abs(q_rot - taps["q"]).max() / np.abs(taps["q"]).max()
            assert e < 2e-2, f"tap q seq {b}: rel err {e}"
            k_g, v_g = case.drafter.read_kv(b, T - 1, 1)       # the step's K (rotated) and V rows
            for got, want, nm in ((k_g, taps["k"], "k"), (v_g, taps["v"], "v")):
                e = np.abs(got[0].cpu().numpy() - want).max() / np.abs(want).max()
                assert e < 2e-2, f"{nm} row of seq {b}: rel err {e}"
    finally:
        case.close()


@pytest.mark.parametrize("T,k", [(1, 1), (1, 5), (2, 3), (129, 2), (128, 4), (257, 1)])
def test_edge_lengths(T, k):
    wl = hi.scaled(hi.workload("mini_mha_b1"), text_len=T, k=k, seed=3000 + T + k)
    case = Case(wl)
    try:
        res = check_draft_parity(case)
        check_kv_parity(case, res["ref"])
        check_verify_parity(case, res["ids_o"])
    finally:
        case.close()


def test_qkv_bias_and_residual_projection():
    wl = hi.workload("mini_gqa_b3")
    rng = np.random.default_rng(5)
    D = wl.dims
    extra = {"bq": hi.round_to_bf16(rng.standard_normal(D.q_dim).astype(np.float32) * 0.5),
             "bk": hi.round_to_bf16(rng.standard_normal(D.kv_dim).astype(np.float32) * 0.5),
             "bv": hi.round_to_bf16(rng.standard_normal(D.kv_dim).astype(np.float32) * 0.5)}
    case = Case(wl, extra_weights=extra)
    try:
        res = check_draft_parity(case)
        check_kv_parity(case, res["ref"])
    finally:
        case.close()


def test_residual_projection_matrix():
    import torch
    from paper_2509_23928_b200 import Drafter
    from tests.harness import dev_weights
    import oracle
    wl = hi.workload("mini_mha_b1")
    D = wl.dims
    W = hi.make_weights(D, wl.seed)
    rp = hi.round_to_bf16(np.random.default_rng(6).standard_normal((D.d, D.d)).astype(np.float32) * 0.05)
    ids, hidden, cu = hi.make_prompt(wl)
    resid = hi.make_residuals(wl)
    o = oracle.Oracle(D, W)
    ref = o.run_batch(ids, hidden, cu, wl.k, resid, resid_proj=rp)[0]
    dW = dev_weights(W, "bf16")
    dW["resid_proj"] = to_dev(rp, "bf16")
    dr = Drafter(D, dW, 1, 64, 8)
    try:
        d_resid = to_dev(resid, "bf16")
        dr.prefill(torch.from_numpy(ids).cuda(), to_dev(hidden, "bf16"), [int(x) for x in cu], resid0=d_resid[0])
        f = torch.from_numpy(ref["ids"][None].astype(np.int32)).cuda()
        _, logits = dr.draft(1, wl.k, d_resid, forced_ids=f, want_logits=True)
        torch.cuda.synchronize()
        assert row_rel_err(logits[0].cpu().numpy(), ref["logits"]).max() < 2e-2
    finally:
        dr.close()


def test_no_residual_equals_zero_residual():
    import torch
    wl = hi.workload("mini_mha_b1")
    case = Case(wl)
    try:
        case.drafter.prefill(case.d_ids, case.d_hidden, [int(x) for x in case.cu], resid0=None)
        ids_a, la = case.drafter.draft(1, 3, None, want_logits=True)
        case.gpu_restore()
        z = torch.zeros_like(case.d_resid)
        case.drafter.prefill(case.d_ids, case.d_hidden, [int(x) for x in case.cu], start_pos=[0], resid0=z[0])
        ids_b, lb = case.drafter.draft(1, 3, z, want_logits=True)
        torch.cuda.synchronize()
        assert torch.equal(ids_a, ids_b) and torch.equal(la, lb)
    finally:
        case.close()


def test_run_to_run_determinism():
    wl = hi.workload("mini_gqa_b16_ragged")
    case = Case(wl)
    try:
        case.gpu_prefill()
        ids_a, la = case.gpu_draft()
        case.gpu_restore()
        ids_b, lb = case.gpu_draft()
        np.testing.assert_array_equal(ids_a, ids_b)
        np.testing.assert_array_equal(la, lb)
    finally:
        case.close()


def test_slots_subset_and_order():
    """Sequences may sit in any slots, in any order, and calls may address a subset."""
    import torch
    wl = hi.workload("mini_mha_b5_ragged")
    case = Case(wl)
    try:
        ref = case.oracle_run()
        perm = [3, 0, 4, 1, 2]
        # prefill sequence b into slot perm[b]
        case.drafter.prefill(case.d_ids, case.d_hidden, [int(x) for x in case.cu], slots=perm, resid0=case.d_resid[0])
        sub = [1, 3]                                  # draft only sequences 1 and 3, listed in reverse
        slots = [perm[3], perm[1]]
        ids = case.drafter.draft(2, wl.k, case.d_resid, slots=slots)
        torch.cuda.synchronize()
        ids = ids.cpu().numpy()
        for row, b in enumerate([3, 1]):
            first_bad = next((s for s in range(wl.k) if ids[row, s] != ref[b]["ids"][s]), None)
            assert first_bad is None or ref[b]["gaps"][first_bad] < 1e-2
        assert case.drafter.kv_len(perm[3])[0] == case.lens[3] - 1 + wl.k
        assert case.drafter.kv_len(perm[0])[0] == case.lens[0] - 1      # untouched
    finally:
        case.close()


def test_multi_round_loop_with_refresh_matches_oracle():
    """draft -> verify -> prefill(start_pos) refresh -> draft, compared with the oracle doing the same."""
    import torch
    wl = hi.workload("mini_mha_b1")
    case = Case(wl, max_len=128)
    try:
        o, D = case.oracle, wl.dims
        k = 4
        rho = o.fold_residuals(case.resid)
        T = int(case.lens[0])
        Kc, Vc = o.new_cache(128)
        o.prefill(case.ids, case.hidden, rho[0], Kc, Vc)
        case.gpu_prefill()
        pend_h, pend_id = case.hidden[-1], int(case.ids[-1])
        rng = np.random.default_rng(77)
        for rnd in range(3):
            ref = o.draft(T - 1, pend_id, pend_h, k, rho, Kc, Vc)
            f = torch.from_numpy(ref["ids"][None].astype(np.int32)).cuda()
            ids_g, logits_g = case.drafter.draft(1, k, case.d_resid, forced_ids=f, want_logits=True)
            torch.cuda.synchronize()
            assert row_rel_err(logits_g[0].cpu().numpy(), ref["logits"]).max() < 2e-2, f"round {rnd}"
            planted = np.array([[2, 0, 4][rnd]])
            logits, _ = hi.make_target_logits(hi.scaled(wl, k=k, seed=wl.seed + rnd), ref["ids"][None], planted)
            acc, nxt, kv = case.drafter.verify(f, to_dev(logits, wl.logits_dtype))
            torch.cuda.synchronize()
            n, nx, kvl = o.verify(ref["ids"], logits[0], T)
            assert (int(acc[0]), int(nxt[0]), int(kv[0])) == (n, nx, kvl)
            # the target now supplies hidden states for the n+1 new tokens; refresh rows T.. with them
            new_ids = np.array(list(ref["ids"][:n]) + [nx], np.int32)
            new_hidden = hi.round_to_bf16(rng.standard_normal((n + 1, D.d)).astype(np.float32))
            o.prefill(new_ids, new_hidden, rho[0], Kc, Vc, start_pos=T)
            case.drafter.prefill(torch.from_numpy(new_ids).cuda(), to_dev(new_hidden, "bf16"), [0, n + 1],
                                 start_pos=[T], resid0=case.d_resid[0])
            T += n + 1
            pend_h, pend_id = new_hidden[-1], int(new_ids[-1])
            assert case.drafter.kv_len(0) == (T - 1, True)
        k_g, v_g = case.drafter.read_kv(0, 0, T - 1)
        torch.cuda.synchronize()
        assert np.abs(k_g.cpu().numpy() - Kc[:T - 1]).max() / np.abs(Kc[:T - 1]).max() < 1e-2
        assert np.abs(v_g.cpu().numpy() - Vc[:T - 1]).max() / np.abs(Vc[:T - 1]).max() < 1e-2
    finally:
        case.close()


def test_verify_ties_bf16_and_unaligned_vocab():
    """bf16 logits make exact ties common: the lowest index must win on both sides."""
    import torch
    wl = hi.scaled(hi.workload("mini_gqa_b3"), k=3)         # vocab 5031: rows are not 16-byte aligned
    case = Case(wl)
    try:
        case.gpu_prefill()
        ids_g, _ = case.gpu_draft(3, want_logits=False)
        V = wl.dims.vocab
        rng = np.random.default_rng(8)
        logits = hi.round_to_bf16(rng.integers(-3, 4, size=(3, 4, V)).astype(np.float32))   # massive ties
        d_logits = to_dev(logits, "bf16")
        d_ids = torch.from_numpy(ids_g).cuda()
        acc, nxt, kv = case.drafter.verify(d_ids, d_logits)
        torch.cuda.synchronize()
        for b in range(3):
            n, nx, kvl = case.oracle.verify(ids_g[b], logits[b], int(case.lens[b]))
            assert (int(acc[b]), int(nxt[b]), int(kv[b])) == (n, nx, kvl)
            assert nx == int(np.argmax(logits[b, n]))
    finally:
        case.close()


def test_host_side_errors_do_not_launch():
    import torch
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload("c1_tiny_f32_b1")
    case = Case(wl, max_len=40, max_k=4)
    try:
        dr = case.drafter
        n0 = dr.launch_count()
        out = torch.empty((1, 4), dtype=torch.int32, device="cuda")
        with pytest.raises(HivisError) as e:                     # draft before prefill
            dr.draft(1, 4, case.d_resid, out_ids=out)
        assert e.value.code == -4
        with pytest.raises(HivisError) as e:                     # k beyond max_k
            dr.draft(1, 5, case.d_resid)
        assert e.value.code == -5
        with pytest.raises(HivisError) as e:                     # slot out of range
            dr.draft(1, 2, case.d_resid, slots=[3])
        assert e.value.code == -1
        with pytest.raises(HivisError) as e:                     # duplicate slot / too many sequences
            dr.prefill(case.d_ids, case.d_hidden, [0, 16, 32], resid0=None)
        assert e.value.code == -5
        with pytest.raises(HivisError) as e:                     # batched row counts: one out of range, nothing changes
            dr.set_kv_len_batch([10 ** 6])
        assert e.value.code == -5
        with pytest.raises(HivisError) as e:                     # misaligned pointer
            dr.prefill(case.d_ids[1:], case.d_hidden, [0, 31])
        assert e.value.code == -1
        assert dr.launch_count() == n0
        case.gpu_prefill()                                       # 31 rows + pending
        with pytest.raises(HivisError) as e:                     # would overflow max_len = 40 ... 31 + 4 fits; shrink
            dr.set_kv_len(0, 41)
        assert e.value.code == -5
        dr.set_kv_len(0, 38, restore_pending=True)
        with pytest.raises(HivisError) as e:
            dr.draft(1, 4, case.d_resid)                         # 38 + 4 > 40
        assert e.value.code == -5
        dr.set_kv_len(0, 31, restore_pending=True)
        ids = dr.draft(1, 4, case.d_resid)
        logits = torch.zeros((1, 4, wl.dims.vocab), device="cuda")
        with pytest.raises(HivisError) as e:                     # verify with another k
            dr.verify(ids[:, :3].contiguous(), logits)
        assert e.value.code == -4
        with pytest.raises(HivisError) as e:                     # second draft without a pending pair
            dr.draft(1, 4, case.d_resid)
        assert e.value.code == -4
        case.gpu_restore()
        n1 = dr.launch_count()
        with pytest.raises(HivisError) as e:                     # appending while a pair is still pending
            dr.prefill(case.d_ids, case.d_hidden, [0, 4])
        assert e.value.code == -4 and dr.launch_count() == n1
    finally:
        case.close()


# ---------------------------------------------------------------------------------------------------
# Full-size workloads, in the launch configuration the benchmark times.  The CUDA path runs the whole
# batch; the oracle (fp64, one sequence at a time) is run on sampled sequences: the shortest, the longest
# and one more.  Every sampled sequence is compared completely: free-running ids (top-2-gap rule),
# teacher-forced logits of every step, appended K/V rows and the verification outputs.
# ---------------------------------------------------------------------------------------------------
def _sampled_full_size(name, n_samples):
    import torch
    wl = hi.workload(name)
    case = Case(wl)                       # builds the oracle object too; nothing is computed yet
    try:
        B, k = wl.batch, wl.k
        lens = case.lens
        order = np.argsort(lens, kind="stable")
        picks = [int(order[0]), int(order[-1])] + [int(b) for b in order[1:-1][:: max(1, (B - 2) // max(1, n_samples - 2))]]
        picks = sorted(set(picks))[:n_samples] if B > 1 else [0]
        case.gpu_prefill()
        ids_g, logits_g = case.gpu_draft(k)                               # free running, whole batch
        rho = case.oracle.fold_residuals(case.resid)
        refs = {}
        for b in picks:
            lo, hi_ = int(case.cu[b]), int(case.cu[b + 1])
            T = hi_ - lo
            Kc, Vc = case.oracle.new_cache(T + k)
            case.oracle.prefill(case.ids[lo:hi_], case.hidden[lo:hi_], rho[0], Kc, Vc)
            r = case.oracle.draft(T - 1, int(case.ids[hi_ - 1]), case.hidden[hi_ - 1], k, rho, Kc, Vc)
            r["K"], r["V"], r["T"] = Kc, Vc, T
            refs[b] = r
            for s in range(k):
                if ids_g[b, s] != r["ids"][s]:
                    assert r["gaps"][s] < 1e-2, f"seq {b} step {s}: id {ids_g[b, s]} != {r['ids'][s]}, gap {r['gaps'][s]}"
                    break
                err = row_rel_err(logits_g[b, s], r["logits"][s])
                assert err <= 2e-2, f"free run seq {b} step {s}: logits rel err {err}"
        # teacher forcing: sampled sequences follow the oracle's ids, the others their own free-running ids
        forced = ids_g.copy()
        for b in picks:
            forced[b] = refs[b]["ids"]
        case.gpu_restore()
        ids_f, logits_f = case.gpu_draft(k, forced=forced)
        case.drafter.status()
        for b in picks:
            r = refs[b]
            err = row_rel_err(logits_f[b], r["logits"])
            assert err.max() <= 2e-2, f"teacher-forced seq {b}: logits rel err {err.max()}"
            bad = (ids_f[b] != r["ids"]) & (r["gaps"] >= 1e-2)
            assert not bad.any(), f"teacher-forced ids of seq {b} differ outside the gap zone"
            n = r["T"] - 1 + k
            k_g, v_g = case.drafter.read_kv(b, 0, n)
            torch.cuda.synchronize()
            for got, want in ((k_g, r["K"][:n]), (v_g, r["V"][:n])):
                e = np.abs(got.cpu().numpy() - want).max() / np.abs(want).max()
                assert e <= 1e-2, f"cache of seq {b}: rel err {e}"
        # verification on the whole batch: planted accept lengths, sampled sequences against the oracle
        logits_t, planted = hi.make_target_logits(wl, forced)
        acc, nxt, kv = case.drafter.verify(torch.from_numpy(forced).cuda(), to_dev(logits_t, wl.logits_dtype))
        torch.cuda.synchronize()
        acc, nxt, kv = acc.cpu().numpy(), nxt.cpu().numpy(), kv.cpu().numpy()
        np.testing.assert_array_equal(acc, planted)
        for b in picks:
            assert (int(acc[b]), int(nxt[b]), int(kv[b])) == case.oracle.verify(forced[b], logits_t[b], int(lens[b]))
        # properties that hold for every sequence at any size
        assert ((0 <= acc) & (acc <= k)).all()
        np.testing.assert_array_equal(kv, lens + np.minimum(acc, k - 1))
        np.testing.assert_array_equal(nxt, logits_t[np.arange(B), acc].argmax(-1))
        assert ((0 <= ids_g) & (ids_g < wl.dims.vocab)).all()
    finally:
        case.close()


def test_full_size_c2_llava_b1():
    _sampled_full_size("c2_llava_b1", 1)


def test_full_size_c3_llava_b16_ragged_sampled():
    _sampled_full_size("c3_llava_b16_ragged", 3)


def test_full_size_c4_qwen_b8_sampled():
    _sampled_full_size("c4_qwen_b8", 2)


def test_full_size_c5a_llava_b16_text_only_sampled():
    _sampled_full_size("c5a_llava_b16_text_only", 2)


def test_full_size_c5b_llava_b16_naive_kv_sampled():
    """704 cached positions per sequence: 22 full blocks and a tail per key, uniform batch (the key-aligned
    split of the attention units over the warps)."""
    _sampled_full_size("c5b_llava_b16_naive_kv", 2)


@pytest.mark.parametrize("name,tc", [("mini_mha_b1", False), ("mini_mha_b1", True), ("mini_gqa_b16_ragged", True)])
def test_device_waits_run_out_cleanly_and_context_recovers(name, tc):
    """Failure detection without a fault: the grid barriers of one draft are made impossible to complete,
    every device-side wait runs into its (shortened) limit, the kernel returns by itself, hivis_status
    reports HIVIS_ERR_TIMEOUT, and the same context then drafts correctly again."""
    import time
    import torch
    from paper_2509_23928_b200 import HivisError
    wl = hi.workload(name)
    case = Case(wl)
    try:
        dr = case.drafter
        dr.set_tc_kernel(tc)
        case.gpu_prefill()
        dr.set_wait_limit_us(2000)
        dr.miss_next_barrier()
        t0 = time.perf_counter()
        dr.draft(wl.batch, wl.k, case.d_resid)
        torch.cuda.synchronize()
        assert time.perf_counter() - t0 < 10.0
        with pytest.raises(HivisError) as e:
            dr.status()
        assert e.value.code == -7
        dr.status()                                       # the error word was cleared
        dr.set_wait_limit_us(1000000)
        ref = case.oracle_run()
        ids_o = np.stack([r["ids"] for r in ref])
        case.gpu_restore()
        ids_f, logits_f = case.gpu_draft(forced=ids_o)
        dr.status()
        err = row_rel_err(logits_f, np.stack([r["logits"] for r in ref]))
        assert err.max() <= 2e-2
    finally:
        case.close()


def test_small_prefill_calls_on_both_prefix_build_paths():
    """A refresh of 24 pairs (more than one pass of the 16-pairs kernels, far fewer than a 128-pair tile) through the
    tensor-core prefix build and through the per-pass kernels, against the oracle; a 9-pair call takes the per-pass
    kernels whatever the option says."""
    import torch
    wl = hi.workload("mini_mha_b1")
    case = Case(wl, max_len=160)
    try:
        o, D = case.oracle, wl.dims
        rho = o.fold_residuals(case.resid)
        T = int(case.lens[0])
        rng = np.random.default_rng(5)
        for n_new in (24, 9):
            # the continuation repeats the pending pair (its row was never cached) and starts at its row
            new_ids = np.concatenate([case.ids[-1:], rng.integers(0, D.vocab, n_new - 1)]).astype(np.int32)
            new_hidden = np.concatenate([case.hidden[-1:], hi.round_to_bf16(rng.standard_normal((n_new - 1, D.d)).astype(np.float32))])
            Kc, Vc = o.new_cache(160)
            o.prefill(case.ids, case.hidden, rho[0], Kc, Vc)
            o.prefill(new_ids, new_hidden, rho[0], Kc, Vc, start_pos=T - 1)
            got = {}
            for opt in (True, False):
                case.drafter.set_tc_prefill(opt)
                case.drafter.reset(0)
                case.gpu_prefill()
                n0 = case.drafter.launch_count()
                case.drafter.prefill(torch.from_numpy(new_ids).cuda(), to_dev(new_hidden, "bf16"), [0, n_new], start_pos=[T - 1],
                                     resid0=case.d_resid[0])
                launches = case.drafter.launch_count() - n0
                case.drafter.status()
                rows = T - 1 + n_new - 1
                k_g, v_g = case.drafter.read_kv(0, 0, rows)
                torch.cuda.synchronize()
                got[opt] = (k_g.cpu().numpy(), v_g.cpu().numpy(), launches)
                for g, want, nm in ((got[opt][0], Kc, "K"), (got[opt][1], Vc, "V")):
                    e = np.abs(g - want[:rows]).max() / np.abs(want[:rows]).max()
                    assert e <= 1e-2, f"{n_new} pairs, tensor-core path {opt}: {nm} rel err {e}"
            if n_new > 16:
                assert got[True][2] != got[False][2]            # two different sets of launches
            else:
                assert got[True][2] == got[False][2]            # a single pass either way
        case.drafter.set_tc_prefill(True)
    finally:
        case.close()
