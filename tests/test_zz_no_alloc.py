"""hivis_verify_noalloc against hivis_verify and against the CPU oracle's verification.

hivis_verify_noalloc is the greedy verification for callers that are not allowed to allocate device
memory (a plug-in inside a server whose pool owns the GPU, code running after allocation has been
closed): its scratch is a fixed array inside the library.  Because every call shares that array and
it keeps the last call's contents, the check is made on two calls in a row with different logits.
This file sorts last so that a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest

import hivis_inputs as hi
from tests.harness import Case, to_dev

pytestmark = pytest.mark.gpu


def _reference_verify(case, d_ids, logits_np, wl):
    """The existing entry point on freshly drafted slots: (accept, next, kv_len) as numpy."""
    t = case.torch
    case.gpu_restore()
    case.drafter.draft(wl.batch, wl.k, case.d_resid)          # hivis_verify must follow a draft
    acc, nxt, kv = case.drafter.verify(d_ids, to_dev(logits_np, wl.logits_dtype))
    t.cuda.synchronize()
    return acc.cpu().numpy(), nxt.cpu().numpy(), kv.cpu().numpy()


@pytest.mark.parametrize("name", ["mini_gqa_b16_ragged", "mini_gqa_b3"])
def test_noalloc_verify_matches_context_verify_twice_in_a_row(name):
    import torch
    from paper_2509_23928_b200 import hivis_verify_noalloc, HIVIS_BF16, HIVIS_F32
    wl = hi.workload(name)                      # f32 logits (aligned rows) / bf16 logits, vocab 5031 (unaligned rows)
    case = Case(wl)
    try:
        B, k, V = wl.batch, wl.k, wl.dims.vocab
        case.gpu_prefill()
        ids_np, _ = case.gpu_draft(want_logits=False)
        d_ids = torch.from_numpy(ids_np).cuda()
        # two different sets of target logits: planted accept lengths, then heavy exact ties
        logits_a, planted = hi.make_target_logits(wl, ids_np)
        rng = np.random.default_rng(11)
        logits_b = rng.integers(-3, 4, size=(B, k + 1, V)).astype(np.float32)     # exact in bf16 too
        want_a = _reference_verify(case, d_ids, logits_a, wl)
        want_b = _reference_verify(case, d_ids, logits_b, wl)
        assert (want_a[0] == planted).all()
        # what the oracle's greedy verification gives for each sequence (Sec. 2.1), independent of the CUDA path
        oracle_a = [case.oracle.verify(ids_np[b], logits_a[b], int(case.lens[b])) for b in range(B)]
        oracle_b = [case.oracle.verify(ids_np[b], logits_b[b], int(case.lens[b])) for b in range(B)]

        ldt = HIVIS_BF16 if wl.logits_dtype == "bf16" else HIVIS_F32
        rows_before = torch.from_numpy((case.lens - 1).astype(np.int32)).cuda()
        d_a, d_b = to_dev(logits_a, wl.logits_dtype), to_dev(logits_b, wl.logits_dtype)
        outs = [[torch.full((B,), -7, dtype=torch.int32, device="cuda") for _ in range(3)] for _ in range(3)]
        # three calls back to back on one stream, no synchronisation in between: a, b, a again
        for (acc, nxt, kv), d_log in zip(outs, (d_a, d_b, d_a)):
            hivis_verify_noalloc(B, k, V, d_ids, d_log, ldt, rows_before, acc, nxt, kv)
        torch.cuda.synchronize()
        for (acc, nxt, kv), want, orc in zip(outs, (want_a, want_b, want_a), (oracle_a, oracle_b, oracle_a)):
            acc, nxt, kv = acc.cpu().numpy(), nxt.cpu().numpy(), kv.cpu().numpy()
            np.testing.assert_array_equal(acc, want[0])
            np.testing.assert_array_equal(nxt, want[1])
            np.testing.assert_array_equal(kv, want[2])
            for b in range(B):
                assert (int(acc[b]), int(nxt[b]), int(kv[b])) == orc[b], f"seq {b} against the oracle"
        # without the row counts
        acc, nxt = outs[0][0].fill_(-7), outs[0][1].fill_(-7)
        hivis_verify_noalloc(B, k, V, d_ids, d_b, ldt, None, acc, nxt, None)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(acc.cpu().numpy(), want_b[0])
        np.testing.assert_array_equal(nxt.cpu().numpy(), want_b[1])
    finally:
        case.close()


def test_noalloc_verify_rejects_sizes_beyond_its_fixed_array():
    import torch
    from paper_2509_23928_b200 import hivis_verify_noalloc, hivis_last_error, HivisError, HIVIS_F32
    buf = torch.zeros(4096, dtype=torch.int32, device="cuda")
    logits = torch.zeros(4096, dtype=torch.float32, device="cuda")
    for B, k in ((65, 2), (2, 17), (0, 2), (2, 0)):
        with pytest.raises(HivisError) as e:
            hivis_verify_noalloc(B, k, 8, buf, logits, HIVIS_F32, None, buf, buf, None)
        assert e.value.code == -5
        assert "hivis_verify_noalloc" in hivis_last_error(None)
    with pytest.raises(HivisError) as e:                         # row counts without an output for them
        hivis_verify_noalloc(1, 1, 8, buf, logits, HIVIS_F32, buf, buf, buf, None)
    assert e.value.code == -1
