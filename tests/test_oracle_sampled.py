"""Pins for the oracle's speculative-sampling verification (oracle/sampled.py): nothing here touches the CUDA path."""
import numpy as np
import pytest
import torch

import oracle
from oracle import sampled as osmp


def test_softmax_with_temperature_against_torch():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(300) * 4
    for T in (1.0, 0.7, 2.5):
        np.testing.assert_allclose(osmp.softmax_t(x, T), torch.softmax(torch.from_numpy(x) / T, 0).numpy(), rtol=1e-12, atol=1e-15)


def test_one_step_of_speculative_sampling_reproduces_the_target_distribution():
    """The theorem behind the rule (Leviathan et al., Chen et al.): drafting x ~ q, accepting with min(1, p/q) and
    otherwise drawing from the normalised max(0, p - q) yields a token distributed exactly as p.  Checked in closed
    form from the oracle's own ratio and residual - a wrong sign, a missing normalisation or p and q swapped breaks it."""
    rng = np.random.default_rng(2)
    for V in (2, 5, 17):
        for _ in range(5):
            p = osmp.softmax_t(rng.standard_normal(V) * 2, 1.0)
            q = osmp.softmax_t(rng.standard_normal(V) * 2, 1.0)
            acc = np.array([q[x] * osmp.accept_ratio(p, q, x) for x in range(V)])
            r = osmp.residual(p, q)
            out = acc + (1.0 - acc.sum()) * r / r.sum()
            np.testing.assert_allclose(out, p, rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(1.0 - acc.sum(), r.sum(), rtol=1e-10, atol=1e-14)     # rejection mass = residual mass


def test_inverse_cdf_against_cumsum_search_and_frequencies():
    mass = np.array([0.0, 2.0, 0.0, 1.0, 1.0, 0.0])
    assert [osmp.inverse_cdf(mass, u)[0] for u in (0.0, 0.49, 0.5, 0.74, 0.75, 0.999)] == [1, 1, 3, 3, 4, 4]
    assert osmp.inverse_cdf(mass, 1.0)[0] == 4                       # rounding past the end: the last token with mass
    rng = np.random.default_rng(3)
    w = rng.random(40)
    us = (np.arange(200000) + 0.5) / 200000
    c = np.cumsum(w)
    want = np.searchsorted(c, us * c[-1], side="right")
    got = np.array([osmp.inverse_cdf(w, u)[0] for u in us[::997]])
    np.testing.assert_array_equal(got, want[::997])
    freq = np.bincount(want, minlength=40) / us.size
    np.testing.assert_allclose(freq, w / w.sum(), atol=2e-5)


def test_identical_distributions_accept_everything_and_draw_the_bonus_from_p():
    rng = np.random.default_rng(4)
    k, V = 4, 50
    logits = rng.standard_normal((k + 1, V))
    ids = rng.integers(0, V, k)
    u = rng.random(k)
    n, nxt, kv, _ = osmp.verify_sampled(ids, logits[:k], logits, 1.0, u, 0.3, base_len=10)
    assert (n, kv) == (k, 10 + k - 1)
    assert nxt == osmp.inverse_cdf(osmp.softmax_t(logits[k], 1.0), 0.3)[0]


def test_rejection_position_residual_draw_and_rollback():
    k, V = 3, 6
    tl = np.zeros((k + 1, V)); dl = np.zeros((k, V))
    dl[1, 2] = 5.0                                  # the drafter is far too sure of token 2 at step 1
    tl[1, 4] = 3.0                                  # the target prefers token 4 there
    ids = np.array([0, 2, 1])
    p1, q1 = osmp.softmax_t(tl[1], 1.0), osmp.softmax_t(dl[1], 1.0)
    a1 = p1[2] / q1[2]
    assert a1 < 0.05
    # u below the ratio: accepted; above: rejected at step 1, next drawn from max(0, p - q), where token 2 has no mass
    n, nxt, kv, _ = osmp.verify_sampled(ids, dl, tl, 1.0, np.array([0.5, a1 * 0.5, 0.5]), 0.9, 7)
    assert n == 3
    n, nxt, kv, _ = osmp.verify_sampled(ids, dl, tl, 1.0, np.array([0.5, a1 * 1.5, 0.5]), 0.0, 7)
    assert (n, kv) == (1, 8) and nxt != 2
    r = osmp.residual(p1, q1)
    assert r[2] == 0.0 and nxt == int(np.nonzero(r > 0)[0][0])
    # step 0: uniform against uniform is always accepted (ratio 1), whatever u < 1
    assert osmp.verify_sampled(ids, dl, tl, 1.0, np.array([0.999999, 2.0, 0.0]), 0.5, 7)[0] == 1


def test_low_temperature_tends_to_greedy_verification():
    dims = type("D", (), dict(d=8, n_q_heads=1, n_kv_heads=1, head_dim=8, ffn=8, vocab=64, rms_eps=1e-5, rope_base=1e4))
    rng = np.random.default_rng(5)
    k, V = 4, 64
    o = oracle.Oracle(dims, {n: np.zeros(s, np.float32) for n, s in
                             dict(embed=(V, 8), lm_head=(V, 8), fc=(8, 16), norm1=(8,), wq=(8, 8), wk=(8, 8), wv=(8, 8), wo=(8, 8),
                                  norm2=(8,), w_gate=(8, 8), w_up=(8, 8), w_down=(8, 8)).items()})
    for trial in range(20):
        tl = rng.standard_normal((k + 1, V)).astype(np.float32)
        ids = tl[:k].argmax(1).astype(np.int32)
        planted = trial % (k + 1)
        if planted < k:
            ids[planted] = (ids[planted] + 1) % V
        dl = rng.standard_normal((k, V)).astype(np.float32)
        dl[np.arange(k), ids] += 4.0                                  # the drafter drew its own favourites
        n, nxt, kv, _ = osmp.verify_sampled(ids, dl, tl, 1e-3, rng.random(k) * 0.98 + 0.01, rng.random(), 20)
        assert (n, nxt, kv) == o.verify(ids, tl, 20)


# ------------------------------------------------------------------------------------------ drafting at T > 0
def test_gumbel_max_draws_follow_the_softmax():
    """The sampling rule against the distribution it must realise: over many seeded uniform draws the token
    frequencies match softmax(logits / T) within four standard deviations (a Gumbel sign error, T multiplied instead of
    divided, or noise missing on one entry fails), and two tokens give the logistic closed form."""
    rng = np.random.default_rng(11)
    logits = np.array([1.5, -0.3, 0.2, 2.0, -1.0, 0.7])
    for T in (1.0, 0.5, 2.0):
        n = 60000
        u = rng.random((n, logits.size))
        toks = np.argmax(logits[None, :] / T + osmp.gumbel(u), axis=1)
        for i in range(0, n, 7919):                                  # the function itself on a sample of the draws
            assert osmp.sample_gumbel(logits, T, u[i])[0] == toks[i]
        freq = np.bincount(toks, minlength=logits.size) / n
        q = osmp.softmax_t(logits, T)
        assert np.all(np.abs(freq - q) < 4 * np.sqrt(q * (1 - q) / n) + 1e-4), (T, freq, q)
    # V = 2: token 0 wins iff l0/T - l1/T > g1 - g0, and g1 - g0 is logistic: P(token 0) = sigmoid((l0 - l1) / T);
    # on the boundary u1 = u0 ** exp(-(l0 - l1) / T) the two perturbed values are equal and the lower index wins
    l0, l1, T = 0.4, -0.9, 0.8
    u0 = 0.37
    u1_edge = u0 ** np.exp(-(l0 - l1) / T)
    assert osmp.sample_gumbel([l0, l1], T, [u0, u1_edge * (1 - 1e-9)])[0] == 0
    assert osmp.sample_gumbel([l0, l1], T, [u0, min(u1_edge * (1 + 1e-6), 1 - 1e-12)])[0] == 1
    tok, gap = osmp.sample_gumbel([l0, l1], T, [u0, u0])              # equal noise: the larger logit, gap = (l0 - l1) / T
    assert tok == 0 and abs(gap - (l0 - l1) / T) < 1e-12


def test_sampled_chain_with_constant_noise_is_the_greedy_chain_and_follows_its_own_tokens():
    """Equal uniform numbers shift every logit by the same amount, so the sampled chain must coincide with the pinned
    greedy chain (ids, logits, cache rows); with real noise every step's logits must equal the pinned chain
    teacher-forced along the tokens that were drawn (a wrong residual row, a stale feature or token fails)."""
    from tests.test_oracle_tree import setup, chain
    dims, W, o, ids, hidden, rho, Kc, Vc = setup(seed=3, T=6)
    k, T = 4, len(ids)
    u = np.full((k, dims.vocab), 0.42)
    K1, V1 = Kc.copy(), Vc.copy()
    got_ids, got_logits, gaps = osmp.draft_sampled(o, T - 1, int(ids[-1]), hidden[-1], k, rho, K1, V1, 0.7, u)
    ref, K2, V2 = chain(o, ids, hidden, rho, [], k)
    np.testing.assert_array_equal(got_ids, ref["ids"])
    np.testing.assert_allclose(got_logits, ref["logits"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(K1[:T - 1 + k], K2[:T - 1 + k], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(V1[:T - 1 + k], V2[:T - 1 + k], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gaps, ref["gaps"] / 0.7, rtol=1e-9)

    rng = np.random.default_rng(5)
    u = rng.random((k, dims.vocab))
    T_hot = float(np.ptp(ref["logits"][0]))                       # hot enough for the noise to matter
    K1, V1 = Kc.copy(), Vc.copy()
    s_ids, s_logits, _ = osmp.draft_sampled(o, T - 1, int(ids[-1]), hidden[-1], k, rho, K1, V1, T_hot, u)
    assert not np.array_equal(s_ids, ref["ids"])                     # the noise moved at least one token (seeded)
    forced, K3, V3 = chain(o, ids, hidden, rho, list(s_ids), k)
    np.testing.assert_allclose(s_logits, forced["logits"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(K1[:T - 1 + k], K3[:T - 1 + k], rtol=1e-12, atol=1e-12)
    for s in range(k):
        assert s_ids[s] == osmp.sample_gumbel(s_logits[s], T_hot, u[s])[0]
