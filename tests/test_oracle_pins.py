"""Pins for the CPU oracle: closed forms, invariants, library special cases, brute force.

Nothing here touches the CUDA path.  Each test is chosen so that a plausible slip in the
oracle (dropped term, wrong sign or index, transposed operand) breaks it.
"""
import itertools
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import hivis_inputs as hi
import oracle
from hivis_inputs import DrafterDims


def small_dims(**kw):
    base = dict(d=32, n_q_heads=4, n_kv_heads=2, head_dim=8, ffn=40, vocab=50, rms_eps=1e-5,
                rope_base=10000.0, dtype="f32", n_resid=4)
    base.update(kw)
    return DrafterDims(**base)


def rand_weights(dims, seed=0, scale=0.3, bias=False):
    rng = np.random.default_rng(seed)
    W = {n: (rng.standard_normal(s) * scale).astype(np.float32) for n, s in dims.weight_shapes().items()}
    W["norm1"] = (1 + 0.1 * rng.standard_normal(dims.d)).astype(np.float32)
    W["norm2"] = (1 + 0.1 * rng.standard_normal(dims.d)).astype(np.float32)
    if bias:
        W["bq"] = rng.standard_normal(dims.q_dim).astype(np.float32)
        W["bk"] = rng.standard_normal(dims.kv_dim).astype(np.float32)
        W["bv"] = rng.standard_normal(dims.kv_dim).astype(np.float32)
    return W


@pytest.fixture(scope="module")
def orc():
    dims = small_dims()
    return oracle.Oracle(dims, rand_weights(dims), "f64")


# ------------------------------------------------------------------ fusion (Sec. 3.2; Algorithm 1, the fusion step)
def test_fuse_equals_two_products(orc):
    d = orc.dims.d
    rng = np.random.default_rng(1)
    f, rho, tok = rng.standard_normal(d), rng.standard_normal(d), 17
    fc = orc._keep["fc"].astype(np.float64)
    w1_t, w2_t = fc[:, :d], fc[:, d:]          # paper's w1, w2 transposed
    e = orc._keep["embed"][tok].astype(np.float64)
    want = f @ w1_t.T + e @ w2_t.T + rho
    np.testing.assert_allclose(orc.fuse(f, tok, rho), want, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.fuse(f, tok, None), want - rho, rtol=1e-12, atol=1e-12)


def test_fuse_halves_are_not_swapped():
    dims = small_dims()
    W = rand_weights(dims)
    W0 = dict(W); W0["fc"] = W["fc"].copy(); W0["fc"][:, dims.d:] = 0   # w2 = 0: ids cannot matter
    o = oracle.Oracle(dims, W0)
    f = np.random.default_rng(2).standard_normal(dims.d)
    np.testing.assert_array_equal(o.fuse(f, 3), o.fuse(f, 44))
    W1 = dict(W); W1["fc"] = W["fc"].copy(); W1["fc"][:, :dims.d] = 0   # w1 = 0: hidden cannot matter
    o = oracle.Oracle(dims, W1)
    np.testing.assert_array_equal(o.fuse(f, 3), o.fuse(2 * f + 1, 3))
    assert np.abs(o.fuse(f, 3) - o.fuse(f, 44)).max() > 1e-3


def test_fold_residuals(orc):
    d = orc.dims.d
    rng = np.random.default_rng(3)
    r = rng.standard_normal((4, d)).astype(np.float32)
    w = rng.standard_normal((d, d)).astype(np.float32)
    np.testing.assert_allclose(orc.fold_residuals(r, w), r.astype(np.float64) @ w.astype(np.float64).T,
                               rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(orc.fold_residuals(r, None), r.astype(np.float64))


# ------------------------------------------------------------------ RMSNorm
def test_rmsnorm_unit_rms_and_scale_invariance(orc):
    x = np.random.default_rng(4).standard_normal(64) * 7
    y = orc.rmsnorm(x, np.ones(64), 0.0)
    assert abs(np.sqrt(np.mean(y ** 2)) - 1) < 1e-12
    np.testing.assert_allclose(orc.rmsnorm(13.0 * x, np.ones(64), 0.0), y, rtol=1e-12)


def test_rmsnorm_matches_torch(orc):
    rng = np.random.default_rng(5)
    x, g = rng.standard_normal(48), rng.standard_normal(48).astype(np.float32)
    want = F.rms_norm(torch.tensor(x), (48,), torch.tensor(g, dtype=torch.float64), 1e-5).numpy()
    np.testing.assert_allclose(orc.rmsnorm(x, g, 1e-5), want, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ RoPE closed forms
def test_rope_position_zero_is_identity(orc):
    x = np.random.default_rng(6).standard_normal(3 * 16)
    np.testing.assert_array_equal(orc.rope(x, 3, 16, 10000.0, 0), x)


def test_rope_one_hot_gives_cos_sin(orc):
    dh, base, pos = 16, 10000.0, 7
    for i in range(dh // 2):
        x = np.zeros(dh); x[i] = 1.0
        y = orc.rope(x, 1, dh, base, pos)
        th = pos * base ** (-2.0 * i / dh)
        want = np.zeros(dh); want[i] = math.cos(th); want[i + dh // 2] = math.sin(th)
        np.testing.assert_allclose(y, want, atol=1e-15)
        x = np.zeros(dh); x[i + dh // 2] = 1.0
        y = orc.rope(x, 1, dh, base, pos)
        want = np.zeros(dh); want[i] = -math.sin(th); want[i + dh // 2] = math.cos(th)
        np.testing.assert_allclose(y, want, atol=1e-15)


def test_rope_is_complex_rotation_and_relative(orc):
    dh, base, H = 32, 500.0, 2
    rng = np.random.default_rng(7)
    q, k = rng.standard_normal(H * dh), rng.standard_normal(H * dh)
    inv = base ** (-2.0 * np.arange(dh // 2) / dh)

    def cplx(x, pos):
        xh = x.reshape(H, dh)
        z = (xh[:, :dh // 2] + 1j * xh[:, dh // 2:]) * np.exp(1j * pos * inv)
        return np.concatenate([z.real, z.imag], axis=1).reshape(-1)

    np.testing.assert_allclose(orc.rope(q, H, dh, base, 11), cplx(q, 11), atol=1e-14)
    np.testing.assert_allclose(np.linalg.norm(orc.rope(q, H, dh, base, 123)), np.linalg.norm(q), rtol=1e-13)
    a = orc.rope(q, H, dh, base, 9).reshape(H, dh) @ orc.rope(k, H, dh, base, 4).reshape(H, dh).T
    b = orc.rope(q, H, dh, base, 9 + 30).reshape(H, dh) @ orc.rope(k, H, dh, base, 4 + 30).reshape(H, dh).T
    np.testing.assert_allclose(np.diag(a), np.diag(b), atol=1e-12)   # depends on p - t only


# ------------------------------------------------------------------ attention
def test_attend_matches_torch_sdpa_gqa(orc):
    D = orc.dims
    L = 9
    rng = np.random.default_rng(8)
    q = rng.standard_normal(orc.qw)
    Kc, Vc = rng.standard_normal((L, orc.kvw)), rng.standard_normal((L, orc.kvw))
    G = D.n_q_heads // D.n_kv_heads
    tq = torch.tensor(q).view(1, D.n_q_heads, 1, D.head_dim)
    tk = torch.tensor(Kc).view(L, D.n_kv_heads, D.head_dim).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    tv = torch.tensor(Vc).view(L, D.n_kv_heads, D.head_dim).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    want = F.scaled_dot_product_attention(tq, tk, tv).reshape(-1).numpy()
    np.testing.assert_allclose(orc.attend(q, Kc, Vc, L), want, rtol=1e-12, atol=1e-13)
    # only the first `length` rows may be read
    np.testing.assert_allclose(orc.attend(q, Kc, Vc, 4),
                               F.scaled_dot_product_attention(tq, tk[:, :, :4], tv[:, :, :4]).reshape(-1).numpy(),
                               rtol=1e-12, atol=1e-13)


def test_attend_single_row_returns_v0(orc):
    D = orc.dims
    rng = np.random.default_rng(9)
    q, Kc, Vc = rng.standard_normal(orc.qw), rng.standard_normal((1, orc.kvw)), rng.standard_normal((1, orc.kvw))
    G = D.n_q_heads // D.n_kv_heads
    want = np.repeat(Vc.reshape(D.n_kv_heads, D.head_dim), G, axis=0).reshape(-1)
    np.testing.assert_allclose(orc.attend(q, Kc, Vc, 1), want, rtol=1e-15)


def test_attend_large_scores_do_not_overflow(orc):
    rng = np.random.default_rng(10)
    q = rng.standard_normal(orc.qw) * 1e3
    Kc, Vc = rng.standard_normal((6, orc.kvw)) * 1e3, rng.standard_normal((6, orc.kvw))
    out = orc.attend(q, Kc, Vc, 6)
    assert np.isfinite(out).all()


# ------------------------------------------------------------------ SwiGLU
def test_mlp_closed_forms():
    dims = small_dims()
    W = rand_weights(dims)
    y = np.random.default_rng(11).standard_normal(dims.d)
    W0 = dict(W); W0["w_down"] = np.zeros_like(W["w_down"])
    g, _ = oracle.Oracle(dims, W0).mlp(y)
    np.testing.assert_array_equal(g, y)                      # W_d = 0  =>  g = y
    o = oracle.Oracle(dims, W)
    g, act = o.mlp(y)
    m = F.rms_norm(torch.tensor(y), (dims.d,), torch.tensor(W["norm2"], dtype=torch.float64), dims.rms_eps)
    gate = torch.tensor(W["w_gate"], dtype=torch.float64) @ m
    up = torch.tensor(W["w_up"], dtype=torch.float64) @ m
    want_act = F.silu(gate) * up
    np.testing.assert_allclose(act, want_act.numpy(), rtol=1e-12, atol=1e-14)
    want = torch.tensor(y) + torch.tensor(W["w_down"], dtype=torch.float64) @ want_act
    np.testing.assert_allclose(g, want.numpy(), rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ argmax
def test_argmax_first_maximum_and_gap(orc):
    x = np.array([0.5, 3.0, -1.0, 3.0, 2.0, 3.0])
    i, gap = orc.argmax(x)
    assert i == int(np.argmax(x)) == 1 and gap == 0.0
    x = np.array([0.5, -3.0, 7.25, 3.0])
    i, gap = orc.argmax(x)
    assert i == 2 and gap == 4.25
    rng = np.random.default_rng(12)
    for _ in range(50):
        x = rng.integers(0, 6, size=40).astype(np.float64)
        assert orc.argmax(x)[0] == int(np.argmax(x))
    x = np.array([1.0, np.nan, 0.5])
    assert orc.argmax(x)[0] == 0                               # a NaN never wins


# ------------------------------------------------------------------ whole layer
def numpy_drafter(dims, W, ids, hidden, k, rho, forced=None):
    """Independent float64 restatement of Algorithm 1's draft loop: full-sequence matrix
    form with an explicit causal mask, no cache, written separately from the C++ oracle."""
    W = {n: np.asarray(v, np.float64) for n, v in W.items()}
    d, H, Hk, dh = dims.d, dims.n_q_heads, dims.n_kv_heads, dims.head_dim
    half = dh // 2
    X = [np.concatenate([hidden[p].astype(np.float64), W["embed"][ids[p]]]) for p in range(len(ids))]
    rows = [0] * len(ids)
    out_ids, out_logits = [], []

    def norm(x, g):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + dims.rms_eps) * g

    def rot(x, nh):                                           # x [L, nh*dh]
        L = x.shape[0]
        xh = x.reshape(L, nh, dh)
        ang = np.arange(L)[:, None] * dims.rope_base ** (-2.0 * np.arange(half) / dh)[None, :]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        a, b = xh[..., :half], xh[..., half:]
        return np.concatenate([a * c - b * s, b * c + a * s], -1)

    for s in range(k):
        Xm = np.stack(X)                                      # [L, 2d]
        L = Xm.shape[0]
        U = Xm @ W["fc"].T + rho[rows]
        A = norm(U, W["norm1"])
        Q = rot(A @ W["wq"].T + (W["bq"] if "bq" in W else 0), H)
        K = rot(A @ W["wk"].T + (W["bk"] if "bk" in W else 0), Hk)
        Vv = (A @ W["wv"].T + (W["bv"] if "bv" in W else 0)).reshape(L, Hk, dh)
        K = np.repeat(K, H // Hk, axis=1); Vv = np.repeat(Vv, H // Hk, axis=1)
        S = np.einsum("phi,thi->hpt", Q, K) / math.sqrt(dh)
        S = np.where(np.tril(np.ones((L, L), bool))[None], S, -np.inf)
        P = np.exp(S - S.max(-1, keepdims=True)); P /= P.sum(-1, keepdims=True)
        O = np.einsum("hpt,thi->phi", P, Vv).reshape(L, H * dh)
        Y = U + O @ W["wo"].T
        M = norm(Y, W["norm2"])
        gate = M @ W["w_gate"].T
        Gf = Y + ((gate / (1 + np.exp(-gate))) * (M @ W["w_up"].T)) @ W["w_down"].T
        logits = W["lm_head"] @ Gf[-1]
        tok = int(np.argmax(logits))
        out_ids.append(tok); out_logits.append(logits)
        nxt = tok if forced is None else int(forced[s])
        X.append(np.concatenate([Gf[-1], W["embed"][nxt]]))
        rows.append(min(s + 1, rho.shape[0] - 1))
    return np.array(out_ids), np.stack(out_logits)


@pytest.mark.parametrize("bias", [False, True])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (4, 1)])
def test_incremental_equals_bruteforce_equals_numpy(hq, hkv, bias):
    dims = small_dims(d=24, n_q_heads=hq, n_kv_heads=hkv, head_dim=6, ffn=20, vocab=31)
    W = rand_weights(dims, seed=20 + hq + hkv, scale=0.4, bias=bias)
    rng = np.random.default_rng(21)
    T, k = 6, 5
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((3, dims.d)).astype(np.float32)
    o = oracle.Oracle(dims, W)
    inc = o.run_batch(ids, hidden, np.array([0, T]), k, resid)[0]
    bf = o.draft_bruteforce(ids, hidden, k, o.fold_residuals(resid))
    ref_ids, ref_logits = numpy_drafter(dims, W, ids, hidden, k, resid.astype(np.float64))
    np.testing.assert_array_equal(inc["ids"], bf["ids"])
    np.testing.assert_array_equal(inc["ids"], ref_ids)
    np.testing.assert_allclose(inc["logits"], bf["logits"], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(inc["logits"], ref_logits, rtol=1e-9, atol=1e-10)
    # teacher forcing feeds the forced token, still reports the argmax
    forced = rng.integers(0, dims.vocab, k).astype(np.int32)
    incf = o.run_batch(ids, hidden, np.array([0, T]), k, resid, forced_ids=forced[None])[0]
    _, ref_logits_f = numpy_drafter(dims, W, ids, hidden, k, resid.astype(np.float64), forced)
    np.testing.assert_allclose(incf["logits"], ref_logits_f, rtol=1e-9, atol=1e-10)
    bff = o.draft_bruteforce(ids, hidden, k, o.fold_residuals(resid), forced)
    np.testing.assert_allclose(incf["logits"], bff["logits"], rtol=1e-10, atol=1e-11)


def test_layer_reduces_to_two_gemvs_when_wo_wd_zero():
    dims = small_dims()
    W = rand_weights(dims)
    W["wo"] = np.zeros_like(W["wo"]); W["w_down"] = np.zeros_like(W["w_down"])
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(22)
    T, k = 3, 1
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((4, dims.d)).astype(np.float32)
    out = o.run_batch(ids, hidden, np.array([0, T]), k, resid)[0]
    x = np.concatenate([hidden[-1], W["embed"][ids[-1]]]).astype(np.float64)
    want = W["lm_head"].astype(np.float64) @ (W["fc"].astype(np.float64) @ x + resid[0])
    np.testing.assert_allclose(out["logits"][0], want, rtol=1e-11, atol=1e-12)


def test_t1_and_k1_are_legal():
    dims = small_dims()
    W = rand_weights(dims)
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(23)
    ids = rng.integers(0, dims.vocab, 1).astype(np.int32)
    hidden = rng.standard_normal((1, dims.d)).astype(np.float32)
    resid = rng.standard_normal((4, dims.d)).astype(np.float32)
    a = o.run_batch(ids, hidden, np.array([0, 1]), 1, resid)[0]
    b = o.draft_bruteforce(ids, hidden, 1, o.fold_residuals(resid))
    np.testing.assert_array_equal(a["ids"], b["ids"])
    ref_ids, ref_logits = numpy_drafter(dims, W, ids, hidden, 1, resid.astype(np.float64))
    np.testing.assert_allclose(a["logits"], ref_logits, rtol=1e-9, atol=1e-10)


# ------------------------------------------------------------------ residual schedule ("Training Setup": reuse r^3)
def _golden_lines(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    return [l.strip() for l in open(path) if l.strip() and not l.startswith("#")]


def test_residual_row_schedule_follows_reuse_rule():
    want_rows = [int(x) for x in _golden_lines("residual_schedule_R4_k7.txt")[0].split()]
    assert want_rows == [0, 1, 2, 3, 3, 3, 3]
    dims = small_dims()
    W = rand_weights(dims)
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(24)
    T, k = 4, 7
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((4, dims.d)).astype(np.float32)
    got = o.run_batch(ids, hidden, np.array([0, T]), k, resid)[0]
    # chain the positions by hand with the row list taken from the paper's rule
    rho = resid.astype(np.float64)
    Kc, Vc = o.new_cache(T + k)
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    f, tok = hidden[-1].astype(np.float64), int(ids[-1])
    lm = W["lm_head"].astype(np.float64)
    for s in range(k):
        g = o.position(f, tok, rho[want_rows[s]], T - 1 + s, Kc, Vc)
        logits = lm @ g
        np.testing.assert_allclose(got["logits"][s], logits, rtol=1e-10, atol=1e-11)
        tok, f = int(np.argmax(logits)), g
        assert tok == got["ids"][s]


def test_single_residual_row_and_zero_residual():
    dims = small_dims()
    W = rand_weights(dims)
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(25)
    T, k = 4, 5
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    r1 = rng.standard_normal((1, dims.d)).astype(np.float32)
    a = o.run_batch(ids, hidden, np.array([0, T]), k, r1)[0]
    b = o.run_batch(ids, hidden, np.array([0, T]), k, np.repeat(r1, 4, 0))[0]
    np.testing.assert_array_equal(a["logits"], b["logits"])            # R = 1: row 0 everywhere
    z = o.run_batch(ids, hidden, np.array([0, T]), k, np.zeros((4, dims.d), np.float32))[0]
    ref_ids, ref_logits = numpy_drafter(dims, W, ids, hidden, k, np.zeros((1, dims.d)))
    np.testing.assert_allclose(z["logits"], ref_logits, rtol=1e-9, atol=1e-10)
    assert np.abs(z["logits"] - a["logits"]).max() > 1e-3


# ------------------------------------------------------------------ text-only KV bookkeeping
def test_cache_rows_written_are_exactly_text_positions():
    dims = small_dims()
    o = oracle.Oracle(dims, rand_weights(dims))
    rng = np.random.default_rng(26)
    T, k = 5, 3
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((4, dims.d)).astype(np.float32)
    rho = o.fold_residuals(resid)
    Kc, Vc = o.new_cache(T + k + 2)
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    written = np.abs(Kc).sum(1) > 0
    assert written.tolist() == [True] * (T - 1) + [False] * (k + 3)    # T-1 rows + 1 pending pair = T
    o.draft(T - 1, int(ids[-1]), hidden[-1], k, rho, Kc, Vc)
    written = np.abs(Kc).sum(1) > 0
    assert written.tolist() == [True] * (T + k - 1) + [False] * 3      # n_cached == T + k - 1


# ------------------------------------------------------------------ refresh of drafted rows (Algorithm 1, after verification; Eq. 2)
@pytest.mark.parametrize("n_new", [1, 2, 4])
def test_prefill_at_a_start_position_equals_a_prefill_of_the_whole_pair_list(n_new):
    """After a round the accepted tokens come back with TARGET features: every prefix position carries a target
    feature and r^0 (Eq. 2), so rows T.. of the cache are rebuilt from true-feature pairs at their own positions.
    Prefill T pairs, draft k (which fills rows T-1..T+k-2 with self-fed rows), refresh from start_pos = T - 1 with
    the old pending pair followed by n_new new pairs; the next draft must equal the brute-force recompute and the
    numpy restatement on the whole updated pair list.  A refresh that rotated K by p instead of start_pos + p, or
    stored its rows at p, fails here."""
    dims = small_dims(d=24, n_q_heads=4, n_kv_heads=2, head_dim=6, ffn=20, vocab=31)
    W = rand_weights(dims, seed=41, scale=0.4, bias=True)
    o = oracle.Oracle(dims, W)
    rng = np.random.default_rng(42 + n_new)
    T, k = 5, 4
    ids = rng.integers(0, dims.vocab, T).astype(np.int32)
    hidden = rng.standard_normal((T, dims.d)).astype(np.float32)
    resid = rng.standard_normal((3, dims.d)).astype(np.float32)
    rho = o.fold_residuals(resid)
    Kc, Vc = o.new_cache(T + n_new + 2 * k)
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    o.draft(T - 1, int(ids[-1]), hidden[-1], k, rho, Kc, Vc)             # rows T-1 .. T+k-2 now hold drafted rows
    drafted_rows = Kc[T - 1:T + k - 1].copy()
    new_ids = rng.integers(0, dims.vocab, n_new).astype(np.int32)
    new_hidden = rng.standard_normal((n_new, dims.d)).astype(np.float32)
    # the refresh: the old pending pair (its row was written by draft step 0 from the same inputs) and the new pairs
    ref_ids = np.concatenate([ids[-1:], new_ids])
    ref_hidden = np.concatenate([hidden[-1:], new_hidden])
    o.prefill(ref_ids, ref_hidden, rho[0], Kc, Vc, start_pos=T - 1)
    all_ids, all_hidden = np.concatenate([ids, new_ids]), np.concatenate([hidden, new_hidden])
    L = T + n_new
    # rows 0..L-2 are exactly those of one prefill of the whole list; rows beyond were not touched
    K2, V2 = o.new_cache(T + n_new + 2 * k)
    o.prefill(all_ids, all_hidden, rho[0], K2, V2)
    np.testing.assert_array_equal(Kc[:L - 1], K2[:L - 1])
    np.testing.assert_array_equal(Vc[:L - 1], V2[:L - 1])
    if n_new < k:
        np.testing.assert_array_equal(Kc[L - 1:T + k - 1], drafted_rows[n_new:])
    if n_new > 1:                                    # the refreshed rows differ from the self-fed rows they replaced
        assert np.abs(Kc[T:L - 1] - drafted_rows[1:n_new]).max() > 1e-3
    # the next draft from the refreshed cache
    got = o.draft(L - 1, int(all_ids[-1]), all_hidden[-1], k, rho, Kc, Vc)
    bf = o.draft_bruteforce(all_ids, all_hidden, k, rho)
    ref_tok, ref_logits = numpy_drafter(dims, W, all_ids, all_hidden, k, resid.astype(np.float64))
    np.testing.assert_array_equal(got["ids"], bf["ids"])
    np.testing.assert_array_equal(got["ids"], ref_tok)
    np.testing.assert_allclose(got["logits"], bf["logits"], rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(got["logits"], ref_logits, rtol=1e-9, atol=1e-10)


# ------------------------------------------------------------------ verification (Sec. 2.1)
def test_verify_all_match_patterns_bruteforce():
    dims = small_dims()
    o = oracle.Oracle(dims, rand_weights(dims))
    rng = np.random.default_rng(27)
    V = 23
    for k in (1, 2, 3, 4):
        for pattern in itertools.product([0, 1], repeat=k):
            draft = rng.integers(0, V, k).astype(np.int32)
            logits = rng.standard_normal((k + 1, V)).astype(np.float32)
            tgt = np.argmax(logits, 1)
            for j in range(k):                      # make row j agree / disagree as the pattern says
                if pattern[j]:
                    draft[j] = tgt[j]
                elif draft[j] == tgt[j]:
                    draft[j] = (tgt[j] + 1) % V
            want_n = 0
            while want_n < k and pattern[want_n]:
                want_n += 1
            n, nxt, kv = o.verify(draft, logits, base_len=10)
            assert n == want_n and 0 <= n <= k
            assert nxt == tgt[n]
            assert kv == 10 + min(n, k - 1)


def test_verify_ties_take_lowest_index_and_planted_lengths():
    dims = small_dims()
    o = oracle.Oracle(dims, rand_weights(dims))
    logits = np.zeros((3, 8), np.float32)
    logits[0, [2, 5]] = 1.0; logits[1, [4, 6]] = 2.0; logits[2, 7] = 1.0
    assert o.verify(np.array([2, 4]), logits, 3) == (2, 7, 4)
    assert o.verify(np.array([5, 4]), logits, 3) == (0, 2, 3)
    assert o.verify(np.array([2, 6]), logits, 3) == (1, 4, 4)
    wl = hi.scaled(hi.workload("tiny_f32_b4_ragged"), batch=9, k=6)
    draft = np.random.default_rng(28).integers(0, wl.dims.vocab, (9, 6)).astype(np.int32)
    planted = np.array([0, 1, 2, 3, 4, 5, 6, 0, 6])
    logits, planted = hi.make_target_logits(wl, draft, planted)
    for b in range(9):
        n, nxt, kv = o.verify(draft[b], logits[b], 20)
        assert n == planted[b] and nxt == int(np.argmax(logits[b, n]))


# ------------------------------------------------------------------ losslessness of the draft-verify loop
def test_draft_verify_loop_reproduces_target_greedy_stream():
    """With greedy verification the emitted stream equals the target's own greedy stream,
    whatever the drafter proposes (the paper's losslessness claim)."""
    dims = small_dims()
    W = rand_weights(dims, seed=31)
    o = oracle.Oracle(dims, W)
    V, d, k = dims.vocab, dims.d, 4
    rng = np.random.default_rng(32)
    tab = rng.standard_normal((V, V)).astype(np.float32)

    def target_logits(prefix):                      # toy deterministic target: depends on last two tokens
        a, b = prefix[-1], prefix[-2] if len(prefix) > 1 else 0
        return tab[a] + 0.5 * np.roll(tab[b], 3)

    def target_hidden(prefix):                      # any fixed function of the prefix
        r = np.random.default_rng(1000 + 7 * len(prefix) + int(prefix[-1]))
        return r.standard_normal(d).astype(np.float32)

    prompt = [int(t) for t in rng.integers(0, V, 5)]
    plain = list(prompt)
    for _ in range(40):
        plain.append(int(np.argmax(target_logits(plain))))

    resid = rng.standard_normal((4, d)).astype(np.float32)
    rho = o.fold_residuals(resid)
    seq = list(prompt)
    seq.append(int(np.argmax(target_logits(seq))))              # target prefill emits the first token
    Kc, Vc = o.new_cache(200)
    # pairs: (hidden of token p, id of token p+1)
    ids = np.array(seq[1:], np.int32)
    hidden = np.stack([target_hidden(seq[:p + 1]) for p in range(len(seq) - 1)])
    o.prefill(ids, hidden, rho[0], Kc, Vc)
    T = len(ids)
    pend_h, pend_id = hidden[-1], int(ids[-1])
    accepted_hist = []
    while len(seq) < len(plain):
        out = o.draft(T - 1, pend_id, pend_h, k, rho, Kc, Vc)
        draft = out["ids"]
        rows = np.stack([target_logits(seq + [int(t) for t in draft[:j]]) for j in range(k + 1)])
        n, nxt, kv = o.verify(draft, rows, T)
        accepted_hist.append(n)
        new_tokens = [int(t) for t in draft[:n]] + [nxt]
        # refresh: overwrite the self-fed rows with true-feature pairs, last pair pending
        base = list(seq)
        new_ids, new_hidden = [], []
        for t in new_tokens:
            new_hidden.append(target_hidden(base)); new_ids.append(t); base.append(t)
        seq = base
        o.prefill(np.array(new_ids, np.int32), np.stack(new_hidden), rho[0], Kc, Vc, start_pos=T)
        T += len(new_tokens)
        pend_h, pend_id = new_hidden[-1], new_ids[-1]
    assert seq[:len(plain)] == plain
    assert all(0 <= n <= k for n in accepted_hist)


# ------------------------------------------------------------------ f32 build agrees with f64 build
def test_f32_build_close_to_f64_and_golden():
    wl = hi.workload("c1_tiny_f32_b1")
    W = hi.make_weights(wl.dims, wl.seed)
    ids, hid, cu = hi.make_prompt(wl)
    r = hi.make_residuals(wl)
    a = oracle.Oracle(wl.dims, W, "f64").run_batch(ids, hid, cu, wl.k, r)[0]
    b = oracle.Oracle(wl.dims, W, "f32").run_batch(ids, hid, cu, wl.k, r)[0]
    assert np.abs(a["logits"] - b["logits"]).max() < 2e-6
    np.testing.assert_array_equal(a["ids"], b["ids"])


def test_oracle_has_not_drifted_from_frozen_tiny_run():
    import json, os
    doc = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "c1_tiny_oracle.json")))
    wl = hi.workload(doc["workload"])
    W = hi.make_weights(wl.dims, wl.seed)
    ids, hid, cu = hi.make_prompt(wl)
    o = oracle.Oracle(wl.dims, W, "f64")
    out = o.run_batch(ids, hid, cu, wl.k, hi.make_residuals(wl))[0]
    assert [int(t) for t in out["ids"]] == doc["draft_ids"]
    np.testing.assert_allclose(out["logits"][:, :8], np.array(doc["logits_head"]), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(np.abs(out["logits"]).sum(1), np.array(doc["logits_abs_sum"]), rtol=1e-9)
    logits, planted = hi.make_target_logits(wl, out["ids"][None])
    assert o.verify(out["ids"], logits[0], out["T"]) == (doc["accept"], doc["next"], doc["kv_len"])
    assert doc["accept"] == doc["planted_accept"]
