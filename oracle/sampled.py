"""Speculative sampling at temperature T > 0: verification of a chained draft against the target's distributions.
TEST INFRASTRUCTURE ONLY (see the package header).

Sec. 2.1 of the paper states the rule in words (the target accepts the drafted tokens that are consistent with its
distribution, rejects the first that is not together with all that follow, and re-draws the next token "accordingly";
when everything is accepted it draws a new token from its own distribution) and refers to the speculative sampling
of Leviathan et al. and Chen et al. for it.  Written out, with p_j = softmax(target logits row j / T),
q_j = softmax(drafter logits row j / T), x_j the token drafted at step j and the uniform numbers given as inputs:

  accept x_j while  u_accept[j] < min(1, p_j(x_j) / q_j(x_j));   n = number accepted (0..k)
  n < k:  next ~ r / sum(r),  r = max(0, p_n - q_n)      (the residual distribution)
  n = k:  next ~ p_k                                       (the bonus token)
  the draw is the inverse CDF at u_sample: the first token whose cumulative mass exceeds u_sample * total mass.

The drafter's cache keeps base_len + min(n, k-1) rows, as in greedy verification.

Drafting at T > 0 (the paper evaluates T = 1 besides greedy decoding, "Inference Setup"): every chained step draws its
token from q = softmax(logits / T) instead of taking the maximum.  The draw is written as the Gumbel-max rule, which
turns one uniform number per vocabulary entry (given as input) into an exact sample of q:

  token = argmax_i ( logits_i / T - log(-log u_i) ),  u_i uniform in (0, 1), lowest index among equal values.
"""
from __future__ import annotations

import numpy as np


def softmax_t(logits, temperature: float) -> np.ndarray:
    x = np.asarray(logits, np.float64) / float(temperature)
    x = x - x.max()
    e = np.exp(x)
    return e / e.sum()


def accept_ratio(p: np.ndarray, q: np.ndarray, token: int) -> float:
    """min(1, p(x) / q(x)) (1 whenever p(x) >= q(x) > 0; 0 for a token neither side gives any mass)."""
    if p[token] >= q[token]:
        return 1.0 if (p[token] > 0.0 or q[token] > 0.0) else 0.0
    return p[token] / q[token]


def residual(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """max(0, p - q), not normalised."""
    return np.maximum(p - q, 0.0)


def inverse_cdf(mass: np.ndarray, u: float):
    """First index whose cumulative mass exceeds u * total; the last index with positive mass if rounding leaves none.
    Also returns how far (relative to the total) u * total lies from the nearest step of the cumulative sum."""
    c = np.cumsum(np.asarray(mass, np.float64))
    total = c[-1]
    t = u * total
    idx = int(np.searchsorted(c, t, side="right"))
    if idx >= mass.size:
        idx = int(np.nonzero(mass > 0)[0][-1])
    gap = float(np.min(np.abs(c - t)) / total) if total > 0 else 0.0
    return idx, gap


def verify_sampled(draft_ids, draft_logits, target_logits, temperature, u_accept, u_sample, base_len: int):
    """One sequence.  draft_ids [k], draft_logits [k, V], target_logits [k+1, V], u_accept [k], u_sample scalar.
    Returns (n, next, kv_len, (accept margin, draw margin)): the smallest distance of an acceptance number from its
    ratio, and the distance (relative to the total mass) of u_sample * total from the nearest step of the cumulative
    sum - an implementation whose probabilities are off by less decides the same."""
    draft_ids = np.asarray(draft_ids)
    k = draft_ids.size
    margin = np.inf
    n = 0
    while n < k:
        p, q = softmax_t(target_logits[n], temperature), softmax_t(draft_logits[n], temperature)
        a = accept_ratio(p, q, int(draft_ids[n]))
        if a < 1.0 or u_accept[n] >= 1.0:
            margin = min(margin, abs(float(u_accept[n]) - a))
        if not (u_accept[n] < a):
            break
        n += 1
    p = softmax_t(target_logits[n], temperature)
    mass = residual(p, softmax_t(draft_logits[n], temperature)) if n < k else p
    if mass.sum() <= 0.0:            # p == q exactly: nothing is left over, and such a position is never rejected
        mass = p
    nxt, gap = inverse_cdf(mass, float(u_sample))
    return n, nxt, base_len + min(n, k - 1), (margin, gap)


def gumbel(u) -> np.ndarray:
    """Standard Gumbel noise from uniform numbers in (0, 1): -log(-log u)."""
    u = np.asarray(u, np.float64)
    with np.errstate(divide="ignore"):
        return -np.log(-np.log(u))


def sample_gumbel(logits, temperature: float, u):
    """The token drawn from softmax(logits / T) with the uniform numbers u [V], and the gap between the largest and the
    second largest perturbed value (an implementation whose perturbed logits are off by less than half of it draws the
    same token)."""
    z = np.asarray(logits, np.float64) / float(temperature) + gumbel(u)
    tok = int(np.argmax(z))                                  # first maximum
    rest = np.delete(z, tok)
    gap = float(z[tok] - rest.max()) if rest.size else np.inf
    return tok, gap


def draft_sampled(o, n_cached: int, pend_id: int, pend_hidden, k: int, rho, Kc, Vc, temperature: float, u):
    """k chained draft steps of one sequence (Algorithm 1, the drafting loop; Eq. 2) in which the token of every step is
    drawn from softmax(logits / T) by the Gumbel-max rule; u [k, V].  Step 0 runs the pending pair at row n_cached,
    step s >= 1 the pair (layer output of step s-1, token drawn at step s-1) with residual row min(s, R-1); every step
    appends its K/V row to Kc / Vc (modified in place).  Returns ids [k], the unperturbed logits [k, V] and the gaps [k]."""
    lm = o._keep["lm_head"].astype(o.rt)
    R = rho.shape[0]
    f, tok = np.asarray(pend_hidden, o.rt), int(pend_id)
    ids, gaps, logits = np.empty(k, np.int32), np.empty(k), np.empty((k, lm.shape[0]))
    for s in range(k):
        g = o.position(f, tok, rho[min(s, R - 1)], n_cached + s, Kc, Vc)
        logits[s] = lm @ g
        tok, gaps[s] = sample_gumbel(logits[s], temperature, u[s])
        ids[s] = tok
        f = g
    return ids, logits, gaps
