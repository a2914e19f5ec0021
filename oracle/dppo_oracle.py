"""Float64 CPU oracle of the DPPO per-token loss path (numpy, one row at a time).

TEST INFRASTRUCTURE ONLY: never imported by the product package; it shares no
code with the CUDA library.  Everything is evaluated in float64 on the stored
input values (fp32 / bf16 values are upcast exactly by the caller), with no
blocking, fusion or reordering beyond what the definitions state.

What each function restates (paper: "Rethinking the Trust Region in LLM
Reinforcement Learning", DPPO):

* ``log_softmax_row``           pi(.|s_t) is a distribution over the vocabulary (Sec. 3).
* ``ratio``                     r_t = pi(a_t)/mu(a_t)                      (Eq. ppo-clip).
* ``binary_tv`` / ``binary_kl`` Bernoulli collapse on the sampled token    (Eq. binary_tv, Eq. binary_kl).
* ``topk_reduced``              A'_t = TopK(mu, K) u {a_t} plus "other"    (Sec. 4.4, Top-K Approximation).
* ``topk_tv`` / ``topk_kl``     divergences of the reduced categoricals    (Eq. topk_tv, Eq. topk_kl).
* ``full_tv`` / ``full_kl``     exact full-vocabulary divergences          (App. B definitions).
* ``exact_divergence_row``      what the approximations stand in for, from two logits rows: full TV, full KL(mu||pi)
                                (App. B) and the entropy of pi (a run metric of App. E).
* ``dppo_mask``                 asymmetric trust-region mask               (Eq. dppo_obj).
* ``dppo_row`` / ``dppo_loss_fwd_bwd``  surrogate and its logits-gradient   (Eq. dppo_obj, Eq. unified_grad; C = inf unless is_cap is given).
* ``ppo_clip_mask``             ratio-clipping mask of the PPO / GRPO baseline (App. C.1 mask definitions; Eq. ppo-clip).
* ``minimal_mask``              the ablation mask of Sec. 5.3: negative samples whose probability dropped by >= delta.
* variant ``GIVEN_D``           Eq. dppo_obj with the per-token divergence handed in by the caller (e.g. the exact
                                full-vocabulary TV or KL of ``exact_divergence_row``, which the Binary / Top-K forms
                                approximate, Sec. 4.4): the mask rule and everything after it are unchanged.
* ``dppo_fused_lmhead_fwd_bwd`` the same applied to logits = H W with the chain rule into H and W.
* ``dppo_fused_lmhead_sampled`` the same, with the two gradients evaluated only on chosen columns of dW and rows of
                                dHidden (for checks at sizes where the full [T, V] gradient does not fit the host).

Readings of points the paper leaves open (each is listed in the design notes):
the library *minimises*, so loss = -s * sum_t M_t r_t A_t with a caller scale s
(default 1/N_valid); M_t is a constant with respect to the logits; comparisons
are strict as printed; r_t >< 1 is decided as log pi(a_t) >< log mu(a_t);
x*log(x/y) = 0 when x = 0 and +inf when x > 0 = y; "other" masses are clamped
to [0, 1]; the sampled token is never counted twice when it is in the top-K
list, where the list's stored probability is used for it.

Parity pins: every function above is pinned by tests/test_oracle_pins.py
(printed worked example, closed forms, App. B invariants, library routines,
finite differences, brute force); nothing here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BINARY_TV, BINARY_KL, TOPK_TV, TOPK_KL, PPO_CLIP, MINIMAL_MASK, GIVEN_D = 0, 1, 2, 3, 4, 5, 6
VARIANT_NAMES = {BINARY_TV: "binary_tv", BINARY_KL: "binary_kl", TOPK_TV: "topk_tv", TOPK_KL: "topk_kl", PPO_CLIP: "ppo_clip", MINIMAL_MASK: "minimal_mask",
                 GIVEN_D: "given_d"}


def _f64(x):
    return np.asarray(x, dtype=np.float64)


def log_softmax_row(z):
    """log pi_j = z_j - lse, lse = m + log sum_j exp(z_j - m), m = max_j z_j.

    Returns (log_pi[V], lse).  Two plain sweeps over one logits row (Sec. 3:
    the policy is a categorical distribution over the vocabulary).
    """
    z = _f64(z)
    m = np.max(z)
    S = np.sum(np.exp(z - m))
    lse = m + np.log(S)
    return z - lse, lse


def ratio(log_pi_a, mu_logp):
    """r_t = pi(a_t|s_t) / mu(a_t|s_t)  (Eq. ppo-clip), from the two log-probs."""
    return float(np.exp(float(log_pi_a) - float(mu_logp)))


def _xlogx_over_y(x, y):
    """x * log(x / y) with 0*log(0/y) = 0 and x*log(x/0) = +inf for x > 0."""
    x = float(x)
    y = float(y)
    if x == 0.0:
        return 0.0
    if y == 0.0:
        return float("inf")
    return x * (np.log(x) - np.log(y))


def binary_tv(mu_a, pi_a):
    """Eq. binary_tv: | mu(a_t) - pi(a_t) |."""
    return abs(float(mu_a) - float(pi_a))


def binary_kl(mu_a, pi_a):
    """Eq. binary_kl: KL between the Bernoulli collapses (mu(a), 1-mu(a)) and (pi(a), 1-pi(a))."""
    mu_a = float(mu_a)
    pi_a = float(pi_a)
    return _xlogx_over_y(mu_a, pi_a) + _xlogx_over_y(1.0 - mu_a, 1.0 - pi_a)


def topk_reduced(pi, a, mu_a, topk_ids, topk_p):
    """Reduced categoricals over A''_t = A'_t u {other} (Sec. 4.4, Top-K Approximation).

    A'_t is the *set* of the stored top-K ids of mu joined with the sampled id a.
    p_mu(a') is the stored top-K probability for list members (also for a when it
    is a member) and mu_a for a otherwise; p_pi(a') = pi[a'].  "other" is one
    minus the sum over A'_t, clamped to [0, 1]; when A'_t already is the whole
    vocabulary the bucket is empty and both masses are exactly 0.
    Returns (p_mu, p_pi): two float64 arrays of length |A'_t| + 1, "other" last.
    """
    pi = _f64(pi)
    ids = [int(i) for i in np.asarray(topk_ids).reshape(-1)]
    ps = [float(p) for p in _f64(topk_p).reshape(-1)]
    members = {}
    for i, p in zip(ids, ps):
        if i not in members:          # a duplicated id is a caller error; first entry wins
            members[i] = p
    if int(a) not in members:
        members[int(a)] = float(mu_a)
    keys = list(members.keys())
    p_mu = np.array([members[i] for i in keys], dtype=np.float64)
    p_pi = np.array([pi[i] for i in keys], dtype=np.float64)
    if len(keys) == pi.shape[0]:      # A'_t is the whole vocabulary: nothing is left to aggregate
        other_mu = other_pi = 0.0
    else:
        other_mu = min(1.0, max(0.0, 1.0 - float(np.sum(p_mu))))
        other_pi = min(1.0, max(0.0, 1.0 - float(np.sum(p_pi))))
    return np.append(p_mu, other_mu), np.append(p_pi, other_pi)


def topk_tv(p_mu, p_pi):
    """Eq. topk_tv: one half of the L1 distance of the reduced distributions."""
    return 0.5 * float(np.sum(np.abs(_f64(p_mu) - _f64(p_pi))))


def topk_kl(p_mu, p_pi):
    """Eq. topk_kl: sum_a p_mu(a) log(p_mu(a)/p_pi(a)) over the reduced vocabulary."""
    return float(sum(_xlogx_over_y(x, y) for x, y in zip(_f64(p_mu), _f64(p_pi))))


def full_tv(mu, pi):
    """Exact TV over the whole vocabulary: 1/2 sum_a |mu(a) - pi(a)|  (App. B)."""
    return 0.5 * float(np.sum(np.abs(_f64(mu) - _f64(pi))))


def full_kl(mu, pi):
    """Exact KL(mu || pi) over the whole vocabulary  (App. B)."""
    return float(sum(_xlogx_over_y(x, y) for x, y in zip(_f64(mu), _f64(pi))))


def exact_divergence_row(z, z_mu):
    """Full-vocabulary quantities of one state from the trainer's and the rollout policy's logits rows:
    TV = 1/2 sum |mu - pi|, KL(mu || pi) = sum mu log(mu / pi)  (App. B definitions) and the entropy
    -sum pi log pi of the trainer policy.  Returns (tv, kl, entropy)."""
    log_pi, _ = log_softmax_row(z)
    log_mu, _ = log_softmax_row(z_mu)
    pi, mu = np.exp(log_pi), np.exp(log_mu)
    tv = full_tv(mu, pi)
    with np.errstate(invalid="ignore"):              # 0 * log 0 = 0 (entries with probability zero)
        kl = float(np.sum(np.where(mu > 0, mu * (log_mu - log_pi), 0.0)))   # log domain: no 0/0 on underflow
        ent = -float(np.sum(np.where(pi > 0, pi * log_pi, 0.0)))
    return tv, kl, ent


def dppo_mask(adv, log_pi_a, mu_logp, D, delta):
    """Eq. dppo_obj: M = 0 iff (A>0 and r>1 and D>delta) or (A<0 and r<1 and D>delta); else 1.

    r >< 1 is decided in the log domain (log pi(a) >< log mu(a)); all comparisons strict.
    """
    adv = float(adv)
    up = float(log_pi_a) > float(mu_logp)
    down = float(log_pi_a) < float(mu_logp)
    away = (adv > 0.0 and up) or (adv < 0.0 and down)
    return 0 if (away and float(D) > float(delta)) else 1


def ppo_clip_mask(adv, r, eps_low, eps_high):
    """App. C.1, GRPO mask: M = 0 iff (A > 0 and r > 1 + eps_high) or (A < 0 and r < 1 - eps_low); else 1.
    It is the set where the clipped objective of Eq. ppo-clip has zero gradient."""
    adv, r = float(adv), float(r)
    blocked = (adv > 0.0 and r - 1.0 > float(eps_high)) or (adv < 0.0 and 1.0 - r > float(eps_low))
    return 0 if blocked else 1


def minimal_mask(adv, mu_a, pi_a, delta):
    """Sec. 5.3 (source of instability): M = 0 iff A < 0 and mu(a) - pi(a) >= delta; else 1."""
    return 0 if (float(adv) < 0.0 and float(mu_a) - float(pi_a) >= float(delta)) else 1


def divergence(variant, pi, a, mu_logp, topk_ids=None, topk_p=None):
    """D_t of one row for the chosen approximation, given pi[V] (float64 probabilities)."""
    mu_a = float(np.exp(float(mu_logp)))
    pi_a = float(pi[int(a)])
    if variant == BINARY_TV:
        return binary_tv(mu_a, pi_a)
    if variant == BINARY_KL:
        return binary_kl(mu_a, pi_a)
    if variant in (TOPK_TV, TOPK_KL):
        if topk_ids is None:
            topk_ids, topk_p = [], []
        p_mu, p_pi = topk_reduced(pi, a, mu_a, topk_ids, topk_p)
        return topk_tv(p_mu, p_pi) if variant == TOPK_TV else topk_kl(p_mu, p_pi)
    raise ValueError(f"unknown variant {variant}")


def dppo_row(z, a, mu_logp, adv, variant, delta, scale, topk_ids=None, topk_p=None, want_grad=True,
             is_cap=None, eps_low=None, given_D=None):
    """All per-token quantities of one valid row.

    Returns a dict: lse, log_pi_a, r, D, M, loss (= -s*M*w*A), g (= s*M*w*A) with the weight
    w = min(r, C) of Eq. unified_grad (C = is_cap; None or inf: w = r, which is Eq. dppo_obj) and,
    if want_grad, dlogits[V] = g * (pi - onehot(a)): Eq. unified_grad, i.e. the derivative of the
    loss term with M and the truncated weight held constant (d log pi(a)/dz_j = 1[j=a] - pi_j).
    variant PPO_CLIP: D = |r - 1| and the mask is ppo_clip_mask with eps_high = delta and eps_low
    (default: delta), the baseline the paper compares against.  variant MINIMAL_MASK: D = mu(a) - pi(a)
    (signed) and the mask of Sec. 5.3.  variant GIVEN_D: D = given_D (the caller's divergence of this token), mask
    of Eq. dppo_obj.
    """
    log_pi, lse = log_softmax_row(z)
    pi = np.exp(log_pi)
    a = int(a)
    log_pi_a = float(log_pi[a])
    r = ratio(log_pi_a, mu_logp)
    if variant == PPO_CLIP:
        D = abs(r - 1.0)
        M = ppo_clip_mask(adv, r, delta if eps_low is None else eps_low, delta)
    elif variant == MINIMAL_MASK:
        mu_a = float(np.exp(float(mu_logp)))
        D = mu_a - float(pi[a])                      # signed drop of the sampled token's probability
        M = minimal_mask(adv, mu_a, pi[a], delta)
    elif variant == GIVEN_D:
        D = float(given_D)
        M = dppo_mask(adv, log_pi_a, mu_logp, D, delta)
    else:
        D = divergence(variant, pi, a, mu_logp, topk_ids, topk_p)
        M = dppo_mask(adv, log_pi_a, mu_logp, D, delta)
    w = r if (is_cap is None or not np.isfinite(is_cap) or is_cap <= 0) else min(r, float(is_cap))
    g = float(scale) * M * w * float(adv)
    out = dict(lse=float(lse), log_pi_a=log_pi_a, r=r, D=D, M=M, loss=-g, g=g)
    if want_grad:
        d = g * pi
        d[a] -= g
        out["dlogits"] = d
    return out


def default_scale(T, token_mask):
    """Token-mean normaliser s = 1 / N_valid (0 if no row is valid)."""
    n = int(T) if token_mask is None else int(np.count_nonzero(np.asarray(token_mask)))
    return (1.0 / n) if n > 0 else 0.0


def dppo_loss_fwd_bwd(logits, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV,
                      K=0, delta=0.2, loss_scale=None, mu_topk_ids=None, mu_topk_p=None, want_grad=True,
                      is_cap=None, eps_low=None, given_D=None):
    """The whole path over T rows (Eq. dppo_obj summed over tokens, as a loss to minimise).

    logits [T,V]; sampled_ids, mu_logp, advantages [T]; token_mask [T] or None;
    mu_topk_ids / mu_topk_p [T,K] for the Top-K variants; given_D [T] for GIVEN_D.  loss_scale None means
    1/N_valid.  Rows with token_mask == 0 contribute nothing: D = 0, M = 0, zero
    gradient row.  Returns dict(loss, D[T], M[T], r[T], row_loss[T], dlogits[T,V] or None).
    """
    logits = np.asarray(logits)
    T, V = logits.shape
    s = default_scale(T, token_mask) if loss_scale is None else float(loss_scale)
    D = np.zeros(T)
    M = np.zeros(T, dtype=np.uint8)
    r = np.zeros(T)
    row_loss = np.zeros(T)
    dl = np.zeros((T, V)) if want_grad else None
    for t in range(T):
        if token_mask is not None and not token_mask[t]:
            continue
        ids = ps = None
        if variant in (TOPK_TV, TOPK_KL) and K > 0:
            ids, ps = mu_topk_ids[t][:K], mu_topk_p[t][:K]
        o = dppo_row(logits[t], sampled_ids[t], mu_logp[t], advantages[t], variant, delta, s, ids, ps, want_grad,
                     is_cap, eps_low, None if given_D is None else given_D[t])
        D[t], M[t], r[t], row_loss[t] = o["D"], o["M"], o["r"], o["loss"]
        if want_grad:
            dl[t] = o["dlogits"]
    return dict(loss=float(np.sum(row_loss)), D=D, M=M, r=r, row_loss=row_loss, dlogits=dl, scale=s)


def dppo_fused_lmhead_fwd_bwd(hidden, W, sampled_ids, mu_logp, advantages, token_mask=None,
                              variant=BINARY_TV, delta=0.2, loss_scale=None, K=0, mu_topk_ids=None, mu_topk_p=None,
                              is_cap=None, eps_low=None, given_D=None):
    """LM-head variant: logits = hidden @ W in float64 (never rounded), then the path above,
    then the chain rule: dHidden = dlogits @ W^T, dW = hidden^T @ dlogits.
    """
    H = _f64(hidden)
    Wm = _f64(W)
    z = H @ Wm
    o = dppo_loss_fwd_bwd(z, sampled_ids, mu_logp, advantages, token_mask, variant, K, delta, loss_scale,
                          mu_topk_ids, mu_topk_p, True, is_cap, eps_low, given_D)
    o["dHidden"] = o["dlogits"] @ Wm.T
    o["dW"] = H.T @ o["dlogits"]
    return o


def dppo_fused_lmhead_sampled(hidden, W, sampled_ids, mu_logp, advantages, token_mask=None, variant=BINARY_TV,
                              delta=0.2, loss_scale=None, dW_cols=(), dH_rows=(), K=0, mu_topk_ids=None, mu_topk_p=None,
                              is_cap=None, eps_low=None, row_block=256):
    """The LM-head variant where a full evaluation does not fit: loss, D, M, r for ALL rows, but of the two gradients only
    the columns ``dW_cols`` of dW and the rows ``dH_rows`` of dHidden.  Same definitions as ``dppo_fused_lmhead_fwd_bwd``:
    logits = hidden @ W in float64, row by row through ``dppo_row``; dlogits_tj = g_t (pi_tj - 1[j = a_t]) (Eq. unified_grad);
    dW[:, c] = hidden^T @ dlogits[:, c]; dHidden[t] = dlogits[t] @ W^T.  The logits are formed ``row_block`` rows at a
    time to bound memory; nothing else is blocked.  Returns dict(loss, D, M, r, row_loss, dW_cols [d, len(dW_cols)],
    dlogits_cols [T, len(dW_cols)], dHidden_rows [len(dH_rows), d], dlogits_rows [len(dH_rows), V], scale)."""
    H = _f64(hidden)
    Wm = _f64(W)
    T, V = H.shape[0], Wm.shape[1]
    cols = np.asarray(list(dW_cols), dtype=np.int64)
    rows = [int(t) for t in dH_rows]
    s = default_scale(T, token_mask) if loss_scale is None else float(loss_scale)
    D = np.zeros(T)
    M = np.zeros(T, dtype=np.uint8)
    r = np.zeros(T)
    row_loss = np.zeros(T)
    dl_cols = np.zeros((T, len(cols)))
    dl_rows = np.zeros((len(rows), V))
    for t0 in range(0, T, int(row_block)):
        z = H[t0:t0 + int(row_block)] @ Wm
        for i in range(z.shape[0]):
            t = t0 + i
            if token_mask is not None and not token_mask[t]:
                continue
            ids = ps = None
            if variant in (TOPK_TV, TOPK_KL) and K > 0:
                ids, ps = mu_topk_ids[t][:K], mu_topk_p[t][:K]
            o = dppo_row(z[i], sampled_ids[t], mu_logp[t], advantages[t], variant, delta, s, ids, ps, False, is_cap, eps_low)
            D[t], M[t], r[t], row_loss[t] = o["D"], o["M"], o["r"], o["loss"]
            a = int(sampled_ids[t])
            dl_cols[t] = o["g"] * (np.exp(z[i, cols] - o["lse"]) - (cols == a))
            if t in rows:
                full = o["g"] * np.exp(z[i] - o["lse"])
                full[a] -= o["g"]
                dl_rows[rows.index(t)] = full
    return dict(loss=float(np.sum(row_loss)), D=D, M=M, r=r, row_loss=row_loss, dW_cols=H.T @ dl_cols, dlogits_cols=dl_cols,
                dHidden_rows=dl_rows @ Wm.T, dlogits_rows=dl_rows, scale=s)
