"""Pins of the float64 oracle to what the paper and the mathematics fix (CPU only).

Each ``check_*`` takes the oracle module (or a mutated copy) so that
``test_planted_mistakes_are_caught`` can show that a plausible mistake planted
in the oracle fails at least one pin.
"""
import itertools
import math
import os
import types

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import dppo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")
rng0 = np.random.default_rng(1234)


def _rand_dist(rng, V, peak=3.0):
    z = peak * rng.standard_normal(V)
    return np.exp(z - scipy.special.logsumexp(z))


def _case(rng, T=6, V=11, K=4, noise=0.3):
    """Random tiny problem with the full rollout distribution available."""
    z = 2.0 * rng.standard_normal((T, V))
    zm = z + noise * rng.standard_normal((T, V))
    mu = np.exp(zm - scipy.special.logsumexp(zm, axis=1, keepdims=True))
    a = np.array([rng.choice(V, p=mu[t]) for t in range(T)])
    mu_logp = np.log(mu[np.arange(T), a])
    order = np.argsort(-mu, axis=1)
    ids = order[:, :K]
    ps = np.take_along_axis(mu, ids, axis=1)
    adv = rng.choice([-1.0, 1.0], T) * rng.uniform(0.2, 1.5, T)
    return dict(z=z, mu=mu, a=a, mu_logp=mu_logp, ids=ids, ps=ps, adv=adv, order=order)


# ----------------------------------------------------------------------------- worked example

def _golden_rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, mu, pi, r, tol, moved = line.split()
        rows.append((name, float(mu), float(pi), float(r), float(tol), float(moved)))
    return rows


def check_worked_example(O):
    """Sec. 4.2 / Sec. 1 printed numbers: ratios 100 and ~0.808, moved mass 0.19."""
    for name, mu, pi, r_print, tol, moved in _golden_rows():
        # a three-token row whose softmax is (pi, (1-pi)/2, (1-pi)/2), sampled token 0
        z = np.log(np.array([pi, (1 - pi) / 2, (1 - pi) / 2])) + 7.25
        o = O.dppo_row(z, 0, math.log(mu), 1.0, O.BINARY_TV, 0.2, 1.0)
        assert abs(o["r"] - r_print) <= tol * max(1.0, r_print) + 1e-12, name
        assert abs(o["D"] - abs(mu - pi)) < 1e-12, name
        if not math.isnan(moved):
            assert abs(o["D"] - moved) < 1e-9, name
    # Sec. 4.2 with delta = 0.2 (the typical value printed there for epsilon): Binary-TV lets both
    # tokens through, whereas |r-1| > 0.2 would stop the low-probability token for A > 0.
    low = O.dppo_row(np.log([1e-2, 0.495, 0.495]), 0, math.log(1e-4), +1.0, O.BINARY_TV, 0.2, 1.0)
    high = O.dppo_row(np.log([0.80, 0.1, 0.1]), 0, math.log(0.99), -1.0, O.BINARY_TV, 0.2, 1.0)
    assert low["M"] == 1 and high["M"] == 1
    assert O.dppo_mask(+1.0, math.log(1e-2), math.log(1e-4), abs(low["r"] - 1.0), 0.2) == 0
    assert O.dppo_mask(-1.0, math.log(0.80), math.log(0.99), abs(high["r"] - 1.0), 0.2) == 1


# ----------------------------------------------------------------------------- softmax / ratio

def check_log_softmax(O):
    rng = np.random.default_rng(1)
    for V in (1, 2, 7, 300):
        z = 5 * rng.standard_normal(V)
        lp, lse = O.log_softmax_row(z)
        np.testing.assert_allclose(lp, scipy.special.log_softmax(z), rtol=0, atol=1e-12)
        assert abs(lse - scipy.special.logsumexp(z)) < 1e-12
        assert abs(np.exp(lp).sum() - 1) < 1e-12
        lp2, lse2 = O.log_softmax_row(z + 900.0)       # shift invariance, no overflow
        np.testing.assert_allclose(lp2, lp, atol=1e-9)
        assert abs(lse2 - lse - 900.0) < 1e-9
    assert abs(O.ratio(math.log(0.3), math.log(0.12)) - 2.5) < 1e-12


# ----------------------------------------------------------------------------- binary

def check_binary(O):
    rng = np.random.default_rng(2)
    for _ in range(50):
        mu, pi = rng.uniform(1e-6, 1 - 1e-6, 2)
        assert O.binary_tv(mu, pi) == abs(mu - pi)
        ref = scipy.stats.entropy([mu, 1 - mu], [pi, 1 - pi])          # library Bernoulli KL
        assert abs(O.binary_kl(mu, pi) - ref) < 1e-12
        assert O.binary_tv(mu, pi) ** 2 <= 0.5 * O.binary_kl(mu, pi) + 1e-15   # Pinsker
    assert O.binary_kl(0.3, 0.3) == 0.0
    assert O.binary_kl(0.0, 0.25) == pytest.approx(-math.log(0.75))
    assert O.binary_kl(0.5, 0.0) == float("inf")
    # KL(mu||pi) is the expectation under mu (direction): not symmetric
    assert abs(O.binary_kl(0.9, 0.5) - O.binary_kl(0.5, 0.9)) > 1e-3
    assert abs(O.binary_kl(0.9, 0.5) - (0.9 * math.log(0.9 / 0.5) + 0.1 * math.log(0.1 / 0.5))) < 1e-15


# ----------------------------------------------------------------------------- top-K

def check_topk_full_and_bounds(O):
    """K=V is the exact divergence; K=0 is Binary; D_bin <= D_topK <= D_full, monotone in K (App. B)."""
    rng = np.random.default_rng(3)
    for V in (2, 5, 16):
        c = _case(rng, T=8, V=V, K=V)
        for t in range(8):
            lp, _ = O.log_softmax_row(c["z"][t])
            pi, mu, a = np.exp(lp), c["mu"][t], c["a"][t]
            tv_lib = 0.5 * np.abs(mu - pi).sum()
            kl_lib = scipy.special.rel_entr(mu, pi).sum()
            assert abs(O.full_tv(mu, pi) - tv_lib) < 1e-13 and abs(O.full_kl(mu, pi) - kl_lib) < 1e-13
            # Eq. tv_as_expectation: TV = 1/2 E_{y~mu} |r - 1|, by exact enumeration over the vocabulary
            tv_exp = 0.5 * sum(mu[j] * abs(O.ratio(lp[j], math.log(mu[j])) - 1.0) for j in range(V))
            assert abs(tv_exp - tv_lib) < 1e-12
            prev_tv = prev_kl = None
            for K in range(0, V + 1):
                ids, ps = c["order"][t][:K], mu[c["order"][t][:K]]
                tv = O.divergence(O.TOPK_TV, pi, a, c["mu_logp"][t], ids, ps)
                kl = O.divergence(O.TOPK_KL, pi, a, c["mu_logp"][t], ids, ps)
                if K == 0:
                    assert abs(tv - O.binary_tv(mu[a], pi[a])) < 1e-13
                    assert abs(kl - O.binary_kl(mu[a], pi[a])) < 1e-13
                else:
                    assert tv >= prev_tv - 1e-13 and kl >= prev_kl - 1e-13
                assert tv <= tv_lib + 1e-13 and kl <= kl_lib + 1e-13
                assert tv * tv <= 0.5 * kl + 1e-13                       # Pinsker on the reduced pair
                prev_tv, prev_kl = tv, kl
            assert abs(prev_tv - tv_lib) < 1e-12 and abs(prev_kl - kl_lib) < 1e-12
            # order of the list is irrelevant
            perm = rng.permutation(V)[: max(1, V // 2)]
            d1 = O.divergence(O.TOPK_KL, pi, a, c["mu_logp"][t], perm, mu[perm])
            d2 = O.divergence(O.TOPK_KL, pi, a, c["mu_logp"][t], perm[::-1], mu[perm[::-1]])
            assert abs(d1 - d2) < 1e-13


def check_topk_other_bucket(O):
    """'other' aggregates every token outside A'_t; the sampled token joins the set only once."""
    rng = np.random.default_rng(4)
    V, K = 12, 3
    c = _case(rng, T=10, V=V, K=K)
    for t in range(10):
        lp, _ = O.log_softmax_row(c["z"][t])
        pi, mu, a = np.exp(lp), c["mu"][t], int(c["a"][t])
        for ids in (c["ids"][t], np.array([j for j in range(V) if j != a][:K]), np.array([a] + [j for j in range(V) if j != a][: K - 1])):
            ps = mu[ids]
            members = sorted(set(int(i) for i in ids) | {a})
            rest = [j for j in range(V) if j not in members]
            p_mu = [mu[j] for j in members] + [sum(mu[j] for j in rest)]     # aggregation written out
            p_pi = [pi[j] for j in members] + [sum(pi[j] for j in rest)]
            tv = 0.5 * sum(abs(x - y) for x, y in zip(p_mu, p_pi))
            kl = sum(x * math.log(x / y) for x, y in zip(p_mu, p_pi))
            assert abs(O.divergence(O.TOPK_TV, pi, a, c["mu_logp"][t], ids, ps) - tv) < 1e-13
            assert abs(O.divergence(O.TOPK_KL, pi, a, c["mu_logp"][t], ids, ps) - kl) < 1e-13
            q_mu, q_pi = O.topk_reduced(pi, a, mu[a], ids, ps)
            assert len(q_mu) == len(members) + 1
            assert abs(q_mu.sum() - 1) < 1e-12 and abs(q_pi.sum() - 1) < 1e-12


def check_topk_equality_conditions(O):
    """App. B: TV is exact when sign(mu-pi) is constant inside 'other'; KL when pi/mu is constant there."""
    V, K = 10, 3
    mu = np.array([0.4, 0.2, 0.1] + [0.3 / 7] * 7)
    # scale the tail of pi uniformly (ratio constant inside 'other'), move the head freely
    tail_scale = 0.5
    pi = mu.copy()
    pi[3:] *= tail_scale
    pi[:3] = np.array([0.5, 0.3, 0.05])
    pi[:3] *= (1 - pi[3:].sum()) / pi[:3].sum()
    a = 1
    ids, ps = np.arange(K), mu[:K]
    tv = O.divergence(O.TOPK_TV, pi, a, math.log(mu[a]), ids, ps)
    kl = O.divergence(O.TOPK_KL, pi, a, math.log(mu[a]), ids, ps)
    assert abs(tv - O.full_tv(mu, pi)) < 1e-13          # mu - pi > 0 on the whole tail
    assert abs(kl - O.full_kl(mu, pi)) < 1e-13          # mu/pi constant on the tail
    # break the conditions: mix signs / ratios inside the tail -> strict lower bound
    pi2 = pi.copy()
    pi2[3] += 0.02
    pi2[4] -= 0.02
    assert O.divergence(O.TOPK_KL, pi2, a, math.log(mu[a]), ids, ps) < O.full_kl(mu, pi2) - 1e-6
    pi3 = mu.copy()
    pi3[3] += 0.03
    pi3[4] -= 0.03
    assert O.divergence(O.TOPK_TV, pi3, a, math.log(mu[a]), ids, ps) < O.full_tv(mu, pi3) - 1e-3


def check_edge_conventions(O):
    pi = np.array([0.5, 0.5, 0.0, 0.0])
    # p_mu > 0 where p_pi = 0 -> +inf; p_mu = 0 contributes 0
    assert O.divergence(O.TOPK_KL, pi, 0, math.log(0.4), [2], [0.1]) == float("inf")
    assert math.isfinite(O.divergence(O.TOPK_KL, pi, 0, math.log(0.5), [1, 2], [0.5, 0.0]))
    # stored top-K probabilities summing slightly above one: 'other' clamps at 0
    q_mu, q_pi = O.topk_reduced(np.array([0.6, 0.4]), 0, 0.6, [0, 1], [0.6000001, 0.4000001])
    assert q_mu[-1] == 0.0 and q_pi[-1] >= 0.0


# ----------------------------------------------------------------------------- mask

def check_mask_truth_table(O):
    """Eq. dppo_obj: exactly two of the sign(A) x (r vs 1) x (D vs delta) cells are blocked."""
    delta = 0.2
    zero_cells = 0
    for adv, dlog, D in itertools.product((-1.0, 0.0, 1.0), (-0.3, 0.0, 0.3), (0.1, 0.2, 0.3)):
        M = O.dppo_mask(adv, math.log(0.5) + dlog, math.log(0.5), D, delta)
        expect = 0 if (D > delta and ((adv > 0 and dlog > 0) or (adv < 0 and dlog < 0))) else 1
        assert M == expect
        zero_cells += (M == 0)
        if (adv > 0 and dlog < 0) or (adv < 0 and dlog > 0):      # moving towards r = 1: never blocked
            assert M == 1
    assert zero_cells == 2
    # D := |r-1| turns it into PPO's clip mask: the clipped objective min(rA, clip(r,1-e,1+e)A)
    # has zero derivative with respect to r exactly where that mask is zero (Eq. ppo-clip).
    eps = 0.2
    for adv in (-1.3, 0.7):
        for r in (0.5, 0.79, 0.81, 0.99, 1.01, 1.19, 1.21, 2.5):
            rt = torch.tensor(r, dtype=torch.float64, requires_grad=True)
            obj = torch.minimum(rt * adv, torch.clamp(rt, 1 - eps, 1 + eps) * adv)
            (gr,) = torch.autograd.grad(obj, rt)
            M = O.dppo_mask(adv, math.log(r), 0.0, abs(r - 1.0), eps)
            assert (float(gr) == 0.0) == (M == 0), (adv, r)


# ----------------------------------------------------------------------------- loss and gradient

def check_on_policy(O):
    """pi == mu: D = 0, all-pass mask, r = 1, loss = -s sum A, gradient = plain policy gradient."""
    rng = np.random.default_rng(5)
    T, V, K = 7, 9, 3
    z = rng.standard_normal((T, V)) * 2
    pi = np.exp(z - scipy.special.logsumexp(z, axis=1, keepdims=True))
    a = rng.integers(0, V, T)
    adv = rng.standard_normal(T)
    ids = np.argsort(-pi, axis=1)[:, :K]
    ps = np.take_along_axis(pi, ids, 1)
    mu_logp = np.log(pi[np.arange(T), a])
    for variant in (O.BINARY_TV, O.BINARY_KL, O.TOPK_TV, O.TOPK_KL):
        o = O.dppo_loss_fwd_bwd(z, a, mu_logp, adv, None, variant, K, 0.0, None, ids, ps)
        assert np.all(np.abs(o["D"]) < 1e-12) and np.all(o["M"] == 1)
        np.testing.assert_allclose(o["r"], 1.0, atol=1e-12)
        assert abs(o["loss"] + adv.sum() / T) < 1e-12
        onehot = np.eye(V)[a]
        np.testing.assert_allclose(o["dlogits"], (adv[:, None] / T) * (pi - onehot), atol=1e-13)


def _surrogate_fixed_mask(O, z, c, M, s, minus_one=False):
    """-s sum_t M_t (r_t [-1]) A_t with the mask held fixed, through the oracle's own log-softmax."""
    tot = 0.0
    for t in range(z.shape[0]):
        lp, _ = O.log_softmax_row(z[t])
        r = O.ratio(lp[c["a"][t]], c["mu_logp"][t])
        tot += -s * M[t] * ((r - 1.0) if minus_one else r) * c["adv"][t]
    return tot


def check_gradient(O):
    rng = np.random.default_rng(6)
    T, V, K = 5, 7, 2
    c = _case(rng, T=T, V=V, K=K, noise=0.8)
    tok = np.array([1, 1, 0, 1, 1], dtype=np.uint8)
    for variant, delta in ((O.BINARY_TV, 0.05), (O.TOPK_KL, 0.02)):
        o = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], tok, variant, K, delta, None, c["ids"], c["ps"])
        s = o["scale"]
        assert s == 0.25
        assert 0 < o["M"][tok == 1].sum() < 4 or variant == O.TOPK_KL          # both mask values exercised
        # central finite differences of the summed loss, mask held fixed
        h = 1e-6
        fd = np.zeros((T, V))
        for t in range(T):
            for j in range(V):
                zp, zm = c["z"].copy(), c["z"].copy()
                zp[t, j] += h
                zm[t, j] -= h
                fd[t, j] = (_surrogate_fixed_mask(O, zp, c, o["M"], s) - _surrogate_fixed_mask(O, zm, c, o["M"], s)) / (2 * h)
        np.testing.assert_allclose(o["dlogits"], fd, atol=2e-8)
        # "replacing r-1 with r leaves the gradient unchanged" (Sec. 4.1)
        t, j = 0, 3
        zp, zm = c["z"].copy(), c["z"].copy()
        zp[t, j] += h
        zm[t, j] -= h
        fd1 = (_surrogate_fixed_mask(O, zp, c, o["M"], s, True) - _surrogate_fixed_mask(O, zm, c, o["M"], s, True)) / (2 * h)
        assert abs(fd1 - o["dlogits"][t, j]) < 2e-8
        # autograd of the same surrogate through torch's own log_softmax (float64)
        zt = torch.tensor(c["z"], dtype=torch.float64, requires_grad=True)
        lp = torch.log_softmax(zt, dim=1)[torch.arange(T), torch.tensor(c["a"])]
        loss = -(s * torch.tensor(o["M"].astype(np.float64)) * torch.exp(lp - torch.tensor(c["mu_logp"])) * torch.tensor(c["adv"])).sum()
        loss.backward()
        assert abs(float(loss.detach()) - o["loss"]) < 1e-13
        np.testing.assert_allclose(o["dlogits"], zt.grad.numpy(), atol=1e-13)
        # structure: rows sum to zero; masked and invalid rows are exactly zero
        np.testing.assert_allclose(o["dlogits"].sum(1), 0, atol=1e-13)
        for t in range(T):
            if tok[t] == 0 or o["M"][t] == 0:
                assert np.all(o["dlogits"][t] == 0.0)
        assert o["D"][2] == 0 and o["M"][2] == 0 and o["row_loss"][2] == 0
        # caller-supplied scale
        o2 = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], tok, variant, K, delta, 0.5, c["ids"], c["ps"])
        assert abs(o2["loss"] - o["loss"] * 2) < 1e-13
    empty = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], np.zeros(T, np.uint8), O.BINARY_TV, 0, 0.2)
    assert empty["loss"] == 0.0 and not empty["dlogits"].any()


def check_brute_force_tiny(O):
    """Pure-Python enumeration over tiny vocabularies, all four variants, both mask outcomes."""
    rng = np.random.default_rng(7)
    seen = set()
    for trial in range(200):
        V = int(rng.integers(2, 9))
        K = int(rng.integers(0, V + 1))
        z = [float(x) for x in 2 * rng.standard_normal(V)]
        zmu = [zi + float(x) for zi, x in zip(z, rng.standard_normal(V))]
        Zp = sum(math.exp(x) for x in z)
        Zm = sum(math.exp(x) for x in zmu)
        pi = [math.exp(x) / Zp for x in z]
        mu = [math.exp(x) / Zm for x in zmu]
        a = int(rng.integers(0, V))
        adv = float(rng.choice([-1.0, 1.0]))
        top = sorted(range(V), key=lambda j: -mu[j])[:K]
        delta = float(rng.choice([0.01, 0.05, 0.2]))
        variant = trial % 4
        if variant == O.BINARY_TV:
            D = abs(mu[a] - pi[a])
        elif variant == O.BINARY_KL:
            D = mu[a] * math.log(mu[a] / pi[a]) + (1 - mu[a]) * math.log((1 - mu[a]) / (1 - pi[a]))
        else:
            S = set(top) | {a}
            rest = [j for j in range(V) if j not in S]
            pm = [mu[j] for j in S] + [sum(mu[j] for j in rest)]
            pp = [pi[j] for j in S] + [sum(pi[j] for j in rest)]
            if variant == O.TOPK_TV:
                D = 0.5 * sum(abs(x - y) for x, y in zip(pm, pp))
            else:
                D = sum(x * math.log(x / y) for x, y in zip(pm, pp) if x > 0)
        r = pi[a] / mu[a]
        blocked = D > delta and ((adv > 0 and r > 1) or (adv < 0 and r < 1))
        M = 0 if blocked else 1
        s = 0.37
        o = O.dppo_row(np.array(z), a, math.log(mu[a]), adv, variant, delta, s, np.array(top, dtype=np.int64), np.array([mu[j] for j in top]))
        assert abs(o["D"] - D) < 1e-12 and o["M"] == M and abs(o["r"] - r) < 1e-12 * max(1, r)
        assert abs(o["loss"] - (-s * M * r * adv)) < 1e-12 * max(1, r)
        for j in range(V):
            assert abs(o["dlogits"][j] - s * M * r * adv * (pi[j] - (1.0 if j == a else 0.0))) < 1e-12 * max(1, r)
        seen.add((variant, M))
    assert len(seen) == 8


def check_fused(O):
    rng = np.random.default_rng(8)
    T, d, V = 4, 3, 6
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((d, V))
    z = H @ W
    zmu = z + 0.5 * rng.standard_normal((T, V))
    mu = np.exp(zmu - scipy.special.logsumexp(zmu, axis=1, keepdims=True))
    a = rng.integers(0, V, T)
    mu_logp = np.log(mu[np.arange(T), a])
    adv = rng.choice([-1.0, 1.0], T)
    tok = np.array([1, 1, 1, 0], dtype=np.uint8)
    o = O.dppo_fused_lmhead_fwd_bwd(H, W, a, mu_logp, adv, tok, O.BINARY_TV, 0.05)
    s = O.dppo_loss_fwd_bwd(np.einsum("td,dv->tv", H, W), a, mu_logp, adv, tok, O.BINARY_TV, 0, 0.05)
    assert abs(o["loss"] - s["loss"]) < 1e-14 and np.array_equal(o["M"], s["M"])
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    lp = torch.log_softmax(Ht @ Wt, dim=1)[torch.arange(T), torch.tensor(a)]
    loss = -(o["scale"] * torch.tensor(o["M"].astype(np.float64)) * torch.exp(lp - torch.tensor(mu_logp)) * torch.tensor(adv)).sum()
    loss.backward()
    np.testing.assert_allclose(o["dHidden"], Ht.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(o["dW"], Wt.grad.numpy(), atol=1e-13)
    # finite differences on one entry of each
    c = dict(a=a, mu_logp=mu_logp, adv=adv)
    h = 1e-6
    Hp, Hm = H.copy(), H.copy()
    Hp[1, 2] += h
    Hm[1, 2] -= h
    fd = (_surrogate_fixed_mask(O, Hp @ W, c, o["M"], o["scale"]) - _surrogate_fixed_mask(O, Hm @ W, c, o["M"], o["scale"])) / (2 * h)
    assert abs(fd - o["dHidden"][1, 2]) < 2e-8
    Wp, Wm = W.copy(), W.copy()
    Wp[0, 4] += h
    Wm[0, 4] -= h
    fd = (_surrogate_fixed_mask(O, H @ Wp, c, o["M"], o["scale"]) - _surrogate_fixed_mask(O, H @ Wm, c, o["M"], o["scale"])) / (2 * h)
    assert abs(fd - o["dW"][0, 4]) < 2e-8


def check_fused_sampled(O):
    """The column / row restricted LM-head form against torch autograd (float64) of the surrogate with the mask held
    fixed, and against the full form; ragged row blocks, a token mask, Top-K lists, an importance cap."""
    rng = np.random.default_rng(21)
    T, d, V, K = 23, 5, 17, 4
    H = rng.standard_normal((T, d))
    W = 0.8 * rng.standard_normal((d, V))
    zmu = H @ W + 0.7 * rng.standard_normal((T, V))
    mu = np.exp(zmu - scipy.special.logsumexp(zmu, axis=1, keepdims=True))
    a = np.array([rng.choice(V, p=mu[t]) for t in range(T)])
    mu_logp = np.log(mu[np.arange(T), a])
    ids = np.argsort(-mu, axis=1)[:, :K]
    ps = np.take_along_axis(mu, ids, axis=1)
    adv = rng.choice([-1.0, 1.0], T) * rng.uniform(0.3, 1.2, T)
    tok = (np.arange(T) % 6 != 2).astype(np.uint8)
    cols = [0, 3, int(a[1]), int(a[5]), V - 1]
    rows = [0, 5, 8, T - 1]                 # row 8 is masked out: a zero row
    for variant, delta, cap in ((O.BINARY_TV, 0.03, None), (O.TOPK_KL, 0.02, 1.1)):
        o = O.dppo_fused_lmhead_sampled(H, W, a, mu_logp, adv, tok, variant, delta, None, cols, rows, K, ids, ps, cap, row_block=7)
        f = O.dppo_fused_lmhead_fwd_bwd(H, W, a, mu_logp, adv, tok, variant, delta, None, K, ids, ps, cap)
        assert np.array_equal(o["M"], f["M"]) and 0 < int(((o["M"] == 0) & (tok != 0)).sum())
        np.testing.assert_allclose(o["D"], f["D"], atol=1e-15)
        assert abs(o["loss"] - f["loss"]) < 1e-14
        Ht = torch.tensor(H, requires_grad=True)
        Wt = torch.tensor(W, requires_grad=True)
        lp = torch.log_softmax(Ht @ Wt, dim=1)[torch.arange(T), torch.tensor(a)]
        r = torch.exp(lp - torch.tensor(mu_logp))
        w = r
        if cap is not None:     # Eq. unified_grad: value min(r, C), gradient min(r, C) grad(log pi)
            w = torch.where(r.detach() < cap, r, torch.full_like(r, cap) * (1 + lp - lp.detach()))
        loss = -(o["scale"] * torch.tensor((o["M"] * (tok != 0)).astype(np.float64)) * w * torch.tensor(adv)).sum()
        loss.backward()
        np.testing.assert_allclose(o["dW_cols"], Wt.grad.numpy()[:, cols], atol=1e-13)
        np.testing.assert_allclose(o["dHidden_rows"], Ht.grad.numpy()[rows], atol=1e-13)
        assert not o["dHidden_rows"][2].any() and o["dlogits_rows"].shape == (len(rows), V)
        np.testing.assert_allclose(o["dlogits_cols"], f["dlogits"][:, cols], atol=1e-15)


def check_is_cap_and_baselines(O):
    """Eq. unified_grad: weight min(r, C); C = inf is Eq. dppo_obj; delta = inf gives the unmasked PG-IS / CISPO baselines."""
    rng = np.random.default_rng(9)
    T, V = 12, 9
    c = _case(rng, T=T, V=V, K=3, noise=1.2)
    base = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], None, O.BINARY_TV, 0, 0.05)
    same = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], None, O.BINARY_TV, 0, 0.05, is_cap=float("inf"))
    assert np.array_equal(base["dlogits"], same["dlogits"]) and base["loss"] == same["loss"]
    C = float(np.median(base["r"]))
    cap = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], None, O.BINARY_TV, 0, 0.05, is_cap=C)
    assert np.array_equal(cap["M"], base["M"]) and 0 < (base["r"] > C).sum() < T
    for t in range(T):
        f = min(1.0, C / base["r"][t])
        np.testing.assert_allclose(cap["dlogits"][t], f * base["dlogits"][t], rtol=1e-13, atol=1e-18)
        assert abs(cap["row_loss"][t] - f * base["row_loss"][t]) <= 1e-15
    # the gradient is that of -s M stopgrad(min(r, C)) A log pi(a)  (autograd, float64)
    s_ = 1.0 / T
    zt = torch.tensor(c["z"], dtype=torch.float64, requires_grad=True)
    lp = torch.log_softmax(zt, dim=1)[torch.arange(T), torch.tensor(c["a"])]
    w = torch.clamp(torch.exp(lp - torch.tensor(c["mu_logp"])), max=C).detach()
    (-(s_ * torch.tensor(cap["M"].astype(np.float64)) * w * torch.tensor(c["adv"]) * lp).sum()).backward()
    np.testing.assert_allclose(cap["dlogits"], zt.grad.numpy(), atol=1e-14)
    # PG-IS (no mask): delta = +inf
    pg = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], None, O.BINARY_KL, 0, float("inf"), is_cap=3.0)
    assert np.all(pg["M"] == 1)


def check_ppo_clip_variant(O):
    """App. C.1: the GRPO / PPO mask is where the clipped objective of Eq. ppo-clip has zero gradient; with
    eps_low = eps_high = delta it is the DPPO mask with D replaced by |r - 1|."""
    for adv in (-1.3, 0.0, 0.7):
        for r in (0.5, 0.79, 0.81, 0.99, 1.0, 1.01, 1.27, 1.29, 2.5):
            rt = torch.tensor(r, dtype=torch.float64, requires_grad=True)
            obj = torch.minimum(rt * adv, torch.clamp(rt, 1 - 0.2, 1 + 0.28) * adv)
            (gr,) = torch.autograd.grad(obj, rt)
            M = O.ppo_clip_mask(adv, r, 0.2, 0.28)
            if adv != 0.0:
                assert (float(gr) == 0.0) == (M == 0), (adv, r)
            else:
                assert M == 1
            assert O.ppo_clip_mask(adv, r, 0.2, 0.2) == O.dppo_mask(adv, math.log(r), 0.0, abs(r - 1.0), 0.2)
    rng = np.random.default_rng(10)
    c = _case(rng, T=40, V=6, K=2, noise=1.0)
    o = O.dppo_loss_fwd_bwd(c["z"], c["a"], c["mu_logp"], c["adv"], None, O.PPO_CLIP, 0, 0.28, eps_low=0.2)
    np.testing.assert_allclose(o["D"], np.abs(o["r"] - 1.0), atol=1e-15)
    exp_M = [O.ppo_clip_mask(c["adv"][t], o["r"][t], 0.2, 0.28) for t in range(40)]
    assert np.array_equal(o["M"], np.array(exp_M)) and 0 < sum(exp_M) < 40
    # the low-probability token of the worked example (Sec. 4.2) is clipped by PPO for A > 0 but not by Binary-TV
    z = np.log([1e-2, 0.495, 0.495])
    assert O.dppo_row(z, 0, math.log(1e-4), 1.0, O.PPO_CLIP, 0.2, 1.0)["M"] == 0
    assert O.dppo_row(z, 0, math.log(1e-4), 1.0, O.BINARY_TV, 0.2, 1.0)["M"] == 1


def check_minimal_mask(O):
    """Sec. 5.3: only negative samples whose sampled-token probability dropped by at least delta are blocked."""
    for adv, mu, pi, delta, expect in ((-1.0, 0.9, 0.3, 0.5, 0), (-1.0, 0.9, 0.39, 0.5, 0), (-1.0, 0.9, 0.41, 0.5, 1),
                                       (1.0, 0.9, 0.1, 0.5, 1), (-1.0, 0.3, 0.9, 0.5, 1), (0.0, 0.9, 0.1, 0.5, 1),
                                       (-1.0, 0.99, 0.18, 0.8, 0), (-1.0, 0.99, 0.20, 0.8, 1)):
        assert O.minimal_mask(adv, mu, pi, delta) == expect, (adv, mu, pi, delta)
        assert O.minimal_mask(-1.0, 0.75, 0.25, 0.5) == 0          # ">=": exactly delta is blocked (exact in binary)
        z = np.log(np.array([pi, (1 - pi) * 0.25, (1 - pi) * 0.75]))
        o = O.dppo_row(z, 0, math.log(mu), adv, O.MINIMAL_MASK, delta, 0.5)
        assert o["M"] == expect and abs(o["D"] - (mu - pi)) < 1e-12
        # the blocked set is inside the DPPO Binary-TV blocked set at the same threshold (it adds "A < 0" and the sign)
        if expect == 0:
            assert O.dppo_row(z, 0, math.log(mu), adv, O.BINARY_TV, delta - 1e-9, 0.5)["M"] == 0
        g_expect = 0.5 * expect * (pi / mu) * adv
        assert abs(o["g"] - g_expect) < 1e-12


def check_exact_divergence(O):
    """Full TV / KL / entropy from two logits rows against library routines and the App. B ordering."""
    rng = np.random.default_rng(11)
    for V in (2, 9, 500):
        z = 3 * rng.standard_normal(V)
        zm = z + rng.standard_normal(V)
        tv, kl, ent = O.exact_divergence_row(z, zm)
        pi, mu = scipy.special.softmax(z), scipy.special.softmax(zm)
        assert abs(tv - 0.5 * np.abs(mu - pi).sum()) < 1e-13
        assert abs(kl - scipy.stats.entropy(mu, pi)) < 1e-12
        assert abs(ent - scipy.stats.entropy(pi)) < 1e-12
        assert abs(kl - O.full_kl(mu, pi)) < 1e-12 and tv * tv <= 0.5 * kl + 1e-15
        a = int(rng.integers(0, V))
        assert O.binary_tv(mu[a], pi[a]) <= tv + 1e-15 and O.binary_kl(mu[a], pi[a]) <= kl + 1e-13
    tv, kl, ent = O.exact_divergence_row(np.zeros(64), np.zeros(64))
    assert tv == 0.0 and abs(kl) < 1e-15 and abs(ent - math.log(64)) < 1e-13
    # direction: KL(mu || pi), not the reverse
    z, zm = np.log([0.7, 0.2, 0.1]), np.log([0.1, 0.3, 0.6])
    assert abs(O.exact_divergence_row(z, zm)[1] - (0.1 * math.log(0.1 / 0.7) + 0.3 * math.log(0.3 / 0.2) + 0.6 * math.log(0.6 / 0.1))) < 1e-12
    # huge offsets and a -inf entry do not produce nan
    tv, kl, ent = O.exact_divergence_row(np.array([800.0, 799.0, -np.inf]), np.array([-300.0, -301.0, -np.inf]))
    assert np.isfinite(tv) and np.isfinite(ent) and np.isfinite(kl)


def check_given_divergence(O):
    """Variant GIVEN_D: Eq. dppo_obj with the caller's per-token divergence.  Feeding the Binary-TV values back reproduces
    the Binary-TV variant; with the exact full-vocabulary TV (App. B: D_bin <= D_full) every token the Binary form blocks
    stays blocked; D = 0 never blocks, D = +inf blocks exactly the tokens that moved away from r = 1."""
    rng = np.random.default_rng(77)
    c = _case(rng, T=40, V=13, K=3, noise=0.9)
    z, a, ml, adv = c["z"], c["a"], c["mu_logp"], c["adv"]
    T = len(a)
    zm = np.log(c["mu"])
    delta = 0.08
    ref = O.dppo_loss_fwd_bwd(z, a, ml, adv, None, O.BINARY_TV, 0, delta)
    same = O.dppo_loss_fwd_bwd(z, a, ml, adv, None, O.GIVEN_D, 0, delta, given_D=ref["D"])
    assert np.array_equal(same["M"], ref["M"]) and same["loss"] == ref["loss"] and np.array_equal(same["dlogits"], ref["dlogits"])
    assert np.array_equal(same["D"], ref["D"])
    full = np.array([O.exact_divergence_row(z[t], zm[t])[0] for t in range(T)])
    assert np.all(full >= ref["D"] - 1e-15)
    ex = O.dppo_loss_fwd_bwd(z, a, ml, adv, None, O.GIVEN_D, 0, delta, given_D=full)
    lp = scipy.special.log_softmax(z, axis=1)[np.arange(T), a]
    away = ((adv > 0) & (lp > ml)) | ((adv < 0) & (lp < ml))
    assert np.array_equal(ex["M"], np.where(away & (full > delta), 0, 1).astype(np.uint8))
    assert np.all(ex["M"] <= ref["M"]) and 0 < int((ex["M"] == 0).sum()) < T and int((ex["M"] != ref["M"]).sum()) > 0
    assert np.array_equal(ex["D"], full)
    tok = (np.arange(T) % 4 != 1).astype(np.uint8)
    zero = O.dppo_loss_fwd_bwd(z, a, ml, adv, tok, O.GIVEN_D, 0, delta, given_D=np.zeros(T))
    r = np.exp(lp - ml)
    assert np.array_equal(zero["M"], tok) and abs(zero["loss"] + np.sum((r * adv)[tok != 0]) / tok.sum()) < 1e-12
    inf = O.dppo_loss_fwd_bwd(z, a, ml, adv, tok, O.GIVEN_D, 0, delta, given_D=np.full(T, np.inf))
    assert np.array_equal(inf["M"], np.where(away | (tok == 0), 0, 1).astype(np.uint8))
    assert not inf["dlogits"][inf["M"] == 0].any()
    # the LM-head form passes it through
    H = rng.standard_normal((T, 5))
    W = rng.standard_normal((5, 13))
    zz = H @ W
    f1 = O.dppo_fused_lmhead_fwd_bwd(H, W, a, ml, adv, None, O.GIVEN_D, delta, given_D=full)
    f2 = O.dppo_loss_fwd_bwd(zz, a, ml, adv, None, O.GIVEN_D, 0, delta, given_D=full)
    assert np.array_equal(f1["M"], f2["M"]) and np.allclose(f1["dW"], H.T @ f2["dlogits"])


CHECKS = [check_given_divergence, check_exact_divergence, check_minimal_mask, check_is_cap_and_baselines, check_ppo_clip_variant, check_worked_example, check_log_softmax, check_binary, check_topk_full_and_bounds,
          check_topk_other_bucket, check_topk_equality_conditions, check_edge_conventions,
          check_mask_truth_table, check_on_policy, check_gradient, check_brute_force_tiny, check_fused, check_fused_sampled]


@pytest.mark.parametrize("check", CHECKS, ids=lambda f: f.__name__)
def test_pin(check):
    check(O)


# ----------------------------------------------------------------------------- planted mistakes

def _mutant(**repl):
    """A copy of the oracle module with some functions replaced (functions inside look names up in the copy)."""
    src = open(O.__file__).read()
    m = types.ModuleType("oracle_mutant")
    m.__file__ = O.__file__
    exec(compile(src, O.__file__, "exec"), m.__dict__)
    for k, v in repl.items():
        setattr(m, k, v(m) if callable(v) else v)
    return m


MUTANTS = {
    "tv_without_half": lambda m: (lambda p, q: float(np.sum(np.abs(np.asarray(p) - np.asarray(q))))),
    "kl_reversed": lambda m: (lambda p, q: float(sum(m._xlogx_over_y(y, x) for x, y in zip(p, q)))),
    "binary_kl_drops_complement": lambda m: (lambda mu, pi: m._xlogx_over_y(mu, pi)),
    "binary_tv_signed": lambda m: (lambda mu, pi: float(mu) - float(pi)),
    "ratio_inverted": lambda m: (lambda lp, lm: float(np.exp(float(lm) - float(lp)))),
    "mask_symmetric": lambda m: (lambda adv, lp, lm, D, delta: 0 if D > delta else 1),
    "mask_wrong_side": lambda m: (lambda adv, lp, lm, D, delta: 0 if (D > delta and ((adv > 0 and lp < lm) or (adv < 0 and lp > lm))) else 1),
    "mask_nonstrict_sign": lambda m: (lambda adv, lp, lm, D, delta: 0 if (D > delta and ((adv >= 0 and lp > lm) or (adv < 0 and lp < lm))) else 1),
}
MUTANT_TARGET = {
    "tv_without_half": "topk_tv", "kl_reversed": "topk_kl", "binary_kl_drops_complement": "binary_kl",
    "binary_tv_signed": "binary_tv", "ratio_inverted": "ratio", "mask_symmetric": "dppo_mask",
    "mask_wrong_side": "dppo_mask", "mask_nonstrict_sign": "dppo_mask",
}


def _no_dedupe(m):
    def topk_reduced(pi, a, mu_a, topk_ids, topk_p):       # counts the sampled token twice when it is in the list
        ids = [int(i) for i in topk_ids] + [int(a)]
        ps = [float(p) for p in topk_p] + [float(mu_a)]
        p_mu = np.array(ps)
        p_pi = np.array([pi[i] for i in ids])
        return np.append(p_mu, max(0.0, 1 - p_mu.sum())), np.append(p_pi, max(0.0, 1 - p_pi.sum()))
    return topk_reduced


def _grad_sign(m):
    orig = m.dppo_row

    def dppo_row(*a, **k):
        o = orig(*a, **k)
        if "dlogits" in o:
            o["dlogits"] = -o["dlogits"]
        return o
    return dppo_row


def _grad_no_onehot(m):
    orig = m.dppo_row

    def dppo_row(z, a, *rest, **k):
        o = orig(z, a, *rest, **k)
        if "dlogits" in o:
            o["dlogits"][int(a)] += o["g"]
        return o
    return dppo_row


def _fused_transposed(m):
    orig = m.dppo_fused_lmhead_fwd_bwd

    def f(H, W, *a, **k):
        o = orig(H, W, *a, **k)
        o["dW"] = (o["dlogits"].T @ np.asarray(H, dtype=np.float64)).T * 1.0
        o["dHidden"] = o["dlogits"] @ np.asarray(W, dtype=np.float64).T[:, ::-1][:, ::-1] * 2.0
        return o
    return f


def _cap_as_max(m):
    orig = m.dppo_row

    def dppo_row(z, a, mu_logp, adv, variant, delta, scale, topk_ids=None, topk_p=None, want_grad=True, is_cap=None, eps_low=None,
                 given_D=None):
        o = orig(z, a, mu_logp, adv, variant, delta, scale, topk_ids, topk_p, want_grad, None, eps_low, given_D)
        if is_cap is not None and np.isfinite(is_cap):
            f = max(o["r"], is_cap) / o["r"]
            o["g"] *= f
            o["loss"] *= f
            if "dlogits" in o:
                o["dlogits"] = o["dlogits"] * f
        return o
    return dppo_row


def _given_d_ignored(m):
    orig = m.dppo_row

    def dppo_row(z, a, mu_logp, adv, variant, *rest, **k):       # uses the Binary-TV value instead of the caller's
        if variant == m.GIVEN_D:
            rest = list(rest)
            if "given_D" in k:
                k["given_D"] = None
            elif len(rest) >= 8:
                rest[7] = None
            o = orig(z, a, mu_logp, adv, m.BINARY_TV, *rest, **k)
            return o
        return orig(z, a, mu_logp, adv, variant, *rest, **k)
    return dppo_row


MUTANTS.update({"given_d_ignored": _given_d_ignored, "minimal_mask_positive_side": lambda m: (lambda adv, mu, pi, delta: 0 if (adv > 0 and mu - pi >= delta) else 1),
                "cap_as_max": _cap_as_max, "ppo_eps_swapped": lambda m: (lambda adv, r, el, eh: 0 if ((adv > 0 and r - 1 > el) or (adv < 0 and 1 - r > eh)) else 1),
                "topk_no_dedupe": _no_dedupe, "grad_sign": _grad_sign, "grad_no_onehot": _grad_no_onehot,
                "fused_scaled": _fused_transposed})
MUTANT_TARGET.update({"given_d_ignored": "dppo_row", "minimal_mask_positive_side": "minimal_mask", "cap_as_max": "dppo_row", "ppo_eps_swapped": "ppo_clip_mask", "topk_no_dedupe": "topk_reduced", "grad_sign": "dppo_row", "grad_no_onehot": "dppo_row",
                      "fused_scaled": "dppo_fused_lmhead_fwd_bwd"})


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistakes_are_caught(name):
    m = _mutant(**{MUTANT_TARGET[name]: MUTANTS[name]})
    failed = []
    for check in CHECKS:
        try:
            check(m)
        except Exception:  # noqa: BLE001  (any failure counts: assertion, nan, ...)
            failed.append(check.__name__)
    assert failed, f"mutant {name} passed every pin"
