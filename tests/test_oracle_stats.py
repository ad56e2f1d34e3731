"""Pins for the oracle's monitors and optional steps: token entropy, the approximate-KL and
clip-fraction monitors of the policy step, and masked advantage whitening.

The paper (Section 2.1) says the actor is trained to raise reward while limiting its deviation from
the old policy, and prints no formula; these quantities are how that deviation is watched.  The
pins are what each definition fixes: closed forms, invariances, special cases that reduce to a
float64 torch routine, and brute force on small inputs.
"""
import math

import numpy as np
import pytest
import torch


def _bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------------------------------ entropy

def test_entropy_of_uniform_logits_is_log_V(oracle):
    for V in (2, 1000, 32000, 50272):
        for c in (0.0, -3.5, 7.0):
            z = np.full((1, 2, V), c)
            h = oracle.token_entropy(z, [2])
            assert np.abs(h - math.log(V)).max() < 1e-11
            hb = oracle.token_entropy(_bits(torch.from_numpy(z)), [2])
            assert np.abs(hb - math.log(V)).max() < 1e-11


def test_entropy_one_hot_spike_closed_form(oracle):
    # one logit M, the other V-1 logits 0: p = e^M / (e^M + V - 1), the rest q = 1 / (e^M + V - 1)
    V = 777
    for M in (0.5, 4.0, 12.0, 40.0):
        z = np.zeros((1, 1, V))
        z[0, 0, 5] = M
        Z = math.exp(M) + (V - 1)
        p, q = math.exp(M) / Z, 1.0 / Z
        want = -p * math.log(p) - (V - 1) * q * math.log(q)
        # (at M = 40 the entropy itself is 1e-13: log-sum-exp of 40 + 3e-15 rounds in float64, hence the absolute slack)
        assert oracle.token_entropy(z, [1])[0, 0] == pytest.approx(want, rel=1e-12, abs=1e-13)


def test_entropy_two_entries_is_the_binary_entropy(oracle):
    for d in (0.0, 0.3, 2.0, 9.0):
        z = np.array([[[d, 0.0]]])
        p = 1.0 / (1.0 + math.exp(-d))
        want = -(p * math.log(p) + (1 - p) * math.log1p(-p))
        assert oracle.token_entropy(z, [1])[0, 0] == pytest.approx(want, rel=1e-12)


def test_entropy_against_torch_float64_and_shift_invariance(oracle):
    g = torch.Generator().manual_seed(11)
    z = (torch.randn((3, 5, 300), generator=g, dtype=torch.float64) * 3).to(torch.bfloat16)
    lengths = [5, 2, 0]
    h = oracle.token_entropy(_bits(z), lengths)
    lp = torch.log_softmax(z.double(), -1)
    want = -(lp.exp() * lp).sum(-1).numpy()
    valid = np.arange(5)[None, :] < np.array(lengths)[:, None]
    assert np.abs(h - want)[valid].max() < 1e-12
    assert (h[~valid] == 0).all()
    # float64 entry, shifted by a constant (a naive exp would overflow at +800)
    z64 = z.double().numpy()
    assert np.abs(oracle.token_entropy(z64 + 800.0, lengths) - h).max() < 1e-11
    # entropy lies in [0, log V] and is largest for the flattest row
    assert (h[valid] > 0).all() and (h[valid] < math.log(300)).all()


def test_entropy_neg_inf_is_a_deleted_entry(oracle):
    rng = np.random.default_rng(3)
    V = 64
    z = rng.normal(0, 3, size=(1, 4, V))
    dead = np.array([1, 7, 8, 30, 63])
    keep = np.setdiff1d(np.arange(V), dead)
    zi = z.copy()
    zi[..., dead] = -np.inf
    assert np.abs(oracle.token_entropy(zi, [4]) - oracle.token_entropy(np.ascontiguousarray(z[..., keep]), [4])).max() < 1e-13


def test_entropy_strided_view(oracle):
    g = torch.Generator().manual_seed(5)
    full = (torch.randn((2, 9, 50), generator=g) * 2).to(torch.bfloat16)
    view = full[:, 3:7]
    h = oracle.token_entropy(_bits(view), [4, 3])
    hc = oracle.token_entropy(_bits(view.contiguous()), [4, 3])
    assert np.array_equal(h, hc)


# ------------------------------------------------------------------------------------------ monitors

def test_stats_on_policy_are_zero(oracle):
    rng = np.random.default_rng(0)
    lp = rng.normal(-3, 1, (3, 6))
    adv = rng.normal(0, 1, (3, 6))
    kl, cf = oracle.ppo_stats(lp, lp, adv, [6, 3, 0], 0.2)
    assert kl == 0.0 and cf == 0.0


def test_stats_constant_log_ratio_closed_form(oracle):
    # lp_new - lp_old = d everywhere: approx_kl = e^d - 1 - d; every token is clipped iff the ratio left the
    # interval on the side that A makes worse
    lp_old = np.full((2, 4), -2.0)
    for d in (0.05, -0.05, 0.3, -0.4):
        for sign in (1.0, -1.0):
            adv = np.full((2, 4), sign)
            kl, cf = oracle.ppo_stats(lp_old + d, lp_old, adv, [4, 2], 0.2)
            assert kl == pytest.approx(math.expm1(d) - d, rel=1e-12, abs=1e-16)
            rho = math.exp(d)
            clipped = (sign > 0 and rho > 1.2) or (sign < 0 and rho < 0.8)
            assert cf == (1.0 if clipped else 0.0)


def test_stats_four_sign_and_side_cases_and_padding(oracle):
    # one token of each kind in a sequence of 4, plus a padded position with wild values
    lp_old = np.zeros((1, 5))
    lp_new = np.log(np.array([[1.5, 1.5, 0.5, 0.5, 9.0]]))
    adv = np.array([[+1.0, -1.0, +1.0, -1.0, 3.0]])
    kl, cf = oracle.ppo_stats(lp_new, lp_old, adv, [4], 0.2)
    # clipped and worse: (A>0, rho>1+eps) and (A<0, rho<1-eps) only
    assert cf == pytest.approx(2 / 4)
    want_kl = np.mean([(r - 1) - math.log(r) for r in (1.5, 1.5, 0.5, 0.5)])
    assert kl == pytest.approx(want_kl, rel=1e-12)
    # the clip fraction is the share of tokens with a zero policy gradient
    out = oracle.ppo_loss_from_logprobs(lp_new, lp_old, adv, np.zeros((1, 5)), np.zeros((1, 5)), np.zeros((1, 5)),
                                        [4], 0.2, 0.2, 1.0)
    assert cf == pytest.approx(np.mean(out.g[0, :4] == 0))


def test_stats_brute_force_random(oracle):
    rng = np.random.default_rng(7)
    B, T = 5, 9
    lengths = np.array([9, 0, 4, 1, 7])
    lp_old = rng.normal(-3, 1, (B, T))
    lp_new = lp_old + rng.normal(0, 0.25, (B, T))
    adv = rng.normal(0, 1, (B, T))
    kl, cf = oracle.ppo_stats(lp_new, lp_old, adv, lengths, 0.2)
    tot, ncl, n = 0.0, 0, 0
    for b in range(B):
        for t in range(lengths[b]):
            r = math.exp(lp_new[b, t] - lp_old[b, t])
            tot += r - 1 - (lp_new[b, t] - lp_old[b, t])
            ncl += (-adv[b, t] * min(max(r, 0.8), 1.2)) > (-adv[b, t] * r)
            n += 1
    assert kl == pytest.approx(tot / n, rel=1e-12) and cf == pytest.approx(ncl / n)
    assert kl >= 0.0                                 # the estimator is non-negative term by term
    assert oracle.ppo_stats(lp_new, lp_old, adv, np.zeros(B, int), 0.2) == (0.0, 0.0)


# ------------------------------------------------------------------------------------------ whitening

def _valid(lengths, T):
    return np.arange(T)[None, :] < np.asarray(lengths)[:, None]


def test_whiten_gives_mean_zero_variance_one_over_valid_tokens(oracle):
    rng = np.random.default_rng(1)
    B, T = 6, 11
    lengths = np.array([11, 3, 0, 1, 7, 11])
    adv = rng.normal(2.0, 3.0, (B, T))
    adv[~_valid(lengths, T)] = 1e9                    # padded inputs are ignored
    w = oracle.whiten(adv, lengths, eps=0.0)
    v = w[_valid(lengths, T)]
    assert abs(v.mean()) < 1e-13 and abs(v.var() - 1.0) < 1e-12
    assert (w[~_valid(lengths, T)] == 0).all()
    # the float64 torch routine it reduces to
    a = torch.from_numpy(adv[_valid(lengths, T)])
    want = (a - a.mean()) / torch.sqrt(a.var(unbiased=False))
    assert np.abs(v - want.numpy()).max() < 1e-12


def test_whiten_shift_and_scale_invariance(oracle):
    rng = np.random.default_rng(2)
    adv = rng.normal(0, 1, (3, 8))
    lengths = [8, 5, 2]
    base = oracle.whiten(adv, lengths, eps=0.0)
    assert np.abs(oracle.whiten(adv + 17.0, lengths, eps=0.0) - base).max() < 1e-12
    assert np.abs(oracle.whiten(adv * 4.0, lengths, eps=0.0) - base).max() < 1e-12
    assert np.abs(oracle.whiten(adv * -0.5, lengths, eps=0.0) + base).max() < 1e-12


def test_whiten_eps_and_degenerate_batches(oracle):
    adv = np.array([[3.0, 5.0, 0.0]])
    # two valid tokens 3 and 5: mean 4, population variance 1
    w = oracle.whiten(adv, [2], eps=3.0)
    assert np.allclose(w, [[-0.5, 0.5, 0.0]], atol=1e-15)
    # one valid token: variance 0, the result is 0 for any eps (0/sqrt(eps), and 0 for eps = 0)
    assert (oracle.whiten(adv, [1], eps=1e-8) == 0).all() and (oracle.whiten(adv, [1], eps=0.0) == 0).all()
    # no valid token
    assert (oracle.whiten(adv, [0], eps=1e-8) == 0).all()
    # constant advantages: all zeros
    assert (oracle.whiten(np.full((2, 3), 7.0), [3, 3], eps=1e-8) == 0).all()
