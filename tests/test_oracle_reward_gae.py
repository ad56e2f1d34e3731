"""Pins for the oracle's steps 2 and 3: the KL-penalised per-token reward and GAE.

Section 2.1 of the paper says only that the reference model keeps the reward from diverging, the
reward model scores the sequence and the critic estimates returns.  The pins are closed forms,
special cases and an O(T^2) brute force of the textbook definitions.
"""
import numpy as np
import pytest


def test_reward_special_cases(oracle):
    rng = np.random.default_rng(0)
    B, T = 4, 9
    lengths = np.array([9, 4, 1, 0], dtype=np.int32)
    lp_old = rng.normal(-3, 1, (B, T))
    lp_ref = lp_old + rng.normal(0, 0.3, (B, T))
    score = np.array([0.7, 7.5, -9.0, 3.0])          # two scores outside the clip range
    beta, c = 0.1, 5.0
    r = oracle.kl_reward(lp_old, lp_ref, score, lengths, beta, c)
    clipped = np.array([0.7, 5.0, -5.0, 3.0])
    for b, n in enumerate(lengths):
        assert (r[b, n:] == 0).all()
        if n == 0:
            continue
        # sum over the sequence: -beta * sum kl + clipped score
        kl = (lp_old[b, :n] - lp_ref[b, :n])
        assert r[b, :n].sum() == pytest.approx(-beta * kl.sum() + clipped[b], abs=1e-13)
        # all tokens but the last carry the KL term only; the sign penalises lp_old > lp_ref
        assert np.allclose(r[b, :n - 1], -beta * kl[:n - 1], rtol=0, atol=1e-15)
        assert r[b, n - 1] == pytest.approx(-beta * kl[n - 1] + clipped[b], abs=1e-15)
    # identical policies, or beta = 0: only the clipped score at the last valid token is left
    for rr in (oracle.kl_reward(lp_old, lp_old, score, lengths, beta, c),
               oracle.kl_reward(lp_old, lp_ref, score, lengths, 0.0, c)):
        expect = np.zeros((B, T))
        for b, n in enumerate(lengths):
            if n:
                expect[b, n - 1] = clipped[b]
        assert np.array_equal(rr, expect)


def _brute_force_gae(r, v, n, gamma, lam):
    """A_t = sum_l (gamma*lam)^l delta_{t+l}, written as the double sum it is."""
    vpad = np.concatenate([v[:n], [0.0]])
    delta = r[:n] + gamma * vpad[1:n + 1] - vpad[:n]
    adv = np.zeros(n)
    for t in range(n):
        for l in range(n - t):
            adv[t] += (gamma * lam) ** l * delta[t + l]
    return adv


def test_gae_brute_force_and_padding(oracle):
    rng = np.random.default_rng(1)
    B, T = 5, 33
    lengths = np.array([33, 17, 2, 1, 0], dtype=np.int32)
    r = rng.normal(0, 1, (B, T))
    v = rng.normal(0, 1, (B, T))
    for gamma, lam in ((1.0, 0.95), (0.99, 1.0), (0.9, 0.7), (1.0, 1.0), (0.97, 0.0)):
        adv, ret = oracle.gae(r, v, lengths, gamma, lam)
        for b, n in enumerate(lengths):
            assert np.allclose(adv[b, :n], _brute_force_gae(r[b], v[b], n, gamma, lam), rtol=0, atol=1e-12)
            assert np.allclose(ret[b, :n] - adv[b, :n], v[b, :n], rtol=0, atol=1e-13)   # G - A = V
            assert (adv[b, n:] == 0).all() and (ret[b, n:] == 0).all()


def test_gae_closed_forms(oracle):
    rng = np.random.default_rng(2)
    B, T = 3, 40
    lengths = np.array([40, 25, 1], dtype=np.int32)
    r = rng.normal(0, 1, (B, T))
    v = rng.normal(0, 1, (B, T))
    # gamma = lambda = 1: returns are reward-to-go (no dependence on the values), A = G - V
    adv, ret = oracle.gae(r, v, lengths, 1.0, 1.0)
    for b, n in enumerate(lengths):
        togo = np.cumsum(r[b, :n][::-1])[::-1]
        assert np.allclose(ret[b, :n], togo, rtol=0, atol=1e-12)
        assert np.allclose(adv[b, :n], togo - v[b, :n], rtol=0, atol=1e-12)
    ret_other_values = oracle.gae(r, rng.normal(0, 1, (B, T)), lengths, 1.0, 1.0)[1]
    assert np.allclose(ret_other_values, ret, rtol=0, atol=1e-12)
    # lambda = 1, any gamma: A_t = sum_s gamma^(s-t) r_s - V_t (the values telescope away)
    gamma = 0.99
    adv, _ = oracle.gae(r, v, lengths, gamma, 1.0)
    for b, n in enumerate(lengths):
        for t in range(n):
            disc = sum(gamma ** (s - t) * r[b, s] for s in range(t, n))
            assert adv[b, t] == pytest.approx(disc - v[b, t], abs=1e-12)
    # lambda = 0: one-step TD error, with value 0 after the last valid token
    adv, _ = oracle.gae(r, v, lengths, 0.9, 0.0)
    for b, n in enumerate(lengths):
        vnext = np.concatenate([v[b, 1:n], [0.0]])
        assert np.allclose(adv[b, :n], r[b, :n] + 0.9 * vnext - v[b, :n], rtol=0, atol=1e-14)
    # zero values, constant reward c, q = gamma*lambda: geometric series c (1 - q^(len-t)) / (1 - q)
    c, gamma, lam = 0.3, 0.98, 0.9
    q = gamma * lam
    adv, ret = oracle.gae(np.full((B, T), c), np.zeros((B, T)), lengths, gamma, lam)
    for b, n in enumerate(lengths):
        t = np.arange(n)
        assert np.allclose(adv[b, :n], c * (1 - q ** (n - t)) / (1 - q), rtol=0, atol=1e-13)
        assert np.array_equal(adv[b, :n], ret[b, :n])
    # a one-token response: A_0 = r_0 - V_0
    adv, ret = oracle.gae(r, v, np.array([1, 1, 1], dtype=np.int32), 0.95, 0.9)
    assert np.allclose(adv[:, 0], r[:, 0] - v[:, 0], rtol=0, atol=1e-15)
    assert np.allclose(ret[:, 0], r[:, 0], rtol=0, atol=1e-15)


def test_gae_ignores_padded_inputs(oracle):
    rng = np.random.default_rng(3)
    r = rng.normal(0, 1, (2, 12))
    v = rng.normal(0, 1, (2, 12))
    lengths = np.array([7, 12], dtype=np.int32)
    a0, g0 = oracle.gae(r, v, lengths, 0.99, 0.95)
    r2, v2 = r.copy(), v.copy()
    r2[0, 7:] = 1e6
    v2[0, 7:] = -1e6
    a1, g1 = oracle.gae(r2, v2, lengths, 0.99, 0.95)
    assert np.array_equal(a0, a1) and np.array_equal(g0, g1)
