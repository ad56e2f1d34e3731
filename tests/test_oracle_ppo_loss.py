"""Pins for the oracle's step 4: clipped PPO policy and value loss and their gradients.

Section 2.1 of the paper: the actor is trained to raise reward while limiting its deviation from
the old policy (the clipped surrogate of the PPO paper it cites) and the critic is trained on the
returns.  Pins: float64 autograd of the same loss written with library ops, central finite
differences of the oracle's own loss, special cases with closed forms, and the structure of the
softmax gradient (rows sum to zero, sign pattern, exact zeros where clipping switches it off).
"""
import numpy as np
import pytest
import torch


def _case(seed, B=3, T=12, V=19, sigma_lp=0.25, sigma_v=0.5):
    rng = np.random.default_rng(seed)
    z = rng.normal(0, 2, (B, T, V))
    ids = rng.integers(0, V, (B, T)).astype(np.int64)
    lengths = np.array([T, max(1, T // 2), 0][:B], dtype=np.int32)
    lp_cur = torch.log_softmax(torch.from_numpy(z), -1).gather(
        2, torch.from_numpy(ids)[..., None])[..., 0].numpy()
    lp_old = lp_cur + rng.normal(0, sigma_lp, (B, T))     # wide enough that many tokens clip
    adv = rng.normal(0, 1, (B, T))
    v_old = rng.normal(0, 1, (B, T))
    v_new = v_old + rng.normal(0, sigma_v, (B, T))
    ret = v_old + rng.normal(0, 0.5, (B, T))
    return z, ids, lengths, lp_old, adv, v_new, v_old, ret


def _torch_losses(z, ids, lengths, lp_old, adv, v_new, v_old, ret, eps, eps_v):
    """The two losses in a few lines of float64 library ops (torch.clamp / torch.maximum)."""
    B, T, _ = z.shape
    mask = (torch.arange(T)[None, :] < torch.as_tensor(lengths)[:, None]).double()
    N = mask.sum()
    lp = torch.log_softmax(z, -1).gather(2, torch.as_tensor(ids)[..., None])[..., 0]
    rho = torch.exp(lp - torch.as_tensor(lp_old))
    A = torch.as_tensor(adv)
    l_pg = torch.maximum(-A * rho, -A * torch.clamp(rho, 1 - eps, 1 + eps))
    vo, G = torch.as_tensor(v_old), torch.as_tensor(ret)
    vc = vo + torch.clamp(v_new - vo, -eps_v, eps_v)
    l_vf = 0.5 * torch.maximum((v_new - G) ** 2, (vc - G) ** 2)
    return (l_pg * mask).sum() / N, (l_vf * mask).sum() / N


@pytest.mark.parametrize("seed,grad_scale", [(0, 1.0), (1, 3.5)])
def test_against_float64_autograd(oracle, seed, grad_scale):
    z, ids, lengths, lp_old, adv, v_new, v_old, ret = _case(seed)
    eps, eps_v = 0.2, 0.2
    zt = torch.tensor(z, requires_grad=True)
    vt = torch.tensor(v_new, requires_grad=True)
    lpg, lvf = _torch_losses(zt, ids, lengths, lp_old, adv, vt, v_old, ret, eps, eps_v)
    (grad_scale * lpg).backward()
    (grad_scale * lvf).backward()
    out = oracle.ppo_loss(z, ids, lengths, lp_old, adv, v_new, v_old, ret, eps, eps_v, grad_scale)
    assert out.loss_pg == pytest.approx(lpg.item(), abs=1e-13)
    assert out.loss_vf == pytest.approx(lvf.item(), abs=1e-13)
    B, T, V = z.shape
    dl = oracle.dlogits_rows(z, ids, lengths, out.g, np.arange(B * T)).reshape(B, T, V)
    assert np.abs(dl - zt.grad.numpy()).max() < 1e-13
    assert np.abs(out.dvalues - vt.grad.numpy()).max() < 1e-14
    # the case exercises both branches of both clips
    valid = np.arange(T)[None, :] < lengths[:, None]
    assert (out.g[valid] == 0).any() and (out.g[valid] != 0).any()
    assert (out.dvalues[valid] == 0).any() and (out.dvalues[valid] != 0).any()


def test_finite_differences_of_the_oracle_loss(oracle):
    z, ids, lengths, lp_old, adv, v_new, v_old, ret = _case(2, B=2, T=4, V=11)
    eps, eps_v, h = 0.2, 0.2, 1e-5
    out = oracle.ppo_loss(z, ids, lengths, lp_old, adv, v_new, v_old, ret, eps, eps_v)
    B, T, V = z.shape
    dl = oracle.dlogits_rows(z, ids, lengths, out.g, np.arange(B * T)).reshape(B, T, V)

    def losses(zz, vv):
        o = oracle.ppo_loss(zz, ids, lengths, lp_old, adv, vv, v_old, ret, eps, eps_v)
        return o.loss_pg, o.loss_vf

    for b in range(B):
        for t in range(T):
            for v in range(V):
                zp, zm = z.copy(), z.copy()
                zp[b, t, v] += h
                zm[b, t, v] -= h
                fd = (losses(zp, v_new)[0] - losses(zm, v_new)[0]) / (2 * h)
                assert dl[b, t, v] == pytest.approx(fd, abs=2e-9)
            vp, vm = v_new.copy(), v_new.copy()
            vp[b, t] += h
            vm[b, t] -= h
            fd = (losses(z, vp)[1] - losses(z, vm)[1]) / (2 * h)
            assert out.dvalues[b, t] == pytest.approx(fd, abs=2e-9)


def test_on_policy_special_case(oracle):
    # lp_old = lp_new: rho = 1 everywhere, nothing clips
    z, ids, lengths, _, adv, v_new, v_old, ret = _case(3)
    lp = oracle.gather_logprobs(z, ids, lengths)
    s = 2.0
    out = oracle.ppo_loss(z, ids, lengths, lp, adv, v_old, v_old, ret, 0.2, 0.2, s)
    valid = np.arange(z.shape[1])[None, :] < lengths[:, None]
    N = valid.sum()
    assert out.loss_pg == pytest.approx(-(adv * valid).sum() / N, abs=1e-14)
    assert np.allclose(out.g, -s * adv * valid / N, rtol=0, atol=1e-16)
    # v_new = v_old: the value clip is inactive, plain half squared error
    assert out.loss_vf == pytest.approx(0.5 * (((v_old - ret) ** 2) * valid).sum() / N, abs=1e-14)
    assert np.allclose(out.dvalues, s * (v_old - ret) * valid / N, rtol=0, atol=1e-16)
    # and the logits gradient is -(s A / N)(onehot - softmax)
    B, T, V = z.shape
    dl = oracle.dlogits_rows(z, ids, lengths, out.g, np.arange(B * T)).reshape(B, T, V)
    p = torch.softmax(torch.from_numpy(z), -1).numpy()
    onehot = np.eye(V)[ids]
    assert np.abs(dl - out.g[..., None] * (onehot - p)).max() < 1e-15


def test_clip_switches_the_gradient_off(oracle):
    # one token per sign/side combination; eps = 0.2
    lp_new = np.zeros((1, 4))
    rho = np.array([[1.5, 1.5, 0.5, 0.5]])
    lp_old = lp_new - np.log(rho)
    adv = np.array([[2.0, -2.0, 2.0, -2.0]])
    zeros = np.zeros((1, 4))
    out = oracle.ppo_loss_from_logprobs(lp_new, lp_old, adv, zeros, zeros, zeros, [4], 0.2, 0.2)
    # A>0, rho>1+eps: clipped, no gradient, loss -A(1+eps).  A<0, rho>1+eps: unclipped.
    # A>0, rho<1-eps: unclipped.  A<0, rho<1-eps: clipped, loss -A(1-eps).
    assert out.g[0, 0] == 0 and out.g[0, 3] == 0
    assert out.g[0, 1] == pytest.approx(2.0 * 1.5 / 4) and out.g[0, 2] == pytest.approx(-2.0 * 0.5 / 4)
    assert out.loss_pg == pytest.approx((-2.0 * 1.2 + 2.0 * 1.5 - 2.0 * 0.5 + 2.0 * 0.8) / 4)
    # value clip: v_new far above v_old; the clipped branch is the larger one iff G lies above v_old
    v_old = np.array([[0.0, 0.0]])
    v_new = np.array([[1.0, 1.0]])
    G = np.array([[2.0, -2.0]])
    o = oracle.ppo_loss_from_logprobs(np.zeros((1, 2)), np.zeros((1, 2)), np.zeros((1, 2)),
                                      v_new, v_old, G, [2], 0.2, 0.2)
    # token 0: (1-2)^2 = 1 < (0.2-2)^2 = 3.24 -> clipped, dV = 0; token 1: (1+2)^2 = 9 > (0.2+2)^2 -> dV = (v-G)/N
    assert o.dvalues[0, 0] == 0 and o.dvalues[0, 1] == pytest.approx(3.0 / 2)
    assert o.loss_vf == pytest.approx(0.5 * (3.24 + 9.0) / 2)


def test_gradient_structure(oracle):
    z, ids, lengths, lp_old, adv, v_new, v_old, ret = _case(4, B=3, T=6, V=50)
    out = oracle.ppo_loss(z, ids, lengths, lp_old, adv, v_new, v_old, ret, 0.2, 0.2, 10.0)
    B, T, V = z.shape
    dl = oracle.dlogits_rows(z, ids, lengths, out.g, np.arange(B * T)).reshape(B, T, V)
    for b in range(B):
        for t in range(T):
            row, g = dl[b, t], out.g[b, t]
            if t >= lengths[b] or g == 0:
                assert (row == 0).all()
                continue
            assert abs(row.sum()) < 1e-15 * max(1.0, abs(g)) * V        # rows sum to zero
            assert np.sign(row[ids[b, t]]) == np.sign(g)                # label entry has the sign of g
            others = np.delete(row, ids[b, t])
            assert (np.sign(others) == -np.sign(g)).all()               # every other entry the opposite
    # rows listed in any order, with repeats
    pick = np.array([5, 0, 5, 11])
    sub = oracle.dlogits_rows(z, ids, lengths, out.g, pick)
    assert np.array_equal(sub, dl.reshape(B * T, V)[pick])


def test_bf16_logits_are_widened_exactly(oracle):
    g = torch.Generator().manual_seed(5)
    z16 = (torch.randn((2, 3, 40), generator=g) * 3).to(torch.bfloat16)
    bits = z16.view(torch.int16).numpy().view(np.uint16)
    ids = torch.randint(0, 40, (2, 3), generator=g).numpy()
    lengths = [3, 2]
    rng = np.random.default_rng(5)
    aux = [rng.normal(0, 1, (2, 3)) for _ in range(5)]
    aux[0] = oracle.gather_logprobs(bits, ids, lengths) + 0.05 * aux[0]
    a = oracle.ppo_loss(bits, ids, lengths, *aux, 0.2, 0.2)
    b = oracle.ppo_loss(z16.double().numpy(), ids, lengths, *aux, 0.2, 0.2)
    assert a.loss_pg == b.loss_pg and a.loss_vf == b.loss_vf and np.array_equal(a.g, b.g)
    rows = np.arange(6)
    assert np.array_equal(oracle.dlogits_rows(bits, ids, lengths, a.g, rows),
                          oracle.dlogits_rows(z16.double().numpy(), ids, lengths, a.g, rows))


def test_empty_batch(oracle):
    z, ids, _, lp_old, adv, v_new, v_old, ret = _case(6)
    lengths = np.zeros(3, dtype=np.int32)
    out = oracle.ppo_loss(z, ids, lengths, lp_old, adv, v_new, v_old, ret, 0.2, 0.2)
    assert out.loss_pg == 0 and out.loss_vf == 0
    assert (out.g == 0).all() and (out.dvalues == 0).all()
    assert (oracle.dlogits_rows(z, ids, lengths, out.g, np.arange(4)) == 0).all()
