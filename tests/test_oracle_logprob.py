"""Pins for the oracle's step 1 (log-prob of the generated token) and its bf16 helpers.

The paper (Section 2.1) only names the quantity, so the pins are what the definition
lp = z_y - log sum_v exp z_v fixes: closed forms, invariances, normalisation, the deleted-entry
reading of -inf, and the float64 library routine it reduces to.
"""
import math
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_uniform_logits_give_minus_log_V(oracle):
    # all-equal logits: softmax is uniform, lp = -ln V, whatever the common value and the label
    rows = [l.split() for l in open(os.path.join(GOLDEN, "uniform_logprob.txt")) if l[0] != "#"]
    for V, expect in ((int(a), float(b)) for a, b in rows):
        assert expect == pytest.approx(-math.log(V), rel=0, abs=1e-15)
        for c in (0.0, -3.5, 7.0):
            z = torch.full((1, 2, V), c)
            ids = np.array([[0, V - 1]], dtype=np.int64)
            for arr in (_bits(z), z.double().numpy()):
                lp = oracle.gather_logprobs(arr, ids, [2])
                assert np.abs(lp - expect).max() < 1e-12


def test_one_hot_spike_closed_form(oracle):
    # z_y = M, the rest 0: lp_y = -log1p((V-1) e^-M); for another label u: lp_u = lp_y - M
    V = 777
    for M in (0.5, 4.0, 12.0, 40.0):
        z = np.zeros((1, 2, V))
        z[0, :, 5] = M
        ids = np.array([[5, 6]], dtype=np.int64)
        lp = oracle.gather_logprobs(z, ids, [2])
        lp_y = -math.log1p((V - 1) * math.exp(-M))
        assert lp[0, 0] == pytest.approx(lp_y, abs=1e-13)
        assert lp[0, 1] == pytest.approx(lp_y - M, abs=1e-12)


def test_shift_invariance_and_large_offsets(oracle):
    # adding a constant to a row changes nothing; a naive exp(z) would overflow at +800
    rng = np.random.default_rng(1)
    z = rng.integers(-6, 7, size=(2, 3, 50)).astype(np.float64)
    ids = rng.integers(0, 50, size=(2, 3)).astype(np.int64)
    base = oracle.gather_logprobs(z, ids, [3, 3])
    for c in (64.0, -1024.0, 800.0):
        assert np.abs(oracle.gather_logprobs(z + c, ids, [3, 3]) - base).max() < 1e-12
    # the same through the bf16 entry: small integers plus a power of two stay exact in bf16
    zt = torch.from_numpy(z)
    b0 = oracle.gather_logprobs(_bits(zt), ids, [3, 3])
    b1 = oracle.gather_logprobs(_bits(zt + 64.0), ids, [3, 3])
    assert np.abs(b0 - base).max() < 1e-12 and np.abs(b1 - base).max() < 1e-12


def test_probabilities_sum_to_one(oracle):
    # gathering every label of one row: sum_v exp(lp_v) = 1
    rng = np.random.default_rng(2)
    V = 37
    row = rng.normal(0, 3, size=V)
    z = np.broadcast_to(row, (1, V, V)).copy()
    ids = np.arange(V, dtype=np.int64)[None, :]
    lp = oracle.gather_logprobs(z, ids, [V])
    assert abs(np.exp(lp).sum() - 1.0) < 1e-13
    assert np.argmax(lp) == np.argmax(row)           # the largest logit is the likeliest token


def test_neg_inf_is_a_deleted_entry(oracle):
    rng = np.random.default_rng(3)
    V = 64
    z = rng.normal(0, 3, size=(1, 4, V))
    dead = np.array([1, 7, 8, 30, 63])
    keep = np.setdiff1d(np.arange(V), dead)
    zi = z.copy()
    zi[:, :, dead] = -np.inf
    labels = np.array([[0, 2, 31, 62]], dtype=np.int64)            # none of them deleted
    lp_inf = oracle.gather_logprobs(zi, labels, [4])
    relabel = np.searchsorted(keep, labels)                        # position in the reduced vocabulary
    lp_red = oracle.gather_logprobs(np.ascontiguousarray(z[:, :, keep]), relabel, [4])
    assert np.isfinite(lp_inf).all()
    assert np.abs(lp_inf - lp_red).max() < 1e-13


def test_against_torch_float64_log_softmax(oracle):
    g = torch.Generator().manual_seed(4)
    B, T, V = 3, 5, 211
    z16 = (torch.randn((B, T, V), generator=g) * 3).to(torch.bfloat16)
    ids = torch.randint(0, V, (B, T), generator=g)
    lengths = [5, 2, 0]
    ref = torch.log_softmax(z16.double(), -1).gather(2, ids[..., None])[..., 0].numpy()
    lp = oracle.gather_logprobs(_bits(z16), ids.numpy(), lengths)
    for b, n in enumerate(lengths):
        assert np.abs(lp[b, :n] - ref[b, :n]).max(initial=0.0) < 1e-12
        assert (lp[b, n:] == 0).all()                              # padded positions give 0


def test_strided_view_of_a_longer_tensor(oracle):
    # response rows P-1 .. P+T-2 of a [B,P+T,V] tensor, ids columns P .. P+T-1
    g = torch.Generator().manual_seed(5)
    B, P, T, V = 2, 4, 6, 40
    full = (torch.randn((B, P + T, V), generator=g) * 3).to(torch.bfloat16)
    ids_full = torch.randint(0, V, (B, P + T), generator=g)
    view = _bits(full)[:, P - 1:P - 1 + T]
    ids_view = ids_full.numpy()[:, P:]
    lp = oracle.gather_logprobs(view, ids_view, [6, 3])
    dense = oracle.gather_logprobs(np.ascontiguousarray(view), np.ascontiguousarray(ids_view), [6, 3])
    assert (lp == dense).all()
    ref = torch.log_softmax(full[:, P - 1:P - 1 + T].double(), -1).gather(
        2, ids_full[:, P:, None])[..., 0].numpy()
    assert np.abs(lp[0] - ref[0]).max() < 1e-12 and np.abs(lp[1, :3] - ref[1, :3]).max() < 1e-12


def test_bad_ids_and_lengths_are_reported(oracle):
    z = np.zeros((1, 2, 8))
    with pytest.raises(ValueError):
        oracle.gather_logprobs(z, np.array([[0, 8]], dtype=np.int64), [2])
    with pytest.raises(ValueError):
        oracle.gather_logprobs(z, np.array([[0, 1]], dtype=np.int64), [3])
    # an id outside the vocabulary at a padded position is never looked at
    oracle.gather_logprobs(z, np.array([[0, 99]], dtype=np.int64), [1])


def test_round_bf16_matches_library_rounding(oracle):
    # torch rounds float32 -> bf16 to nearest even; float32 inputs are exact in float64
    g = torch.Generator().manual_seed(6)
    x = torch.cat([
        torch.randn(4000, generator=g) * 10.0 ** torch.randint(-42, 38, (4000,), generator=g).float(),
        torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e-40, -1.0e-45, 3.3e38, 3.4e38,
                      2.0 ** -133, 2.0 ** -134, 1.5 * 2.0 ** -133]),
    ])
    ref = x.to(torch.bfloat16).double().numpy()
    got = oracle.round_bf16(x.double().numpy())
    assert np.array_equal(got, ref)


def test_bf16_ulp(oracle):
    assert oracle.bf16_ulp(1.0) == 2.0 ** -7
    assert oracle.bf16_ulp(1.99) == 2.0 ** -7
    assert oracle.bf16_ulp(2.0) == 2.0 ** -6
    assert oracle.bf16_ulp(-0.75) == 2.0 ** -8
    assert oracle.bf16_ulp(1e-45) == 2.0 ** -133
    x = torch.tensor([0.3, 5.0, 100.0], dtype=torch.bfloat16)
    nxt = (x.view(torch.int16) + 1).view(torch.bfloat16)
    assert np.array_equal(oracle.bf16_ulp(x.double().numpy()), (nxt.double() - x.double()).numpy())
