"""Pins for the oracle's IEEE binary16 (fp16) entry: exact widening, rounding, spacing, and the
steps that take fp16 logits.  (Section 3 of the paper, "Workload and Setting": the model families
are run in 16-bit floating point; bf16 and fp16 are the two such types.)
"""
import numpy as np
import pytest
import torch


def test_f16_widening_is_exact_for_every_bit_pattern(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.f16_to_double(bits)
    want = bits.view(np.float16).astype(np.float64)              # numpy's own binary16
    nan = np.isnan(want)
    assert (np.isnan(got) == nan).all()
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_round_f16_matches_torch_rounding(oracle):
    g = torch.Generator().manual_seed(0)
    mant = torch.rand(4000, generator=g, dtype=torch.float64) + 1.0
    expo = torch.randint(-30, 18, (4000,), generator=g).double()
    sign = torch.randint(0, 2, (4000,), generator=g).double() * 2 - 1
    x = sign * mant * torch.exp2(expo)
    special = torch.tensor([0.0, 1.0, 65504.0, 65519.99, 65520.0, 70000.0, -65520.0, 2.0 ** -24, 2.0 ** -25,
                            1.5 * 2.0 ** -25, 2.0 ** -14, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11,
                            1.0 + 2.0 ** -11 + 2.0 ** -20, 2049.0, 2051.0], dtype=torch.float64)
    # torch converts float64 to fp16 through float32, so the comparison uses values that float32 holds exactly
    x = torch.cat([x, special]).float().double()
    want = x.to(torch.float16).double().numpy()
    got = oracle.round_f16(x.numpy())
    assert np.array_equal(got, want)


def test_f16_ulp_is_the_gap_to_the_next_value(oracle):
    bits = np.array([0x0001, 0x03ff, 0x0400, 0x3c00, 0x3fff, 0x4000, 0x7bfe], dtype=np.uint16)
    x = oracle.f16_to_double(bits)
    nxt = oracle.f16_to_double(bits + 1)
    assert np.array_equal(oracle.f16_ulp(x), nxt - x)
    assert oracle.f16_ulp(0.0) == 2.0 ** -24


def test_steps_on_f16_logits_equal_the_float64_entry(oracle):
    g = torch.Generator().manual_seed(4)
    z16 = (torch.randn((2, 5, 257), generator=g) * 3).to(torch.float16)
    z16[0, 1, 7] = float("-inf")
    ids = torch.randint(0, 257, (2, 5), generator=g).numpy()
    ids[0, 1] = 3
    lengths = [5, 3]
    arr16 = z16.numpy()
    arr64 = z16.double().numpy()
    assert np.array_equal(oracle.gather_logprobs(arr16, ids, lengths), oracle.gather_logprobs(arr64, ids, lengths))
    assert np.array_equal(oracle.token_entropy(arr16, lengths), oracle.token_entropy(arr64, lengths))
    gg = np.random.default_rng(0).normal(0, 1, (2, 5))
    rows = np.arange(10)
    assert np.array_equal(oracle.dlogits_rows(arr16, ids, lengths, gg, rows), oracle.dlogits_rows(arr64, ids, lengths, gg, rows))
    # and against torch's float64 log-softmax of the widened tensor
    lp = torch.log_softmax(z16.double(), -1).gather(2, torch.from_numpy(ids)[..., None])[..., 0].numpy()
    valid = np.arange(5)[None, :] < np.array(lengths)[:, None]
    assert np.abs(oracle.gather_logprobs(arr16, ids, lengths) - lp)[valid].max() < 1e-12


def test_bf16_and_f16_bits_are_not_confused(oracle):
    # the same 16 bits mean different numbers in the two types: 0x3c00 is 1.0 in fp16 and 0.0078125 in bf16
    z = np.array([[[0x3c00, 0x0000]]], dtype=np.uint16)
    ids = np.zeros((1, 1), dtype=np.int64)
    lp_bf16 = oracle.gather_logprobs(z, ids, [1])[0, 0]
    lp_f16 = oracle.gather_logprobs(z.view(np.float16), ids, [1])[0, 0]
    assert lp_f16 == pytest.approx(-np.log1p(np.exp(-1.0)), abs=1e-15)
    assert lp_bf16 == pytest.approx(-np.log1p(np.exp(-0.0078125)), abs=1e-15)
