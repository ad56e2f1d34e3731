"""The entry point for callers that cannot allocate scratch memory, against the regular one.

rlhf_ppo_loss_fwd_bwd_noalloc takes no workspace: its scratch is a fixed array inside the library's
device image, shared by all calls on a device and never cleared between them.  The test calls it
twice in a row through the C ABI, on two different batches (the second smaller than the first, so
that stale contents of the shared array lie beyond what the second call writes), and requires each
call to reproduce the regular entry point: bit-identical, since both run the same kernels.

This file is collected last on purpose, so that a run that stops at the first failure has already
run every other test; it passes on its own in a fresh process as well.
"""
import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _inputs(w):
    """A batch and plausible float32 step-4 inputs made with torch ops (no oracle needed here: the
    comparison is between two entry points of the same library)."""
    batch = inputs.make_batch(w, device=DEV)
    B, T = w.B, w.T
    ws = binding.workspace(B, T, DEV)
    lengths = batch["lengths"]
    mask = torch.arange(T, device=DEV)[None, :] < lengths[:, None]
    lp_cur = binding.gather_logprobs(batch["actor"], batch["ids"], lengths, ws)
    lp_ref = binding.gather_logprobs(batch["ref"], batch["ids"], lengths, ws)
    lp_old = (lp_cur + batch["lp_old_noise"] * mask).contiguous()
    rewards = binding.kl_reward(lp_old, lp_ref, batch["score"], lengths, w.beta_kl, w.reward_clip)
    adv, ret = binding.gae(rewards, batch["values_old"], lengths, w.gamma, w.lam)
    return batch, ws, lp_old, adv, ret


def _both(w, grad_scale):
    batch, ws, lp_old, adv, ret = _inputs(w)
    args = (batch["actor"], batch["ids"], batch["lengths"], lp_old, adv, batch["values_new"],
            batch["values_old"], ret, w.clip_eps, w.value_clip, grad_scale)
    want = binding.ppo_loss_fwd_bwd(*args, ws, binding.PPOOutputs(batch["actor"]))
    assert binding.poll_status(ws) == 0
    got = binding.PPOOutputs(batch["actor"])
    for t in (got.loss, got.dvalues, got.lp_new):
        t.fill_(float("nan"))
    got.dlogits.fill_(float("nan"))
    flags = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    binding.ppo_loss_fwd_bwd_noalloc(*args, got, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    # the tolerances of the parity tests, and in fact bit-identical
    assert torch.isfinite(got.loss).all()
    assert torch.allclose(got.loss, want.loss, rtol=1e-4, atol=1e-4)
    assert torch.equal(got.loss, want.loss)
    assert torch.equal(got.dlogits.view(torch.int16), want.dlogits.view(torch.int16))
    assert torch.equal(got.dvalues, want.dvalues)
    assert torch.equal(got.lp_new, want.lp_new)
    return batch, lp_old, adv, ret


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    big = inputs.scaled(inputs.WORKLOADS["opt"], B=4, T=96, lengths="uniform:40:96")       # V = 50272
    small = inputs.scaled(inputs.WORKLOADS["ragged"], B=6, T=20, V=4096)                     # padded rows, -inf
    _both(big, grad_scale=float(4 * 96))
    _both(small, grad_scale=1.0)


def test_noalloc_reports_device_flags_and_refuses_large_batches():
    w = inputs.scaled(inputs.WORKLOADS["tiny"], B=2, T=8, V=64, lengths="full")
    batch, lp_old, adv, ret = _both(w, grad_scale=1.0)
    # an id outside the vocabulary is flagged through out_device_status, and the flag does not
    # leak into the next call
    bad_ids = batch["ids"].clone()
    bad_ids[1, 3] = w.V + 5
    out = binding.PPOOutputs(batch["actor"])
    flags = torch.zeros(1, dtype=torch.int32, device=DEV)
    args = [batch["actor"], bad_ids, batch["lengths"], lp_old, adv, batch["values_new"],
            batch["values_old"], ret, w.clip_eps, w.value_clip, 1.0]
    binding.ppo_loss_fwd_bwd_noalloc(*args, out, flags)
    assert int(flags.item()) == 16
    assert (out.dlogits[1, 3].view(torch.int16) == 0).all()
    args[1] = batch["ids"]
    binding.ppo_loss_fwd_bwd_noalloc(*args, out, flags)
    assert int(flags.item()) == 0
    # beyond the fixed scratch: refused on the host, nothing launched (no buffer needs to be that large)
    B, T = 2, binding.NOALLOC_MAX_TOKENS // 2 + 1
    with pytest.raises(binding.RlhfError) as err:
        lib = binding.lib()
        p = batch["actor"].data_ptr()
        status = lib.rlhf_ppo_loss_fwd_bwd_noalloc(p, T * 8, 8, p, T, p, p, p, p, p, p, B, T, 8, 0.2, 0.2, 1.0,
                                                   p, p, p, T * 8, 8, p, None, None, None)
        binding._check(status, "rlhf_ppo_loss_fwd_bwd_noalloc")
    assert err.value.status == 8 and "TOO_LARGE" in str(err.value)
