"""What the path costs in device memory, in the paper's terms (reserved / allocated / fragmentation).

The library's calls allocate nothing: neither PyTorch's allocator statistics nor the driver's free
memory move across them when every output buffer is passed in.  Out of place, the loss phase needs one
bf16 [B,T,V] gradient; in place it needs none.  Releasing the allocator cache between the experience
phase and the training phase (the paper's proposal) returns the experience phase's blocks to the driver."""
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs
from paper_2410_15651_b200.memory import PhaseMemory

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda:0")


def _setup(w):
    batch = inputs.make_batch(w, device=DEV)
    ws = binding.workspace(w.B, w.T, DEV)
    exp = binding.Experience(w.B, w.T, DEV)
    return batch, ws, exp


def test_library_calls_allocate_nothing():
    w = inputs.scaled(inputs.WORKLOADS["opt"], B=4, T=64)
    batch, ws, exp = _setup(w)
    out = binding.PPOOutputs(batch["actor"])
    lp_old = torch.zeros((w.B, w.T), device=DEV)
    N = float(batch["lengths"].sum().item())

    def experience():
        binding.experience(batch["actor"], batch["ref"], batch["ids"], batch["lengths"], batch["score"],
                           batch["values_old"], w.beta_kl, w.reward_clip, w.gamma, w.lam, ws, exp)

    def loss():
        binding.ppo_loss_fwd_bwd(batch["actor"], batch["ids"], batch["lengths"], lp_old, exp.adv,
                                 batch["values_new"], batch["values_old"], exp.returns, w.clip_eps, w.value_clip,
                                 N, ws, out)

    experience(); loss()                                  # first calls: module loading, function attributes
    mem = PhaseMemory(DEV)
    mem.run("experience", experience)
    mem.run("loss", loss)
    for name, s in mem.summary().items():
        assert s["allocated_delta"] == 0 and s["reserved_delta"] == 0, (name, s)
        assert s["peak_allocated_over_start"] == 0, (name, s)
        assert s["driver_used_delta"] == 0, (name, s)       # nothing taken from the driver behind torch's back
    assert binding.poll_status(ws) == 0


def test_in_place_gradient_needs_no_logits_sized_buffer_and_empty_cache_releases_the_rest():
    # start from an empty allocator cache, so that this test's tensors do not share segments with blocks that
    # earlier tests left cached (a segment goes back to the driver only when all of it is free)
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    w = inputs.scaled(inputs.WORKLOADS["llama2"], B=4, T=128)
    batch, ws, exp = _setup(w)
    logits_bytes = batch["actor"].numel() * 2
    lp_old = torch.zeros((w.B, w.T), device=DEV)
    N = float(batch["lengths"].sum().item())
    torch.cuda.empty_cache()

    def loss(in_place):
        out = binding.PPOOutputs(batch["actor"], in_place=in_place)
        binding.ppo_loss_fwd_bwd(batch["actor"], batch["ids"], batch["lengths"], lp_old, exp.adv,
                                 batch["values_new"], batch["values_old"], exp.returns, w.clip_eps, w.value_clip,
                                 N, ws, out)
        return out

    mem = PhaseMemory(DEV)
    keep = mem.run("loss out of place", lambda: loss(False))
    s = mem.summary()["loss out of place"]
    assert logits_bytes <= s["allocated_delta"] <= logits_bytes + (1 << 20)      # one bf16 [B,T,V] gradient
    del keep
    # the paper's remedy: the freed gradient block sits in the allocator's cache (reserved, not allocated) until
    # empty_cache() hands it back to the driver
    reserved_cached = torch.cuda.memory_reserved(DEV)
    torch.cuda.empty_cache()
    assert reserved_cached - torch.cuda.memory_reserved(DEV) >= logits_bytes
    keep = mem.run("loss in place", lambda: loss(True))
    s = mem.summary()["loss in place"]
    assert s["allocated_delta"] < (1 << 20) and s["peak_allocated_over_start"] < (1 << 20)
