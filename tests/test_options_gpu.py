"""The optional parts of the CUDA path against the oracle: fp16 logits (every kernel family), token
entropy from the log-prob pass, and the monitors of the policy step.
"""
import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs

from helpers import OracleRun, TOL_LP, bits, close_rel, np32
from test_parity_gpu import DEV, _experience_both_ways, _t, dlogits_properties, run_steps, sample_rows

pytestmark = pytest.mark.gpu


def _f16_batch(w):
    """The workload's batch with both logits tensors converted to fp16 (bf16 values are exact in fp16 here: the
    synthetic logits stay far inside its range; -inf stays -inf)."""
    batch = inputs.make_batch(w, device=DEV)
    batch["actor"] = batch["actor"].to(torch.float16)
    batch["ref"] = batch["ref"].to(torch.float16)
    # add fp16-only precision: values that bf16 cannot hold
    g = torch.Generator(device=DEV).manual_seed(w.seed + 77)
    fin = torch.isfinite(batch["actor"])
    noise = (torch.randn(batch["actor"].shape, generator=g, device=DEV) * 2.0 ** -6).to(torch.float16)
    batch["actor"] = torch.where(fin, batch["actor"] + noise, batch["actor"])
    batch["ref"] = torch.where(fin, batch["ref"] + noise, batch["ref"])
    return batch


@pytest.mark.parametrize("name,kw,in_place", [
    ("tiny", {}, False),                                   # short rows: generic kernel for fp16
    ("tiny", {"V": 1001, "B": 3, "T": 9, "lengths": "uniform:0:9"}, False),      # odd rows
    ("llama2", {"B": 2, "T": 24}, False),                  # exponentials in registers
    ("opt", {"B": 2, "T": 24}, True),                      # registers + tensor memory, in place
    ("gpt2", {"B": 3, "T": 12, "lengths": "uniform:5:12"}, True),               # rows off 16-byte boundaries
    ("ragged", {"B": 5, "T": 6, "V": 57000}, False),      # one block, chunk ring
    ("ragged", {"B": 5, "T": 6, "V": 70000}, False),      # cluster of two blocks, whole-slice buffers
    ("ragged", {"B": 5, "T": 6, "V": 131072}, False),     # cluster of two blocks, chunk ring
    ("ragged", {"B": 5, "T": 6, "V": 150000}, False),     # cluster of three blocks
    ("ragged", {"B": 5, "T": 6, "V": 163840}, True),      # cluster of four blocks, in place
    ("ragged", {"B": 3, "T": 4, "V": 213000}, False),     # cluster of four blocks, chunk ring
    ("ragged", {"B": 3, "T": 4, "V": 262152}, False),     # beyond every cluster: generic kernel for fp16
    ("ragged", {"B": 12, "T": 40, "V": 16384}, False),    # -inf entries, sharpened rows, 32 KB rows
])
def test_fp16_logits_every_step(oracle, name, kw, in_place):
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = _f16_batch(w)
    run = OracleRun(oracle, w, batch)
    out, rep = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], in_place=in_place,
                         all_rows=True)
    assert out.dlogits.dtype == torch.float16
    if not in_place:
        dlogits_properties(run, out, batch["ids"], batch["actor"])
        _experience_both_ways(w, batch, batch["actor"], batch["ref"], batch["ids"])


@pytest.mark.parametrize("name", ["opt", "gpt2"])
def test_fp16_full_size(oracle, name):
    w = inputs.WORKLOADS[name]
    batch = _f16_batch(w)
    run = OracleRun(oracle, w, batch)
    rows = sample_rows(run, 48, seed=w.seed)
    out, rep = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], sample_rows=rows)
    dlogits_properties(run, out, batch["ids"], batch["actor"])
    print(name, "fp16", {k: (round(v, 4) if isinstance(v, float) else v) for k, v in rep.items()})


@pytest.mark.parametrize("name,kw,f16", [
    ("tiny", {}, False), ("tiny", {}, True),
    ("tiny", {"V": 1003, "B": 3, "T": 9, "lengths": "uniform:0:9"}, False),      # rows off 16-byte boundaries
    ("ragged", {"B": 12, "T": 40, "V": 4096}, False),                              # -inf entries, sharpened rows
    ("ragged", {"B": 12, "T": 40, "V": 4096}, True),
    ("llama2", {"B": 4, "T": 64}, False),                                          # peaked rows
    ("opt", {}, False),                                                            # full size
])
def test_entropy_from_the_logprob_pass(oracle, name, kw, f16):
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = _f16_batch(w) if f16 else inputs.make_batch(w, device=DEV)
    ln = batch["lengths"].cpu().numpy()
    ws = binding.workspace(w.B, w.T, DEV)
    ent = torch.full((w.B, w.T), float("nan"), device=DEV)
    lp = binding.gather_logprobs(batch["actor"], batch["ids"], batch["lengths"], ws, out_entropy=ent)
    assert binding.poll_status(ws) == 0
    want = np.zeros((w.B, w.T))
    for b0 in range(0, w.B, 4):
        want[b0:b0 + 4] = oracle.token_entropy(bits(batch["actor"][b0:b0 + 4]), ln[b0:b0 + 4])
    ok, ratio = close_rel(np32(ent), want)
    assert ok, ratio
    valid = np.arange(w.T)[None, :] < ln[:, None]
    assert (np32(ent)[~valid] == 0).all() and (np32(ent)[valid] >= 0).all()
    # the log-probs of the same call agree with those of the plain call (the entropy variant sums in another order)
    plain = binding.gather_logprobs(batch["actor"], batch["ids"], batch["lengths"], ws)
    assert (lp - plain).abs().max().item() <= 1e-5
    # and the fused experience call gives the same entropy for the actor's rows
    exp = binding.Experience(w.B, w.T, DEV)
    ent2 = torch.full((w.B, w.T), float("nan"), device=DEV)
    binding.experience(batch["actor"], batch["ref"], batch["ids"], batch["lengths"], batch["score"], batch["values_old"],
                       w.beta_kl, w.reward_clip, w.gamma, w.lam, ws, exp, out_entropy=ent2)
    assert torch.equal(ent, ent2) and torch.equal(exp.lp_actor, lp)


def test_entropy_closed_forms():
    # uniform rows: ln V; a row with one live entry: 0
    V = 4096
    z = torch.zeros((1, 3, V), dtype=torch.bfloat16, device=DEV)
    z[0, 1] = -3.5
    z[0, 2] = float("-inf")
    z[0, 2, 17] = 2.0
    ids = torch.tensor([[0, 5, 17]], device=DEV)
    lengths = torch.tensor([3], dtype=torch.int32, device=DEV)
    ws = binding.workspace(1, 3, DEV)
    ent = torch.empty((1, 3), device=DEV)
    lp = binding.gather_logprobs(z, ids, lengths, ws, out_entropy=ent)
    assert abs(float(ent[0, 0]) - np.log(V)) < 1e-4 and abs(float(ent[0, 1]) - np.log(V)) < 1e-4
    assert abs(float(ent[0, 2])) < 1e-6 and abs(float(lp[0, 2])) < 1e-6


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"lp_old_sigma": 0.4}), ("opt", {"B": 4}),
                                     ("ragged", {"B": 12, "T": 40, "V": 4096}),
                                     ("tiny", {"lengths": "uniform:0:0"})])
def test_policy_step_monitors(oracle, name, kw):
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    ws = binding.workspace(w.B, w.T, DEV)
    out = binding.PPOOutputs(batch["actor"])
    lp_old, adv = _t(run.lp_old_in), _t(run.adv_in)
    binding.ppo_loss_fwd_bwd(batch["actor"], batch["ids"], batch["lengths"], lp_old, adv, _t(run.values_new_in),
                             _t(run.values_old_in), _t(run.ret_in), w.clip_eps, w.value_clip, run.grad_scale, ws, out)
    stats = binding.ppo_stats(out.lp_new, lp_old, adv, batch["lengths"], w.clip_eps, ws)
    assert binding.poll_status(ws) == 0
    kl, cf = oracle.ppo_stats(run.lp_actor, run.lp_old_in, run.adv_in, run.lengths, w.clip_eps)
    got = np32(stats).astype(np.float64)
    assert abs(got[0] - kl) <= 1e-4 * max(1.0, abs(kl)), (got, kl)
    # tokens within float32 rounding of the edge of the interval may fall on either side
    slack = run.pg_kink.sum() / max(run.N, 1)
    assert abs(got[1] - cf) <= slack + 1e-6, (got, cf, slack)
    if run.N:
        # the clip fraction is the share of valid tokens whose gradient row is all zero
        zero_rows = (out.dlogits.view(torch.int16) == 0).all(-1).cpu().numpy() & run.valid
        assert abs(zero_rows.sum() / run.N - got[1]) <= slack + 1e-6
    again = binding.ppo_stats(out.lp_new, lp_old, adv, batch["lengths"], w.clip_eps, ws)
    assert torch.equal(stats, again)
