"""Stored outputs of the whole path on the tiny workload (tests/golden/tiny_path.json, written by
tests/golden/write_golden.py from the CPU oracle).  On the CPU: the oracle and the seeded generator
still reproduce them.  On the GPU: the CUDA path matches them within the stated tolerances."""
import json
import os

import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import inputs

from helpers import OracleRun, TOL_LP, close_rel

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "tiny_path.json")))


def test_oracle_reproduces_the_stored_values(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device="cpu")
    run = OracleRun(oracle, w, batch)
    assert run.lengths.tolist() == GOLD["lengths"] and run.N == GOLD["N"]
    for name in ("lp_actor", "lp_ref", "rewards", "adv", "ret"):
        assert np.allclose(getattr(run, name), np.array(GOLD[name]), rtol=0, atol=1e-12), name
    assert abs(run.ppo.loss_pg - GOLD["loss_pg"]) < 1e-12 and abs(run.ppo.loss_vf - GOLD["loss_vf"]) < 1e-12
    assert np.allclose(run.ppo.g, np.array(GOLD["g"]), rtol=0, atol=1e-12)
    # what the definitions fix about the stored numbers themselves
    lens = np.array(GOLD["lengths"])
    valid = np.arange(w.T)[None, :] < lens[:, None]
    adv, ret = np.array(GOLD["adv"]), np.array(GOLD["ret"])
    v_old = batch["values_old"].numpy().astype(np.float64)
    assert np.allclose((ret - adv)[valid], v_old[valid], rtol=0, atol=1e-6)       # G - A = V
    assert (np.array(GOLD["lp_actor"])[valid] < 0).all() and (np.array(GOLD["rewards"])[~valid] == 0).all()
    assert all(v == 0 for v in GOLD["dlogits"][-1]) and GOLD["dlogits_rows"][-1] == 31   # the padded row


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_values(oracle):
    from paper_2410_15651_b200 import binding
    dev = "cuda:0"
    w = inputs.WORKLOADS["tiny"]
    cpu = inputs.make_batch(w, device="cpu")
    run = OracleRun(oracle, w, cpu)                      # only for the float32 inputs of each step
    b = {k: v.to(dev) for k, v in cpu.items()}
    ws = binding.workspace(w.B, w.T, dev)
    t = lambda a: torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float32, device=dev)
    lp_a = binding.gather_logprobs(b["actor"], b["ids"], b["lengths"], ws).cpu().numpy()
    lp_r = binding.gather_logprobs(b["ref"], b["ids"], b["lengths"], ws).cpu().numpy()
    assert np.abs(lp_a - np.array(GOLD["lp_actor"])).max() <= TOL_LP
    assert np.abs(lp_r - np.array(GOLD["lp_ref"])).max() <= TOL_LP
    r = binding.kl_reward(t(run.lp_old_in), t(run.lp_ref_in), t(run.score_in), b["lengths"], w.beta_kl, w.reward_clip)
    assert close_rel(r.cpu().numpy(), np.array(GOLD["rewards"]))[0]
    adv, ret = binding.gae(t(run.rewards_in), t(run.values_old_in), b["lengths"], w.gamma, w.lam)
    assert close_rel(adv.cpu().numpy(), np.array(GOLD["adv"]))[0] and close_rel(ret.cpu().numpy(), np.array(GOLD["ret"]))[0]
    out = binding.ppo_loss_fwd_bwd(b["actor"], b["ids"], b["lengths"], t(run.lp_old_in), t(run.adv_in),
                                   t(run.values_new_in), t(run.values_old_in), t(run.ret_in), w.clip_eps,
                                   w.value_clip, float(GOLD["N"]), ws)
    assert binding.poll_status(ws) == 0
    loss = out.loss.cpu().numpy()
    assert close_rel(loss[0], GOLD["loss_pg"])[0] and close_rel(loss[1], GOLD["loss_vf"])[0]
    assert close_rel(out.dvalues.cpu().numpy(), np.array(GOLD["dvalues"]))[0]
    rows, cols = np.array(GOLD["dlogits_rows"]), np.array(GOLD["dlogits_cols"])
    got = out.dlogits.float().cpu().numpy().reshape(w.B * w.T, w.V).astype(np.float64)
    want = np.array(GOLD["dlogits"])
    assert (np.abs(got[rows][:, cols] - want) <= oracle.bf16_ulp(want) + 1e-6).all()
    ids = cpu["ids"].numpy().reshape(-1)
    for i, rr in enumerate(rows):
        wl = GOLD["dlogits_at_label"][i]
        assert abs(got[rr, ids[rr]] - wl) <= oracle.bf16_ulp(wl) + 1e-6
