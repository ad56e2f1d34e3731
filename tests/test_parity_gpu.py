"""CUDA path against the CPU oracle, step by step, on the synthetic workloads.

Each step of the CUDA library is given the same float32 inputs as the oracle (the oracle's own
outputs of the step before, rounded to float32) and compared element by element.  The tiny case
is compared in full; the larger ones in full for every O(B*T) output and on sampled rows for the
bf16 logits gradient, plus properties that hold for every row.
"""
import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs

from helpers import OracleRun, TOL_LP, check_dlogits_rows, close_rel, np32

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _t(a, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype, device=DEV)


def run_steps(oracle, w, batch, run, logits, ref, ids, in_place=False, sample_rows=None, all_rows=False):
    """Run every CUDA step on the oracle-fed inputs and compare.  Returns a dict of error ratios."""
    B, T, V = logits.shape
    lengths = batch["lengths"]
    ws = binding.workspace(B, T, DEV)
    report = {}

    # step 1, actor and reference
    lp_a = binding.gather_logprobs(logits, ids, lengths, ws)
    lp_r = binding.gather_logprobs(ref, ids, lengths, ws)
    for name, got, want in (("lp_actor", lp_a, run.lp_actor), ("lp_ref", lp_r, run.lp_ref)):
        err = np.abs(np32(got).astype(np.float64) - want)
        assert np.isfinite(np32(got)).all(), name
        assert err.max(initial=0.0) <= TOL_LP, (name, err.max())
        assert (np32(got)[~run.valid] == 0).all(), name
        report[name] = err.max(initial=0.0) / TOL_LP

    # step 2
    r = binding.kl_reward(_t(run.lp_old_in), _t(run.lp_ref_in), _t(run.score_in), lengths,
                          w.beta_kl, w.reward_clip)
    ok, report["rewards"] = close_rel(np32(r), run.rewards)
    assert ok, report
    assert (np32(r)[~run.valid] == 0).all()

    # step 3
    adv, ret = binding.gae(_t(run.rewards_in), _t(run.values_old_in), lengths, w.gamma, w.lam)
    ok, report["adv"] = close_rel(np32(adv), run.adv)
    assert ok, report
    ok, report["ret"] = close_rel(np32(ret), run.ret)
    assert ok, report
    assert (np32(adv)[~run.valid] == 0).all() and (np32(ret)[~run.valid] == 0).all()

    # step 4
    src = logits.clone() if in_place else logits
    out = binding.PPOOutputs(src, in_place=in_place)
    # every output starts as NaN: an element the kernels fail to write cannot pass for a zero
    for t_ in (out.loss, out.dvalues, out.lp_new):
        t_.fill_(float("nan"))
    if not in_place:
        out.dlogits.fill_(float("nan"))
    binding.ppo_loss_fwd_bwd(src, ids, lengths, _t(run.lp_old_in), _t(run.adv_in), _t(run.values_new_in),
                             _t(run.values_old_in), _t(run.ret_in), w.clip_eps, w.value_clip,
                             run.grad_scale, ws, out)
    assert binding.poll_status(ws) == 0
    loss = np32(out.loss).astype(np.float64)
    ok, report["loss_pg"] = close_rel(loss[0], run.ppo.loss_pg)
    assert ok, (loss, run.ppo.loss_pg, report)
    ok, report["loss_vf"] = close_rel(loss[1], run.ppo.loss_vf)
    assert ok, (loss, run.ppo.loss_vf, report)
    lp_new = np32(out.lp_new).astype(np.float64)
    assert np.abs(lp_new - run.lp_actor).max(initial=0.0) <= TOL_LP
    assert (lp_new[~run.valid] == 0).all()
    dv = np32(out.dvalues).astype(np.float64)
    keep = ~run.vf_kink
    ok, report["dvalues"] = close_rel(dv[keep], run.ppo.dvalues[keep])
    assert ok, report
    assert (dv[~run.valid] == 0).all()

    rows = np.arange(B * T) if all_rows else np.asarray(sample_rows)
    report["dlogits"], report["dlogits_rows"] = check_dlogits_rows(oracle, run, logits, ids, out.dlogits, rows)
    return out, report


def sample_rows(run, n, seed=0):
    """A mix of valid rows, padded rows and zero-gradient rows."""
    rng = np.random.default_rng(seed)
    flat_valid = np.flatnonzero(run.valid.reshape(-1))
    flat_pad = np.flatnonzero(~run.valid.reshape(-1))
    zero_g = np.flatnonzero((run.ppo.g.reshape(-1) == 0) & run.valid.reshape(-1))
    picks = [rng.choice(flat_valid, size=min(n, flat_valid.size), replace=False)]
    if flat_pad.size:
        picks.append(rng.choice(flat_pad, size=min(max(2, n // 8), flat_pad.size), replace=False))
    if zero_g.size:
        picks.append(zero_g[:4])
    # first and last valid row, and the rows around each sequence end
    picks.append(flat_valid[[0, -1]])
    return np.unique(np.concatenate(picks))


def dlogits_properties(run, out, ids, logits):
    """Properties of the full dlogits tensor that need no oracle row: padded rows are zero, every
    row sums to ~0 (within the bf16 rounding of its entries), the label entry carries the sign of g."""
    B, T, V = logits.shape
    d = out.dlogits
    valid = torch.as_tensor(run.valid, device=d.device)
    for b in range(B):
        db = d[b].float()                                           # [T,V]
        assert torch.isfinite(db).all()
        pad = ~valid[b]
        if pad.any():
            assert (d[b][pad].view(torch.int16) == 0).all()         # exact +0
        rs = db.double().sum(-1).abs()
        if d.dtype == torch.float16:
            # half a step of every entry: relative 2^-11 for normal values, 2^-25 absolute below 2^-14
            lim = 0.5 * db.abs().double().sum(-1) * 2.0 ** -10 + V * 2.0 ** -25 + 1e-5
        else:
            lim = 0.5 * db.abs().double().sum(-1) * 2.0 ** -7 + 1e-5    # sum of half-ulps bound, with slack
        assert (rs <= lim).all(), (b, float((rs / lim).max()))
        g = torch.as_tensor(run.ppo.g[b], device=d.device)
        dy = db.gather(1, ids[b][:, None])[:, 0].double()
        # one_m_py can underflow to 0 for extremely peaked rows; otherwise the sign follows g
        assert ((torch.sign(dy) == torch.sign(g)) | (dy == 0) | torch.as_tensor(run.pg_kink[b], device=d.device)).all()


# --------------------------------------------------------------------------------------------

def test_tiny_full(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    out, rep = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    dlogits_properties(run, out, batch["ids"], batch["actor"])
    # twice the same call: bit-identical results (no atomics on floats, fixed reduction order)
    out2, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    assert torch.equal(out.loss, out2.loss) and torch.equal(out.dlogits, out2.dlogits)


def test_tiny_strided_prompt_view_and_in_place(oracle):
    # logits of the whole sequence [B,P+T,V]; the response rows are a strided view of it
    w = inputs.WORKLOADS["tiny"]
    full = inputs.make_batch(w, device=DEV, with_prompt=True)
    logits = inputs.response_view(w, full["actor"])
    ref = inputs.response_view(w, full["ref"])
    ids = full["ids"][:, w.P:]
    assert not logits.is_contiguous() and not ids.is_contiguous()
    run = OracleRun(oracle, w, full, logits_view=logits, ref_view=ref, ids_view=ids)
    run_steps(oracle, w, full, run, logits, ref, ids, all_rows=True)
    # in place: dlogits overwrite a copy of the logits (contiguous clone of the view)
    run_steps(oracle, w, full, run, logits.contiguous(), ref, ids, in_place=True, all_rows=True)
    # in place on the strided view itself: the prompt rows around it must stay untouched
    full2 = full["actor"].clone()
    view2 = inputs.response_view(w, full2)
    ws = binding.workspace(w.B, w.T, DEV)
    out = binding.PPOOutputs(view2, in_place=True)
    binding.ppo_loss_fwd_bwd(view2, ids, full["lengths"], torch.as_tensor(run.lp_old_in, device=DEV),
                             torch.as_tensor(run.adv_in, device=DEV), torch.as_tensor(run.values_new_in, device=DEV),
                             torch.as_tensor(run.values_old_in, device=DEV), torch.as_tensor(run.ret_in, device=DEV),
                             w.clip_eps, w.value_clip, run.grad_scale, ws, out)
    assert binding.poll_status(ws) == 0
    assert torch.equal(full2[:, :w.P - 1], full["actor"][:, :w.P - 1])
    assert torch.equal(full2[:, w.P - 1 + w.T:], full["actor"][:, w.P - 1 + w.T:])
    check_dlogits_rows(oracle, run, logits, ids, view2, np.arange(w.B * w.T))


def test_tiny_special_cases(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device=DEV)
    # on-policy (rho = 1) and sequence scores outside the reward clip on both sides
    run = OracleRun(oracle, w, batch, on_policy=True, score_override=np.array([7.5, -9.0], dtype=np.float32))
    run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    assert (run.ppo.g[run.valid] != 0).all()
    # grad_scale = 1: the 1/N normalisation is inside the gradient
    run1 = OracleRun(oracle, w, batch, grad_scale=1.0)
    run_steps(oracle, w, batch, run1, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    # a wider old-policy spread so that many tokens are clipped (zero-gradient rows)
    wide = inputs.scaled(w, lp_old_sigma=0.4)
    bw = inputs.make_batch(wide, device=DEV)
    runw = OracleRun(oracle, wide, bw)
    assert (runw.ppo.g[runw.valid] == 0).sum() >= 3
    run_steps(oracle, wide, bw, runw, bw["actor"], bw["ref"], bw["ids"], all_rows=True)


@pytest.mark.parametrize("V", [1000, 1001, 1003, 8, 7, 1, 4099])
def test_small_odd_vocabularies(oracle, V):
    # V not a multiple of 8 makes rows that are not 16-byte aligned
    w = inputs.scaled(inputs.WORKLOADS["tiny"], V=V, B=3, T=9, lengths="uniform:0:9", seed=10 + V)
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)


def test_ragged_small(oracle):
    # the ragged recipe (all-pad, length 1 and 2, -inf entries, sharpened rows; gamma .99, lambda 1) at a small size
    w = inputs.scaled(inputs.WORKLOADS["ragged"], B=12, T=40, V=4096)
    batch = inputs.make_batch(w, device=DEV)
    assert (batch["lengths"][:4].cpu() == torch.tensor([0, 1, 2, 40])).all()
    run = OracleRun(oracle, w, batch)
    out, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    dlogits_properties(run, out, batch["ids"], batch["actor"])
    # deleted (-inf) entries get a zero gradient
    dead = torch.isinf(batch["actor"].float())
    assert dead.any() and (out.dlogits[dead].float() == 0).all()


def test_all_padding_batch(oracle):
    w = inputs.scaled(inputs.WORKLOADS["tiny"], lengths="uniform:0:0")
    batch = inputs.make_batch(w, device=DEV)
    assert int(batch["lengths"].sum()) == 0
    run = OracleRun(oracle, w, batch)
    out, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    assert (out.loss == 0).all() and (out.dlogits.view(torch.int16) == 0).all() and (out.dvalues == 0).all()


def test_gae_long_sequences_closed_form(oracle):
    # T beyond one warp-chunk round, gamma = lambda = 1: returns are reward-to-go (float64 cumsum)
    rng = np.random.default_rng(5)
    B, T = 7, 3000
    lengths = np.array([3000, 2999, 1025, 1024, 33, 1, 0], dtype=np.int32)
    r = rng.normal(0, 1, (B, T)).astype(np.float32)
    v = rng.normal(0, 1, (B, T)).astype(np.float32)
    adv, ret = binding.gae(_t(r), _t(v), _t(lengths, torch.int32), 1.0, 1.0)
    for b, n in enumerate(lengths):
        togo = np.cumsum(r[b, :n][::-1].astype(np.float64))[::-1]
        ok, ratio = close_rel(np32(ret)[b, :n], togo)
        assert ok, (b, ratio)
    for gamma, lam in ((0.99, 0.95), (0.9, 1.0), (1.0, 0.0)):
        adv, ret = binding.gae(_t(r), _t(v), _t(lengths, torch.int32), gamma, lam)
        wa, wr = oracle.gae(r, v, lengths, gamma, lam)
        assert close_rel(np32(adv), wa)[0] and close_rel(np32(ret), wr)[0]


def _experience_both_ways(w, batch, logits, ref, ids, lp_old=None):
    """rlhf_experience against the four separate calls it stands for: bit-identical outputs."""
    B, T, _ = logits.shape
    lengths = batch["lengths"]
    ws = binding.workspace(B, T, DEV)
    lp_a = binding.gather_logprobs(logits, ids, lengths, ws)
    lp_r = binding.gather_logprobs(ref, ids, lengths, ws)
    r = binding.kl_reward(lp_a if lp_old is None else lp_old, lp_r, batch["score"], lengths, w.beta_kl, w.reward_clip)
    adv, ret = binding.gae(r, batch["values_old"], lengths, w.gamma, w.lam)
    out = binding.Experience(B, T, DEV)
    for t in (out.lp_actor, out.lp_ref, out.rewards, out.adv, out.returns):
        t.fill_(float("nan"))
    for _ in range(2):                       # twice: the per-sequence counters in the workspace must come back to zero
        binding.experience(logits, ref, ids, lengths, batch["score"], batch["values_old"], w.beta_kl,
                           w.reward_clip, w.gamma, w.lam, ws, out, lp_old=lp_old)
        assert binding.poll_status(ws) == 0
        for name, got, want in (("lp_actor", out.lp_actor, lp_a), ("lp_ref", out.lp_ref, lp_r),
                                ("rewards", out.rewards, r), ("adv", out.adv, adv), ("returns", out.returns, ret)):
            assert torch.equal(got, want), name
    return out


def test_experience_fused_tiny_and_ragged(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device=DEV)
    out = _experience_both_ways(w, batch, batch["actor"], batch["ref"], batch["ids"])
    # and against the oracle, the KL term taken from the actor log-probs computed in the same call
    ln = batch["lengths"].cpu().numpy()
    from helpers import bits
    o_a = oracle.gather_logprobs(bits(batch["actor"]), batch["ids"].cpu().numpy(), ln)
    o_r = oracle.gather_logprobs(bits(batch["ref"]), batch["ids"].cpu().numpy(), ln)
    o_rw = oracle.kl_reward(np32(out.lp_actor), np32(out.lp_ref), np32(batch["score"]), ln, w.beta_kl, w.reward_clip)
    o_adv, o_ret = oracle.gae(np32(out.rewards), np32(batch["values_old"]), ln, w.gamma, w.lam)
    assert np.abs(np32(out.lp_actor) - o_a).max() <= TOL_LP and np.abs(np32(out.lp_ref) - o_r).max() <= TOL_LP
    assert close_rel(np32(out.rewards), o_rw)[0] and close_rel(np32(out.adv), o_adv)[0] and close_rel(np32(out.returns), o_ret)[0]
    # ragged recipe: empty sequences, lengths 1 and 2, -inf entries; with an explicit lp_old for the KL term
    w2 = inputs.scaled(inputs.WORKLOADS["ragged"], B=12, T=40, V=4096)
    b2 = inputs.make_batch(w2, device=DEV)
    _experience_both_ways(w2, b2, b2["actor"], b2["ref"], b2["ids"])
    lp_old = torch.randn((12, 40), device=DEV) - 5.0
    _experience_both_ways(w2, b2, b2["actor"], b2["ref"], b2["ids"], lp_old=lp_old)
    # all padding
    w3 = inputs.scaled(w, lengths="uniform:0:0")
    b3 = inputs.make_batch(w3, device=DEV)
    o3 = _experience_both_ways(w3, b3, b3["actor"], b3["ref"], b3["ids"])
    assert (o3.rewards == 0).all() and (o3.adv == 0).all() and (o3.returns == 0).all()


@pytest.mark.parametrize("V", [1001, 7])
def test_experience_unaligned_rows_take_the_separate_kernels(V):
    w = inputs.scaled(inputs.WORKLOADS["tiny"], V=V, B=3, T=9, lengths="uniform:0:9", seed=40 + V)
    batch = inputs.make_batch(w, device=DEV)
    _experience_both_ways(w, batch, batch["actor"], batch["ref"], batch["ids"])


def test_experience_strided_views():
    w = inputs.WORKLOADS["tiny"]
    full = inputs.make_batch(w, device=DEV, with_prompt=True)
    _experience_both_ways(w, full, inputs.response_view(w, full["actor"]), inputs.response_view(w, full["ref"]),
                          full["ids"][:, w.P:])


@pytest.mark.parametrize("V,in_place", [(65544, False), (70000, True), (131072, False), (57000, False)])
def test_rows_larger_than_shared_memory(oracle, V, in_place):
    # rows that one block cannot hold twice in whole-row buffers: 131,088 B (one vector more than 128 KB) and 140,000 B
    # go to a cluster of two, exactly 256 KB to two blocks with a chunk ring each, 114,000 B to one such block
    w = inputs.scaled(inputs.WORKLOADS["ragged"], V=V, B=5, T=6, seed=70 + V % 7)
    batch = inputs.make_batch(w, device=DEV)
    batch["lengths"] = torch.tensor([0, 1, 6, 3, 6], dtype=torch.int32, device=DEV)
    # labels in the first, the last and a middle vector of the row
    batch["ids"][2, 0], batch["ids"][2, 1], batch["ids"][2, 2] = 0, V - 1, V // 2
    batch["actor"][2, 1, V - 1] = 3.0
    batch["actor"][2, 2, V // 2] = 2.0
    batch["actor"][2, 0, 0] = 1.0
    batch["ref"][2, :3] = batch["actor"][2, :3]
    run = OracleRun(oracle, w, batch)
    out, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], in_place=in_place, all_rows=True)
    if not in_place:
        dlogits_properties(run, out, batch["ids"], batch["actor"])


@pytest.mark.parametrize("V,in_place", [(32000, False), (50272, True), (4096, False)])
def test_rows_that_leave_the_common_reference_exponent(oracle, V, in_place):
    # The loss kernel sums a row against one reference exponent taken from the row's first 8 logits and falls back to
    # per-thread references when that does not hold.  Rows built to force every branch:
    # first 8 logits all -inf (no reference); first 8 logits far below the rest (entries > 2^64 above the
    # reference: spikes of +60..+90, at the label and elsewhere); first 8 logits far above the rest (everything else
    # more than 100 binades below the reference); -inf inside the first vector only.  V=4096 takes the chunk-ring kernel.
    w = inputs.scaled(inputs.WORKLOADS["llama2"], V=V, B=2, T=6, lengths="uniform:6:6", seed=90 + V % 11)
    batch = inputs.make_batch(w, device=DEV)
    a = batch["actor"]
    a[0, 0, :8] = float("-inf")
    a[0, 1, 1234] = 80.0                              # spike elsewhere
    a[0, 2, int(batch["ids"][0, 2])] = 90.0           # spike at the label
    a[0, 3, :8] = 70.0                                # reference far above the rest of the row
    a[0, 4, 1:5] = float("-inf")
    a[0, 5, :8] = -60.0                               # reference far below: every other entry is ~2^86 above it
    a[1, 0, V - 1] = 75.0
    a[1, 1, :16] = float("-inf")
    for b_, t_ in ((0, 0), (0, 4), (1, 1)):           # the label must not sit on a deleted entry
        if int(batch["ids"][b_, t_]) < 16:
            batch["ids"][b_, t_] = 100
    batch["ref"] = a.clone()
    run = OracleRun(oracle, w, batch)
    out, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], in_place=in_place, all_rows=True)
    if not in_place:
        dlogits_properties(run, out, batch["ids"], batch["actor"])


def test_gpt2_vocabulary_rows_off_16_byte_boundaries(oracle):
    # V = 50257: every row starts 2 bytes further off a 16-byte boundary than the one before it
    w = inputs.scaled(inputs.WORKLOADS["gpt2"], B=3, T=12, lengths="uniform:5:12")
    batch = inputs.make_batch(w, device=DEV)
    batch["ids"][0, 0], batch["ids"][0, 1], batch["ids"][1, 0] = 0, w.V - 1, 7       # labels in the ragged first/last vectors
    batch["actor"][0, 0, 0], batch["actor"][0, 1, w.V - 1], batch["actor"][1, 0, 7] = 4.0, 4.0, 4.0
    run = OracleRun(oracle, w, batch)
    out, _ = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)
    dlogits_properties(run, out, batch["ids"], batch["actor"])
    run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], in_place=True, all_rows=True)
    _experience_both_ways(w, batch, batch["actor"], batch["ref"], batch["ids"])
    # a view that starts in the middle of a row of a larger tensor: odd base address as well
    big = torch.zeros((3, 12, w.V + 5), dtype=torch.bfloat16, device=DEV)
    big[:, :, 3:3 + w.V] = batch["actor"]
    view = big[:, :, 3:3 + w.V]
    ws = binding.workspace(w.B, w.T, DEV)
    lp = binding.gather_logprobs(view, batch["ids"], batch["lengths"], ws)
    assert np.abs(np32(lp).astype(np.float64) - run.lp_actor).max() <= TOL_LP
    # the loss in place on that view: the 3 + 2 entries either side of every row must stay untouched
    big[:, :, :3] = 7.0
    big[:, :, 3 + w.V:] = -7.0
    run_steps(oracle, w, batch, run, view, batch["ref"], batch["ids"], all_rows=True)      # out of place, other layout
    t = lambda a: torch.as_tensor(a, device=DEV)
    outp = binding.PPOOutputs(view, in_place=True)
    binding.ppo_loss_fwd_bwd(view, batch["ids"], batch["lengths"], t(run.lp_old_in), t(run.adv_in), t(run.values_new_in),
                             t(run.values_old_in), t(run.ret_in), w.clip_eps, w.value_clip, run.grad_scale, ws, outp)
    assert binding.poll_status(ws) == 0
    assert (big[:, :, :3] == 7.0).all() and (big[:, :, 3 + w.V:] == -7.0).all()
    check_dlogits_rows(oracle, run, batch["actor"], batch["ids"], view, np.arange(w.B * w.T))


@pytest.mark.parametrize("V", [1000, 50272, 1001])
def test_device_detected_errors_are_flagged_not_faulted(oracle, V):
    # an id outside the vocabulary and lengths outside [0,T]: status flags, the offending token's outputs are 0,
    # everything else is computed as if the lengths had been clamped
    w = inputs.scaled(inputs.WORKLOADS["tiny"], V=V, B=3, T=8, lengths="full", seed=3)
    batch = inputs.make_batch(w, device=DEV)
    ws = binding.workspace(w.B, w.T, DEV)
    good = OracleRun(oracle, w, batch)
    bad_ids = batch["ids"].clone()
    bad_ids[1, 2] = V
    bad_ids[2, 5] = -1
    lp = binding.gather_logprobs(batch["actor"], bad_ids, batch["lengths"], ws)
    assert binding.poll_status(ws) == 16 and binding.poll_status(ws) == 0          # reported once, then cleared
    got = np32(lp).astype(np.float64)
    assert got[1, 2] == 0 and got[2, 5] == 0
    mask = np.ones((3, 8), bool); mask[1, 2] = mask[2, 5] = False
    assert np.abs(got - good.lp_actor)[mask].max() <= TOL_LP
    # lengths: 99 is clamped to T, -4 to 0
    bad_len = torch.tensor([99, -4, 8], dtype=torch.int32, device=DEV)
    lp = binding.gather_logprobs(batch["actor"], batch["ids"], bad_len, ws)
    assert binding.poll_status(ws) == 32
    got = np32(lp).astype(np.float64)
    assert np.abs(got[0] - good.lp_actor[0]).max() <= TOL_LP and (got[1] == 0).all()
    # both at once in the loss: flags are OR-ed; the bad token's gradient row is zero
    out = binding.PPOOutputs(batch["actor"])
    f = lambda a: torch.as_tensor(a, device=DEV)
    binding.ppo_loss_fwd_bwd(batch["actor"], bad_ids, bad_len, f(good.lp_old_in), f(good.adv_in), f(good.values_new_in),
                             f(good.values_old_in), f(good.ret_in), w.clip_eps, w.value_clip, 1.0, ws, out)
    assert binding.poll_status(ws) == (16 | 32)
    assert (out.dlogits[2, 5].view(torch.int16) == 0).all() and (out.dlogits[1].view(torch.int16) == 0).all()
    assert torch.isfinite(out.loss).all() and torch.isfinite(out.dlogits.float()).all()
