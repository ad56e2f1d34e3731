"""Branches of the CUDA path that the step-by-step parity tests do not reach: optional outputs left
out, run-to-run bit identity on the shapes that take each loss kernel, aliasing that the header
allows, the documented behaviour of an out-of-range token id, the whitening step, the bounded wait
that runs out, and a batch cut into shards as a data-parallel job would cut it.
"""
import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs, parallel

from helpers import OracleRun, check_dlogits_rows, close_rel, np32
from test_parity_gpu import DEV, _t

pytestmark = pytest.mark.gpu


def _loss_inputs(run):
    return [_t(a) for a in (run.lp_old_in, run.adv_in, run.values_new_in, run.values_old_in, run.ret_in)]


def _call_loss(w, batch, run, logits, out, ws, grad_scale=None, lengths=None, ids=None, extra=None):
    lp_old, adv, vn, vo, ret = extra if extra is not None else _loss_inputs(run)
    binding.ppo_loss_fwd_bwd(logits, batch["ids"] if ids is None else ids,
                             batch["lengths"] if lengths is None else lengths, lp_old, adv, vn, vo, ret,
                             w.clip_eps, w.value_clip, run.grad_scale if grad_scale is None else grad_scale, ws, out)
    assert binding.poll_status(ws) == 0
    return out


@pytest.mark.parametrize("name,kw", [("tiny", {}),                                   # short rows: chunk-ring kernel
                                     ("tiny", {"V": 1001}),                          # odd rows: generic kernel + separate finalisation
                                     ("llama2", {"B": 2, "T": 24}),                  # exponentials in registers
                                     ("opt", {"B": 2, "T": 24}),                     # registers + tensor memory
                                     ("gpt2", {"B": 2, "T": 12}),                    # rows off 16-byte boundaries
                                     ("large_vocab", {"B": 1, "T": 12}),             # two blocks, chunk ring
                                     ("ragged", {"B": 1, "T": 12, "V": 150000})])    # cluster of three blocks
def test_lp_new_is_optional(oracle, name, kw):
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    ws = binding.workspace(w.B, w.T, DEV)
    full = _call_loss(w, batch, run, batch["actor"], binding.PPOOutputs(batch["actor"]), ws)
    bare = binding.PPOOutputs(batch["actor"], want_lp_new=False)
    assert bare.lp_new is None
    for t_ in (bare.loss, bare.dvalues):
        t_.fill_(float("nan"))
    bare.dlogits.fill_(float("nan"))
    _call_loss(w, batch, run, batch["actor"], bare, ws)
    assert torch.equal(bare.loss, full.loss) and torch.equal(bare.dvalues, full.dvalues)
    assert torch.equal(bare.dlogits.view(torch.int16), full.dlogits.view(torch.int16))
    ok, _ = close_rel(np32(bare.loss)[0], run.ppo.loss_pg)
    assert ok


@pytest.mark.parametrize("name,kw", [("opt", {}),                                    # rows dealt dynamically, 148 blocks
                                     ("llama2", {"B": 8}),
                                     ("ragged", {"B": 6, "T": 64, "V": 57000}),      # 114 KB rows: one block, chunk ring
                                     ("ragged", {"B": 6, "T": 64, "V": 131072}),     # 256 KB rows: two blocks, chunk ring
                                     ("ragged", {"B": 6, "T": 64, "V": 150000}),     # 300 KB rows: cluster of three, whole-slice buffers
                                     ("gpt2", {"B": 4, "T": 64}),                    # rows off 16-byte boundaries
                                     ("ragged", {"B": 12, "T": 40, "V": 4096})])     # chunk-ring kernel
def test_two_runs_are_bit_identical(name, kw):
    # fixed-order reductions, no floating-point atomics: whatever block takes whatever row, and whichever block
    # finishes last, the same bits come out
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = inputs.make_batch(w, device=DEV)
    ws = binding.workspace(w.B, w.T, DEV)
    g = torch.Generator(device=DEV).manual_seed(3)
    f = lambda: torch.randn((w.B, w.T), generator=g, device=DEV)
    lp_old = binding.gather_logprobs(batch["actor"], batch["ids"], batch["lengths"], ws) + 0.05 * f()
    adv, ret = f(), f()
    N = float(batch["lengths"].sum())
    outs = []
    for rep in range(3):
        out = binding.PPOOutputs(batch["actor"])
        out.dlogits.fill_(float("nan"))
        binding.ppo_loss_fwd_bwd(batch["actor"], batch["ids"], batch["lengths"], lp_old, adv, batch["values_new"],
                                 batch["values_old"], ret, w.clip_eps, w.value_clip, N, ws, out)
        assert binding.poll_status(ws) == 0
        outs.append(out)
        if rep == 0:
            # perturb the timing of the next run: something else keeps some SMs busy while it starts
            torch.randn((4096, 4096), device=DEV) @ torch.randn((4096, 4096), device=DEV)
    for o in outs[1:]:
        assert torch.equal(o.loss, outs[0].loss)
        assert torch.equal(o.dvalues, outs[0].dvalues) and torch.equal(o.lp_new, outs[0].lp_new)
        assert torch.equal(o.dlogits.view(torch.int16), outs[0].dlogits.view(torch.int16))
    assert torch.isfinite(outs[0].loss).all()


def test_kl_reward_may_overwrite_an_input(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device=DEV)
    g = torch.Generator(device=DEV).manual_seed(1)
    lp_old = torch.randn((w.B, w.T), generator=g, device=DEV) - 4
    lp_ref = torch.randn((w.B, w.T), generator=g, device=DEV) - 4
    want = binding.kl_reward(lp_old, lp_ref, batch["score"], batch["lengths"], w.beta_kl, w.reward_clip)
    a = lp_old.clone()
    binding.kl_reward(a, lp_ref, batch["score"], batch["lengths"], w.beta_kl, w.reward_clip, out=a)
    b = lp_ref.clone()
    binding.kl_reward(lp_old, b, batch["score"], batch["lengths"], w.beta_kl, w.reward_clip, out=b)
    assert torch.equal(a, want) and torch.equal(b, want)
    ref = oracle.kl_reward(np32(lp_old), np32(lp_ref), np32(batch["score"]), batch["lengths"].cpu().numpy(),
                           w.beta_kl, w.reward_clip)
    assert close_rel(np32(want), ref)[0]


@pytest.mark.parametrize("V", [1000, 32000, 50272])
def test_out_of_range_id_drops_the_policy_term_only(oracle, V):
    # the token still counts in N, and its value-loss term and dvalues entry are those of a valid token
    w = inputs.scaled(inputs.WORKLOADS["tiny"], V=V, B=3, T=8, lengths="full", seed=3)
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch, grad_scale=1.0)
    ws = binding.workspace(w.B, w.T, DEV)
    good = _call_loss(w, batch, run, batch["actor"], binding.PPOOutputs(batch["actor"]), ws)
    bad_ids = batch["ids"].clone()
    bad_ids[1, 2] = V
    out = binding.PPOOutputs(batch["actor"])
    lp_old, adv, vn, vo, ret = _loss_inputs(run)
    binding.ppo_loss_fwd_bwd(batch["actor"], bad_ids, batch["lengths"], lp_old, adv, vn, vo, ret, w.clip_eps,
                             w.value_clip, 1.0, ws, out)
    assert binding.poll_status(ws) == 16
    assert torch.equal(out.dvalues, good.dvalues)                       # value path untouched
    assert torch.equal(out.loss[1], good.loss[1])
    assert (out.dlogits[1, 2].view(torch.int16) == 0).all() and out.lp_new[1, 2] == 0
    keep = torch.ones((3, 8), dtype=torch.bool, device=DEV)
    keep[1, 2] = False
    assert torch.equal(out.dlogits[keep].view(torch.int16), good.dlogits[keep].view(torch.int16))   # N unchanged: same 1/N
    # the policy loss lost exactly that token's term
    o = run.ppo
    rho = np.exp(o.lp_new[1, 2] - run.lp_old_in[1, 2])
    term = max(-run.adv_in[1, 2] * rho, -run.adv_in[1, 2] * min(max(rho, 1 - w.clip_eps), 1 + w.clip_eps))
    assert close_rel(float(out.loss[0]), o.loss_pg - term / run.N)[0]


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("ragged", {"B": 12, "T": 40, "V": 64}), ("opt", {"V": 64}),
                                     ("ragged", {"V": 64})])
def test_whitening_against_the_oracle(oracle, name, kw):
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = inputs.make_batch(w, device=DEV)
    ln = batch["lengths"].cpu().numpy()
    g = torch.Generator(device=DEV).manual_seed(7)
    adv = torch.randn((w.B, w.T), generator=g, device=DEV) * 3 + 2
    adv[torch.arange(w.T, device=DEV)[None, :] >= batch["lengths"][:, None]] = 1e9       # padded inputs are ignored
    ws = binding.workspace(w.B, w.T, DEV)
    for eps in (1e-8, 0.5):
        want = oracle.whiten(np32(adv), ln, eps)
        got = binding.whiten_advantages(adv, batch["lengths"], eps, ws)
        ok, ratio = close_rel(np32(got), want)
        assert ok, ratio
        again = binding.whiten_advantages(adv, batch["lengths"], eps, ws)
        assert torch.equal(got, again)                                   # fixed-order sums
    inplace = adv.clone()
    binding.whiten_advantages(inplace, batch["lengths"], 1e-8, ws, out=inplace)
    assert torch.equal(inplace, binding.whiten_advantages(adv, batch["lengths"], 1e-8, ws))
    # the workspace is left ready for the loss call (its ticket word is back to zero)
    run = OracleRun(oracle, w, batch)
    _call_loss(w, batch, run, batch["actor"], binding.PPOOutputs(batch["actor"]), ws)


def test_whitening_degenerate_batches():
    lengths = torch.tensor([0, 1, 0], dtype=torch.int32, device=DEV)
    adv = torch.tensor([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]], device=DEV)
    ws = binding.workspace(3, 2, DEV)
    assert (binding.whiten_advantages(adv, lengths, 1e-8, ws) == 0).all()          # one valid token: variance 0
    assert (binding.whiten_advantages(adv, lengths, 0.0, ws) == 0).all()
    none = torch.zeros(3, dtype=torch.int32, device=DEV)
    assert (binding.whiten_advantages(adv, none, 1e-8, ws) == 0).all()
    two = torch.tensor([2, 0, 0], dtype=torch.int32, device=DEV)
    got = binding.whiten_advantages(adv, two, 3.0, ws)                             # values 1, 2: mean 1.5, var 0.25
    assert torch.allclose(got[0], torch.tensor([-0.5, 0.5], device=DEV) / (3.25 ** 0.5), atol=1e-6)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_library_usable(oracle):
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    ws = binding.workspace(w.B, w.T, DEV)
    binding.selftest_bounded_wait(ws, 1_000_000)                      # 1 ms: nothing ever arrives at the barrier
    torch.cuda.synchronize()                                          # the call returned and the kernel ended
    assert binding.poll_status(ws) == 64
    assert binding.status_string(64) == "RLHF_ERR_TIMEOUT"
    assert binding.poll_status(ws) == 0                               # reported once
    # the next ordinary calls on the same workspace are clean and correct
    out = _call_loss(w, batch, run, batch["actor"], binding.PPOOutputs(batch["actor"]), ws)
    assert close_rel(np32(out.loss)[0], run.ppo.loss_pg)[0]
    lp = binding.gather_logprobs(batch["actor"], batch["ids"], batch["lengths"], ws)
    assert np.abs(np32(lp) - run.lp_actor).max() <= 1e-4 and binding.poll_status(ws) == 0


@pytest.mark.parametrize("name,kw,shards", [("opt", {"B": 8}, 2), ("tiny", {"B": 5, "lengths": "uniform:0:16"}, 3)])
def test_sequence_shards_reproduce_the_whole_batch(oracle, name, kw, shards):
    # data parallel over sequences: every shard calls the loss with grad_scale * N_local / N_global; its gradient
    # rows are then the whole-batch call's rows, and the token-weighted mean of the shard losses is the batch loss
    w = inputs.scaled(inputs.WORKLOADS[name], **kw)
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    ws = binding.workspace(w.B, w.T, DEV)
    whole = _call_loss(w, batch, run, batch["actor"], binding.PPOOutputs(batch["actor"]), ws)
    lp_old, adv, vn, vo, ret = _loss_inputs(run)
    n_global = run.N
    acc = torch.zeros(2, dtype=torch.float64)
    for r in range(shards):
        b0, b1 = parallel.shard_range(w.B, shards, r)
        if b1 == b0:
            continue
        sl = slice(b0, b1)
        lengths = batch["lengths"][sl].contiguous()
        n_local, _ = parallel.token_counts(lengths)
        gs = parallel.grad_scale_for_global_mean(n_local, n_global, upstream=run.grad_scale)
        logits = batch["actor"][sl]
        out = binding.PPOOutputs(logits)
        binding.ppo_loss_fwd_bwd(logits, batch["ids"][sl], lengths, lp_old[sl].contiguous(), adv[sl].contiguous(),
                                 vn[sl].contiguous(), vo[sl].contiguous(), ret[sl].contiguous(), w.clip_eps,
                                 w.value_clip, gs, ws, out)
        assert binding.poll_status(ws) == 0
        acc += out.loss.double().cpu() * n_local
        if n_local == 0:
            assert (out.dlogits.view(torch.int16) == 0).all()
            continue
        # gradients: grad_scale * N_local / N_global / N_local differs from grad_scale / N_global by float32 rounding
        # only, which moves a bf16 value by at most one step
        d_sh, d_wh = out.dlogits.float(), whole.dlogits[sl].float()
        step = torch.maximum(d_wh.abs(), torch.tensor(1e-30, device=DEV)) * 2.0 ** -7
        assert ((d_sh - d_wh).abs() <= step + 1e-30).all()
        assert torch.allclose(out.dvalues, whole.dvalues[sl], rtol=1e-6, atol=1e-12)
        rows = np.arange((b1 - b0) * w.T)
        sub = OracleRun.__new__(OracleRun)
        sub.valid = run.valid[sl]
        sub.pg_kink = run.pg_kink[sl]
        sub.ppo = type(run.ppo)(0.0, 0.0, run.ppo.lp_new[sl], run.ppo.g[sl], run.ppo.dvalues[sl])
        check_dlogits_rows(oracle, sub, logits, batch["ids"][sl], out.dlogits, rows)      # and against the oracle
    total = acc / n_global
    assert close_rel(total[0].item(), run.ppo.loss_pg)[0] and close_rel(total[1].item(), run.ppo.loss_vf)[0]
    assert close_rel(total[0].item(), float(whole.loss[0]))[0]


@pytest.mark.parametrize("V", [8192, 8200, 16384, 32768, 32776, 45056, 53248, 57344, 65536, 65544, 98304, 106496, 106504, 114688,
                               131072, 131080, 150000, 163840, 212992, 213000, 262144, 262152])
def test_vocabulary_sizes_around_the_kernel_boundaries(oracle, V):
    # 16 KB rows (the first size of the on-chip-exponentials kernel), rows that fill a thread's register-held vectors
    # exactly and by one more vector (tensor memory), the last size one block holds twice in whole-row buffers (53248)
    # and the sizes that one block takes through the chunk ring (57344, 65536: eight full chunks), the first that needs
    # a cluster of two with whole-slice buffers (65544), the last of those (106496 = 208 KB) and the sizes that two
    # blocks take through the chunk ring (106504 ... 131072), clusters of three (131080, 150000) and four (163840,
    # 212992: the last size whole-slice buffers hold), the chunk ring in a cluster of four beyond that (213000, 262144:
    # 512 KB, eight full chunks per block), and rows beyond everything (262152), which the plain chunk ring streams twice
    from test_parity_gpu import run_steps
    w = inputs.scaled(inputs.WORKLOADS["ragged"], V=V, B=3, T=5, seed=200 + V % 13)
    batch = inputs.make_batch(w, device=DEV)
    batch["lengths"] = torch.tensor([5, 0, 3], dtype=torch.int32, device=DEV)
    batch["ids"][0, 0], batch["ids"][0, 1] = 0, V - 1               # labels in the first and the last vector
    batch["actor"][0, 0, 0], batch["actor"][0, 1, V - 1] = 2.0, 3.0
    batch["ref"][0, :2] = batch["actor"][0, :2]
    run = OracleRun(oracle, w, batch)
    run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"], all_rows=True)


@pytest.mark.parametrize("V", [32000, 50272, 128256])
def test_all_padding_and_prompt_views_on_the_main_loss_kernel(oracle, V):
    from test_parity_gpu import run_steps
    # no valid token at all: every row is zero-filled, both losses are 0
    w0 = inputs.scaled(inputs.WORKLOADS["llama2"], V=V, B=2, T=4, P=3, lengths="uniform:0:0")
    b0 = inputs.make_batch(w0, device=DEV)
    run0 = OracleRun(oracle, w0, b0)
    out, _ = run_steps(oracle, w0, b0, run0, b0["actor"], b0["ref"], b0["ids"], all_rows=True)
    assert (out.loss == 0).all() and (out.dlogits.view(torch.int16) == 0).all() and (out.dvalues == 0).all()
    # the response rows as a strided view of a [B,P+T,V] tensor, out of place and in place on the view itself
    w = inputs.scaled(inputs.WORKLOADS["llama2"], V=V, B=2, T=4, P=3, lengths="uniform:2:4")
    full = inputs.make_batch(w, device=DEV, with_prompt=True)
    logits, ref, ids = inputs.response_view(w, full["actor"]), inputs.response_view(w, full["ref"]), full["ids"][:, w.P:]
    assert not logits.is_contiguous()
    run = OracleRun(oracle, w, full, logits_view=logits, ref_view=ref, ids_view=ids)
    run_steps(oracle, w, full, run, logits, ref, ids, all_rows=True)
    full2 = full["actor"].clone()
    view2 = inputs.response_view(w, full2)
    ws = binding.workspace(w.B, w.T, DEV)
    out2 = binding.PPOOutputs(view2, in_place=True)
    lp_old, adv, vn, vo, ret = _loss_inputs(run)
    binding.ppo_loss_fwd_bwd(view2, ids, full["lengths"], lp_old, adv, vn, vo, ret, w.clip_eps, w.value_clip,
                             run.grad_scale, ws, out2)
    assert binding.poll_status(ws) == 0
    assert torch.equal(full2[:, :w.P - 1], full["actor"][:, :w.P - 1])            # the prompt rows around it are untouched
    assert torch.equal(full2[:, w.P - 1 + w.T:], full["actor"][:, w.P - 1 + w.T:])
    check_dlogits_rows(oracle, run, logits, ids, view2, np.arange(w.B * w.T))
