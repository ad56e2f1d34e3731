"""Shared test plumbing: runs the CPU oracle over a synthetic batch and compares the CUDA path
with it under the stated tolerances.

Tolerances (fp32 arithmetic on the GPU against float64 on the CPU):
  log-probs                      |d| <= 1e-4
  rewards, advantages, returns,
  dvalues, losses                |d| <= 1e-4 * max(1, |x|)
  dlogits (bf16 / fp16)          |d| <= ulp(x) + 1e-6, ulp the spacing of the output type at x
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2410_15651_b200 import inputs

TOL_LP = 1e-4
TOL_REL = 1e-4


def bits(x: torch.Tensor) -> np.ndarray:
    """What the oracle takes for a 16-bit logits tensor (copied to the CPU if needed, strides preserved): uint16 bit
    patterns for bf16, a numpy float16 array for fp16."""
    x = x.cpu() if x.is_cuda else x
    if x.dtype == torch.float16:
        return x.numpy()
    return inputs.bf16_bits(x)


def np32(x: torch.Tensor) -> np.ndarray:
    return x.detach().cpu().numpy()


def close_rel(got, want, tol=TOL_REL):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    lim = tol * np.maximum(1.0, np.abs(want))
    return bool((err <= lim).all()), float((err / lim).max(initial=0.0))


def oracle_gather_chunked(oracle, logits: torch.Tensor, ids: torch.Tensor, lengths: np.ndarray,
                          seq_chunk: int = 4) -> np.ndarray:
    """Step 1 of the oracle over a (possibly device-resident, possibly strided) logits view,
    copying a few sequences at a time to the host."""
    B, T, _ = logits.shape
    out = np.zeros((B, T), dtype=np.float64)
    ids_np = ids.cpu().numpy()
    for b0 in range(0, B, seq_chunk):
        b1 = min(B, b0 + seq_chunk)
        out[b0:b1] = oracle.gather_logprobs(bits(logits[b0:b1]), ids_np[b0:b1], lengths[b0:b1])
    return out


class OracleRun:
    """Every step of the path on the CPU, each step fed with float32-rounded outputs of the step
    before it -- the same float32 arrays the CUDA functions are given, so each step is compared
    on identical inputs."""

    def __init__(self, oracle, w: inputs.Workload, batch: dict, logits_view=None, ref_view=None,
                 ids_view=None, on_policy: bool = False, score_override=None, grad_scale=None):
        f32 = lambda a: np.asarray(a, dtype=np.float32)
        self.w = w
        actor = batch["actor"] if logits_view is None else logits_view
        ref = batch["ref"] if ref_view is None else ref_view
        ids = batch["ids"] if ids_view is None else ids_view
        self.lengths = batch["lengths"].cpu().numpy().astype(np.int32)
        self.N = int(self.lengths.sum())
        self.lp_actor = oracle_gather_chunked(oracle, actor, ids, self.lengths)
        self.lp_ref = oracle_gather_chunked(oracle, ref, ids, self.lengths)
        noise = np32(batch["lp_old_noise"]).astype(np.float64)
        valid = np.arange(w.T)[None, :] < self.lengths[:, None]
        self.valid = valid
        self.lp_old_in = f32(np.where(valid, self.lp_actor + (0.0 if on_policy else 1.0) * noise, 0.0))
        self.lp_ref_in = f32(self.lp_ref)
        self.score_in = f32(np32(batch["score"]) if score_override is None else score_override)
        self.rewards = oracle.kl_reward(self.lp_old_in, self.lp_ref_in, self.score_in, self.lengths,
                                        w.beta_kl, w.reward_clip)
        self.rewards_in = f32(self.rewards)
        self.values_old_in = np32(batch["values_old"])
        self.values_new_in = np32(batch["values_new"])
        self.adv, self.ret = oracle.gae(self.rewards_in, self.values_old_in, self.lengths, w.gamma, w.lam)
        self.adv_in, self.ret_in = f32(self.adv), f32(self.ret)
        self.grad_scale = float(self.N if grad_scale is None else grad_scale)
        self.ppo = oracle.ppo_loss_from_logprobs(
            self.lp_actor, self.lp_old_in, self.adv_in, self.values_new_in, self.values_old_in,
            self.ret_in, self.lengths, w.clip_eps, w.value_clip, self.grad_scale)
        # tokens whose clip decision sits on a kink: either branch is a correct float32 answer
        rho = np.exp(self.lp_actor - self.lp_old_in)
        self.pg_kink = valid & ((np.abs(rho - (1 - w.clip_eps)) < 2e-4) | (np.abs(rho - (1 + w.clip_eps)) < 2e-4))
        v, vo, G = (self.values_new_in.astype(np.float64), self.values_old_in.astype(np.float64),
                    self.ret_in.astype(np.float64))
        vc = vo + np.clip(v - vo, -w.value_clip, w.value_clip)
        e1, e2 = (v - G) ** 2, (vc - G) ** 2
        self.vf_kink = valid & (np.abs(e1 - e2) < 1e-4 * np.maximum(1.0, e1)) & (e1 != e2)


def check_dlogits_rows(oracle, run: OracleRun, logits: torch.Tensor, ids: torch.Tensor,
                       dlogits: torch.Tensor, rows: np.ndarray, chunk: int = 64):
    """Compare the listed rows (flat b*T+t) of the CUDA dlogits with the oracle, element by element.
    Returns (worst error / tolerance, number of rows compared)."""
    B, T, V = logits.shape
    worst, n = 0.0, 0
    ids_np = ids.cpu().numpy()
    rows = np.asarray(rows, dtype=np.int64)
    rows = rows[~run.pg_kink.reshape(-1)[rows]]
    for i in range(0, rows.size, chunk):
        rr = rows[i:i + chunk]
        bsel = torch.as_tensor(rr // T, device=logits.device)
        tsel = torch.as_tensor(rr % T, device=logits.device)
        z = logits[bsel, tsel][:, None, :]                                  # [n,1,V]
        sub_ids = ids_np[rr // T, rr % T][:, None]
        sub_len = (run.valid.reshape(-1)[rr]).astype(np.int32)
        sub_g = run.ppo.g.reshape(-1)[rr][:, None]
        want = oracle.dlogits_rows(bits(z), np.ascontiguousarray(sub_ids), sub_len, sub_g,
                                   np.arange(rr.size))
        got = dlogits[bsel, tsel].float().cpu().numpy().astype(np.float64)
        lim = (oracle.f16_ulp(want) if dlogits.dtype == torch.float16 else oracle.bf16_ulp(want)) + 1e-6
        err = np.abs(got - want)
        assert np.isfinite(got).all()
        ratio = float((err / lim).max(initial=0.0))
        if ratio > 1.0:
            k = np.unravel_index(np.argmax(err / lim), err.shape)
            raise AssertionError(f"dlogits row {rr[k[0]]} v={k[1]}: got {got[k]!r} want {want[k]!r} "
                                 f"(err/tol = {ratio:.3f}, g = {sub_g[k[0], 0]!r})")
        worst = max(worst, ratio)
        n += rr.size
        # rows the oracle says are all zero must be exact (+0) zeros
        zero_rows = (sub_len == 0) | (sub_g[:, 0] == 0)
        if zero_rows.any():
            raw = dlogits[bsel, tsel].view(torch.int16).cpu().numpy()
            assert (raw[zero_rows] == 0).all()
    return worst, n
