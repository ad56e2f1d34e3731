"""Seeded synthetic inputs for the token-level PPO path.

This module only draws random tensors with the shapes and value distributions of the workloads;
it holds none of the method's arithmetic (no softmax, no log-prob, no reward, no loss) and is
the one module that both the CUDA path and the CPU oracle's tests may import.

The workloads stand in for the paper's (Section 3, "Workload and Setting", and the additional
results in Appendix C): OPT and Llama-2 actors, whose vocabularies (50272 and 32000) fix V, with
batch sizes and sequence lengths of the order the paper's frameworks run.  No dataset or trained
weight is used: logits are Gaussian, so that what matters for the path -- the shape, the bf16
type, the spread of the softmax, the ragged response lengths -- is reproduced.

Token ids "sampled from the softmax" are drawn with the Gumbel-max construction,
argmax_v(z_v + G_v) with G_v standard Gumbel, which needs no normalisation.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    T: int
    V: int
    P: int = 0                       # prompt length (layout only)
    logit_sigma: float = 3.0
    ref_sigma: float = 0.1
    spike: float = 0.0               # added to one random token per row (peaked rows)
    ids: str = "uniform"             # "uniform" | "softmax"
    lengths: str = "full"            # "full" | "uniform:lo:hi" | "mixture"
    temp_rows: float = 0.0           # fraction of rows multiplied by 1/temperature
    temperature: float = 1.0
    neg_inf_rows: float = 0.0        # fraction of rows that carry -inf entries
    neg_inf_frac: float = 0.0        # fraction of entries set to -inf on those rows
    beta_kl: float = 0.1
    gamma: float = 1.0
    lam: float = 0.95
    clip_eps: float = 0.2
    value_clip: float = 0.2
    reward_clip: float = 5.0
    lp_old_sigma: float = 0.05
    value_new_sigma: float = 0.2
    seed: int = 0


# The five configurations: a tiny case, an OPT-shaped and a Llama-2-shaped batch, a large-vocabulary
# stress case and a ragged edge case.
WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", B=2, P=8, T=16, V=1000, lengths="uniform:8:16", seed=0),
    "opt": Workload("opt", B=16, P=256, T=256, V=50272, ids="softmax",
                    lengths="uniform:128:256", seed=1),
    "llama2": Workload("llama2", B=32, P=512, T=512, V=32000, spike=8.0, ids="softmax",
                       lengths="uniform:64:512", seed=2),
    "large_vocab": Workload("large_vocab", B=64, T=512, V=128256, logit_sigma=4.0, ref_sigma=0.2,
                            lengths="full", seed=3),
    # beyond the five configurations: the paper's second model family, GPT-2 (vocabulary 50257: rows are
    # 100,514 bytes long, so consecutive rows start 2 bytes further off a 16-byte boundary)
    "gpt2": Workload("gpt2", B=16, P=256, T=256, V=50257, ids="softmax", lengths="uniform:128:256", seed=5),
    "ragged": Workload("ragged", B=128, T=1024, V=50272, lengths="mixture", temp_rows=0.5,
                       temperature=0.3, neg_inf_rows=0.25, neg_inf_frac=0.01,
                       gamma=0.99, lam=1.0, seed=4),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (e.g. fewer sequences for a quick case)."""
    return replace(w, **kw)


def _gen(device, seed: int, name: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + zlib.crc32(name.encode())) % (2 ** 63 - 1))
    return g


def _draw_lengths(w: Workload, device) -> torch.Tensor:
    g = _gen("cpu", w.seed, "lengths")
    if w.lengths == "full":
        out = torch.full((w.B,), w.T, dtype=torch.int32)
    elif w.lengths.startswith("uniform:"):
        lo, hi = (int(x) for x in w.lengths.split(":")[1:])
        lo, hi = min(lo, w.T), min(hi, w.T)
        out = torch.randint(lo, hi + 1, (w.B,), generator=g, dtype=torch.int32)
    elif w.lengths == "mixture":
        # 0 (all pad) w.p. 0.05, 1 w.p. 0.15, 2 w.p. 0.15, uniform[3,T] w.p. 0.65
        u = torch.rand((w.B,), generator=g)
        long_len = torch.randint(min(3, w.T), w.T + 1, (w.B,), generator=g, dtype=torch.int32)
        out = long_len.clone()
        out[u < 0.35] = 2
        out[u < 0.20] = 1
        out[u < 0.05] = 0
        out = out.clamp(max=w.T)
        if w.B >= 4:                       # every kind of row is present whatever the draw
            out[0], out[1], out[2], out[3] = 0, 1, 2, w.T
    else:
        raise ValueError(w.lengths)
    return out.to(device)


def make_batch(w: Workload, device="cpu", with_prompt: bool = False,
               seq_chunk: Optional[int] = None) -> Dict[str, torch.Tensor]:
    """Draw one batch.  Returned tensors (all on `device`):

    actor, ref    bf16 [B,T,V], or [B,P+T,V] with `with_prompt` (then row P-1+t predicts response
                  token t, and `ids` is [B,P+T] with the response ids in columns P..P+T-1)
    ids           int64
    lengths       int32 [B] valid response length per sequence (trailing pad)
    values_old, values_new, lp_old_noise   fp32 [B,T]
    score         fp32 [B]

    `lp_old_noise` is the N(0, sigma^2) term that the caller adds to the current log-probs to make
    the old-policy log-probs; the log-probs themselves are not computed here.
    """
    dev = torch.device(device)
    B, T, V = w.B, w.T, w.V
    rows_per_seq = (w.P + T) if with_prompt else T
    first = (w.P - 1) if with_prompt else 0          # tensor row that predicts response token 0
    if with_prompt and w.P < 1:
        raise ValueError("with_prompt needs P >= 1")
    actor = torch.empty((B, rows_per_seq, V), dtype=torch.bfloat16, device=dev)
    ref = torch.empty_like(actor)
    ids_resp = torch.empty((B, T), dtype=torch.int64, device=dev)
    g_act, g_ref, g_ids, g_aux = (_gen(dev, w.seed, n) for n in ("actor", "ref", "ids", "aux"))
    chunk = seq_chunk or max(1, min(B, (1 << 26) // max(1, rows_per_seq * V)))
    for b0 in range(0, B, chunk):
        b1 = min(B, b0 + chunk)
        nb = b1 - b0
        z = torch.randn((nb, rows_per_seq, V), generator=g_act, device=dev) * w.logit_sigma
        if w.spike != 0.0:
            pos = torch.randint(0, V, (nb, rows_per_seq, 1), generator=g_aux, device=dev)
            z.scatter_add_(2, pos, torch.full_like(pos, w.spike, dtype=z.dtype))
        if w.temp_rows > 0.0:
            hot = torch.rand((nb, rows_per_seq, 1), generator=g_aux, device=dev) < w.temp_rows
            z = torch.where(hot, z / w.temperature, z)
        resp = z[:, first:first + T, :]
        if w.ids == "softmax":
            u = torch.rand(resp.shape, generator=g_ids, device=dev).clamp_(1e-12, 1.0 - 1e-7)
            y = (resp - torch.log(-torch.log(u))).argmax(dim=2)
            del u
        else:
            y = torch.randint(0, V, (nb, T), generator=g_ids, device=dev)
        ids_resp[b0:b1] = y
        if w.neg_inf_rows > 0.0:
            rows_hit = torch.rand((nb, rows_per_seq, 1), generator=g_aux, device=dev) < w.neg_inf_rows
            hit = (torch.rand(z.shape, generator=g_aux, device=dev) < w.neg_inf_frac) & rows_hit
            keep = torch.zeros_like(hit[:, first:first + T, :])
            keep.scatter_(2, y.unsqueeze(2), True)
            hit[:, first:first + T, :] &= ~keep           # never delete the generated token
            z = z.masked_fill(hit, float("-inf"))
            del hit, keep
        a16 = z.to(torch.bfloat16)
        actor[b0:b1] = a16
        noise = torch.randn(z.shape, generator=g_ref, device=dev) * w.ref_sigma
        ref[b0:b1] = (a16.float() + noise).to(torch.bfloat16)      # -inf stays -inf
        del z, noise, a16
    if with_prompt:
        g_p = _gen(dev, w.seed, "prompt_ids")
        ids = torch.randint(0, V, (B, w.P + T), generator=g_p, device=dev)
        ids[:, w.P:] = ids_resp
    else:
        ids = ids_resp
    g_s = _gen(dev, w.seed, "small")
    values_old = torch.randn((B, T), generator=g_s, device=dev)
    values_new = values_old + w.value_new_sigma * torch.randn((B, T), generator=g_s, device=dev)
    score = torch.randn((B,), generator=g_s, device=dev)
    lp_old_noise = w.lp_old_sigma * torch.randn((B, T), generator=g_s, device=dev)
    return {
        "actor": actor, "ref": ref, "ids": ids, "lengths": _draw_lengths(w, dev),
        "values_old": values_old, "values_new": values_new, "score": score,
        "lp_old_noise": lp_old_noise,
    }


def response_view(w: Workload, full: torch.Tensor) -> torch.Tensor:
    """The [B,T,...] view of a [B,P+T,...] tensor made with `with_prompt`: logits rows P-1..P+T-2
    (the rows that predict the response tokens)."""
    return full[:, w.P - 1:w.P - 1 + w.T]


def bf16_bits(x: torch.Tensor):
    """numpy uint16 view (bit patterns) of a CPU bf16 tensor, strides preserved."""
    import numpy as np
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.view(torch.int16).numpy().view(np.uint16)
