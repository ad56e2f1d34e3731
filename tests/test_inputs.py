"""The seeded input generator: shapes, types, determinism and the structure each workload asks for."""
import torch

from paper_2410_15651_b200 import inputs


def _small(name, **kw):
    base = dict(B=6, T=24, V=512)
    base.update(kw)
    return inputs.scaled(inputs.WORKLOADS[name], **base)


def test_shapes_types_and_determinism():
    w = inputs.WORKLOADS["tiny"]
    a = inputs.make_batch(w)
    b = inputs.make_batch(w)
    assert a["actor"].shape == (2, 16, 1000) and a["actor"].dtype == torch.bfloat16
    assert a["ids"].dtype == torch.int64 and a["lengths"].dtype == torch.int32
    for k in a:
        assert torch.equal(a[k], b[k]), k
    assert ((a["lengths"] >= 8) & (a["lengths"] <= 16)).all()
    c = inputs.make_batch(inputs.scaled(w, seed=7))
    assert not torch.equal(a["actor"], c["actor"])
    # reference logits are the actor's plus small noise
    d = (a["ref"].float() - a["actor"].float()).abs()
    assert 0 < d.mean() < 0.3


def test_prompt_layout():
    w = inputs.WORKLOADS["tiny"]
    full = inputs.make_batch(w, with_prompt=True)
    assert full["actor"].shape == (2, 24, 1000) and full["ids"].shape == (2, 24)
    view = inputs.response_view(w, full["actor"])
    assert view.shape == (2, 16, 1000)
    assert view.data_ptr() == full["actor"].data_ptr() + (w.P - 1) * w.V * 2


def test_softmax_ids_prefer_large_logits():
    w = _small("llama2", P=0)
    b = inputs.make_batch(w)
    z = b["actor"].float()
    picked = z.gather(2, b["ids"][..., None])[..., 0]
    # sampled tokens sit far above the row mean; with a +8 spike most rows pick a top logit
    assert (picked > z.mean(-1) + 3.0).float().mean() > 0.9
    assert (z.max(-1).values > 8.0).float().mean() > 0.9


def test_ragged_workload_structure():
    w = _small("ragged", B=40, T=32)
    b = inputs.make_batch(w)
    L = b["lengths"]
    assert L[0] == 0 and L[1] == 1 and L[2] == 2 and L[3] == w.T
    assert ((L >= 0) & (L <= w.T)).all()
    z = b["actor"].float()
    ninf = torch.isinf(z) & (z < 0)
    assert ninf.any() and not torch.isnan(z).any()
    assert not ninf.gather(2, b["ids"][..., None]).any()          # never at the generated token
    assert torch.equal(torch.isinf(b["ref"].float()), ninf)       # deleted entries stay deleted
    assert not ninf.all(-1).any()                                 # no row loses every entry
    finite = torch.where(ninf, torch.zeros_like(z), z)
    spread = finite.std(-1)
    assert (spread > 7).any() and (spread < 5).any()              # some rows sharpened by 1/0.3
