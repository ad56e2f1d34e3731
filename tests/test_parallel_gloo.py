"""The data-parallel host logic on two gloo ranks (CPU): sharding by sequence, the global token
normaliser passed through grad_scale, and the combination of the per-rank losses.  The arithmetic
of each shard is done by the CPU oracle, so the test states what the multi-GPU run must reproduce:
per-shard calls with the adjusted grad_scale give exactly the gradients of the whole-batch call."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case():
    rng = np.random.default_rng(11)
    B, T, V = 5, 9, 33
    z = rng.normal(0, 2, (B, T, V))
    ids = rng.integers(0, V, (B, T)).astype(np.int64)
    lengths = np.array([9, 4, 0, 7, 1], dtype=np.int32)
    arrs = [rng.normal(0, 1, (B, T)) for _ in range(5)]       # lp_old offset, adv, v_new, v_old, ret
    return z, ids, lengths, arrs


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2410_15651_b200 import parallel
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        z, ids, lengths, arrs = _case()
        lp = oracle.gather_logprobs(z, ids, lengths)
        lp_old = lp + 0.2 * arrs[0]
        b0, b1 = parallel.shard_range(len(lengths), world, rank)
        sl = slice(b0, b1)
        n_local, n_global = parallel.token_counts(torch.as_tensor(lengths[sl]))
        assert n_global == int(lengths.sum()) and n_local == int(lengths[sl].sum())
        upstream = 3.0
        gs = parallel.grad_scale_for_global_mean(n_local, n_global, upstream)
        loc = oracle.ppo_loss(z[sl], ids[sl], lengths[sl], lp_old[sl], arrs[1][sl], arrs[2][sl], arrs[3][sl],
                              arrs[4][sl], 0.2, 0.2, gs)
        glob = oracle.ppo_loss(z, ids, lengths, lp_old, arrs[1], arrs[2], arrs[3], arrs[4], 0.2, 0.2, upstream)
        # per-rank gradients with the adjusted grad_scale are the whole-batch gradients of the rank's sequences
        assert np.allclose(loc.g, glob.g[sl], rtol=0, atol=1e-15)
        assert np.allclose(loc.dvalues, glob.dvalues[sl], rtol=0, atol=1e-15)
        both = parallel.combine_losses(torch.tensor([loc.loss_pg, loc.loss_vf], dtype=torch.float64), n_local, n_global)
        assert abs(both[0].item() - glob.loss_pg) < 1e-13 and abs(both[1].item() - glob.loss_vf) < 1e-13
        # timing helpers: max and sum over ranks
        assert parallel.max_over_ranks(10.0 + rank) == 10.0 + world - 1
        assert parallel.sum_over_ranks(float(n_local)) == float(n_global)
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_rank_data_parallel_losses(tmp_path, oracle):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(world))


def test_shard_range_covers_everything():
    from paper_2410_15651_b200 import parallel
    for n in (0, 1, 5, 16, 17):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
