"""CUDA path against the CPU oracle at the full sizes of the OPT-shaped, Llama-2-shaped,
large-vocabulary, ragged and GPT-2-shaped (rows off 16-byte boundaries) workloads, in the launch
configuration the benchmark times.

Every O(B*T) output (log-probs of all rows for actor and reference, rewards, advantages, returns,
dvalues, both losses) is compared in full: the oracle computes all of them.  The bf16 logits
gradient is compared element by element on every row for the OPT-, Llama-2- and GPT-2-shaped workloads
(out of place), and for the others on a sample of rows (some 600 for the ragged workload; valid,
padded, zero-gradient, first and last, and for the large-vocabulary workload, whose rows are dealt statically to 74 clusters of two
blocks with a ring of 13 chunk slots each (a slice takes 8, so a cluster's i-th row starts at slot
8i mod 13), the first 1024 valid rows, which cover every block at every ring offset and both
phases of every slot's barriers, and the last 148, the end of every cluster's work); every row is
also checked through properties that need no oracle row.
"""
import numpy as np
import pytest
import torch

from paper_2410_15651_b200 import binding, inputs

from helpers import OracleRun
from test_parity_gpu import DEV, _experience_both_ways, dlogits_properties, run_steps, sample_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,in_place", [("opt", False), ("opt", True), ("llama2", False),
                                           ("large_vocab", False), ("ragged", False), ("gpt2", False), ("gpt2", True)])
def test_full_size(oracle, name, in_place):
    w = inputs.WORKLOADS[name]
    batch = inputs.make_batch(w, device=DEV)
    run = OracleRun(oracle, w, batch)
    rows = sample_rows(run, 48, seed=w.seed)
    if name == "large_vocab":
        flat_valid = np.flatnonzero(run.valid.reshape(-1))
        rows = np.unique(np.concatenate([rows, flat_valid[:1024], flat_valid[-148:]]))
    if name == "ragged":
        rows = np.unique(np.concatenate([rows, sample_rows(run, 600, seed=w.seed + 1)]))
    every_row = name in ("opt", "llama2", "gpt2") and not in_place
    out, rep = run_steps(oracle, w, batch, run, batch["actor"], batch["ref"], batch["ids"],
                         in_place=in_place, sample_rows=rows, all_rows=every_row)
    dlogits_properties(run, out, batch["ids"], batch["actor"])
    if not in_place:
        _experience_both_ways(w, batch, batch["actor"], batch["ref"], batch["ids"])
    print(name, {k: (round(v, 4) if isinstance(v, float) else v) for k, v in rep.items()})
    del batch, out
    torch.cuda.empty_cache()
