"""Writes the stored expected values under tests/golden/.  Calls only the CPU oracle (and the
seeded input generator); never the CUDA library.  Run from the repository root:

    python tests/golden/write_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def uniform_logprob():
    # Step 1 on all-equal logits.  The definition gives -ln V; the test compares the stored values
    # with that closed form.  Vocabulary sizes: the tiny case, Llama-2, OPT, and the large one.
    lines = ["# V  log-prob of any token when all V logits are equal (oracle, float64)\n",
             "# definition: Section 2.1 names the actor/reference log-probabilities; closed form -ln V\n"]
    for V in (1000, 32000, 50272, 128256):
        z = np.zeros((1, 1, V))
        lp = oracle.gather_logprobs(z, np.zeros((1, 1), dtype=np.int64), [1])[0, 0]
        lines.append(f"{V} {float(lp)!r}\n")
    with open(os.path.join(HERE, "uniform_logprob.txt"), "w") as f:
        f.writelines(lines)


def tiny_path():
    """Every output of the path on the tiny workload (inputs drawn on the CPU, seed 0), step by step as
    the tests run it: each step is fed the float32-rounded outputs of the step before."""
    import json
    sys.path.insert(0, os.path.join(os.path.dirname(HERE)))
    from helpers import OracleRun
    from paper_2410_15651_b200 import inputs
    w = inputs.WORKLOADS["tiny"]
    batch = inputs.make_batch(w, device="cpu")
    run = OracleRun(oracle, w, batch)
    rows = np.array([0, 5, 17, 31])                      # three valid rows and a padded one
    dl = oracle.dlogits_rows(inputs.bf16_bits(batch["actor"]), batch["ids"].numpy(), run.lengths, run.ppo.g, rows)
    cols = np.array([0, 1, 499, 998, 999])
    out = {
        "_comment": "written by tests/golden/write_golden.py from the CPU oracle; tiny workload (B=2,T=16,V=1000), "
                    "definitions of Section 2.1 as read in the oracle's header; grad_scale = N",
        "lengths": run.lengths.tolist(), "N": run.N,
        "lp_actor": run.lp_actor.tolist(), "lp_ref": run.lp_ref.tolist(),
        "rewards": run.rewards.tolist(), "adv": run.adv.tolist(), "ret": run.ret.tolist(),
        "loss_pg": run.ppo.loss_pg, "loss_vf": run.ppo.loss_vf,
        "g": run.ppo.g.tolist(), "dvalues": run.ppo.dvalues.tolist(),
        "dlogits_rows": rows.tolist(), "dlogits_cols": cols.tolist(),
        "dlogits": dl[:, cols].tolist(),
        "dlogits_at_label": [float(dl[i, batch["ids"].numpy().reshape(-1)[r]]) for i, r in enumerate(rows)],
    }
    with open(os.path.join(HERE, "tiny_path.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    uniform_logprob()
    tiny_path()
    print("golden files written")
