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


if __name__ == "__main__":
    uniform_logprob()
    print("golden files written")
