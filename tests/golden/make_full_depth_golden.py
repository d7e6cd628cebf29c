"""Writes tests/golden/c2_full_depth.txt: what the CPU oracle computes for the 7B-shaped workload (C2) at FULL
depth on its seeded prompt.  Calls only the oracle and the seeded input generator; takes several minutes and a
few GB of memory (weights are generated layer by layer and dropped again).

    python tests/golden/make_full_depth_golden.py

Stored: the root mean square of the last position's logits, its 32 largest logits with their indices, the logits
at 64 evenly spaced indices, and for layers 0, 15 and 31 the root mean square and 16 evenly spaced entries of the
last position's H_attn and H_ffn (Eq. 1-2)."""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.join(HERE, "..", ".."))

import tpi_synth as S                                   # noqa: E402
from tests.helpers import make_oracle                   # noqa: E402


def main():
    shape = S.CONFIGS["C2"]
    toks = S.prompt_tokens(shape)
    orc = make_oracle(shape, cache=12)
    logits = orc.forward(toks)
    out = ["# oracle values for workload C2 (7B-shaped, bf16 weights and KV, N-independent), full depth, "
           f"prompt of {len(toks)} seeded tokens; written by tests/golden/make_full_depth_golden.py",
           f"logits_rms {np.sqrt(np.mean(logits * logits)):.17g}"]
    top = np.argsort(-logits, kind="stable")[:32]
    for i in top:
        out.append(f"top {int(i)} {logits[i]:.17g}")
    for i in np.linspace(0, shape.vocab - 1, 64).astype(int):
        out.append(f"logit {int(i)} {logits[i]:.17g}")
    for l in (0, 15, 31):
        for key in ("attn", "ffn"):
            hrow = orc.taps[(l, key)][-1]
            out.append(f"hidden_rms {l} {key} {np.sqrt(np.mean(hrow * hrow)):.17g}")
            for i in np.linspace(0, shape.hidden - 1, 16).astype(int):
                out.append(f"hidden {l} {key} {int(i)} {hrow[i]:.17g}")
    with open(os.path.join(HERE, "c2_full_depth.txt"), "w") as f:
        f.write("\n".join(out) + "\n")
    print("written", len(out), "lines")


if __name__ == "__main__":
    main()
