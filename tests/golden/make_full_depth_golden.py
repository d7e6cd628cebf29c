"""Writes tests/golden/<workload>_full_depth.txt: what the CPU oracle computes for a workload at FULL depth on its seeded
prompt.  Calls only the oracle and the seeded input generator; on 8 cores C2 takes ~4 minutes, C3 ~30 minutes, C5 ~1 hour,
with up to ~25 GB of memory (weights are generated layer by layer and dropped again).

    python tests/golden/make_full_depth_golden.py            # C2: 7B shape, 128-token prompt
    python tests/golden/make_full_depth_golden.py C3         # 8B shape, its 4096-token prompt
    python tests/golden/make_full_depth_golden.py C5         # 70B shape, 512-token prompt

Stored, for the last prompt position: the root mean square of the logits, the 32 largest logits with their indices,
the logits at 64 evenly spaced indices, and for the first, the middle and the last layer the root mean square and 16
evenly spaced entries of H_attn and H_ffn (Eq. 1-2).  Then the same logit records (prefix "d") for ONE decode step on
top of the prompt, fed with the oracle's own greedy token (the GPU test teacher-forces the same token)."""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.join(HERE, "..", ".."))

import tpi_synth as S                                   # noqa: E402
from tests.helpers import make_oracle                   # noqa: E402


def logit_records(out, prefix, logits, vocab):
    out.append(f"{prefix}logits_rms {np.sqrt(np.mean(logits * logits)):.17g}")
    for i in np.argsort(-logits, kind="stable")[:32]:
        out.append(f"{prefix}top {int(i)} {logits[i]:.17g}")
    for i in np.linspace(0, vocab - 1, 64).astype(int):
        out.append(f"{prefix}logit {int(i)} {logits[i]:.17g}")


def main():
    name = sys.argv[1] if len(sys.argv) > 1 else "C2"
    shape = S.CONFIGS[name]
    toks = S.prompt_tokens(shape)
    orc = make_oracle(shape, cache=12)
    logits = orc.forward(toks)
    L = shape.n_layers
    out = [f"# oracle values for workload {name} ({shape.name}, {shape.dtype} weights and KV, N-independent), full depth, "
           f"prompt of {len(toks)} seeded tokens; written by tests/golden/make_full_depth_golden.py"]
    logit_records(out, "", logits, shape.vocab)
    for l in (0, L // 2 - 1, L - 1):
        for key in ("attn", "ffn"):
            hrow = orc.taps[(l, key)][-1]
            out.append(f"hidden_rms {l} {key} {np.sqrt(np.mean(hrow * hrow)):.17g}")
            for i in np.linspace(0, shape.hidden - 1, 16).astype(int):
                out.append(f"hidden {l} {key} {int(i)} {hrow[i]:.17g}")
    if name != "C2":      # C2's file predates the decode records and is kept as it was written
        feed = int(np.argmax(logits))
        out.append(f"dfeed {feed}")
        logit_records(out, "d", orc.forward([feed]), shape.vocab)
    with open(os.path.join(HERE, f"{name.lower()}_full_depth.txt"), "w") as f:
        f.write("\n".join(out) + "\n")
    print("written", len(out), "lines")


if __name__ == "__main__":
    main()
