"""Writes tests/golden/c1_oracle.json: per-utterance losses, subset and gradient norms of the
float64 oracle on the seeded c1 batch.  Calls only the oracle and the input generator."""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import pruned_ctc_oracle as O  # noqa: E402
from paper_2609_33645_b200 import workloads as wl  # noqa: E402

batch = wl.make_batch(wl.CONFIGS["c1"])
ref = O.pruned_ctc_reference(batch.hidden, batch.W, None, batch.targets, batch.input_lengths,
                             batch.target_lengths, batch.blank)
out = dict(
    source="oracle/pruned_ctc_oracle.py on workloads.CONFIGS['c1'] (seed 1001); Section 3.1 Eq. ctc, Eq. grad-full",
    loss=[float(x) for x in ref["loss"]], K=int(ref["K"]), U=[int(x) for x in ref["U"]],
    dH_fro=float(np.linalg.norm(ref["dH"])), dW_fro=float(np.linalg.norm(ref["dW"])),
    dW_row_blank=[float(x) for x in ref["dW"][0, :8]],
)
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_oracle.json"), "w") as f:
    json.dump(out, f, indent=1)
print("written")
