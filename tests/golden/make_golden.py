"""Writes tests/golden/cfg1_round.json: the integer outputs of one cfg1 round (temperature 1 and 0)
as computed by the CPU oracle alone on the seeded cfg1 inputs.  Run from the repository root:

    python tests/golden/make_golden.py

The paper prints no worked numeric example, so this fixture is oracle-written (never taken from the
CUDA path); it guards the oracle and the input generator against silent drift and gives the GPU
test a second, stored reference.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import goodspeed_oracle as orc          # noqa: E402
from paper_2512_09963_b200 import workloads as wl   # noqa: E402


def main():
    out = {"source": "oracle/goodspeed_oracle.py on workloads.make_step(cfg1); eta=0.1 beta=0.5 C=10, "
                     "alpha_hat(0)=0.5, X(0)=1"}
    for key, tau in (("tau1", 1.0), ("tau0", 0.0)):
        inp = wl.make_step(wl.CONFIGS["cfg1"], tau=tau)
        res = orc.ref_verify_round(inp, np.full(4, 0.5), np.ones(4), 0.1, 0.5, 10)
        out[key] = {
            "accepted": [int(v) for v in res["accepted"]],
            "out_tok": [int(v) for v in res["out_tok"]],
            "S_next": [int(v) for v in res["S_next"]],
            "min_abs_accept_margin": float(np.min(np.abs(res["margin_acc"]))),
            "input_checksum": float(inp["target_logits_f32"].double().sum() + inp["q_probs"].double().sum()
                                    + inp["draft_tok"].double().sum()),
        }
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_round.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()
