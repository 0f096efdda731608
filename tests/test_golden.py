"""The stored cfg1 fixture is reproduced by the oracle on freshly generated inputs."""
import json
import os

import numpy as np

from oracle import goodspeed_oracle as orc
from paper_2512_09963_b200 import workloads as wl


def test_oracle_reproduces_stored_cfg1_round():
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "cfg1_round.json")))
    for key, tau in (("tau1", 1.0), ("tau0", 0.0)):
        inp = wl.make_step(wl.CONFIGS["cfg1"], tau=tau)
        chk = float(inp["target_logits_f32"].double().sum() + inp["q_probs"].double().sum()
                    + inp["draft_tok"].double().sum())
        assert abs(chk - gold[key]["input_checksum"]) < 1e-3, "the seeded inputs changed"
        res = orc.ref_verify_round(inp, np.full(4, 0.5), np.ones(4), 0.1, 0.5, 10)
        assert [int(v) for v in res["accepted"]] == gold[key]["accepted"]
        assert [int(v) for v in res["out_tok"]] == gold[key]["out_tok"]
        assert [int(v) for v in res["S_next"]] == gold[key]["S_next"]
        # no decision of the fixture sits near a tie, so the GPU must match it exactly
        assert gold[key]["min_abs_accept_margin"] > 1e-4
