"""The synthetic input generator: shapes, dtypes, determinism and the stated distributions."""
import numpy as np
import torch

from oracle import goodspeed_oracle as orc
from paper_2512_09963_b200 import workloads as wl


def test_cfg1_shapes_and_determinism():
    a = wl.make_step(wl.CONFIGS["cfg1"])
    b = wl.make_step(wl.CONFIGS["cfg1"])
    assert a["Q"].shape == (14, 4, 64) and a["K"].shape[1:] == (2, 64) and a["W"].shape == (256, 1024)
    assert a["q_probs"].shape == (10, 1024) and a["draft_tok"].shape == (10,)
    assert a["cu_q"].tolist() == [0, 2, 5, 9, 14]
    assert all(64 <= p <= 128 for p in a["prefix"])
    assert int(a["cu_kv"][-1]) == int(sum(a["prefix"]) + 14)
    for k in ("Q", "K", "V", "H", "W", "q_probs", "draft_tok", "u_accept", "u_sample"):
        assert torch.equal(a[k], b[k]), k
    assert torch.allclose(a["q_probs"].sum(dim=1), torch.ones(10), atol=1e-5)
    u = a["u_accept"].numpy()
    assert np.all((u > 0) & (u < 1))
    assert abs(float(a["target_logits_f32"].std()) - 1.0) < 0.1      # W ~ N(0, 1/d) gives unit logits
    c = wl.make_step(wl.CONFIGS["cfg1"], round_idx=1)
    assert not torch.equal(a["H"], c["H"])


def test_shrunken_configs_keep_structure():
    c2 = wl.shrink(wl.CONFIGS["cfg2"], d=128, V=2000, prefix_scale=0.02)
    s = wl.make_step(c2)
    assert s["Q"].dtype == torch.bfloat16 and s["Q"].shape[1:] == (64, 128) and s["K"].shape[1:] == (8, 128)
    assert np.all((s["gamma"] >= 1) & (s["gamma"] <= 8)) and len(s["gamma"]) == 8
    assert np.all((s["sigma"] >= 0.2) & (s["sigma"] <= 1.5))
    c3 = wl.shrink(wl.CONFIGS["cfg3"], d=128, V=2000, prefix_scale=0.05)
    s = wl.make_step(c3, allocator=orc.ref_schedule_greedy)
    assert s["gamma"].sum() == 256 and s["gamma"].min() >= 1 and s["gamma"].max() <= 16
    full = wl.draw_prefix(wl.CONFIGS["cfg3"])
    assert full.min() >= 128 and full.max() <= 8192 and 500 < np.median(full) < 2100
    c4 = wl.CONFIGS["cfg4"]
    g = wl.draw_gamma(c4)
    assert len(g) == 16 and g.min() >= 2 and g.max() <= 8


def test_noise_level_sets_acceptance_and_calibration_inverts_it():
    sig = np.array([0.0, 0.2, 0.5, 1.0, 2.0])
    ov = wl.overlap_table(4000, 0.7, sig, rows=4)
    assert abs(ov[0] - 1.0) < 1e-12 and np.all(np.diff(ov) < 0)
    want = np.array([0.9, 0.6, 0.4])
    s = wl.calibrate_sigma(want, 4000, 0.7)
    got = wl.overlap_table(4000, 0.7, s, rows=8)
    assert np.all(np.abs(got - want) < 0.05)
    al = wl.draw_true_alpha(wl.CONFIGS["cfg5"], 0)
    assert len(al) == 16 and np.all((al > 0) & (al < 1))
    assert not np.allclose(al, wl.draw_true_alpha(wl.CONFIGS["cfg5"], 1))
