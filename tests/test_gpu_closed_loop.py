"""Closed-loop scheduling (the fifth workload): the library and the oracle run Algorithm 1 in
lock-step, round after round, on the same generated inputs.  Small layer shapes for hundreds of
rounds, the full Qwen3-32B-shaped layer for a few rounds."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import goodspeed_oracle as orc
from paper_2512_09963_b200 import workloads as wl
from paper_2512_09963_b200.closed_loop import ClosedLoop, run_closed_loop, jain

import parity_utils as pu

pytestmark = pytest.mark.gpu


def lockstep(cfg, rounds, check_tensors_every=1):
    state = {"alpha": np.full(cfg.N, 0.5), "X": np.ones(cfg.N), "flips": 0, "sample_ties": 0}

    def on_round(t, loop, inp, O, logits):
        host = {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in inp.items()}
        tau = float(np.float32(inp["tau"]))
        host["tau"] = tau
        ref = orc.ref_verify_round(host, state["alpha"], state["X"], loop.eta, loop.beta, loop.C,
                                   loop.s_min.cpu().numpy(), loop.s_max.cpu().numpy())
        if t % check_tensors_every == 0:
            pu.assert_close_rel(O, ref["O"], f"round {t} attention")
            pu.assert_close_rel(logits, ref["logits"], f"round {t} logits")
        Tq = host["Q"].shape[0]
        G = Tq - cfg.N
        got = {"accepted": loop.accepted.cpu().numpy(), "out_tok": loop.out_tok[:Tq].cpu().numpy(),
               "n_out": loop.n_out.cpu().numpy(), "ratio": loop.ratio[:G].cpu().numpy(),
               "p_tok": loop.p_tok[:G].cpu().numpy()}
        slack = pu.chain_slack(logits, ref["logits"], tau)
        log = pu.compare_accept(got, ref, ref["logits"], host["q_probs"], host["cu_q"].numpy(), host["u_sample"],
                                tau, cfg.V, slack=slack)
        state["flips"] += len(log["accept_near_ties"])
        state["sample_ties"] += len(log["sample_near_ties"])
        if log["accept_near_ties"]:
            # a logged near-tie flipped a count: take the oracle's estimator state and allocation
            loop.alpha_hat.copy_(torch.from_numpy(ref["alpha_hat"]).to(loop.alpha_hat.device))
            loop.X.copy_(torch.from_numpy(ref["X"]).to(loop.X.device))
            loop.S_next.copy_(torch.from_numpy(ref["S_next"].astype(np.int32)).to(loop.S_next.device))
        else:
            np.testing.assert_allclose(loop.alpha_hat.cpu().numpy(), ref["alpha_hat"], atol=1e-4)
            np.testing.assert_allclose(loop.X.cpu().numpy(), ref["X"], atol=1e-9)
            S_gpu = loop.S_next.cpu().numpy()
            if not np.array_equal(S_gpu, ref["S_next"]):
                # estimator rounding moved a near-tied marginal: both allocations must be optimal
                o1 = orc.ref_sched_objective(ref["X"], ref["alpha_hat"], S_gpu)
                o2 = orc.ref_sched_objective(ref["X"], ref["alpha_hat"], ref["S_next"])
                assert S_gpu.sum() == ref["S_next"].sum() and abs(o1 - o2) <= 1e-6 * abs(o2)
                loop.S_next.copy_(torch.from_numpy(ref["S_next"].astype(np.int32)).to(loop.S_next.device))
            # keep the two state machines on identical numbers (the library's are fp32-derived)
            loop.alpha_hat.copy_(torch.from_numpy(ref["alpha_hat"]).to(loop.alpha_hat.device))
        state["alpha"], state["X"] = ref["alpha_hat"], ref["X"]
        assert int(loop.S_next.sum().item()) <= loop.C

    rep = run_closed_loop(cfg, rounds, on_round=on_round)
    return rep, state


def test_closed_loop_small_shapes_300_rounds():
    cfg = dataclasses.replace(wl.CONFIGS["cfg5"], name="cfg5_small", d=128, V=4096, Hq=8, Hkv=1, hd=128,
                              prefix_lo=96, prefix_hi=96, N=8, C=40)
    rep, state = lockstep(cfg, 300, check_tensors_every=25)
    assert state["flips"] <= 3, state
    assert 0.5 < rep["jain"] <= 1.0
    assert all(x >= 1.0 for x in rep["goodput_per_server"])
    # estimates track the truth: after 100 rounds in the last epoch alpha_hat is near the calibrated rate
    err = np.abs(np.asarray(rep["final_alpha_hat"]) - np.asarray(rep["true_alpha_last_epoch"]))
    assert np.median(err) < 0.15, err


def test_closed_loop_full_shapes_few_rounds():
    rep, state = lockstep(wl.CONFIGS["cfg5"], 3)
    assert rep["rounds"] == 3 and len(rep["goodput_per_server"]) == 16
    assert state["flips"] <= 1


def test_policies_goodspeed_beats_fixed_and_random_in_utility():
    """Sec. V compares GoodSpeed with Fixed-S and Random-S on the utility of the mean goodput,
    sum_i log x_bar_i.  Same simulated servers, same rounds, the library's round on the GPU; only the
    rule for S(t+1) differs.  Stationary, spread-out acceptance rates (one epoch)."""
    cfg = dataclasses.replace(wl.CONFIGS["cfg5"], name="cfg5_policies", d=128, V=4096, Hq=8, Hkv=1, hd=128,
                              prefix_lo=96, prefix_hi=96, N=8, C=40)
    rounds = 100
    util = {}
    for pol in ("goodspeed", "fixed", "random"):
        rep = run_closed_loop(cfg, rounds, policy=pol, curve_every=20)
        util[pol] = rep["utility_sum_log"]
        assert rep["policy"] == pol and len(rep["utility_curve"]) == 5
        assert all(x >= 1.0 for x in rep["goodput_per_server"])          # every server gets its bonus/correction token
    assert util["goodspeed"] >= util["fixed"] - 1e-9, util
    assert util["goodspeed"] > util["random"], util


def test_decaying_steps_run_and_converge():
    """Assumption 3 (steps with divergent sum, convergent sum of squares): the loop runs with
    (t+1)^-0.6 steps and the goodput estimate X stays within the range of per-round goodputs."""
    cfg = dataclasses.replace(wl.CONFIGS["cfg5"], name="cfg5_decay", d=128, V=4096, Hq=8, Hkv=1, hd=128,
                              prefix_lo=96, prefix_hi=96, N=8, C=40)
    rep = run_closed_loop(cfg, 60, step_decay=0.6)
    assert rep["step_decay"] == 0.6 and 0.5 < rep["jain"] <= 1.0


def test_growing_paged_caches():
    """Sec. III-A: every round's output tokens join the server's prefix.  The caches live in a page
    pool (pages handed out in shuffled order as they are needed) and attention reads them through
    the block table; the oracle gets the same keys and values gathered into its contiguous layout."""
    cfg = dataclasses.replace(wl.CONFIGS["cfg5"], name="cfg5_grow", d=128, V=4096, Hq=8, Hkv=1, hd=128,
                              prefix_lo=100, prefix_hi=100, N=6, C=30)
    seen = {"rounds": 0, "grown": 0}

    def on_round(t, loop, inp, O, logits):
        lens = (inp["cu_kv"][1:] - inp["cu_kv"][:-1]).cpu().numpy() - (inp["gamma"] + 1)
        assert np.array_equal(lens, loop.len)
        if t % 4 == 0:
            K, V = loop.gather_contiguous(inp)
            ref = orc.ref_attention(inp["Q"].cpu(), K.cpu(), V.cpu(), inp["cu_q"].cpu(), inp["cu_kv"].cpu())
            pu.assert_close_rel(O, ref, f"round {t} attention over paged caches")
        seen["rounds"] += 1

    rep = run_closed_loop(cfg, 40, on_round=on_round, grow=True, max_len=700)
    assert seen["rounds"] == 40
    total_out = np.asarray(rep["goodput_per_server"]) * 40
    final = np.asarray(rep["final_cache_len"])
    # every cache grew by exactly its output tokens until it hit the cap
    cap = 700 - (cfg.C + 1)
    assert np.array_equal(final, np.minimum(100 + np.rint(total_out).astype(np.int64), cap))
    assert final.max() > 128 * 2          # caches crossed page boundaries
