"""Closed-loop scheduling (the fifth workload): the library and the oracle run Algorithm 1 in
lock-step, round after round, on the same generated inputs.  Small layer shapes for hundreds of
rounds with the oracle's whole round beside every one; the full Qwen3-32B-shaped layer for a few
rounds the same way, and for all 1000 rounds with the oracle's acceptance, estimator and scheduler
steps beside every round and its attention / LM head beside six of them."""
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


def _full_tensor_check(t, Q, K, V, cu_q, cu_kv, H, W, O, logits):
    """Attention and LM head of one round against the oracle's definitions, every element."""
    pu.assert_close_rel(O, orc.ref_attention(Q, K, V, cu_q, cu_kv), f"round {t} attention")
    Vn = W.shape[1]
    worst = 0.0
    for c0 in range(0, Vn, 8192):
        cols = np.arange(c0, min(Vn, c0 + 8192))
        worst = max(worst, pu.assert_close_rel(logits[:, cols], orc.ref_lm_head(H, W, cols=cols),
                                               f"round {t} logits, columns {c0}.."))
    return worst


def test_closed_loop_thousand_rounds_at_full_shapes():
    """The fifth workload as stated: 1000 rounds, 16 servers, budget 128, the Qwen3-32B-shaped layer.
    The library runs the closed loop on the GPU by itself; beside it the oracle takes its steps of
    every round -- temperature softmax, acceptance, correction / bonus token (Sec. II-A2), estimator
    updates (Eq. updatealpha, Eq. updateX), next allocation (Eq. goodspeed_sched) -- on the logits the
    GPU produced, widened to fp64: identical logits on both sides, so the strict 1e-5 band applies
    with no slack.  Attention and the LM head are compared in full on rounds 0, 1, 99, 100, 500, 999.
    The oracle's per-round work (half a second of numpy) runs on a pool of threads behind the GPU
    loop; the order-dependent part (estimators, allocation) is checked in round order.
    Two oracle state machines are kept: one restarts every round from the library's previous state
    (a one-step check: estimators to 2e-6, the allocation bit-exact on identical inputs), one runs
    free for all 1000 rounds and only takes over a count after a logged near-tie (drift check)."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    cfg = wl.CONFIGS["cfg5"]
    rounds, full_rounds = 1000, {0, 1, 99, 100, 500, 999}
    N, C, V = cfg.N, cfg.C, cfg.V
    tau = float(np.float32(cfg.tau))
    workers = min(12, max(2, (os.cpu_count() or 4) - 2))
    pool = ThreadPoolExecutor(max_workers=workers)
    pending = []
    st = {"prev_a": np.full(N, 0.5), "prev_X": np.ones(N), "free_a": np.full(N, 0.5), "free_X": np.ones(N),
          "flips": [], "draw_ties": [], "free_alloc_differs": 0, "checked": 0, "full": [], "W_host": None}

    def verify(rec):
        ref = rec["fut"].result()
        log = pu.compare_accept(rec["got"], ref, rec["logits"], rec["q_probs"], rec["cu_q"], rec["u_sample"], tau, V)
        flipped = {i for i, _, _ in log["accept_near_ties"]}
        st["flips"] += [(rec["t"],) + x for x in log["accept_near_ties"]]
        st["draw_ties"] += [(rec["t"],) + x for x in log["sample_near_ties"]]
        keep = np.array([i not in flipped for i in range(N)])
        # one step from the library's previous state
        a1, X1 = orc.ref_ema(st["prev_a"], st["prev_X"], ref["ratio"], ref["accepted"], rec["cu_q"], rec["eta"], rec["beta"])
        np.testing.assert_allclose(rec["alpha_hat"], a1, rtol=0, atol=2e-6, err_msg=f"round {rec['t']} alpha_hat")
        np.testing.assert_allclose(rec["X"][keep], X1[keep], rtol=0, atol=1e-9, err_msg=f"round {rec['t']} X")
        S1 = orc.ref_schedule_greedy(rec["X"], rec["alpha_hat"], C, rec["s_min"], rec["s_max"])
        assert np.array_equal(rec["S_next"], S1), f"round {rec['t']}: allocation on identical estimates"
        assert rec["S_next"].sum() <= C
        st["prev_a"], st["prev_X"] = rec["alpha_hat"], rec["X"]
        # the free-running oracle: its own state all the way; a logged near-tie hands it the library's count
        acc = ref["accepted"].copy()
        for i in flipped:
            acc[i] = rec["got"]["accepted"][i]
        st["free_a"], st["free_X"] = orc.ref_ema(st["free_a"], st["free_X"], ref["ratio"], acc, rec["cu_q"],
                                                 rec["eta"], rec["beta"])
        np.testing.assert_allclose(rec["alpha_hat"], st["free_a"], rtol=0, atol=1e-4, err_msg=f"round {rec['t']} drift of alpha_hat")
        np.testing.assert_allclose(rec["X"], st["free_X"], rtol=0, atol=1e-6, err_msg=f"round {rec['t']} drift of X")
        S2 = orc.ref_schedule_greedy(st["free_X"], st["free_a"], C, rec["s_min"], rec["s_max"])
        if not np.array_equal(S2, rec["S_next"]):     # estimator rounding moved a near-tied marginal: both must be optimal
            st["free_alloc_differs"] += 1
            o1 = orc.ref_sched_objective(st["free_X"], st["free_a"], rec["S_next"])
            o2 = orc.ref_sched_objective(st["free_X"], st["free_a"], S2)
            assert S2.sum() == rec["S_next"].sum() and abs(o1 - o2) <= 1e-6 * abs(o2)
        if rec["full"] is not None:
            st["full"].append((rec["t"], rec["full"].result()))
        st["checked"] += 1

    def on_round(t, loop, inp, O, logits):
        Tq = inp["Q"].shape[0]
        G = Tq - N
        lg, qp = logits.cpu(), inp["q_probs"].cpu()
        cu_q = inp["cu_q"].cpu().numpy()
        tok, ua, us = inp["draft_tok"].cpu(), inp["u_accept"].cpu(), inp["u_sample"].cpu()
        rec = {"t": t, "logits": lg, "q_probs": qp, "cu_q": cu_q, "u_sample": us, "eta": loop.eta, "beta": loop.beta,
               "s_min": loop.s_min.cpu().numpy(), "s_max": loop.s_max.cpu().numpy(),
               "got": {"accepted": loop.accepted.cpu().numpy(), "out_tok": loop.out_tok[:Tq].cpu().numpy(),
                       "n_out": loop.n_out.cpu().numpy(), "ratio": loop.ratio[:G].cpu().numpy(),
                       "p_tok": loop.p_tok[:G].cpu().numpy()},
               "alpha_hat": loop.alpha_hat.cpu().numpy().copy(), "X": loop.X.cpu().numpy().copy(),
               "S_next": loop.S_next.cpu().numpy().copy(), "full": None}
        rec["fut"] = pool.submit(orc.ref_spec_accept, lg, qp, tok, cu_q, ua, us, tau)
        if t in full_rounds:
            if st["W_host"] is None:
                st["W_host"] = loop.W.cpu()
            rec["full"] = pool.submit(_full_tensor_check, t, inp["Q"].cpu(), inp["K"].cpu(), inp["V"].cpu(), cu_q,
                                      inp["cu_kv"].cpu().numpy(), inp["H"].cpu(), st["W_host"], O.cpu(), lg)
        pending.append(rec)
        while len(pending) > 2 * workers:
            verify(pending.pop(0))

    try:
        rep = run_closed_loop(cfg, rounds, on_round=on_round)
        while pending:
            verify(pending.pop(0))
    finally:
        pool.shutdown(wait=True, cancel_futures=True)
    assert st["checked"] == rounds and sorted(t for t, _ in st["full"]) == sorted(full_rounds)
    # near-ties are rare on identical logits: the band is 1e-5 wide and a round has ~128 decisions
    assert len(st["flips"]) <= 8, st["flips"]
    assert rep["rounds"] == rounds and len(rep["goodput_per_server"]) == N
    assert all(x >= 1.0 for x in rep["goodput_per_server"]) and 0.5 < rep["jain"] <= 1.0
    print("cfg5, 1000 rounds at full shapes:", {"jain": rep["jain"], "utility_sum_log": rep["utility_sum_log"],
                                                  "goodput_per_server": rep["goodput_per_server"],
                                                  "verified_tokens_per_s": rep["verified_tokens_per_s"],
                                                  "goodput_tokens_per_s": rep["goodput_tokens_per_s"],
                                                  "gpu_ms_per_round": rep["gpu_ms_per_round"]})
    print("logged accept near-ties (round, server, position, |u - p/q|):", st["flips"])
    print("logged draw near-ties (round, server, library token, oracle token, CDF distance):", st["draw_ties"])
    print("rounds whose allocation differs from the free-running oracle's at equal objective:", st["free_alloc_differs"],
          "; worst full-tensor error/bound:", st["full"])


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
