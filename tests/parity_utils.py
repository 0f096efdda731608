"""Comparison rules between the CUDA library and the CPU oracle (used by the GPU tests, the
smoke check and the benchmark's self-check).

Integer results (accepted counts, token ids, allocations) must be identical, except decisions
the oracle itself flags as near-ties:
  * an accept/reject decision whose |u - p/q| < 1e-5 in the oracle;
  * a correction/bonus draw where u lies within 1e-5 (in CDF units) of the interval of the
    token the library emitted, measured on the oracle's fp64 CDF.
After a logged accept/reject flip the rest of that server's outputs legitimately diverge and
are skipped.  Every such decision is printed (pytest -s shows the lines) and returned in the log.  Probabilities are compared to 1e-5 absolute, attention outputs and logits to
2e-2 relative to max(|ref|, rms(ref row)).
"""
from __future__ import annotations

import numpy as np

from oracle import goodspeed_oracle as orc

NEAR_TIE = 1e-5
PROB_ATOL = 1e-5
REL_TOL = 2e-2


def np64(t):
    return t.detach().cpu().double().numpy() if hasattr(t, "detach") else np.asarray(t, dtype=np.float64)


def assert_close_rel(got, ref, what, rel=REL_TOL):
    """|got - ref| <= rel * max(|ref|, rms of ref's last-dim row)."""
    got, ref = np64(got), np64(ref)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    bound = rel * np.maximum(np.abs(ref), rms)
    err = np.abs(got - ref)
    bad = err > bound
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} elements outside {rel} relative; "
                           f"worst err {err.max():.3e}, worst err/bound {np.max(err / np.maximum(bound, 1e-300)):.3f}")
    return float(np.max(err / np.maximum(bound, 1e-300)))


def chain_slack(gpu_logits, ref_logits, tau):
    """Extra probability tolerance when the two sides ran on their OWN logits (library: bf16
    products accumulated in fp32 on the tensor cores; oracle: fp64).  A logit error e moves
    log p(s) = l_s/tau - logsumexp(l/tau) by at most 2e/tau, and p, min(1, p/q) <= 1, so the
    probabilities move by at most 2e/tau.  e is the largest observed logit difference."""
    e = float(np.max(np.abs(np64(gpu_logits) - np64(ref_logits))))
    return 2.0 * e / tau if tau > 0 else 0.0


def compare_accept(gpu, ref, logits, q_probs, cu_q, u_sample, tau, V, slack=0.0):
    """gpu: dict of numpy arrays accepted/out_tok/n_out/ratio/p_tok from the library;
    ref: ref_spec_accept output on the same inputs.  slack widens the probability tolerance and
    the near-tie band (see chain_slack); it is 0 when both sides read identical logits.
    Returns a log dict."""
    PROB_ATOL_, NEAR_TIE_ = PROB_ATOL + slack, NEAR_TIE + slack
    cu_q = np.asarray(cu_q, dtype=np.int64)
    N = len(cu_q) - 1
    log = {"accept_near_ties": [], "sample_near_ties": [], "sample_exact": 0, "servers": N}
    u_sample = np64(u_sample)      # logits and q_probs rows are widened only where a draw has to be re-examined
    for i in range(N):
        r0 = cu_q[i]
        gamma = int(cu_q[i + 1] - r0 - 1)
        g0 = r0 - i
        a_g, a_r = int(gpu["accepted"][i]), int(ref["accepted"][i])
        assert 0 <= a_g <= gamma, f"server {i}: accepted {a_g} outside [0,{gamma}]"
        assert int(gpu["n_out"][i]) == a_g + 1
        np.testing.assert_allclose(gpu["ratio"][g0:g0 + gamma], ref["ratio"][g0:g0 + gamma], rtol=0,
                                   atol=PROB_ATOL_, err_msg=f"ratio, server {i}")
        np.testing.assert_allclose(gpu["p_tok"][g0:g0 + gamma], ref["p_tok"][g0:g0 + gamma], rtol=0,
                                   atol=PROB_ATOL_, err_msg=f"p_tok, server {i}")
        seg = gpu["out_tok"][r0:r0 + gamma + 1]
        assert np.all(seg[a_g + 1:] == -1), f"server {i}: padding after the last token"
        assert 0 <= seg[a_g] < V, f"server {i}: emitted id {seg[a_g]} outside the vocabulary"
        if a_g != a_r:
            j = min(a_g, a_r)
            marg = abs(ref["margin_acc"][g0 + j])
            assert marg < NEAR_TIE_, (f"server {i}: accepted {a_g} vs oracle {a_r}, decision {j} has "
                                     f"|u - p/q| = {marg:.3e}")
            log["accept_near_ties"].append((i, j, float(marg)))
            print(f"near-tie (accept): server {i} draft position {j}: |u - p/q| = {marg:.3e}; "
                  f"library accepted {a_g}, oracle {a_r}")
            continue
        assert np.array_equal(seg[:a_g], ref["out_tok"][r0:r0 + a_g]), f"server {i}: accepted tokens"
        tok_g, tok_r = int(seg[a_g]), int(ref["out_tok"][r0 + a_r])
        if tok_g == tok_r:
            log["sample_exact"] += 1
            continue
        # not the oracle's token: is u within NEAR_TIE of the emitted token's CDF interval?
        p = orc.ref_softmax_T(np64(logits[r0 + a_r]), tau)
        w = orc.ref_residual(p, np64(q_probs[g0 + a_r])) if a_r < gamma else p
        F = np.cumsum(w)
        R = F[-1]
        lo = (F[tok_g - 1] if tok_g > 0 else 0.0) / R
        hi = F[tok_g] / R
        dist = max(0.0, lo - u_sample[i], u_sample[i] - hi)
        assert w[tok_g] > 0 and dist < NEAR_TIE_, (
            f"server {i}: emitted {tok_g}, oracle {tok_r}; u={u_sample[i]:.8f} is {dist:.3e} away from "
            f"the emitted token's CDF interval [{lo:.8f},{hi:.8f}]")
        log["sample_near_ties"].append((i, tok_g, tok_r, float(dist)))
        print(f"near-tie (draw): server {i}: library token {tok_g}, oracle token {tok_r}; u is {dist:.3e} "
              f"(CDF units) from the library token's interval")
    return log


def log_for_json(log):
    """The near-tie log as plain lists: which decisions differed from the oracle's, and by how little."""
    return {"servers": log["servers"], "sample_exact": log["sample_exact"],
            "accept_near_ties": [{"server": int(i), "draft_position": int(j), "abs_u_minus_ratio": m}
                                 for i, j, m in log["accept_near_ties"]],
            "sample_near_ties": [{"server": int(i), "library_token": int(a), "oracle_token": int(b),
                                  "cdf_distance": d} for i, a, b, d in log["sample_near_ties"]]}


def gpu_accept_dict(rnd):
    """Copies a VerifyRound's acceptance outputs to numpy."""
    return {k: getattr(rnd, k).detach().cpu().numpy() for k in ("accepted", "out_tok", "n_out", "ratio", "p_tok")}
