"""Plain fp64 CPU restatement of one GoodSpeed verification round.

TEST INFRASTRUCTURE ONLY.  This module exists to check the CUDA library; it is
slow on purpose and shares no code, table or constant with the CUDA path.  Only
the test-suite, the smoke check and the benchmark's reported CPU baseline may
import it.  Nothing in the product package imports it.

Everything is numpy float64.  Inputs stored in bf16/fp32 are widened exactly
before use.  Each function names the passage of the paper it restates:

* ref_attention      -- Sec. II-A2 ("the target model computes the probabilities
                        of candidate tokens in parallel"); the paper gives no
                        attention formula, the textbook scaled-dot-product
                        definition with grouped KV heads is written out.
* ref_lm_head        -- Sec. II-A1, P_M = softmax(W h): the W h product.
* ref_dequant_w4     -- Sec. V names an AWQ-INT4 target: the 4-bit head weight, dequantised by
                        its definition (scale * (code - zero)), then ref_lm_head as before.
* ref_softmax_T      -- Sec. II-A1 softmax; temperature 0 is the "greedy
                        sampling ... argmax" case of the same paragraph.
* ref_spec_accept    -- Sec. II-A2: accept s_j iff r_j <= p_j(s_j)/q_j(s_j);
                        m = first rejection; correction from
                        normalise(max(0, p_{m+1}-q_{m+1})) or bonus from p_{S+1}.
* ref_ema            -- Eq. (updatealpha) and Eq. (updateX), Sec. III-C.
* ref_mu             -- expected goodput mu_i(k), Sec. III-B.
* ref_schedule_*     -- GoodSpeed-sched, Eq. (goodspeed_sched), Sec. III-C.

Pins (see tests/test_oracle_*.py): closed forms, invariants, brute force and
exact enumeration; no function below is "parity unpinned".
"""
from __future__ import annotations

import itertools
import numpy as np

F64 = np.float64


def _f64(x):
    """Widen any array-like (numpy, or a torch CPU tensor incl. bfloat16) to float64."""
    if hasattr(x, "detach"):  # torch tensor, without importing torch here
        x = x.detach().cpu().double().numpy()
    return np.asarray(x, dtype=F64)


def _i64(x):
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.asarray(x, dtype=np.int64)


# --------------------------------------------------------------------------- #
# a1  verify attention                                                         #
# --------------------------------------------------------------------------- #
def ref_attention(Q, K, V, cu_q, cu_kv, scale=None):
    """Attention of each server's gamma_i+1 new positions over its own cache.

    Q [T_q, H_q, hd]; K, V [sum L_kv, H_kv, hd]; server i owns query rows
    cu_q[i]:cu_q[i+1] and key rows cu_kv[i]:cu_kv[i+1].  The last
    n_i = cu_q[i+1]-cu_q[i] keys of a server are the new positions themselves, so
    new position t (0-based) sees keys 0 .. L_i+t with L_i = L_kv,i - n_i.
    Query head h reads KV head h // (H_q/H_kv).  scale defaults to 1/sqrt(hd).
    Returns O [T_q, H_q, hd] float64.
    """
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    cu_q, cu_kv = _i64(cu_q), _i64(cu_kv)
    Tq, Hq, hd = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(F64(hd))
    O = np.zeros_like(Q)
    for i in range(len(cu_q) - 1):
        q0, q1 = cu_q[i], cu_q[i + 1]
        k0, k1 = cu_kv[i], cu_kv[i + 1]
        n_new = q1 - q0
        L = (k1 - k0) - n_new
        for h in range(Hq):
            g = h // G
            for t in range(n_new):
                visible = L + t + 1
                keys = K[k0:k0 + visible, g, :]
                vals = V[k0:k0 + visible, g, :]
                s = scale * (keys @ Q[q0 + t, h, :])
                w = np.exp(s - s.max())
                w = w / w.sum()
                O[q0 + t, h, :] = w @ vals
    return O


# --------------------------------------------------------------------------- #
# a2  LM head                                                                  #
# --------------------------------------------------------------------------- #
def ref_lm_head(H, W, cols=None):
    """logits[r, v] = sum_c H[r, c] * W[c, v]  (W stored [d, V]).

    cols, if given, selects the vocabulary columns to compute (the definition is
    column-separable, so sampled columns of a huge head can be checked one by one).
    """
    H = _f64(H)
    if cols is not None:
        cols = _i64(cols)
        if hasattr(W, "detach"):
            W = W.detach().cpu()[:, cols]
        else:
            W = np.asarray(W)[:, cols]
    return H @ _f64(W)


def ref_dequant_w4(qweight, scales, zeros, group):
    """The head weight of a 4-bit checkpoint, W[k, v] = scale[k // group, v] * (code[k, v] - zero[k // group, v]).

    The paper's larger target is an AWQ-INT4 model (Sec. V) and gives no storage format; the format is
    the library's, restated here from its definition: qweight [d/8, V] holds eight 4-bit codes per
    32-bit word along d, the code of row 8w + j in bits [4n, 4n+4) of word [w, v] with
    n = (j >> 1) + 4 (j & 1); scales [d/group, V]; zeros [d/group, V] in 0..15.  Returns W [d, V] float64
    (exact: no rounding of the product).
    """
    qw = _i64(qweight) & 0xFFFFFFFF
    scales, zeros = _f64(scales), _f64(zeros)
    d8, V = qw.shape
    W = np.empty((8 * d8, V))
    for w in range(d8):
        for j in range(8):
            n = (j >> 1) + 4 * (j & 1)
            k = 8 * w + j
            code = (qw[w] >> (4 * n)) & 15
            W[k] = scales[k // group] * (code.astype(F64) - zeros[k // group])
    return W


# --------------------------------------------------------------------------- #
# a3  temperature softmax, acceptance, correction / bonus token               #
# --------------------------------------------------------------------------- #
def ref_softmax_T(logits_row, tau):
    """p = softmax(logits / tau); tau == 0 is the one-hot at the lowest-index argmax."""
    x = _f64(logits_row)
    if tau == 0:
        p = np.zeros_like(x)
        p[int(np.argmax(x))] = 1.0  # numpy argmax returns the first maximum
        return p
    z = (x - x.max()) / F64(tau)
    e = np.exp(z)
    return e / e.sum()


def ref_ratio(p_s, q_s):
    """p(s)/q(s) with the q(s)=0 convention: p>0 -> certain accept, p=0 -> certain reject."""
    if q_s > 0:
        return p_s / q_s
    return np.inf if p_s > 0 else 0.0


def ref_residual(p, q):
    """Unnormalised correction distribution max(0, p - q); falls back to p if it has no mass."""
    r = np.maximum(p - q, 0.0)
    if r.sum() <= 0.0:
        r = p.copy()
    return r


def ref_inverse_cdf(weights, u):
    """Smallest v with sum_{w<=v} weights[w] > u * sum(weights); ascending token id.

    Returns (v, margin) where margin is the distance, in units of the total mass,
    from the threshold to the nearer edge of token v's CDF interval.
    """
    F = np.cumsum(weights)
    R = F[-1]
    thr = F64(u) * R
    hit = np.nonzero(F > thr)[0]
    if len(hit) == 0:  # rounding left no index: last token that has mass
        v = int(np.nonzero(weights > 0)[0][-1])
    else:
        v = int(hit[0])
    lo = F[v - 1] if v > 0 else 0.0
    margin = min(thr - lo, F[v] - thr) / R
    return v, float(margin)


def ref_spec_accept(logits, q_probs, draft_tok, cu_q, u_accept, u_sample, tau):
    """One acceptance pass over all servers.

    Row layout: server i owns logits rows cu_q[i] .. cu_q[i+1]-1 (gamma_i + 1 rows);
    row cu_q[i]+j is the target distribution of draft position j+1 (row gamma_i is
    the bonus distribution).  The per-draft arrays (q_probs rows, draft_tok,
    u_accept, ratio, p_tok) use offset cu_q[i] - i.

    Returns a dict with
      accepted [N]   a_i, number of accepted draft tokens
      out_tok  [T_q] first a_i+1 slots of each server's segment valid, rest -1
      n_out    [N]   a_i + 1
      ratio    [Gamma] min(1, p/q) of EVERY draft position (Eq. updatealpha sums to S_i)
      p_tok    [Gamma] p_j(s_j)
      margin_acc [Gamma] u_j - p/q (signed; only decisions up to the first rejection matter)
      margin_smp [N]   distance of the sampling threshold to a CDF step
      resampled  [N]   1 if the last token is a correction, 0 if it is the bonus
    """
    logits = _f64(logits)
    q_probs = _f64(q_probs)
    draft_tok, cu_q = _i64(draft_tok), _i64(cu_q)
    u_accept, u_sample = _f64(u_accept), _f64(u_sample)
    N = len(cu_q) - 1
    Tq = logits.shape[0]
    Gamma = Tq - N
    out = dict(
        accepted=np.zeros(N, np.int64), out_tok=np.full(Tq, -1, np.int64),
        n_out=np.zeros(N, np.int64), ratio=np.zeros(Gamma), p_tok=np.zeros(Gamma),
        margin_acc=np.zeros(Gamma), margin_smp=np.zeros(N), resampled=np.zeros(N, np.int64))
    for i in range(N):
        r0 = cu_q[i]
        gamma = cu_q[i + 1] - r0 - 1
        g0 = r0 - i
        m = gamma
        rejected = False
        for j in range(gamma):
            p = ref_softmax_T(logits[r0 + j], tau)
            s = draft_tok[g0 + j]
            rho = ref_ratio(p[s], q_probs[g0 + j, s])
            out["p_tok"][g0 + j] = p[s]
            out["ratio"][g0 + j] = min(1.0, rho)
            out["margin_acc"][g0 + j] = u_accept[g0 + j] - rho
            if not rejected and u_accept[g0 + j] > rho:
                m, rejected = j, True
        out["accepted"][i] = m
        out["n_out"][i] = m + 1
        out["out_tok"][r0:r0 + m] = draft_tok[g0:g0 + m]
        p = ref_softmax_T(logits[r0 + m], tau)
        if m < gamma:
            w = ref_residual(p, q_probs[g0 + m])
            out["resampled"][i] = 1
        else:
            w = p
        tok, marg = ref_inverse_cdf(w, u_sample[i])
        out["out_tok"][r0 + m] = tok
        out["margin_smp"][i] = marg
    return out


# --------------------------------------------------------------------------- #
# a4  estimators                                                               #
# --------------------------------------------------------------------------- #
def ref_ema(alpha_hat, X, ratio, accepted, cu_q, eta, beta, alpha_min=1e-3, alpha_max=0.999):
    """alpha_hat_i <- (1-eta) alpha_hat_i + eta * mean_j min(1, p_j/q_j)   (Eq. updatealpha)
    X_i         <- (1-beta) X_i + beta * (a_i + 1)                         (Eq. updateX)
    A server with gamma_i = 0 keeps its alpha_hat; alpha_hat is clamped to
    [alpha_min, alpha_max] (Assumption 2 needs alpha_hat <= alpha_max < 1).
    """
    alpha_hat, X, ratio = _f64(alpha_hat).copy(), _f64(X).copy(), _f64(ratio)
    accepted, cu_q = _i64(accepted), _i64(cu_q)
    for i in range(len(cu_q) - 1):
        gamma = cu_q[i + 1] - cu_q[i] - 1
        g0 = cu_q[i] - i
        if gamma > 0:
            obs = ratio[g0:g0 + gamma].sum() / F64(gamma)
            a = (1.0 - eta) * alpha_hat[i] + eta * obs
            alpha_hat[i] = min(max(a, alpha_min), alpha_max)
        X[i] = (1.0 - beta) * X[i] + beta * F64(accepted[i] + 1)
    return alpha_hat, X


# --------------------------------------------------------------------------- #
# a5  gradient scheduler                                                       #
# --------------------------------------------------------------------------- #
def ref_mu(alpha, S):
    """Expected tokens per round, (1 - alpha^(S+1)) / (1 - alpha)."""
    alpha = F64(alpha)
    return (1.0 - alpha ** (S + 1)) / (1.0 - alpha)


def ref_sched_objective(X, alpha_hat, S):
    """sum_i grad U_i(X_i) * x_hat_i(S_i) with U_i = log, i.e. grad = 1/X_i."""
    X, alpha_hat = _f64(X), _f64(alpha_hat)
    return float(sum(ref_mu(alpha_hat[i], int(S[i])) / X[i] for i in range(len(X))))


def ref_schedule_greedy(X, alpha_hat, C, s_min=None, s_max=None):
    """Maximise the GoodSpeed-sched objective by marginal allocation.

    The objective is separable and each term is concave in S_i, with marginal gain
    Delta_i(s) = alpha_hat_i^(s+1) / X_i for raising S_i from s to s+1.  Start at
    s_min, then hand out the remaining budget one token at a time to the largest
    marginal (lowest index on ties) among servers below s_max.  Delta_i(s+1) is
    obtained from Delta_i(s) by one multiplication with alpha_hat_i, starting from
    Delta_i(0) = alpha_hat_i / X_i, so the value sequence is reproducible bit for bit.
    """
    X, alpha_hat = _f64(X), _f64(alpha_hat)
    N = len(X)
    s_min = np.zeros(N, np.int64) if s_min is None else _i64(s_min)
    s_max = np.full(N, C, np.int64) if s_max is None else _i64(s_max)
    S = s_min.copy()
    delta = np.empty(N)
    for i in range(N):
        dlt = alpha_hat[i] / X[i]
        for _ in range(int(S[i])):
            dlt = dlt * alpha_hat[i]
        delta[i] = dlt
    budget = int(C) - int(S.sum())
    while budget > 0:
        best = -1
        for i in range(N):
            if S[i] < s_max[i] and (best < 0 or delta[i] > delta[best]):
                best = i
        if best < 0:
            break
        S[best] += 1
        delta[best] = delta[best] * alpha_hat[best]
        budget -= 1
    return S


def ref_schedule_bruteforce(X, alpha_hat, C, s_min=None, s_max=None):
    """Enumerate every feasible S (tiny N, C only); returns (best S, best objective)."""
    N = len(X)
    s_min = [0] * N if s_min is None else [int(v) for v in s_min]
    s_max = [C] * N if s_max is None else [int(v) for v in s_max]
    best, best_val = None, -np.inf
    for S in itertools.product(*[range(s_min[i], s_max[i] + 1) for i in range(N)]):
        if sum(S) > C:
            continue
        val = ref_sched_objective(X, alpha_hat, S)
        if val > best_val:
            best, best_val = S, val
    return np.array(best, np.int64), best_val


# --------------------------------------------------------------------------- #
# one whole round                                                              #
# --------------------------------------------------------------------------- #
def ref_verify_round(inp, alpha_hat, X, eta, beta, C, s_min=None, s_max=None,
                     alpha_min=1e-3, alpha_max=0.999, logits=None):
    """Attention, head, acceptance, estimator update and next allocation for one round.

    inp is a dict with Q, K, V, H, W, cu_q, cu_kv, q_probs, draft_tok, u_accept,
    u_sample, tau.  If logits is given it replaces H @ W (used where the head is
    checked separately on sampled columns).
    """
    res = {}
    res["O"] = ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
    res["logits"] = ref_lm_head(inp["H"], inp["W"]) if logits is None else _f64(logits)
    acc = ref_spec_accept(res["logits"], inp["q_probs"], inp["draft_tok"], inp["cu_q"],
                          inp["u_accept"], inp["u_sample"], inp["tau"])
    res.update(acc)
    res["alpha_hat"], res["X"] = ref_ema(alpha_hat, X, acc["ratio"], acc["accepted"],
                                         inp["cu_q"], eta, beta, alpha_min, alpha_max)
    res["S_next"] = ref_schedule_greedy(res["X"], res["alpha_hat"], C, s_min, s_max)
    return res
