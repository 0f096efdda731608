"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these re-types an oracle formula: each uses a closed form, an invariant,
a special case with a known answer, exact rational arithmetic, or brute force.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import goodspeed_oracle as orc


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ attention
def _ragged(gammas, prefixes):
    n_new = np.asarray(gammas) + 1
    cu_q = np.concatenate([[0], np.cumsum(n_new)])
    cu_kv = np.concatenate([[0], np.cumsum(np.asarray(prefixes) + n_new)])
    return cu_q, cu_kv


def test_attention_zero_query_is_mean_of_visible_values():
    """Q = 0 gives uniform weights, so row t equals the mean of exactly the first
    L_i + t + 1 value rows of ITS server: pins the causal count, the per-server
    key offset and the kv-head mapping."""
    r = rng(1)
    gam, pre = [0, 2, 3], [5, 1, 4]
    cu_q, cu_kv = _ragged(gam, pre)
    Hq, Hkv, hd = 4, 2, 8
    Q = np.zeros((cu_q[-1], Hq, hd))
    K = r.standard_normal((cu_kv[-1], Hkv, hd))
    V = r.standard_normal((cu_kv[-1], Hkv, hd))
    O = orc.ref_attention(Q, K, V, cu_q, cu_kv)
    for i in range(3):
        for t in range(gam[i] + 1):
            for h in range(Hq):
                want = V[cu_kv[i]:cu_kv[i] + pre[i] + t + 1, h // 2, :].mean(axis=0)
                np.testing.assert_allclose(O[cu_q[i] + t, h], want, rtol=0, atol=1e-13)


def test_attention_sharp_scores_select_one_key():
    """Keys are scaled one-hot directions; a query aligned with direction c makes the
    softmax collapse on the single visible key carrying c, so O is that key's value."""
    hd, L = 16, 10
    cu_q, cu_kv = _ragged([2], [L])
    K = np.zeros((L + 3, 1, hd))
    for k in range(L + 3):
        K[k, 0, k % hd] = 1.0
    V = rng(2).standard_normal((L + 3, 1, hd))
    Q = np.zeros((3, 2, hd))
    Q[0, 0, 3] = 4000.0   # key 3 (prefix)
    Q[1, 1, 11] = 4000.0  # key 11 = second new position, visible to t=1
    Q[2, 0, 12] = 4000.0  # key 12 = own position of t=2
    O = orc.ref_attention(Q, K, V, cu_q, cu_kv)
    np.testing.assert_allclose(O[0, 0], V[3, 0], atol=1e-12)
    np.testing.assert_allclose(O[1, 1], V[11, 0], atol=1e-12)
    np.testing.assert_allclose(O[2, 0], V[12, 0], atol=1e-12)
    # t = 0 may not see key 11 (a later draft position): weight stays uniform over 0..10.
    Q2 = np.zeros((3, 2, hd))
    Q2[0, 0, 11] = 4000.0
    O2 = orc.ref_attention(Q2, K, V, cu_q, cu_kv)
    np.testing.assert_allclose(O2[0, 0], V[:11, 0].mean(axis=0), atol=1e-12)


def test_attention_two_key_closed_form_and_scale():
    """One query over two keys: weight on key 0 is sigmoid(scale * (q.k0 - q.k1))."""
    hd = 4
    cu_q, cu_kv = _ragged([0], [1])  # prefix 1 + own position = 2 keys
    q = np.array([0.3, -1.2, 0.5, 2.0])
    K = np.array([[0.1, 0.2, 0.3, 0.4], [1.0, -1.0, 0.5, 0.25]]).reshape(2, 1, hd)
    V = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]]).reshape(2, 1, hd)
    O = orc.ref_attention(q.reshape(1, 1, hd), K, V, cu_q, cu_kv)
    d = (q @ K[0, 0] - q @ K[1, 0]) / np.sqrt(hd)   # default scale 1/sqrt(hd)
    w0 = 1.0 / (1.0 + np.exp(-d))
    np.testing.assert_allclose(O[0, 0], [w0, 1 - w0, 0, 0], atol=1e-14)
    O3 = orc.ref_attention(q.reshape(1, 1, hd), K, V, cu_q, cu_kv, scale=3.0)
    w0 = 1.0 / (1.0 + np.exp(-3.0 * (q @ K[0, 0] - q @ K[1, 0])))
    np.testing.assert_allclose(O3[0, 0], [w0, 1 - w0, 0, 0], atol=1e-14)


def test_attention_causality_and_server_isolation():
    r = rng(3)
    gam, pre = [3, 2], [6, 7]
    cu_q, cu_kv = _ragged(gam, pre)
    Q = r.standard_normal((cu_q[-1], 4, 8))
    K = r.standard_normal((cu_kv[-1], 2, 8))
    V = r.standard_normal((cu_kv[-1], 2, 8))
    O = orc.ref_attention(Q, K, V, cu_q, cu_kv)
    K2, V2 = K.copy(), V.copy()
    last = cu_kv[1] - 1          # server 0's last new position
    K2[last] += 5.0
    V2[last] -= 3.0
    O2 = orc.ref_attention(Q, K2, V2, cu_q, cu_kv)
    assert np.array_equal(O[:3], O2[:3])          # earlier queries unchanged, bit for bit
    assert not np.allclose(O[3], O2[3])           # the last one sees it
    assert np.array_equal(O[4:], O2[4:])          # other server untouched
    # constant values -> output is that constant (weights sum to one)
    Vc = np.broadcast_to(r.standard_normal((1, 2, 8)), V.shape)
    Oc = orc.ref_attention(Q, K, Vc, cu_q, cu_kv)
    for h in range(4):
        np.testing.assert_allclose(Oc[:, h], np.broadcast_to(Vc[0, h // 2], (cu_q[-1], 8)), atol=1e-13)


# -------------------------------------------------------------------- LM head
def test_lm_head_selection_matrix_and_python_loops():
    r = rng(4)
    T, d, V = 3, 5, 7
    H = r.standard_normal((T, d))
    W = np.zeros((d, V))
    picks = [4, 0, 2, 2, 1, 3, 0]                 # column v copies hidden component picks[v]
    for v, c in enumerate(picks):
        W[c, v] = 1.0
    np.testing.assert_array_equal(orc.ref_lm_head(H, W), H[:, picks])
    W = r.standard_normal((d, V))
    want = [[sum(float(H[t, c]) * float(W[c, v]) for c in range(d)) for v in range(V)] for t in range(T)]
    np.testing.assert_allclose(orc.ref_lm_head(H, W), want, rtol=1e-14)
    np.testing.assert_allclose(orc.ref_lm_head(H, W, cols=[6, 1]), np.asarray(want)[:, [6, 1]], rtol=1e-14)


def test_dequant_w4_hand_written_words():
    """The 4-bit weight format on words written out by hand: nibble n of a word holds the code of row
    offset j with n = (j >> 1) + 4 (j & 1), so 0x76543210 (nibble n holds n) reads, in row order,
    0 4 1 5 2 6 3 7.  Two groups of 8 rows with different scales and zero points, two columns."""
    qweight = np.array([[0x76543210, 0xFFFF0000],
                        [0x89ABCDEF, 0x00000001]], dtype=np.uint32).view(np.int32)
    scales = np.array([[0.5, 2.0], [0.25, 1.0]])
    zeros = np.array([[3, 8], [8, 0]], dtype=np.uint8)
    W = orc.ref_dequant_w4(qweight, scales, zeros, group=8)
    assert W.shape == (16, 2)
    np.testing.assert_array_equal(W[:8, 0], [-1.5, 0.5, -1.0, 1.0, -0.5, 1.5, 0.0, 2.0])       # 0.5 (code - 3)
    np.testing.assert_array_equal(W[8:, 0], [1.75, 0.75, 1.5, 0.5, 1.25, 0.25, 1.0, 0.0])      # 0.25 ((15 11 14 10 13 9 12 8) - 8)
    np.testing.assert_array_equal(W[:8, 1], [-16.0, 14.0] * 4)                                 # 2 ((0 15 0 15 ...) - 8)
    np.testing.assert_array_equal(W[8:, 1], [1.0, 0, 0, 0, 0, 0, 0, 0])
    # the head on it is the plain product with the dequantised weight
    H = rng(21).standard_normal((3, 16))
    np.testing.assert_allclose(orc.ref_lm_head(H, W), H @ W, rtol=1e-14)


# -------------------------------------------------------------------- softmax
def test_softmax_closed_forms():
    p = orc.ref_softmax_T(np.array([1.5, -0.5]), 0.5)
    np.testing.assert_allclose(p[0], 1 / (1 + np.exp(-(1.5 + 0.5) / 0.5)), rtol=1e-15)
    x = rng(5).standard_normal(50)
    for tau in (0.3, 0.7, 1.0, 2.5):
        p = orc.ref_softmax_T(x, tau)
        assert abs(p.sum() - 1) < 1e-14
        np.testing.assert_allclose(orc.ref_softmax_T(x + 123.0, tau), p, rtol=1e-12)
        # log-odds of any pair equal the logit gap over tau
        np.testing.assert_allclose(np.log(p[3] / p[17]), (x[3] - x[17]) / tau, rtol=1e-12)
    p0 = orc.ref_softmax_T(x, 0.0)
    assert p0.sum() == 1.0 and p0[np.argmax(x)] == 1.0
    np.testing.assert_allclose(orc.ref_softmax_T(x, 1e-4), p0, atol=1e-12)  # tau -> 0+ limit
    xt = np.array([0.0, 2.0, 2.0, 1.0])
    assert orc.ref_softmax_T(xt, 0.0)[1] == 1.0     # lowest index on ties


# ------------------------------------------------------------- accept / sample
def _one_server(p_rows, q_rows, toks, u_acc, u_smp, tau=1.0):
    logits = np.log(np.asarray(p_rows, dtype=np.float64))
    gamma = len(toks)
    cu_q = np.array([0, gamma + 1])
    return orc.ref_spec_accept(logits, np.asarray(q_rows, dtype=np.float64).reshape(gamma, -1),
                               np.asarray(toks), cu_q, np.asarray(u_acc), np.asarray([u_smp]), tau)


def test_accept_hand_worked_case():
    """p1=(.5,.3,.2) q1=(.2,.6,.2): token 1 has ratio 0.5.  u=.4 accepts, u=.6 rejects and the
    correction distribution is max(0,p-q)=(.3,0,0)/.3 -> always token 0."""
    p1, q1 = [0.5, 0.3, 0.2], [0.2, 0.6, 0.2]
    p2 = [0.1, 0.1, 0.8]
    acc = _one_server([p1, p2], [q1], [1], [0.4], 0.15)
    assert acc["accepted"][0] == 1 and acc["n_out"][0] == 2
    assert list(acc["out_tok"]) == [1, 1]             # bonus from p2: cdf .1,.2,1 -> u=.15 -> token 1
    np.testing.assert_allclose(acc["ratio"], [0.5], rtol=1e-12)
    np.testing.assert_allclose(acc["p_tok"], [0.3], rtol=1e-12)
    assert acc["resampled"][0] == 0
    rej = _one_server([p1, p2], [q1], [1], [0.6], 0.999)
    assert rej["accepted"][0] == 0 and list(rej["out_tok"]) == [0, -1] and rej["resampled"][0] == 1
    # boundary: u == ratio accepts (r_j <= p/q)
    rho = float(acc["ratio"][0])                      # 0.5 up to the rounding of exp(log(.))
    eq = _one_server([p1, p2], [q1], [1], [rho], 0.5)
    assert eq["accepted"][0] == 1
    above = _one_server([p1, p2], [q1], [1], [np.nextafter(rho, 1.0)], 0.5)
    assert above["accepted"][0] == 0
    # token 0 has ratio 2.5 -> clipped to 1 in the estimator input, always accepted
    up = _one_server([p1, p2], [q1], [0], [0.999999], 0.5)
    assert up["accepted"][0] == 1 and up["ratio"][0] == 1.0


def test_accept_stops_at_first_rejection_but_rates_cover_all_positions():
    p = [[0.25, 0.75], [0.5, 0.5], [0.9, 0.1], [0.5, 0.5]]
    q = [[0.5, 0.5], [0.5, 0.5], [0.3, 0.7]]
    out = _one_server(p, q, [0, 1, 1], [0.9, 0.2, 0.0001], 0.3)   # ratios .5, 1, 1/7
    assert out["accepted"][0] == 0                               # first is rejected (0.9 > 0.5)
    np.testing.assert_allclose(out["ratio"], [0.5, 1.0, 0.1 / 0.7], rtol=1e-12)
    out = _one_server(p, q, [0, 1, 1], [0.4, 0.99, 0.5], 0.3)
    assert out["accepted"][0] == 2 and list(out["out_tok"][:2]) == [0, 1]
    # correction at position 3: max(0,(.9,.1)-(.3,.7)) = (.6,0) -> token 0
    assert out["out_tok"][2] == 0 and out["out_tok"][3] == -1


def test_identical_draft_is_always_accepted_and_bounds():
    r = rng(6)
    V, gam = 11, [0, 1, 4, 2]
    cu_q = np.concatenate([[0], np.cumsum(np.asarray(gam) + 1)])
    logits = r.standard_normal((cu_q[-1], V))
    tau = 0.7
    q = np.stack([orc.ref_softmax_T(logits[cu_q[i] + j], tau) for i in range(4) for j in range(gam[i])])
    tok = r.integers(0, V, size=sum(gam))
    out = orc.ref_spec_accept(logits, q, tok, cu_q, r.uniform(0, 1, sum(gam)), r.uniform(0, 1, 4), tau)
    assert list(out["accepted"]) == gam
    assert np.all(out["resampled"] == 0)
    # random drafts: 0 <= a_i <= gamma_i, ids in range, n_out = a+1, valid slots only
    q = r.dirichlet(np.ones(V), size=sum(gam))
    out = orc.ref_spec_accept(logits, q, tok, cu_q, r.uniform(0, 1, sum(gam)), r.uniform(0, 1, 4), tau)
    for i in range(4):
        a = out["accepted"][i]
        assert 0 <= a <= gam[i] and out["n_out"][i] == a + 1
        seg = out["out_tok"][cu_q[i]:cu_q[i + 1]]
        assert np.all((seg[:a + 1] >= 0) & (seg[:a + 1] < V)) and np.all(seg[a + 1:] == -1)


def test_temperature_zero_is_greedy_prefix_match():
    r = rng(7)
    V = 9
    for trial in range(40):
        gam = [int(g) for g in r.integers(0, 5, size=3)]
        cu_q = np.concatenate([[0], np.cumsum(np.asarray(gam) + 1)])
        logits = r.standard_normal((cu_q[-1], V))
        greedy = logits.argmax(axis=1)
        q = r.dirichlet(np.ones(V), size=sum(gam)) if sum(gam) else np.zeros((0, V))
        tok = []
        for i in range(3):      # drafts agree with greedy for a random prefix, then deviate
            agree = r.integers(0, gam[i] + 1)
            for j in range(gam[i]):
                g = greedy[cu_q[i] + j]
                tok.append(g if j < agree else (g + 1 + r.integers(0, V - 1)) % V)
        tok = np.asarray(tok, dtype=np.int64)
        out = orc.ref_spec_accept(logits, q, tok, cu_q, r.uniform(0, 1, sum(gam)), r.uniform(0, 1, 3), 0.0)
        for i in range(3):
            g0 = cu_q[i] - i
            match = 0
            while match < gam[i] and tok[g0 + match] == greedy[cu_q[i] + match]:
                match += 1
            assert out["accepted"][i] == match
            assert out["out_tok"][cu_q[i] + match] == greedy[cu_q[i] + match]


def test_zero_draft_probability_convention():
    out = _one_server([[0.5, 0.5], [0.5, 0.5]], [[1.0, 0.0]], [1], [0.99], 0.1)
    assert out["accepted"][0] == 1 and out["ratio"][0] == 1.0       # p>0, q=0: accept
    logits = np.array([[0.0, -np.inf], [0.0, 0.0]])
    out = orc.ref_spec_accept(logits, np.array([[1.0, 0.0]]), np.array([1]), np.array([0, 2]),
                              np.array([1e-9]), np.array([0.5]), 1.0)
    assert out["accepted"][0] == 0 and out["ratio"][0] == 0.0       # p=0, q=0: reject


def test_inverse_cdf_convention():
    w = np.array([0.0, 0.2, 0.0, 0.3, 0.5, 0.0])
    assert orc.ref_inverse_cdf(w, 0.0)[0] == 1          # zero-mass token 0 can never be drawn
    assert orc.ref_inverse_cdf(w, 0.1999)[0] == 1
    assert orc.ref_inverse_cdf(w, 0.2)[0] == 3          # strict >: exactly on a step moves on
    assert orc.ref_inverse_cdf(w, 0.4999)[0] == 3
    assert orc.ref_inverse_cdf(w, 0.9999999)[0] == 4    # trailing zero-mass token never drawn
    v, m = orc.ref_inverse_cdf(w, 0.35)
    assert v == 3 and abs(m - 0.15) < 1e-12
    # scale invariance: unnormalised weights give the same draw
    assert orc.ref_inverse_cdf(7.0 * w, 0.35)[0] == 3


def test_inverse_cdf_without_an_index_takes_the_last_token_with_mass():
    """Threshold at (or, by rounding, beyond) the total mass: no prefix sum exceeds it, and the draw
    is the last token that has mass, never a trailing zero-mass token.  Expected values by hand."""
    w = np.array([0.0, 0.2, 0.0, 0.3, 0.5, 0.0])           # prefix sums .0 .2 .2 .5 1. 1.: none > 1.0
    v, m = orc.ref_inverse_cdf(w, 1.0)
    assert v == 4 and m == 0.0
    assert orc.ref_inverse_cdf(np.array([3.0, 1.0, 0.0, 0.0]), 1.0)[0] == 1
    assert orc.ref_inverse_cdf(np.array([0.0, 0.0, 2.0]), 1.0)[0] == 2
    # a threshold beyond the total (u > 1 stands in for rounding) behaves the same
    assert orc.ref_inverse_cdf(w, 1.0 + 1e-9)[0] == 4


def test_residual_without_mass_falls_back_to_the_target_distribution():
    """A draft row with q >= p everywhere leaves max(0, p - q) without mass; the correction token is
    then drawn from p itself.  q = 1.5 p (unnormalised on purpose) gives ratio 2/3 for every token."""
    p = np.array([0.2, 0.3, 0.5])
    q = 1.5 * p
    np.testing.assert_array_equal(orc.ref_residual(p, q), p)
    np.testing.assert_array_equal(orc.ref_residual(p, p), p)           # q == p: the same fall-back
    # one element with mass left: the ordinary residual, not the fall-back
    np.testing.assert_allclose(orc.ref_residual(p, np.array([0.3, 0.45, 0.4])), [0.0, 0.0, 0.1], atol=1e-15)
    # through the whole acceptance pass: u_accept = 0.9 > 2/3 rejects the first draft token, and the
    # correction token follows p's CDF (.2, .5, 1.)
    p2 = [0.6, 0.3, 0.1]
    for u_smp, want in ((0.1, 0), (0.35, 1), (0.6, 2), (0.999, 2)):
        out = _one_server([p, p2], [q], [1], [0.9], u_smp)
        assert out["accepted"][0] == 0 and out["resampled"][0] == 1
        np.testing.assert_allclose(out["ratio"], [2.0 / 3.0], rtol=1e-12)
        assert list(out["out_tok"]) == [want, -1]
    # u_accept below 2/3 accepts and the bonus token comes from the second row
    out = _one_server([p, p2], [q], [1], [0.6], 0.65)
    assert out["accepted"][0] == 1 and list(out["out_tok"]) == [1, 1]


def _exact_output_law(p1, q1, p2_of, q2_of, V):
    """P(first output token = x) and P(s1 accepted, second output token = y), obtained by
    integrating the oracle's own decisions over the uniforms exactly: accept has measure
    min(1, ratio); the correction draw has the measure of each token's CDF interval."""
    first = np.zeros(V)
    second = np.zeros((V, V))
    for s1 in range(V):
        if q1[s1] == 0:
            continue
        acc1 = min(1.0, orc.ref_ratio(p1[s1], q1[s1]))
        first[s1] += q1[s1] * acc1
        res = orc.ref_residual(p1, q1)
        first += q1[s1] * (1 - acc1) * res / res.sum()
        p2, q2 = p2_of[s1], q2_of[s1]
        for s2 in range(V):
            if q2[s2] == 0:
                continue
            acc2 = min(1.0, orc.ref_ratio(p2[s2], q2[s2]))
            second[s1, s2] += q1[s1] * acc1 * q2[s2] * acc2
            res2 = orc.ref_residual(p2, q2)
            second[s1] += q1[s1] * acc1 * q2[s2] * (1 - acc2) * res2 / res2.sum()
    return first, second


@pytest.mark.parametrize("V", [2, 3, 5])
def test_output_distribution_equals_target_exactly(V):
    r = rng(100 + V)
    for trial in range(20):
        p1, q1 = r.dirichlet(np.ones(V)), r.dirichlet(np.ones(V))
        if trial % 4 == 0:
            q1[r.integers(V)] = 0.0
            q1 /= q1.sum()
        p2_of, q2_of = r.dirichlet(np.ones(V), size=V), r.dirichlet(np.ones(V), size=V)
        first, second = _exact_output_law(p1, q1, p2_of, q2_of, V)
        np.testing.assert_allclose(first, p1, atol=1e-12)
        # given the first draft token x was accepted, the next output follows p2(.|x)
        p_acc = np.array([min(p1[x], q1[x]) for x in range(V)])
        np.testing.assert_allclose(second, p_acc[:, None] * p2_of, atol=1e-12)


def test_output_distribution_through_full_oracle_on_uniform_grid():
    """Same claim through ref_spec_accept itself: a stratified grid over (u_accept, u_sample)
    for every draft token weighted by q; the histogram matches p within the grid error."""
    r = rng(11)
    V, K = 4, 256
    p1, q1 = r.dirichlet(np.ones(V)), r.dirichlet(np.ones(V))
    p2 = r.dirichlet(np.ones(V))
    logits = np.log(np.stack([p1, p2]))
    grid = (np.arange(K) + 0.5) / K
    hist = np.zeros(V)
    acc_rate = 0.0
    for s in range(V):
        for ua in grid:
            # the draw is piecewise constant in u_sample: evaluate the K strata at once
            for us in grid[:: K // 32]:
                o = orc.ref_spec_accept(logits, q1[None, :], np.array([s]), np.array([0, 2]),
                                        np.array([ua]), np.array([us]), 1.0)
                hist[o["out_tok"][0]] += q1[s] / (K * 32)
            acc_rate += q1[s] * o["ratio"][0] / K
    np.testing.assert_allclose(hist, p1, atol=2.0 * V / 32)
    # expected clipped ratio under s ~ q is the overlap sum_v min(p, q)  (definition of alpha)
    np.testing.assert_allclose(acc_rate, np.minimum(p1, q1).sum(), atol=1e-12)


# ------------------------------------------------------------------ estimators
def test_mu_is_capped_geometric_series():
    for a, S in [(Fraction(1, 2), 3), (Fraction(9, 10), 7), (Fraction(1, 3), 0), (Fraction(4, 5), 16)]:
        exact = sum(a ** k for k in range(S + 1))
        assert abs(orc.ref_mu(float(a), S) - float(exact)) < 1e-13
    assert abs(orc.ref_mu(0.5, 3) - 1.875) < 1e-15
    # Monte-Carlo: tokens produced = accepted run (each accept w.p. alpha, at most S) + 1
    r = rng(12)
    alpha, S, n = 0.7, 5, 200_000
    acc = r.uniform(size=(n, S)) < alpha
    produced = np.where(acc.all(axis=1), S, np.argmin(acc, axis=1)) + 1
    assert abs(produced.mean() - orc.ref_mu(alpha, S)) < 4 * produced.std() / np.sqrt(n)


def test_ema_closed_form_and_conventions():
    cu_q = np.array([0, 3, 4])           # gamma = 2, 0
    ratio = np.array([0.25, 0.75])
    a_hat, X = np.array([0.9, 0.4]), np.array([2.0, 5.0])
    eta, beta = 0.1, 0.5
    for t in range(1, 30):
        a_hat, X = orc.ref_ema(a_hat, X, ratio, np.array([1, 0]), cu_q, eta, beta)
        np.testing.assert_allclose(a_hat[0], 0.5 + (1 - eta) ** t * (0.9 - 0.5), rtol=1e-12)
        np.testing.assert_allclose(X[0], 2.0, rtol=1e-12)                       # a+1 = 2 = X(0)
        np.testing.assert_allclose(X[1], 1.0 + (1 - beta) ** t * (5.0 - 1.0), rtol=1e-12)
        assert a_hat[1] == 0.4                                                  # gamma = 0: untouched
    a_hat, _ = orc.ref_ema(np.array([0.999]), np.array([1.0]), np.array([1.0]), np.array([1]),
                           np.array([0, 2]), 0.5, 0.5)
    assert a_hat[0] == 0.999                                                    # clamp at alpha_max
    a_hat, _ = orc.ref_ema(np.array([0.001]), np.array([1.0]), np.array([0.0]), np.array([0]),
                           np.array([0, 2]), 0.5, 0.5)
    assert a_hat[0] == 0.001


# ------------------------------------------------------------------- scheduler
def test_objective_matches_rational_arithmetic():
    X = [Fraction(3, 2), Fraction(5, 4)]
    al = [Fraction(1, 2), Fraction(3, 4)]
    S = [2, 3]
    exact = sum(sum(al[i] ** k for k in range(S[i] + 1)) / X[i] for i in range(2))
    got = orc.ref_sched_objective([float(x) for x in X], [float(a) for a in al], S)
    assert abs(got - float(exact)) < 1e-14


@pytest.mark.parametrize("N,C", [(2, 5), (3, 6), (4, 8), (4, 3)])
def test_greedy_matches_brute_force(N, C):
    r = rng(1000 * N + C)
    for trial in range(25):
        X = r.uniform(0.5, 6.0, N)
        al = r.uniform(0.05, 0.98, N)
        S = orc.ref_schedule_greedy(X, al, C)
        Sb, best = orc.ref_schedule_bruteforce(X, al, C)
        assert S.sum() == C and np.all(S >= 0)
        assert abs(orc.ref_sched_objective(X, al, S) - best) <= 1e-12 * abs(best)
        if trial % 3 == 0:      # box constraints
            lo = r.integers(0, 2, N)
            hi = lo + r.integers(0, 3, N)
            S = orc.ref_schedule_greedy(X, al, C, lo, hi)
            if lo.sum() <= C:
                Sb, best = orc.ref_schedule_bruteforce(X, al, C, lo, hi)
                assert np.all(S >= lo) and np.all(S <= hi) and S.sum() <= C
                assert abs(orc.ref_sched_objective(X, al, S) - best) <= 1e-12 * abs(best)


def test_scheduler_special_cases():
    # identical servers: the uniform split (the Fixed-S policy, S_i = C/N)
    S = orc.ref_schedule_greedy(np.full(4, 2.0), np.full(4, 0.8), 12)
    assert list(S) == [3, 3, 3, 3]
    # remainder goes to the lowest indices
    assert list(orc.ref_schedule_greedy(np.full(4, 2.0), np.full(4, 0.8), 14)) == [4, 4, 3, 3]
    # scaling every X by a constant does not move the allocation
    r = rng(13)
    X, al = r.uniform(1, 6, 8), r.uniform(0.3, 0.95, 8)
    assert np.array_equal(orc.ref_schedule_greedy(X, al, 40), orc.ref_schedule_greedy(8.0 * X, al, 40))
    # a starved server (X -> 0+) is served first and most
    X2 = X.copy()
    X2[5] = 1e-9
    S2 = orc.ref_schedule_greedy(X2, al, 40)
    assert S2[5] == S2.max() and S2[5] > orc.ref_schedule_greedy(X, al, 40)[5]
    # with budget 1 the token goes to argmax alpha_i / X_i
    assert np.argmax(orc.ref_schedule_greedy(X, al, 1)) == np.argmax(al / X)
    # caps bind: everyone at s_max leaves budget unspent
    S = orc.ref_schedule_greedy(X, al, 100, np.zeros(8, int), np.full(8, 3))
    assert list(S) == [3] * 8
    # marginal gains really are alpha^(s+1)/X: objective increments along the greedy path
    Xs, als = np.array([1.3, 2.1]), np.array([0.9, 0.6])
    prev = orc.ref_sched_objective(Xs, als, [0, 0])
    Sprev = np.zeros(2, int)
    for c in range(1, 8):
        S = orc.ref_schedule_greedy(Xs, als, c)
        i = int(np.argmax(S - Sprev))
        cur = orc.ref_sched_objective(Xs, als, S)
        np.testing.assert_allclose(cur - prev, als[i] ** (Sprev[i] + 1) / Xs[i], rtol=1e-10)
        prev, Sprev = cur, S


def test_closed_loop_beats_fixed_and_random_allocation():
    """Heterogeneous stationary acceptance rates: after a few hundred rounds the utility of the
    time-averaged goodput under the gradient scheduler is at least that of Fixed-S and Random-S
    (the qualitative outcome of the paper's utility-convergence experiment)."""
    r = rng(14)
    N, C, T = 8, 32, 600
    alpha = np.array([0.95, 0.9, 0.85, 0.8, 0.6, 0.5, 0.35, 0.2])

    def run(policy):
        a_hat, X = np.full(N, 0.5), np.ones(N)
        S = np.full(N, C // N)
        tot = np.zeros(N)
        rr = np.random.default_rng(99)
        for t in range(T):
            acc = np.zeros(N, int)
            ratios = []
            for i in range(N):
                ok = rr.uniform(size=S[i]) < alpha[i]
                acc[i] = S[i] if ok.all() else int(np.argmin(ok))
                ratios.append(np.full(S[i], alpha[i]))   # observed clipped ratios average alpha_i
            cu_q = np.concatenate([[0], np.cumsum(S + 1)])
            a_hat, X = orc.ref_ema(a_hat, X, np.concatenate(ratios) if S.sum() else np.zeros(0),
                                   acc, cu_q, 0.1, 0.05)
            tot += acc + 1
            if policy == "goodspeed":
                S = orc.ref_schedule_greedy(X, a_hat, C)
            elif policy == "random":
                cuts = np.sort(rr.integers(0, C + 1, N - 1))
                S = np.diff(np.concatenate([[0], cuts, [C]]))
            # fixed: unchanged
        return np.log(tot / T).sum()

    u_gs, u_fix, u_rnd = run("goodspeed"), run("fixed"), run("random")
    assert u_gs >= u_fix - 1e-9 and u_gs >= u_rnd - 1e-9
