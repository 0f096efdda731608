"""Parity of the CUDA library (through its C ABI) against the fp64 CPU oracle on the same seeded
inputs.  Small cases compare every element; the full-size configurations compare everything the
oracle can compute in seconds (attention and acceptance in full, the LM head on sampled columns
plus the complete chain where the host has the memory for it)."""
import numpy as np
import pytest
import torch

from oracle import goodspeed_oracle as orc
from paper_2512_09963_b200 import binding as B
from paper_2512_09963_b200 import workloads as wl
from paper_2512_09963_b200.runner import VerifyRound

import parity_utils as pu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def to_dev(inp):
    return {k: (v.to(DEV) if isinstance(v, torch.Tensor) else v) for k, v in inp.items()}


def tau32(tau):
    """The library takes the temperature as fp32; the oracle gets the same value."""
    return float(np.float32(tau))


def run_accept_only(inp, update=False):
    """spec_accept on the generator's fp32 logits: both sides read identical logits."""
    d = to_dev(inp)
    logits = d["target_logits_f32"].contiguous()
    Tq, V = logits.shape
    N = d["cu_q"].numel() - 1
    rnd = VerifyRound(N=N, Tq=Tq, total_kv=1, max_kv_len=1, Hq=1, Hkv=1, hd=8, d=8, V=V,
                      dtype=torch.float32, C=0, device=DEV)
    rnd.accept(d["q_probs"], d["draft_tok"], d["cu_q"], d["u_accept"], d["u_sample"], inp["tau"],
               logits=logits, update=update)
    torch.cuda.synchronize()
    assert int(rnd.d_status.item()) == 0
    return rnd


def check_accept(inp, rnd):
    tau = tau32(inp["tau"])
    ref = orc.ref_spec_accept(inp["target_logits_f32"], inp["q_probs"], inp["draft_tok"], inp["cu_q"],
                              inp["u_accept"], inp["u_sample"], tau)
    log = pu.compare_accept(pu.gpu_accept_dict(rnd), ref, inp["target_logits_f32"], inp["q_probs"],
                            inp["cu_q"].cpu().numpy(), inp["u_sample"], tau, inp["target_logits_f32"].shape[1])
    return ref, log


# ------------------------------------------------------------------ cfg1: the whole round
@pytest.mark.parametrize("tau", [1.0, 0.0])
def test_cfg1_full_round(tau):
    cfg = wl.CONFIGS["cfg1"]
    inp = wl.make_step(cfg, tau=tau)
    d = to_dev(inp)
    rnd = VerifyRound.for_inputs(d, C=10)
    rnd.run(d)
    torch.cuda.synchronize()
    assert int(rnd.d_status.item()) == 0
    ref = orc.ref_verify_round(inp, np.full(cfg.N, 0.5), np.ones(cfg.N), 0.1, 0.5, 10)
    pu.assert_close_rel(rnd.O, ref["O"], "attention output")
    pu.assert_close_rel(rnd.logits, ref["logits"], "logits")
    log = pu.compare_accept(pu.gpu_accept_dict(rnd), ref, ref["logits"], inp["q_probs"],
                            inp["cu_q"].numpy(), inp["u_sample"], tau32(tau), cfg.V)
    assert not log["accept_near_ties"] and not log["sample_near_ties"], log
    np.testing.assert_allclose(rnd.alpha_hat.cpu().numpy(), ref["alpha_hat"], atol=1e-6)
    np.testing.assert_allclose(rnd.X.cpu().numpy(), ref["X"], atol=1e-12)
    assert np.array_equal(rnd.S_next.cpu().numpy(), ref["S_next"])
    # fp32 path: far tighter than the bf16 bar
    pu.assert_close_rel(rnd.logits, ref["logits"], "logits (fp32 bar)", rel=1e-4)
    pu.assert_close_rel(rnd.O, ref["O"], "attention (fp32 bar)", rel=1e-4)


def test_cfg1_matches_stored_golden():
    """The oracle-written fixture (tests/golden) and the library agree on the integer outputs."""
    import json, os
    path = os.path.join(os.path.dirname(__file__), "golden", "cfg1_round.json")
    gold = json.load(open(path))
    for tau_key, tau in (("tau1", 1.0), ("tau0", 0.0)):
        inp = wl.make_step(wl.CONFIGS["cfg1"], tau=tau)
        d = to_dev(inp)
        rnd = VerifyRound.for_inputs(d, C=10)
        rnd.run(d)
        torch.cuda.synchronize()
        assert rnd.accepted.cpu().tolist() == gold[tau_key]["accepted"]
        assert rnd.out_tok.cpu().tolist() == gold[tau_key]["out_tok"]
        assert rnd.S_next.cpu().tolist() == gold[tau_key]["S_next"]


def test_round_without_dependent_launch_is_bit_identical():
    """Programmatic dependent launch only moves kernel start-up earlier: a whole round (split
    attention with tickets included) gives the same bits with the attribute switched off."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=256, V=8192, prefix_scale=0.25, name="round_pdl")
    inp = wl.make_step(cfg)
    d = to_dev(inp)
    B.gs_verify_attn_configure(2)                 # two-tile splits: partial results, tickets, merges
    try:
        outs = []
        for on in (True, False):
            B.gs_set_dependent_launch(on)
            rnd = VerifyRound.for_inputs(d, C=4 * cfg.N)
            rnd.run(d, fused=True)
            torch.cuda.synchronize()
            assert int(rnd.d_status.item()) == 0
            outs.append({k: getattr(rnd, k).clone() for k in ("O", "logits", "accepted", "out_tok", "ratio", "S_next")})
    finally:
        B.gs_set_dependent_launch(True)
        B.gs_verify_attn_configure(0)
    for k in outs[0]:
        assert torch.equal(outs[0][k], outs[1][k]), k
    pu.assert_close_rel(outs[0]["O"], orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "attention")


# ------------------------------------------------------------------ spec_accept
ACCEPT_CASES = [
    # name, base cfg, V, tau   (V spans several 4096-chunks plus a ragged tail, or breaks the 16-byte path)
    ("cfg2-shaped", "cfg2", 20000, 0.7),
    ("cfg3-shaped", "cfg3", 12000, 1.0),
    ("cfg4-shaped", "cfg4", 9000, 1.0),
    ("odd-V", "cfg2", 4099, 0.7),
    ("tiny-V", "cfg2", 5, 1.0),
    ("greedy", "cfg3", 12000, 0.0),
    ("cold", "cfg4", 8192, 0.05),
]


@pytest.fixture(params=[0, 1], ids=["cluster-finish", "ticket-finish"])
def finish_variant(request):
    """Both second-pass kernels of gs_spec_accept: a cluster per server (where the shape allows
    it) and the ticket kernel."""
    B.gs_spec_accept_select(request.param)
    yield request.param
    B.gs_spec_accept_select(0)


@pytest.mark.parametrize("name,base,V,tau", ACCEPT_CASES + [("two-slices", "cfg2", 8, 1.0),
                                                            ("ragged-slices", "cfg3", 30004, 0.7)])
def test_spec_accept_small(name, base, V, tau, finish_variant):
    cfg = wl.shrink(wl.CONFIGS[base], V=V, d=64, prefix_scale=0.01, name=f"{base}_acc_{V}")
    inp = wl.make_step(cfg, tau=tau, synthetic_logits=True, allocator=orc.ref_schedule_greedy)
    rnd = run_accept_only(inp)
    ref, log = check_accept(inp, rnd)
    # identical logits on both sides: flips must be rare
    assert len(log["accept_near_ties"]) <= 1
    assert len(log["sample_near_ties"]) <= max(1, cfg.N // 8)
    # run it again: bit-identical outputs (fixed summation order, no float atomics)
    first = {k: v.copy() for k, v in pu.gpu_accept_dict(rnd).items()}
    rnd2 = run_accept_only(inp)
    for k, v in pu.gpu_accept_dict(rnd2).items():
        assert np.array_equal(v, first[k]), k


def test_spec_accept_without_dependent_launch():
    """The programmatic-dependent-launch attribute is launch plumbing: results are identical without it."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=20000, d=64, prefix_scale=0.01, name="cfg2_acc_20000")
    inp = wl.make_step(cfg, tau=0.7, synthetic_logits=True)
    with_pdl = pu.gpu_accept_dict(run_accept_only(inp))
    B.gs_set_dependent_launch(False)
    try:
        rnd = run_accept_only(inp)
        check_accept(inp, rnd)
        for k, v in pu.gpu_accept_dict(rnd).items():
            assert np.array_equal(v, with_pdl[k]), k
    finally:
        B.gs_set_dependent_launch(True)


def test_spec_accept_zero_length_drafts_and_single_server(finish_variant):
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=10000, d=64, prefix_scale=0.01, name="acc_gamma0")
    inp = wl.make_step(cfg, gamma=[0, 3, 0, 0, 5, 1, 0, 2], synthetic_logits=True)
    rnd = run_accept_only(inp)
    ref, _ = check_accept(inp, rnd)
    assert rnd.accepted.cpu().tolist()[0] == 0 and rnd.n_out.cpu().tolist()[0] == 1
    cfg1 = wl.shrink(wl.CONFIGS["cfg2"], V=10000, d=64, N=1, prefix_scale=0.01, name="acc_single")
    inp = wl.make_step(cfg1, gamma=[7], synthetic_logits=True)
    check_accept(inp, run_accept_only(inp))
    inp = wl.make_step(cfg1, gamma=[0], synthetic_logits=True)     # Gamma = 0: no draft arrays at all
    check_accept(inp, run_accept_only(inp))


def test_spec_accept_identical_draft_accepts_everything():
    cfg = wl.shrink(wl.CONFIGS["cfg4"], V=8200, d=64, prefix_scale=0.01, name="acc_same")
    inp = wl.make_step(cfg, sigma=np.zeros(cfg.N), synthetic_logits=True)
    rnd = run_accept_only(inp)
    # q == p up to fp32 rounding of the generator's softmax: ratios are 1 within 1e-5
    assert np.all(rnd.ratio.cpu().numpy() > 1 - 1e-4)
    check_accept(inp, rnd)


def test_spec_accept_estimators_and_device_status():
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=6000, d=64, prefix_scale=0.01, name="acc_ema")
    inp = wl.make_step(cfg, synthetic_logits=True)
    rnd = run_accept_only(inp, update=True)
    ref, _ = check_accept(inp, rnd)
    a_hat, X = orc.ref_ema(np.full(cfg.N, 0.5), np.ones(cfg.N), ref["ratio"], ref["accepted"],
                           inp["cu_q"].numpy(), 0.1, 0.5)
    if np.array_equal(rnd.accepted.cpu().numpy(), ref["accepted"]):
        np.testing.assert_allclose(rnd.alpha_hat.cpu().numpy(), a_hat, atol=1e-6)
        np.testing.assert_allclose(rnd.X.cpu().numpy(), X, atol=1e-12)
    # a draft token outside the vocabulary: flagged on the device, treated as a rejection
    bad = dict(inp)
    bad["draft_tok"] = inp["draft_tok"].clone()
    bad["draft_tok"][0] = cfg.V + 7
    d = to_dev(bad)
    r2 = VerifyRound(N=cfg.N, Tq=d["target_logits_f32"].shape[0], total_kv=1, max_kv_len=1, Hq=1, Hkv=1,
                     hd=8, d=8, V=cfg.V, dtype=torch.float32, C=0, device=DEV)
    r2.accept(d["q_probs"], d["draft_tok"], d["cu_q"], d["u_accept"], d["u_sample"], inp["tau"],
              logits=d["target_logits_f32"], update=False)
    torch.cuda.synchronize()
    assert int(r2.d_status.item()) == 1      # GS_ERR_INVALID_ARG
    assert int(r2.accepted[0].item()) == 0
    # decreasing offsets: flagged, nothing written for that server, no fault
    d2 = to_dev(inp)
    cu = d2["cu_q"].clone()
    cu[1] = cu[2] + 1
    r3 = VerifyRound(N=cfg.N, Tq=d2["target_logits_f32"].shape[0], total_kv=1, max_kv_len=1, Hq=1, Hkv=1,
                     hd=8, d=8, V=cfg.V, dtype=torch.float32, C=0, device=DEV)
    r3.accept(d2["q_probs"], d2["draft_tok"], cu, d2["u_accept"], d2["u_sample"], inp["tau"],
              logits=d2["target_logits_f32"], update=False)
    torch.cuda.synchronize()
    assert int(r3.d_status.item()) == 2      # GS_ERR_SHAPE


@pytest.mark.parametrize("V", [20000, 8, 4099], ids=["slices", "tiny-V", "odd-V"])
def test_spec_accept_residual_without_mass_draws_from_target(V, finish_variant):
    """A rejected draft row with q >= p everywhere (q = 1.5 p, unnormalised on purpose): the ratio is
    2/3 for every token, u_accept = 0.95 rejects, max(0, p - q) has no mass and the correction token
    is drawn from p itself -- the second pass of the cluster kernel, the whole-row scan of the ticket
    kernel.  Servers 0, 2 and 5 take that path at their first draft position; the others run as usual."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=V, d=64, prefix_scale=0.01, name=f"acc_nomass_{V}")
    inp = wl.make_step(cfg, tau=0.7, gamma=[3, 1, 8, 2, 5, 4, 7, 6], synthetic_logits=True)
    tau = tau32(inp["tau"])
    cu_q = inp["cu_q"].numpy()
    for k in ("q_probs", "u_accept", "draft_tok"):
        inp[k] = inp[k].clone()
    for i in (0, 2, 5):
        r0, g0 = int(cu_q[i]), int(cu_q[i]) - i
        p = torch.softmax(inp["target_logits_f32"][r0].double() / tau, dim=0)
        inp["q_probs"][g0] = (1.5 * p).float()
        inp["u_accept"][g0] = 0.95
        inp["draft_tok"][g0] = int(torch.argmax(p))          # a token with mass, so that p/q is 2/3 and not 0/0
    rnd = run_accept_only(inp)
    ref, log = check_accept(inp, rnd)
    for i in (0, 2, 5):
        r0, g0 = int(cu_q[i]), int(cu_q[i]) - i
        p = orc.ref_softmax_T(pu.np64(inp["target_logits_f32"][r0]), tau)
        assert np.maximum(p - pu.np64(inp["q_probs"][g0]), 0.0).sum() == 0.0      # the case is really reached
        assert ref["accepted"][i] == 0 and ref["resampled"][i] == 1
        assert int(rnd.accepted[i].item()) == 0
        assert abs(float(rnd.ratio[g0].item()) - 2.0 / 3.0) < 1e-5
    assert not log["accept_near_ties"]
    # the three fall-back draws follow p's CDF: they equal the oracle's tokens unless flagged as near-ties
    assert log["sample_exact"] + len(log["sample_near_ties"]) == cfg.N


def _padded(n, dtype, fill):
    """A tensor of n elements in the middle of a canary-filled buffer: (view, whole buffer)."""
    buf = torch.full((n + 128,), fill, dtype=dtype, device=DEV)
    return buf[64:64 + n], buf


@pytest.mark.parametrize("bad", ["all-rows-in-server-0", "no-rows-in-server-0"])
def test_spec_accept_malformed_offsets_touch_nothing(bad, finish_variant):
    """Offsets that do not decrease but leave a server without a row must only set the device status: no read or write outside the arrays.  Outputs sit inside canary-filled
    buffers, which must come back untouched apart from accepted / n_out = 0 of the skipped servers."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=8192, d=64, N=2, prefix_scale=0.01, name="acc_badcu")
    inp = wl.make_step(cfg, gamma=[3, 4], synthetic_logits=True)
    d = to_dev(inp)
    logits = d["target_logits_f32"].contiguous()
    Tq, V = logits.shape
    N, G = 2, Tq - 2
    cu = {"all-rows-in-server-0": [0, Tq, Tq], "no-rows-in-server-0": [0, 0, Tq]}[bad]
    cu_q = torch.tensor(cu, dtype=torch.int32, device=DEV)
    i32, f32 = torch.int32, torch.float32
    acc, acc_b = _padded(N, i32, -77)
    tok, tok_b = _padded(Tq, i32, -77)
    nout, nout_b = _padded(N, i32, -77)
    ratio, ratio_b = _padded(G, f32, -77.0)
    ptok, ptok_b = _padded(G, f32, -77.0)
    marg, marg_b = _padded(G + N, f32, -77.0)
    st = torch.zeros(1, dtype=i32, device=DEV)
    ws = torch.empty(B.gs_spec_accept_workspace(N, Tq, V), dtype=torch.uint8, device=DEV)
    B.gs_spec_accept(logits, d["q_probs"], d["draft_tok"], cu_q, d["u_accept"], d["u_sample"], 0.7,
                     acc, tok, nout, ratio, ptok, marg, None, None, ws=ws, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 2                                   # GS_ERR_SHAPE
    for view, buf, n in ((acc, acc_b, N), (tok, tok_b, Tq), (nout, nout_b, N), (ratio, ratio_b, G),
                         (ptok, ptok_b, G), (marg, marg_b, G + N)):
        assert bool((buf[:64] == -77).all()) and bool((buf[64 + n:] == -77).all())
    assert acc.tolist() == [0, 0] and nout.tolist() == [0, 0]
    assert bool((tok == -77).all()) and bool((ratio == -77).all()) and bool((ptok == -77).all())


def test_bounded_wait_runs_out_and_reports_timeout():
    """A device-side wait that nothing will ever complete gives up after its limit: the kernel writes
    GS_ERR_TIMEOUT to the device status and ends normally; the context stays usable (a scheduler call
    right after it gives the right answer)."""
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    waited = torch.zeros(1, dtype=torch.int64, device=DEV)
    B.gs_selftest_wait_timeout(3000, st, waited)                 # 3 ms
    torch.cuda.synchronize()
    assert int(st.item()) == 6                                   # GS_ERR_TIMEOUT
    assert 3_000_000 <= int(waited.item()) < 500_000_000
    assert "wait" in B.gs_status_str(6)
    X = torch.tensor([1.0, 2.0, 4.0], dtype=torch.float64, device=DEV)
    al = torch.tensor([0.5, 0.9, 0.7], dtype=torch.float64, device=DEV)
    S = torch.empty(3, dtype=torch.int32, device=DEV)
    st2 = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.gs_schedule(X, al, 12, S, None, None, st2)
    torch.cuda.synchronize()
    assert int(st2.item()) == 0
    assert np.array_equal(S.cpu().numpy(), orc.ref_schedule_greedy(X.cpu().numpy(), al.cpu().numpy(), 12))


# ------------------------------------------------------------------ scheduler
@pytest.fixture(params=[0, 1], ids=["rank-kernel", "greedy-kernel"])
def schedule_variant(request):
    """Both scheduler kernels: ranks by bisection (N <= 32) and the token-by-token greedy."""
    B.gs_schedule_select(request.param)
    yield request.param
    B.gs_schedule_select(0)


@pytest.mark.parametrize("N,C", [(1, 5), (4, 10), (8, 64), (16, 128), (32, 256), (32, 600), (33, 64), (100, 300),
                                 (1024, 512), (8, 0)])
def test_schedule_bit_exact(N, C, schedule_variant):
    r = np.random.default_rng(N * 1000 + C)
    for trial in range(8):
        X = r.uniform(0.5, 8.0, N)
        al = r.uniform(0.001, 0.999, N)
        if trial == 1:                      # many exact ties
            X[:] = 2.0
            al[:] = 0.75
        if trial == 4:                      # gains that underflow to zero, and zero / unit rates
            al = r.choice([0.0, 1e-3, 0.5, 1.0], N)
            X = r.choice([1.0, 1e-300, 3.0], N)
        if trial == 5:                      # ties between servers at every step, in groups
            al = r.choice([0.5, 0.25], N)
            X = r.choice([1.0, 2.0, 4.0], N)
        if trial == 6:                      # a rate outside [0, 1]: gains grow, the greedy is still defined
            al[r.integers(0, N)] = 1.25
        if trial == 7:                      # a starved server: its huge gain is served first
            X[r.integers(0, N)] = 1e-12
        lo = hi = None
        if trial in (2, 3, 5):
            lo = r.integers(0, 2, N).astype(np.int32)
            hi = (lo + r.integers(0, 20, N)).astype(np.int32)
            if lo.sum() > C:
                lo[:] = 0
        S = torch.empty(N, dtype=torch.int32, device=DEV)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.gs_schedule(torch.from_numpy(X).to(DEV), torch.from_numpy(al).to(DEV), C, S,
                      None if lo is None else torch.from_numpy(lo).to(DEV),
                      None if hi is None else torch.from_numpy(hi).to(DEV), st)
        torch.cuda.synchronize()
        want = orc.ref_schedule_greedy(X, al, C, lo, hi)
        assert np.array_equal(S.cpu().numpy(), want), (N, C, trial)
        assert int(st.item()) == 0
        assert S.sum().item() <= C


def test_schedule_floor_above_budget_is_flagged():
    N = 4
    S = torch.empty(N, dtype=torch.int32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.gs_schedule(torch.ones(N, dtype=torch.float64, device=DEV), torch.full((N,), 0.5, dtype=torch.float64, device=DEV),
                  3, S, torch.full((N,), 2, dtype=torch.int32, device=DEV), None, st)
    torch.cuda.synchronize()
    assert S.cpu().tolist() == [2, 2, 2, 2] and int(st.item()) == 2


# ------------------------------------------------------------------ attention
def attn_case(cfg, gamma=None):
    gamma = wl.draw_gamma(cfg, allocator=orc.ref_schedule_greedy) if gamma is None else np.asarray(gamma)
    prefix = wl.draw_prefix(cfg)
    return wl.make_attention_inputs(cfg, gamma, prefix)


def run_attn(inp):
    d = to_dev(inp)
    Tq, Hq, hd = d["Q"].shape
    total_kv, Hkv, _ = d["K"].shape
    cu_kv = inp["cu_kv"]
    max_len = int((cu_kv[1:] - cu_kv[:-1]).max())
    N = cu_kv.numel() - 1
    dt = B.GS_F32 if d["Q"].dtype == torch.float32 else B.GS_BF16
    ws = torch.empty(max(256, B.gs_verify_attn_workspace(N, Tq, total_kv, max_len, Hq, Hkv, hd, dt)),
                     dtype=torch.uint8, device=DEV)
    O = torch.full_like(d["Q"], float("nan"))
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.gs_verify_attn(d["Q"], d["K"], d["V"], O, d["cu_q"], d["cu_kv"], max_len, hd ** -0.5, ws, st)
    torch.cuda.synchronize()
    return O, int(st.item())


ATTN_CASES = [
    ("long-split", wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=1.0, N=2, name="attn_long")),  # 2 servers x 2048: many KV splits
    ("cfg2-shaped", wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.15, name="attn2")),       # 307-key prefixes
    ("cfg3-shaped", wl.shrink(wl.CONFIGS["cfg3"], prefix_scale=0.08, name="attn3")),       # ragged 10..655
    ("cfg4-shaped", wl.shrink(wl.CONFIGS["cfg4"], prefix_scale=0.07, N=5, name="attn4")),
]


@pytest.fixture(params=[0, 1, 3], ids=["auto-splits", "one-tile-splits", "three-tile-splits"])
def attn_splits(request):
    """The automatic plan only splits long caches; one- and three-tile splits force partial
    results, tickets and merges (more than eight splits per group included) and CTAs that walk
    through many short items."""
    B.gs_verify_attn_configure(request.param)
    yield request.param
    B.gs_verify_attn_configure(0)


@pytest.mark.parametrize("name,cfg", ATTN_CASES)
def test_attention_small(name, cfg, attn_splits):
    inp = attn_case(cfg)
    O, st = run_attn(inp)
    assert st == 0
    ref = orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
    pu.assert_close_rel(O, ref, f"attention {name}")
    O2, _ = run_attn(inp)
    assert torch.equal(O, O2)                     # deterministic


@pytest.fixture(params=[2, 4, 8, 3], ids=["clusters-of-2", "clusters-of-4", "clusters-of-8", "one-cta-per-group"])
def attn_cluster(request):
    """The cluster kernel forced for any batch: one cluster of that many CTAs per (server, position
    block, KV head) group, parts merged through distributed shared memory."""
    B.gs_verify_attn_select(request.param)
    yield request.param
    B.gs_verify_attn_select(0)


@pytest.mark.parametrize("name,cfg", ATTN_CASES)
def test_attention_cluster_kernel(name, cfg, attn_cluster):
    inp = attn_case(cfg)
    O, st = run_attn(inp)
    assert st == 0
    ref = orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
    pu.assert_close_rel(O, ref, f"attention {name}, cluster kernel variant {attn_cluster}")
    O2, _ = run_attn(inp)
    assert torch.equal(O, O2)                     # deterministic
    B.gs_verify_attn_select(1)                    # the persistent kernel on the same inputs: equal to rounding
    O3, _ = run_attn(inp)
    pu.assert_close_rel(O, O3.float(), "cluster vs persistent kernel", rel=2e-2)


def test_attention_cluster_kernel_edges_groups_pages(attn_cluster):
    """The cluster kernel on the awkward shapes: a single key, empty prefixes, more CTAs than visible
    tiles (parts without work), several position blocks per server, group sizes that do not divide
    128, bad offsets, and paged caches."""
    import dataclasses
    base = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.0, N=4, name="attn_edge")
    for gamma, prefix in (([0, 1, 16, 3], [1, 1, 1, 700]), ([2, 0, 5, 1], [0, 0, 0, 0]), ([40, 17, 0, 33], [300, 5, 1200, 130])):
        inp = wl.make_attention_inputs(base, np.array(gamma), np.array(prefix))
        O, st = run_attn(inp)
        assert st == 0
        pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), f"edge {gamma}")
    for Hq, Hkv in ((40, 8), (7, 1), (128, 1)):
        cfg = dataclasses.replace(wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.12, N=3, name=f"attn_g{Hq}_{Hkv}"), Hq=Hq, Hkv=Hkv)
        inp = wl.make_attention_inputs(cfg, np.array([8, 0, 30]), np.array([245, 130, 300]))
        O, st = run_attn(inp)
        assert st == 0
        pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), f"G={Hq // Hkv}")
    # a server with fewer keys than new positions: flagged, skipped, the other server is still right
    cfg = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.05, N=2, name="attn_bad")
    inp = wl.make_attention_inputs(cfg, np.array([2, 2]), np.array([50, 50]))
    good = orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
    inp["cu_kv"] = inp["cu_kv"].clone()
    inp["cu_kv"][1] = 1
    O, st = run_attn(inp)
    assert st == 2
    assert bool(torch.isnan(O[:3].float()).all())          # server 0's rows were left unwritten


@pytest.mark.parametrize("Hq,Hkv", [(40, 8), (6, 2), (4, 4), (7, 1), (128, 1)],
                         ids=["group-5", "group-3", "no-grouping", "group-7", "group-128"])
def test_attention_group_sizes(Hq, Hkv):
    """Query-to-KV head ratios that do not divide the 128 rows of a score tile (floor(128/G) positions
    per tile, the leftover rows masked), no grouping at all, and one position per tile."""
    import dataclasses
    cfg = dataclasses.replace(wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.12, N=3, name=f"attn_g{Hq}_{Hkv}"),
                              Hq=Hq, Hkv=Hkv)
    inp = wl.make_attention_inputs(cfg, np.array([8, 0, 30]), np.array([245, 130, 300]))
    O, st = run_attn(inp)
    assert st == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), f"G={Hq // Hkv}")


@pytest.mark.parametrize("splits", [0, 2, -2, -4], ids=["auto-splits", "two-tile-splits", "clusters-of-2", "clusters-of-4"])
def test_attention_paged_caches(splits):
    """gs_verify_attn_paged: the caches scattered over a pool of 128-row pages in shuffled order (with
    unused pages in between) give what the contiguous layout gives, i.e. the oracle's attention."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.3, N=5, name="attn_paged")
    gamma, prefix = np.array([3, 0, 8, 1, 5]), np.array([700, 90, 1300, 128, 255])
    inp = wl.make_attention_inputs(cfg, gamma, prefix)
    cu_kv = inp["cu_kv"].numpy()
    N = len(gamma)
    lens = cu_kv[1:] - cu_kv[:-1]
    pages_of = [(int(l) + 127) // 128 for l in lens]
    max_pages = max(pages_of) + 2
    n_pages = sum(pages_of) + 7
    order = np.random.default_rng(3).permutation(n_pages)
    table = np.full((N, max_pages), -1, np.int32)            # unused entries are never read
    K_pool = torch.full((n_pages * 128, cfg.Hkv, cfg.hd), 300.0, dtype=torch.bfloat16)    # stale but finite rows
    V_pool = torch.full_like(K_pool, -70.0)
    nxt = 0
    for i in range(N):
        for t in range(pages_of[i]):
            pg = int(order[nxt]); nxt += 1
            table[i, t] = pg
            lo = cu_kv[i] + t * 128
            n = min(128, cu_kv[i + 1] - lo)
            K_pool[pg * 128: pg * 128 + n] = inp["K"][lo: lo + n]
            V_pool[pg * 128: pg * 128 + n] = inp["V"][lo: lo + n]
    # rows of a server's last page beyond its length hold stale values: they are masked by index
    d = to_dev(inp)
    Tq, Hq, hd = d["Q"].shape
    max_len = int(lens.max())
    B.gs_verify_attn_configure(max(splits, 0))
    B.gs_verify_attn_select(-splits if splits < 0 else 1)
    try:
        ws = torch.empty(max(256, B.gs_verify_attn_paged_workspace(N, Tq, max_len, Hq, cfg.Hkv, hd, B.GS_BF16)),
                         dtype=torch.uint8, device=DEV)
        O = torch.full_like(d["Q"], float("nan"))
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.gs_verify_attn_paged(d["Q"], K_pool.to(DEV), V_pool.to(DEV), O, d["cu_q"], d["cu_kv"],
                               torch.from_numpy(table).to(DEV), max_len, hd ** -0.5, ws, st)
        torch.cuda.synchronize()
        O2, _ = run_attn(inp)          # the contiguous layout under the same split plan
    finally:
        B.gs_verify_attn_configure(0)
        B.gs_verify_attn_select(0)
    assert int(st.item()) == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "paged")
    assert torch.equal(O, O2)          # bit-identical to the contiguous layout (same tiles, same order)


def test_attention_many_short_servers():
    """More items per CTA than the kernel caches descriptors for (700 servers x 8 KV heads over 148
    CTAs), most of them a single tile, a few long ones in between."""
    base = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.0, N=700, name="attn_many")
    r = np.random.default_rng(7)
    gamma = r.integers(0, 4, 700)
    prefix = r.integers(0, 40, 700)
    prefix[[5, 333, 699]] = [1500, 700, 2600]
    inp = wl.make_attention_inputs(base, gamma, prefix)
    O, st = run_attn(inp)
    assert st == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "many servers")


def test_attention_more_servers_than_the_offset_cache():
    """1100 servers: more than the kernel keeps offsets and prefix sums for in shared memory, so the item
    scheduler finds every item by a walk over the offsets in global memory."""
    base = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.0, N=1100, name="attn_1100")
    r = np.random.default_rng(11)
    gamma = r.integers(0, 3, 1100)
    prefix = r.integers(0, 24, 1100)
    prefix[[7, 1099]] = [900, 300]
    inp = wl.make_attention_inputs(base, gamma, prefix)
    O, st = run_attn(inp)
    assert st == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "1100 servers")


def test_attention_edge_shapes():
    base = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.0, N=4, name="attn_edge")   # prefix 1
    inp = wl.make_attention_inputs(base, np.array([0, 1, 16, 3]), np.array([1, 1, 1, 700]))
    O, st = run_attn(inp)
    assert st == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "edge")
    # empty prefix: position t sees only the t+1 new keys
    inp = wl.make_attention_inputs(base, np.array([2, 0, 5, 1]), np.array([0, 0, 0, 0]))
    O, st = run_attn(inp)
    assert st == 0
    pu.assert_close_rel(O, orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]), "no prefix")


def test_attention_causality_and_server_permutation():
    cfg = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.1, N=3, name="attn_prop")
    inp = wl.make_attention_inputs(cfg, np.array([3, 2, 4]), np.array([200, 150, 90]))
    O, _ = run_attn(inp)
    # perturb the K/V of server 0's last new position: only its last query row may change
    inp2 = dict(inp)
    inp2["K"], inp2["V"] = inp["K"].clone(), inp["V"].clone()
    last = int(inp["cu_kv"][1]) - 1
    inp2["K"][last] += 3.0
    inp2["V"][last] -= 2.0
    O2, _ = run_attn(inp2)
    assert torch.equal(O[:3], O2[:3]) and torch.equal(O[4:], O2[4:]) and not torch.equal(O[3], O2[3])
    # swap servers 0 and 2: outputs move with them
    cq, ck = inp["cu_q"].numpy(), inp["cu_kv"].numpy()
    order = [2, 1, 0]
    Q = torch.cat([inp["Q"][cq[i]:cq[i + 1]] for i in order])
    K = torch.cat([inp["K"][ck[i]:ck[i + 1]] for i in order])
    V = torch.cat([inp["V"][ck[i]:ck[i + 1]] for i in order])
    perm = wl.make_attention_inputs(cfg, np.array([4, 2, 3]), np.array([90, 150, 200]))
    perm["Q"], perm["K"], perm["V"] = Q, K, V
    Op, _ = run_attn(perm)
    want = torch.cat([O[cq[i]:cq[i + 1]] for i in order])
    assert torch.equal(Op, want)


def test_attention_bad_offsets_are_flagged():
    cfg = wl.shrink(wl.CONFIGS["cfg2"], prefix_scale=0.05, N=2, name="attn_bad")
    inp = wl.make_attention_inputs(cfg, np.array([2, 2]), np.array([50, 50]))
    inp["cu_kv"] = inp["cu_kv"].clone()
    inp["cu_kv"][1] = 1          # server 0 would have fewer keys than new positions
    O, st = run_attn(inp)
    assert st == 2


# ------------------------------------------------------------------ LM head + acceptance, statistics fused
@pytest.mark.parametrize("T_extra,d,V,tau", [(0, 512, 9000, 0.7), (0, 256, 20000, 1.0), (0, 320, 4104, 0.0),
                                             (150, 256, 8192, 0.7), (288, 256, 8200, 1.0), (512, 192, 4104, 0.7),
                                             (300, 128, 4096, 0.0)],
                         ids=["ragged-V", "wide", "greedy", "many-rows", "288-rows", "512-rows", "greedy-300-rows"])
def test_fused_head_statistics_match_two_pass(T_extra, d, V, tau):
    """gs_lm_head_logits_stats + gs_spec_accept_prestats against the oracle, and against the plain
    pair of calls: logits bit-identical, counts and tokens equal (the statistics group their sums
    differently, so probabilities agree to rounding)."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=d, V=V, prefix_scale=0.02, name=f"fused_{d}_{V}")
    gamma = [8, 1, 3, 0, 6, 2, 7, 4]
    if T_extra == 150:
        cfg = wl.shrink(cfg, N=24, name=cfg.name + "_24")
        gamma = list(np.random.default_rng(5).integers(3, 9, 24))
    elif T_extra:                                     # exactly T_extra verify positions: two MMAs along the rows
        cfg = wl.shrink(cfg, N=32, name=cfg.name + f"_{T_extra}")
        gamma = np.random.default_rng(T_extra).multinomial(T_extra - 32, np.ones(32) / 32)
        assert gamma.sum() + 32 == T_extra
    inp = wl.make_step(cfg, tau=tau, gamma=gamma)
    dev = to_dev(inp)
    plain = VerifyRound.for_inputs(dev, C=4 * cfg.N)
    plain.run(dev)
    fused = VerifyRound.for_inputs(dev, C=4 * cfg.N)
    fused.attn(dev["Q"], dev["K"], dev["V"], dev["cu_q"], dev["cu_kv"])
    ran = fused.head_accept_fused(dev["H"], dev["W"], dev["q_probs"], dev["draft_tok"], dev["cu_q"],
                                  dev["u_accept"], dev["u_sample"], inp["tau"], force=True)
    fused.schedule()
    torch.cuda.synchronize()
    assert ran, "this shape has the fused kernels"
    assert int(fused.d_status.item()) == 0 and int(plain.d_status.item()) == 0
    assert torch.equal(fused.logits, plain.logits)
    t32 = tau32(inp["tau"])
    ref_logits = orc.ref_lm_head(inp["H"], inp["W"])
    ref = orc.ref_spec_accept(ref_logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"],
                              inp["u_sample"], t32)
    slack = pu.chain_slack(fused.logits, ref_logits, t32)
    pu.compare_accept(pu.gpu_accept_dict(fused), ref, ref_logits, inp["q_probs"], inp["cu_q"].numpy(),
                      inp["u_sample"], t32, V, slack=slack)
    a, b = pu.gpu_accept_dict(fused), pu.gpu_accept_dict(plain)
    assert np.array_equal(a["accepted"], b["accepted"]) and np.array_equal(a["out_tok"], b["out_tok"])
    np.testing.assert_allclose(a["ratio"], b["ratio"], atol=2e-6)
    np.testing.assert_allclose(a["p_tok"], b["p_tok"], atol=2e-6)


def test_fused_head_statistics_unsupported_shapes_fall_back():
    """More than 512 rows: no fused kernel, the runner uses the two plain calls and says so."""
    cfg = wl.shrink(wl.CONFIGS["cfg3"], d=128, V=4096, prefix_scale=0.02, name="fused_fallback")
    inp = wl.make_step(cfg, gamma=np.full(32, 16))
    dev = to_dev(inp)
    assert dev["H"].shape[0] > 512
    rnd = VerifyRound.for_inputs(dev, C=256)
    ran = rnd.head_accept_fused(dev["H"], dev["W"], dev["q_probs"], dev["draft_tok"], dev["cu_q"],
                                dev["u_accept"], dev["u_sample"], inp["tau"])
    torch.cuda.synchronize()
    assert not ran and int(rnd.d_status.item()) == 0
    pu.assert_close_rel(rnd.logits, orc.ref_lm_head(inp["H"], inp["W"]), "fallback logits")


# ------------------------------------------------------------------ the round from host buffers
@pytest.mark.parametrize("q_mode", ["in-place", "in-place-only", "copied", "pageable"])
@pytest.mark.parametrize("gamma", [[3, 1, 8, 2, 5, 4, 7, 6], [8, 8, 8, 8, 8, 8, 8, 8]], ids=["44-positions", "72-positions"])
def test_verify_round_host_matches_device_path(gamma, q_mode):
    """gs_verify_round_host gives what the four calls give on device-resident inputs, whether the
    acceptance kernels read the pinned draft distributions where they lie (the default: the first rows of
    every server are copied meanwhile and read on the device; "in-place-only": every row that is needed
    crosses the bus inside the acceptance kernel), the library copies them on its copy stream while attention and the LM head run (in-place reads switched off),
    or the buffer is pageable memory, which can only be copied; two rounds back to back with different
    drafts reuse the staging area."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=256, V=16384, prefix_scale=0.1, name="host_round")
    for round_idx in (0, 1):
        inp = wl.make_step(cfg, round_idx=round_idx, gamma=gamma)     # same shapes, new drafts
        d = to_dev(inp)
        N, Tq = cfg.N, int(inp["cu_q"][-1])
        rnd = VerifyRound.for_inputs(d, C=4 * N)
        # second round of the in-place-only case: the ticket kernel of the acceptance step (which takes no
        # statistics from the LM head, so both sides run the statistics pass) reads the host rows
        ticket = (q_mode == "in-place-only" and round_idx == 1)
        B.gs_spec_accept_select(1 if ticket else 0)
        try:
            rnd.run(d, fused=not ticket)   # the host-buffer round takes the same kernels (statistics from the LM head)
            torch.cuda.synchronize()
        except Exception:
            B.gs_spec_accept_select(0)
            raise
        assert int(rnd.d_status.item()) == 0
        desc = B.RoundDesc(N=N, Tq=Tq, total_kv=d["K"].shape[0], max_kv_len=rnd.max_kv_len, Hq=cfg.Hq, Hkv=cfg.Hkv,
                           hd=cfg.hd, d=cfg.d, V=cfg.V, C=4 * N, dt=B.GS_BF16, scale=cfg.hd ** -0.5,
                           temperature=float(inp["tau"]), eta=0.1, beta=0.5, alpha_min=1e-3, alpha_max=0.999)
        if round_idx == 0:
            ws = torch.empty(B.gs_verify_round_workspace(desc), dtype=torch.uint8, device=DEV)
        pin = {k: inp[k].contiguous().pin_memory() for k in
               ("Q", "H", "q_probs", "draft_tok", "u_accept", "u_sample", "cu_q", "cu_kv")}
        if q_mode == "pageable":
            pin["q_probs"] = inp["q_probs"].contiguous().clone()
        outs = {k: torch.full((n,), -9, dtype=torch.int32).pin_memory() for k, n in
                (("accepted", N), ("out_tok", Tq), ("n_out", N), ("S_next", N), ("status", 1))}
        a_hat = torch.full((N,), 0.5, dtype=torch.float64, device=DEV)
        X = torch.ones(N, dtype=torch.float64, device=DEV)
        B.gs_verify_round_configure({"in-place": 1, "in-place-only": 2, "copied": 0, "pageable": 1}[q_mode])
        try:
            assert B.gs_verify_round_reads_in_place(pin["q_probs"]) == q_mode.startswith("in-place")
            assert (B.gs_verify_round_near_rows(desc) == 0) == (q_mode == "in-place-only")
            B.gs_verify_round_host(desc, pin["Q"], pin["H"], pin["q_probs"], pin["draft_tok"], pin["u_accept"],
                                   pin["u_sample"], pin["cu_q"], pin["cu_kv"], d["K"], d["V"], d["W"], a_hat, X,
                                   None, None, ws, outs["accepted"], outs["out_tok"], outs["n_out"], outs["S_next"],
                                   outs["status"])
            torch.cuda.synchronize()
        finally:
            B.gs_verify_round_configure(True)
            B.gs_spec_accept_select(0)
        assert int(outs["status"][0]) == 0
        for k in ("accepted", "out_tok", "n_out", "S_next"):
            assert torch.equal(outs[k], getattr(rnd, k).cpu()), (round_idx, k)
        assert torch.equal(a_hat, rnd.alpha_hat) and torch.equal(X, rnd.X)


def test_verify_round_host_flags_bad_offsets():
    """Query offsets that leave a server without a row: the host-buffer round (which reads the offsets on
    the host to place its copies of the first draft rows) copies nothing for such a server, every kernel
    skips it, and the device status says GS_ERR_SHAPE; the call after it, with good offsets, is right."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=256, V=16384, N=2, prefix_scale=0.05, name="host_round_bad")
    inp = wl.make_step(cfg, gamma=[3, 4])
    d = to_dev(inp)
    N, Tq = 2, int(inp["cu_q"][-1])
    rnd = VerifyRound.for_inputs(d, C=8)
    rnd.run(d, fused=True)
    torch.cuda.synchronize()
    desc = B.RoundDesc(N=N, Tq=Tq, total_kv=d["K"].shape[0], max_kv_len=rnd.max_kv_len, Hq=cfg.Hq, Hkv=cfg.Hkv,
                       hd=cfg.hd, d=cfg.d, V=cfg.V, C=8, dt=B.GS_BF16, scale=cfg.hd ** -0.5,
                       temperature=float(inp["tau"]), eta=0.1, beta=0.5, alpha_min=1e-3, alpha_max=0.999)
    ws = torch.empty(B.gs_verify_round_workspace(desc), dtype=torch.uint8, device=DEV)
    pin = {k: inp[k].contiguous().pin_memory() for k in
           ("Q", "H", "q_probs", "draft_tok", "u_accept", "u_sample", "cu_q", "cu_kv")}
    good_cu = pin["cu_q"].clone()
    for cu, want_status in (([0, Tq, Tq], 2), (good_cu.tolist(), 0)):
        pin["cu_q"].copy_(torch.tensor(cu, dtype=torch.int32))
        outs = {k: torch.full((n,), -9, dtype=torch.int32).pin_memory() for k, n in
                (("accepted", N), ("out_tok", Tq), ("n_out", N), ("S_next", N), ("status", 1))}
        a_hat = torch.full((N,), 0.5, dtype=torch.float64, device=DEV)
        X = torch.ones(N, dtype=torch.float64, device=DEV)
        B.gs_verify_round_host(desc, pin["Q"], pin["H"], pin["q_probs"], pin["draft_tok"], pin["u_accept"],
                               pin["u_sample"], pin["cu_q"], pin["cu_kv"], d["K"], d["V"], d["W"], a_hat, X,
                               None, None, ws, outs["accepted"], outs["out_tok"], outs["n_out"], outs["S_next"],
                               outs["status"])
        torch.cuda.synchronize()
        assert int(outs["status"][0]) == want_status
        if want_status == 0:
            for k in ("accepted", "out_tok", "n_out", "S_next"):
                assert torch.equal(outs[k], getattr(rnd, k).cpu()), k
        else:
            assert int(outs["accepted"][1]) == 0 and int(outs["n_out"][1]) == 0


# ------------------------------------------------------------------ LM head
@pytest.mark.parametrize("variant", [2, 1], ids=["cta-pairs", "one-cta"])
@pytest.mark.parametrize("T,d,V", [(44, 512, 9000), (96, 1024, 4104), (288, 256, 8192), (1, 64, 8), (130, 136, 1000),
                                   (600, 192, 2056), (257, 320, 520)])
def test_lm_head_small(T, d, V, variant):
    """Both tensor-core kernels (CTA pairs with M = 256, and one CTA per tile) against the oracle:
    ragged vocabulary and row tails, one and two MMAs along the rows, more than 512 rows."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=d, V=V, name=f"head_{T}_{d}_{V}")
    W = wl.make_layer(cfg)["W"]
    H = wl.make_hidden(cfg, T)
    logits = torch.full((T, V), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(256, B.gs_lm_head_workspace(T, d, V, B.GS_BF16)), dtype=torch.uint8, device=DEV)
    B.gs_lm_head_select(variant)
    try:
        B.gs_lm_head_logits(H.to(DEV), W.to(DEV), logits, ws)
        torch.cuda.synchronize()
    finally:
        B.gs_lm_head_select(0)
    ref = orc.ref_lm_head(H, W)
    pu.assert_close_rel(logits, ref, "logits")
    # bf16 products are exact in fp32 and only the accumulation rounds: far inside the 2e-2 bar
    pu.assert_close_rel(logits, ref, "logits (accumulation bar)", rel=2e-4)


# ------------------------------------------------------------------ LM head on 4-bit weights
@pytest.mark.parametrize("T,d,V,group", [(46, 512, 9008, 128), (96, 1024, 4112, 128), (1, 128, 16, 64), (130, 384, 1008, 64),
                                         (256, 256, 2048, 128), (300, 128, 528, 128), (16, 5120, 4096, 128),
                                         (144, 384, 20000, 128), (16, 256, 151552, 128), (46, 256, 151936, 64)])
def test_lm_head_w4_small(T, d, V, group):
    """gs_lm_head_logits_w4 against the oracle's dequantised weight and plain product: ragged vocabulary
    tails, tiles of one to four units (the last two shapes: four units everywhere, and the real vocabulary
    with three and two), one and two accumulator buffers, more than 256 rows (two launches), both group
    sizes, the real model width."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=d, V=V, name=f"w4_{T}_{d}_{V}")
    layer = wl.make_w4_layer(cfg, group)
    H = wl.make_hidden(cfg, T)
    logits = torch.full((T, V), float("nan"), dtype=torch.float32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.gs_lm_head_logits_w4(H.to(DEV), layer["qweight"].to(DEV), layer["scales"].to(DEV), layer["zeros"].to(DEV), group,
                           logits, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    W = orc.ref_dequant_w4(layer["qweight"], layer["scales"], layer["zeros"], group)
    ref = orc.ref_lm_head(H, W)
    pu.assert_close_rel(logits, ref, "logits on 4-bit weights")
    # every weight is rounded to bf16 once (relative error up to 2^-9, mean square a third of that), the
    # products are exact and the errors add up like a random walk: about 1.1e-3 of the row's rms per
    # logit on average; the worst of a few hundred thousand elements reaches about ten times that
    pu.assert_close_rel(logits, ref, "logits on 4-bit weights (rounding bar)", rel=1.5e-2)
    logits2 = torch.empty_like(logits)
    B.gs_lm_head_logits_w4(H.to(DEV), layer["qweight"].to(DEV), layer["scales"].to(DEV), layer["zeros"].to(DEV), group,
                           logits2, st)
    torch.cuda.synchronize()
    assert torch.equal(logits, logits2)


def test_lm_head_w4_feeds_the_acceptance_step():
    """A round whose head weight is 4-bit: gs_lm_head_logits_w4 then gs_spec_accept, against the oracle on
    its own dequantised product for the logits, and on the library's logits for the acceptance step."""
    cfg = wl.shrink(wl.CONFIGS["cfg2"], d=512, V=8192, prefix_scale=0.02, name="w4_round")
    inp = wl.make_step(cfg, gamma=[3, 1, 8, 2, 5, 4, 7, 6])
    layer = wl.make_w4_layer(cfg, 128)
    W = orc.ref_dequant_w4(layer["qweight"], layer["scales"], layer["zeros"], 128)
    # drafts simulated from the 4-bit target's own logits
    logits_sim = torch.from_numpy(orc.ref_lm_head(inp["H"], W)).float()
    q, tok = wl.simulate_drafts(cfg, logits_sim, inp["cu_q"], inp["sigma"], inp["tau"])
    inp["q_probs"], inp["draft_tok"] = q, tok
    d = to_dev(inp)
    rnd = VerifyRound.for_inputs(d, C=64)
    B.gs_lm_head_logits_w4(d["H"], layer["qweight"].to(DEV), layer["scales"].to(DEV), layer["zeros"].to(DEV), 128,
                           rnd.logits, rnd.d_status)
    rnd.accept(d["q_probs"], d["draft_tok"], d["cu_q"], d["u_accept"], d["u_sample"], inp["tau"])
    torch.cuda.synchronize()
    assert int(rnd.d_status.item()) == 0
    tau = tau32(inp["tau"])
    pu.assert_close_rel(rnd.logits, orc.ref_lm_head(inp["H"], W), "logits on 4-bit weights")
    # the acceptance step on the logits the library produced, widened to fp64: identical logits on both
    # sides, so the strict band applies (the weights' bf16 rounding moves a logit by up to 1e-2, which as
    # slack would swallow every decision)
    got_logits = rnd.logits.cpu()
    ref = orc.ref_spec_accept(got_logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"], inp["u_sample"], tau)
    log = pu.compare_accept(pu.gpu_accept_dict(rnd), ref, got_logits, inp["q_probs"], inp["cu_q"].numpy(), inp["u_sample"],
                            tau, cfg.V)
    assert len(log["accept_near_ties"]) <= 1


# ------------------------------------------------------------------ full-size configurations
def _full_round(cfg_name, C, max_head_bytes=40e9):
    cfg = wl.CONFIGS[cfg_name]
    # big tensors are drawn on the device (seconds instead of minutes), then copied to the host
    d = wl.make_step(cfg, allocator=orc.ref_schedule_greedy, device=DEV)
    inp = {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in d.items()}
    rnd = VerifyRound.for_inputs(d, C=C)
    rnd.run(d)
    torch.cuda.synchronize()
    assert int(rnd.d_status.item()) == 0
    tau = tau32(inp["tau"])
    # attention: every element
    ref_O = orc.ref_attention(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
    pu.assert_close_rel(rnd.O, ref_O, f"{cfg_name} attention")
    # LM head: the oracle's full fp64 product, column block by column block
    V = cfg.V
    ref_logits = np.empty((rnd.Tq, V))
    step = 8192
    for c0 in range(0, V, step):
        cols = np.arange(c0, min(V, c0 + step))
        ref_logits[:, cols] = orc.ref_lm_head(inp["H"], inp["W"], cols=cols)
    pu.assert_close_rel(rnd.logits, ref_logits, f"{cfg_name} logits")
    # acceptance, chained: library on its own logits vs oracle on its own logits
    ref = orc.ref_spec_accept(ref_logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"],
                              inp["u_sample"], tau)
    slack = pu.chain_slack(rnd.logits, ref_logits, tau)
    assert slack < 5e-4, slack
    log = pu.compare_accept(pu.gpu_accept_dict(rnd), ref, ref_logits, inp["q_probs"], inp["cu_q"].numpy(),
                            inp["u_sample"], tau, V, slack=slack)
    assert len(log["accept_near_ties"]) <= 1, log
    # acceptance alone on identical logits (the generator's fp32 product)
    rnd_a = run_accept_only(inp)
    _, log2 = check_accept(inp, rnd_a)
    # estimators and next allocation where the counts agree
    a_hat, X = orc.ref_ema(np.full(cfg.N, 0.5), np.ones(cfg.N), ref["ratio"], ref["accepted"],
                           inp["cu_q"].numpy(), 0.1, 0.5)
    if not log["accept_near_ties"]:
        np.testing.assert_allclose(rnd.alpha_hat.cpu().numpy(), a_hat, atol=1e-5)
        np.testing.assert_allclose(rnd.X.cpu().numpy(), X, atol=1e-12)
        S_ref = orc.ref_schedule_greedy(X, a_hat, C)
        S_gpu = rnd.S_next.cpu().numpy()
        if not np.array_equal(S_gpu, S_ref):     # estimator rounding moved a near-tied marginal
            assert S_gpu.sum() == S_ref.sum()
            o1, o2 = orc.ref_sched_objective(X, a_hat, S_gpu), orc.ref_sched_objective(X, a_hat, S_ref)
            assert abs(o1 - o2) <= 1e-6 * abs(o2)
    print(cfg_name, "chain log", log, "accept-only log", log2)


def test_cfg2_full_size():
    _full_round("cfg2", C=64)


def test_cfg3_full_size():
    _full_round("cfg3", C=256)


def test_cfg4_full_size():
    _full_round("cfg4", C=128)


def test_cfg6_paper_scale_full_size():
    _full_round("cfg6", C=20)
