"""Closed-loop harness: Algorithm 1 run round after round with the scheduler in the loop.

The draft servers are simulated (workloads.py): each has a true acceptance rate alpha_i that is
redrawn every `epoch` rounds, and draft noise calibrated to it.  Every round the harness builds the
inputs for the allocation S(t) the scheduler produced in the previous round (gamma_i = S_i(t)),
runs the library's round on the GPU, and feeds S(t+1) back.  It holds no verification arithmetic:
the GPU does the round; the harness only generates inputs and keeps running sums for the report.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

from . import binding as B
from . import workloads as wl


POLICIES = ("goodspeed", "fixed", "random")


class ClosedLoop:
    """policy: who decides S(t+1).  "goodspeed" = the scheduler's allocation (Eq. goodspeed_sched);
    "fixed" = Fixed-S, C/N tokens for every server; "random" = Random-S, the budget thrown at the
    servers uniformly at random (the two baselines of Sec. V).  The estimators are updated in every
    case.  step_decay > 0 shrinks both smoothing steps as (t+1)^-step_decay (Assumption 3 asks for
    steps with divergent sum and convergent sum of squares, e.g. 0.5 < step_decay <= 1).
    grow=True keeps the caches in a pool of 128-row pages and appends every round's output tokens
    (accepted drafts plus the correction or bonus token) to each server's prefix, as Sec. III-A
    describes; attention then runs through gs_verify_attn_paged.  A cache stops growing at max_len."""

    def __init__(self, cfg: wl.VerifyConfig, device="cuda", epoch=100, eta=0.1, beta=0.5, s_min=0,
                 policy="goodspeed", step_decay=0.0, grow=False, max_len=None):
        if policy not in POLICIES:
            raise ValueError(f"policy must be one of {POLICIES}")
        self.cfg, self.dev, self.epoch = cfg, torch.device(device), epoch
        self.eta0, self.beta0, self.step_decay = eta, beta, float(step_decay)
        self.eta, self.beta = eta, beta
        self.policy = policy
        N, C = cfg.N, cfg.C
        self.N, self.C = N, C
        self.max_new = C + 1                                   # a single server can get the whole budget
        self.prefix = int(cfg.prefix_lo)
        dt = wl.torch_dtype(cfg)
        self.W = wl.make_layer(cfg, self.dev)["W"]
        per = self.prefix + self.max_new
        self.grow = bool(grow)
        if not self.grow:
            self.K_pool = wl._normal(cfg, "K_pool", 0, (N, per, cfg.Hkv, cfg.hd), 1.0, dt, self.dev)
            self.V_pool = wl._normal(cfg, "V_pool", 0, (N, per, cfg.Hkv, cfg.hd), 1.0, dt, self.dev)
        else:
            # paged caches: pages are handed out in a shuffled order, one at a time, as a cache needs them
            self.max_len = int(max_len if max_len is not None else self.prefix + 16 * self.max_new)
            self.max_pages = (self.max_len + 127) // 128
            self.n_pages = N * self.max_pages
            self.K_pages = torch.zeros((self.n_pages * 128, cfg.Hkv, cfg.hd), dtype=dt, device=self.dev)
            self.V_pages = torch.zeros_like(self.K_pages)
            self._free = list(wl._rng(cfg, "page_order", 0).permutation(self.n_pages))
            self.table = np.full((N, self.max_pages), -1, np.int32)
            self.len = np.zeros(N, np.int64)
            for i in range(N):                       # the prompt's keys and values
                self._write_rows(i, 0, wl._normal(cfg, f"K_prefix{i}", 0, (self.prefix, cfg.Hkv, cfg.hd), 1.0, dt, self.dev),
                                 wl._normal(cfg, f"V_prefix{i}", 0, (self.prefix, cfg.Hkv, cfg.hd), 1.0, dt, self.dev))
                self.len[i] = self.prefix
        self.s_min = torch.full((N,), int(s_min), dtype=torch.int32, device=self.dev)
        self.s_max = torch.full((N,), C, dtype=torch.int32, device=self.dev)
        self.S = np.full(N, C // N, dtype=np.int64)            # S_i(0) = floor(C/N)
        self._sigma_epoch = -1
        # device state and output buffers sized for the largest round
        Tq_max = C + N
        f32, i32, f64 = torch.float32, torch.int32, torch.float64
        self.alpha_hat = torch.full((N,), 0.5, dtype=f64, device=self.dev)
        self.X = torch.ones(N, dtype=f64, device=self.dev)
        self.O = torch.empty((Tq_max, cfg.Hq, cfg.hd), dtype=dt, device=self.dev)
        self.logits = torch.empty((Tq_max * cfg.V,), dtype=f32, device=self.dev)
        self.accepted = torch.empty(N, dtype=i32, device=self.dev)
        self.out_tok = torch.empty(Tq_max, dtype=i32, device=self.dev)
        self.n_out = torch.empty(N, dtype=i32, device=self.dev)
        self.ratio = torch.empty(max(C, 1), dtype=f32, device=self.dev)
        self.p_tok = torch.empty(max(C, 1), dtype=f32, device=self.dev)
        self.S_next = torch.empty(N, dtype=i32, device=self.dev)
        self.d_status = torch.zeros(1, dtype=i32, device=self.dev)
        gsdt = B.GS_F32 if dt == torch.float32 else B.GS_BF16
        total_kv_max = N * self.prefix + Tq_max
        self.max_kv_len = self.prefix + self.max_new
        ws = lambda n: torch.empty(max(int(n), 256), dtype=torch.uint8, device=self.dev)
        if self.grow:
            self.max_kv_len = self.max_len
            self.ws_attn = ws(B.gs_verify_attn_paged_workspace(N, Tq_max, self.max_kv_len, cfg.Hq, cfg.Hkv, cfg.hd, gsdt))
        else:
            self.ws_attn = ws(B.gs_verify_attn_workspace(N, Tq_max, total_kv_max, self.max_kv_len, cfg.Hq, cfg.Hkv,
                                                         cfg.hd, gsdt))
        self.ws_head = ws(B.gs_lm_head_workspace(Tq_max, cfg.d, cfg.V, gsdt))
        self.ws_acc = ws(B.gs_spec_accept_workspace(N, Tq_max, cfg.V))
        self.stats = ws(B.gs_lm_head_stats_bytes(Tq_max))

    # ---------------------------------------------------------------- inputs of round t
    def true_alpha(self, t):
        return wl.draw_true_alpha(self.cfg, t // self.epoch)

    def sigma(self, t):
        e = t // self.epoch
        if e != self._sigma_epoch:
            self._sigma = wl.calibrate_sigma(self.true_alpha(t), self.cfg.V, self.cfg.tau)
            self._sigma_epoch = e
        return self._sigma

    # ---------------------------------------------------------------- paged caches (grow=True)
    def _rows(self, i, start, n):
        """Pool rows of positions start..start+n-1 of server i (pages are allocated on demand)."""
        pos = np.arange(start, start + n)
        for pg in range(start // 128, (start + n - 1) // 128 + 1) if n > 0 else ():
            if self.table[i, pg] < 0:
                self.table[i, pg] = self._free.pop()
        return torch.from_numpy(self.table[i, pos // 128].astype(np.int64) * 128 + pos % 128).to(self.dev)

    def _write_rows(self, i, start, K_rows, V_rows):
        idx = self._rows(i, start, K_rows.shape[0])
        self.K_pages.index_copy_(0, idx, K_rows)
        self.V_pages.index_copy_(0, idx, V_rows)

    def gather_contiguous(self, inp):
        """K, V of the round in the contiguous layout (for the oracle, which knows no pages)."""
        cu_kv = inp["cu_kv"].cpu().numpy()
        idx = torch.cat([self._rows(i, 0, int(cu_kv[i + 1] - cu_kv[i])) for i in range(self.N)])
        return self.K_pages.index_select(0, idx), self.V_pages.index_select(0, idx)

    def append_outputs(self, n_out):
        """The round's output tokens join the prefixes (their keys and values are the ones the
        round wrote for the accepted positions; what follows is overwritten by the next round)."""
        room = self.max_len - self.max_new
        self.len = np.minimum(self.len + np.asarray(n_out, np.int64), room)

    def make_inputs(self, t, gamma):
        cfg = self.cfg
        gamma = np.asarray(gamma, np.int64)
        n_new = gamma + 1
        cu_q = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
        base_len = self.len if self.grow else np.full(self.N, self.prefix, np.int64)
        cu_kv = np.concatenate([[0], np.cumsum(base_len + n_new)]).astype(np.int32)
        Tq = int(cu_q[-1])
        dt = wl.torch_dtype(cfg)
        if self.grow:
            K_new = wl._normal(cfg, "K_new", t, (Tq, cfg.Hkv, cfg.hd), 1.0, dt, self.dev)
            V_new = wl._normal(cfg, "V_new", t, (Tq, cfg.Hkv, cfg.hd), 1.0, dt, self.dev)
            for i in range(self.N):
                self._write_rows(i, int(self.len[i]), K_new[cu_q[i]:cu_q[i + 1]], V_new[cu_q[i]:cu_q[i + 1]])
            kv = {"K_pool": self.K_pages, "V_pool": self.V_pages,
                  "block_table": torch.from_numpy(self.table.copy()).to(self.dev)}
        else:
            kv = {"K": torch.cat([self.K_pool[i, :self.prefix + int(n_new[i])] for i in range(self.N)]).contiguous(),
                  "V": torch.cat([self.V_pool[i, :self.prefix + int(n_new[i])] for i in range(self.N)]).contiguous()}
        inp = {
            "Q": wl._normal(cfg, "Q", t, (Tq, cfg.Hq, cfg.hd), 1.0, dt, self.dev),
            **kv,
            "cu_q": torch.from_numpy(cu_q).to(self.dev), "cu_kv": torch.from_numpy(cu_kv).to(self.dev),
            "H": wl.make_hidden(cfg, Tq, t, self.dev), "W": self.W, "tau": float(cfg.tau),
            "gamma": gamma,
        }
        logits = wl.library_logits(inp["H"], self.W)
        inp["q_probs"], inp["draft_tok"] = wl.simulate_drafts(cfg, logits, inp["cu_q"], self.sigma(t), cfg.tau, t)
        G = int(gamma.sum())
        inp["u_accept"] = torch.from_numpy(wl.open_uniform(wl._rng(cfg, "u_accept", t), G)).to(self.dev)
        inp["u_sample"] = torch.from_numpy(wl.open_uniform(wl._rng(cfg, "u_sample", t), self.N)).to(self.dev)
        return inp

    def set_round(self, t):
        """Step sizes of round t."""
        if self.step_decay > 0.0:
            f = float(t + 1) ** -self.step_decay
            self.eta, self.beta = self.eta0 * f, self.beta0 * f

    def next_allocation(self, t):
        """S(t+1) under the loop's policy (host integers); gs_schedule has already run."""
        N, C = self.N, self.C
        if self.policy == "goodspeed":
            return self.S_next.cpu().numpy().astype(np.int64)
        if self.policy == "fixed":
            return np.full(N, C // N, dtype=np.int64)
        rng = wl._rng(self.cfg, "random_s", t)
        return np.bincount(rng.integers(0, N, size=C), minlength=N).astype(np.int64)

    # ---------------------------------------------------------------- one round on the GPU
    def gpu_round(self, inp):
        cfg = self.cfg
        Tq = inp["Q"].shape[0]
        G = Tq - self.N
        O = self.O[:Tq]
        logits = self.logits[:Tq * cfg.V].view(Tq, cfg.V)
        if self.grow:
            B.gs_verify_attn_paged(inp["Q"], inp["K_pool"], inp["V_pool"], O, inp["cu_q"], inp["cu_kv"],
                                   inp["block_table"], self.max_kv_len, 1.0 / math.sqrt(cfg.hd), self.ws_attn,
                                   self.d_status)
        else:
            B.gs_verify_attn(inp["Q"], inp["K"], inp["V"], O, inp["cu_q"], inp["cu_kv"], self.max_kv_len,
                             1.0 / math.sqrt(cfg.hd), self.ws_attn, self.d_status)
        # the LM head writes the softmax statistics itself (when the shape has that kernel) and the
        # acceptance step skips its pass over the logits
        n_chunk = None
        if B.gs_lm_head_stats_pays(Tq):
            n_chunk = B.gs_lm_head_logits_stats(inp["H"], inp["W"], logits, inp["tau"], self.stats, self.ws_head,
                                                self.d_status)
        done = False
        if n_chunk is not None:
            done = B.gs_spec_accept_prestats(logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"],
                                             inp["u_sample"], inp["tau"], self.accepted, self.out_tok[:Tq], self.n_out,
                                             self.ratio[:G], self.p_tok[:G], self.stats, n_chunk, None,
                                             self.alpha_hat, self.X, self.eta, self.beta, ws=self.ws_acc,
                                             d_status=self.d_status)
        else:
            B.gs_lm_head_logits(inp["H"], inp["W"], logits, self.ws_head, self.d_status)
        if not done:
            B.gs_spec_accept(logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"], inp["u_sample"],
                             inp["tau"], self.accepted, self.out_tok[:Tq], self.n_out, self.ratio[:G], self.p_tok[:G],
                             None, self.alpha_hat, self.X, self.eta, self.beta, ws=self.ws_acc, d_status=self.d_status)
        B.gs_schedule(self.X, self.alpha_hat, self.C, self.S_next, self.s_min, self.s_max, self.d_status)
        return O, logits


def jain(x):
    x = np.asarray(x, dtype=np.float64)
    return float(x.sum() ** 2 / (len(x) * (x * x).sum()))


def run_closed_loop(cfg: wl.VerifyConfig, rounds: int, device="cuda", on_round=None, policy="goodspeed",
                    step_decay=0.0, curve_every=0, grow=False, max_len=None):
    """Runs `rounds` rounds; returns the report dict.  on_round(t, loop, inp, O, logits) is called after
    each round is enqueued and synchronised (tests use it to compare with the oracle in lock-step).
    curve_every > 0 adds the utility of the running mean goodput, U(x_bar(t)), every that many rounds."""
    loop = ClosedLoop(cfg, device, policy=policy, step_decay=step_decay, grow=grow, max_len=max_len)
    curve = []
    N = cfg.N
    tot = np.zeros(N)
    x_hist, X_hist = [], []
    gpu_ms = 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    drafted = 0
    for t in range(rounds):
        inp = loop.make_inputs(t, loop.S)
        loop.set_round(t)
        e0.record()
        O, logits = loop.gpu_round(inp)
        e1.record()
        torch.cuda.synchronize()
        gpu_ms += e0.elapsed_time(e1)
        assert int(loop.d_status.item()) == 0, "device status"
        if on_round is not None:
            on_round(t, loop, inp, O, logits)
        x = loop.n_out.cpu().numpy().astype(np.float64)
        tot += x
        drafted += int(loop.S.sum())
        x_hist.append(x)
        X_hist.append(loop.X.cpu().numpy().copy())
        loop.S = loop.next_allocation(t)
        if loop.grow:
            loop.append_outputs(x)
        if curve_every > 0 and (t + 1) % curve_every == 0:
            curve.append([t + 1, float(np.log(tot / (t + 1)).sum())])
    xbar = tot / rounds
    xh, Xh = np.asarray(x_hist), np.asarray(X_hist)
    ma = lambda a: np.convolve(a, np.ones(10) / 10, mode="valid") if len(a) >= 10 else a
    est_err = float(np.mean(np.abs(ma(xh.sum(1)) - ma(Xh.sum(1))))) if rounds >= 10 else None
    return {"policy": policy, "step_decay": step_decay, "utility_curve": curve,
            "final_cache_len": [int(v) for v in loop.len] if loop.grow else None,
            "rounds": rounds, "goodput_per_server": [float(v) for v in xbar], "jain": jain(xbar),
            "utility_sum_log": float(np.log(xbar).sum()), "gpu_ms_per_round": gpu_ms / rounds,
            "verified_tokens_per_s": drafted / (gpu_ms * 1e-3), "goodput_tokens_per_s": float(tot.sum()) / (gpu_ms * 1e-3),
            "estimated_vs_realised_goodput_ma10_abs_err": est_err,
            "final_alpha_hat": [float(v) for v in loop.alpha_hat.cpu().numpy()],
            "true_alpha_last_epoch": [float(v) for v in loop.true_alpha(rounds - 1)]}
