"""Buffer management around the four library calls of one verification round.

`VerifyRound` owns the output tensors, the workspaces and the estimator state (all torch
device tensors) for one fixed problem shape and enqueues the round on the current stream.
It holds no arithmetic: every step runs inside libgoodspeed.so.
"""
from __future__ import annotations

import math
from typing import Optional

import torch

from . import binding as B


def _ws(nbytes: int, device) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks; the library asks for 256.
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


class VerifyRound:
    """One verification round (attention, LM head, acceptance + estimators, next allocation)."""

    def __init__(self, *, N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, d, V, dtype, C,
                 eta=0.1, beta=0.5, alpha0=0.5, X0=1.0, alpha_min=1e-3, alpha_max=0.999,
                 device="cuda", want_margin=True):
        self.N, self.Tq, self.V, self.d = N, Tq, V, d
        self.Hq, self.Hkv, self.hd = Hq, Hkv, hd
        self.total_kv, self.max_kv_len = total_kv, max_kv_len
        self.C, self.eta, self.beta = C, eta, beta
        self.alpha_min, self.alpha_max = alpha_min, alpha_max
        self.dtype = dtype
        dt = B.GS_F32 if dtype == torch.float32 else B.GS_BF16
        dev = torch.device(device)
        Gamma = Tq - N
        self.O = torch.empty((Tq, Hq, hd), dtype=dtype, device=dev)
        self.logits = torch.empty((Tq, V), dtype=torch.float32, device=dev)
        self.accepted = torch.empty(N, dtype=torch.int32, device=dev)
        self.out_tok = torch.empty(Tq, dtype=torch.int32, device=dev)
        self.n_out = torch.empty(N, dtype=torch.int32, device=dev)
        self.ratio = torch.empty(max(Gamma, 1), dtype=torch.float32, device=dev)[:Gamma]
        self.p_tok = torch.empty(max(Gamma, 1), dtype=torch.float32, device=dev)[:Gamma]
        self.margin = torch.empty(Gamma + N, dtype=torch.float32, device=dev) if want_margin else None
        self.alpha_hat = torch.full((N,), float(alpha0), dtype=torch.float64, device=dev)
        self.X = torch.full((N,), float(X0), dtype=torch.float64, device=dev)
        self.S_next = torch.empty(N, dtype=torch.int32, device=dev)
        self.d_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws_attn = _ws(B.gs_verify_attn_workspace(N, Tq, total_kv, max_kv_len, Hq, Hkv, hd, dt), dev)
        self.ws_head = _ws(B.gs_lm_head_workspace(Tq, d, V, dt), dev)
        self.ws_acc = _ws(B.gs_spec_accept_workspace(N, Tq, V), dev)
        self.stats = _ws(B.gs_lm_head_stats_bytes(Tq), dev)
        self.scale = 1.0 / math.sqrt(hd)

    # the four steps, separately callable (the benchmark times them one by one as well)
    def attn(self, Q, K, V, cu_q, cu_kv):
        B.gs_verify_attn(Q, K, V, self.O, cu_q, cu_kv, self.max_kv_len, self.scale, self.ws_attn,
                         self.d_status)

    def head(self, H, W):
        B.gs_lm_head_logits(H, W, self.logits, self.ws_head, self.d_status)

    def accept(self, q_probs, draft_tok, cu_q, u_accept, u_sample, tau, logits=None, update=True):
        B.gs_spec_accept(self.logits if logits is None else logits, q_probs, draft_tok, cu_q,
                         u_accept, u_sample, tau, self.accepted, self.out_tok, self.n_out,
                         self.ratio, self.p_tok, self.margin,
                         self.alpha_hat if update else None, self.X if update else None,
                         self.eta, self.beta, self.alpha_min, self.alpha_max,
                         ws=self.ws_acc, d_status=self.d_status)

    def head_accept_fused(self, H, W, q_probs, draft_tok, cu_q, u_accept, u_sample, tau, update=True,
                          force=False) -> bool:
        """LM head with the softmax statistics in its epilogue, then the acceptance step on them (no
        second pass over the logits).  Shapes without such kernels, and shapes where the library
        expects the separate statistics pass to be faster (gs_lm_head_stats_pays; force=True overrides
        that), run the two plain calls.  Returns whether the fused kernels ran."""
        n_chunk = None
        if force or B.gs_lm_head_stats_pays(H.shape[0]):
            n_chunk = B.gs_lm_head_logits_stats(H, W, self.logits, tau, self.stats, self.ws_head, self.d_status)
        if n_chunk is not None:
            if B.gs_spec_accept_prestats(self.logits, q_probs, draft_tok, cu_q, u_accept, u_sample, tau,
                                         self.accepted, self.out_tok, self.n_out, self.ratio, self.p_tok,
                                         self.stats, n_chunk, self.margin,
                                         self.alpha_hat if update else None, self.X if update else None,
                                         self.eta, self.beta, self.alpha_min, self.alpha_max,
                                         ws=self.ws_acc, d_status=self.d_status):
                return True
            self.accept(q_probs, draft_tok, cu_q, u_accept, u_sample, tau, update=update)
            return False
        self.head(H, W)
        self.accept(q_probs, draft_tok, cu_q, u_accept, u_sample, tau, update=update)
        return False

    def schedule(self, s_min: Optional[torch.Tensor] = None, s_max: Optional[torch.Tensor] = None):
        B.gs_schedule(self.X, self.alpha_hat, self.C, self.S_next, s_min, s_max, self.d_status)

    def run(self, inp, s_min=None, s_max=None, fused=False):
        """Enqueue the whole round for the input dict made by workloads.make_step.  fused=True uses
        the LM head that writes the softmax statistics where the shape has one."""
        self.attn(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
        if fused:
            self.head_accept_fused(inp["H"], inp["W"], inp["q_probs"], inp["draft_tok"], inp["cu_q"],
                                   inp["u_accept"], inp["u_sample"], inp["tau"])
        else:
            self.head(inp["H"], inp["W"])
            self.accept(inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"], inp["u_sample"],
                        inp["tau"])
        self.schedule(s_min, s_max)

    @classmethod
    def for_inputs(cls, inp, C, **kw):
        Tq, Hq, hd = inp["Q"].shape
        total_kv, Hkv, _ = inp["K"].shape
        cu_kv = inp["cu_kv"].cpu()
        max_kv_len = int((cu_kv[1:] - cu_kv[:-1]).max())
        d, V = inp["W"].shape
        return cls(N=inp["cu_q"].numel() - 1, Tq=Tq, total_kv=total_kv, max_kv_len=max_kv_len,
                   Hq=Hq, Hkv=Hkv, hd=hd, d=d, V=V, dtype=inp["Q"].dtype, C=C,
                   device=inp["Q"].device, **kw)
