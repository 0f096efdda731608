"""gs_spec_accept_static against gs_spec_accept.

Some users of the library cannot give it a workspace: they run where device memory may not be
allocated (a frozen memory pool, borrowed buffers only).  For them the acceptance pass exists in a
form whose scratch is a fixed array inside the library.  This test calls that form through the C
ABI twice in a row, on two different rounds, and requires every output to equal what the ordinary
entry point gives for the same inputs; the second call also shows that whatever the first left in
the shared array does no harm.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2512_09963_b200 import binding as B
from paper_2512_09963_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
OUTS = ("accepted", "out_tok", "n_out", "ratio", "p_tok", "margin", "alpha_hat", "X")


def _buffers(N, Tq):
    G = Tq - N
    return dict(accepted=torch.full((N,), -7, dtype=torch.int32, device=DEV),
                out_tok=torch.full((Tq,), -7, dtype=torch.int32, device=DEV),
                n_out=torch.full((N,), -7, dtype=torch.int32, device=DEV),
                ratio=torch.full((G,), -7.0, dtype=torch.float32, device=DEV),
                p_tok=torch.full((G,), -7.0, dtype=torch.float32, device=DEV),
                margin=torch.full((G + N,), -7.0, dtype=torch.float32, device=DEV),
                alpha_hat=torch.full((N,), 0.5, dtype=torch.float64, device=DEV),
                X=torch.ones(N, dtype=torch.float64, device=DEV))


def _round(cfg, round_idx, tau):
    inp = wl.make_step(cfg, round_idx=round_idx, tau=tau, synthetic_logits=True)
    return {k: (v.to(DEV) if isinstance(v, torch.Tensor) else v) for k, v in inp.items()}


def test_static_scratch_entry_point_matches_workspace_entry_point():
    cfg = wl.shrink(wl.CONFIGS["cfg2"], V=20000, d=64, prefix_scale=0.01, name="no_alloc")
    for round_idx, tau in ((0, 0.7), (1, 1.0)):            # two calls in a row, different data
        d = _round(cfg, round_idx, tau)
        logits = d["target_logits_f32"].contiguous()
        Tq, V = logits.shape
        N = cfg.N
        assert B.gs_spec_accept_workspace(N, Tq, V) <= B.gs_spec_accept_static_capacity()
        want, got = _buffers(N, Tq), _buffers(N, Tq)
        ws = torch.empty(B.gs_spec_accept_workspace(N, Tq, V), dtype=torch.uint8, device=DEV)
        st_a = torch.zeros(1, dtype=torch.int32, device=DEV)
        st_b = torch.zeros(1, dtype=torch.int32, device=DEV)
        args = (logits, d["q_probs"], d["draft_tok"], d["cu_q"], d["u_accept"], d["u_sample"], tau)
        B.gs_spec_accept(*args, want["accepted"], want["out_tok"], want["n_out"], want["ratio"], want["p_tok"],
                         want["margin"], want["alpha_hat"], want["X"], 0.1, 0.5, ws=ws, d_status=st_a)
        B.gs_spec_accept_static(*args, got["accepted"], got["out_tok"], got["n_out"], got["ratio"], got["p_tok"],
                                got["margin"], got["alpha_hat"], got["X"], 0.1, 0.5, d_status=st_b)
        torch.cuda.synchronize()
        assert int(st_a.item()) == 0 and int(st_b.item()) == 0
        for k in OUTS:      # same kernels, same summation order: identical bits, far inside 1e-5
            assert torch.equal(want[k], got[k]), (round_idx, k)
        assert int(got["accepted"].min()) >= 0 and int(got["n_out"].min()) >= 1


def test_static_scratch_entry_point_rejects_oversized_problems():
    cap = B.gs_spec_accept_static_capacity()
    N, V = 4, 151936
    Tq = 8000                                    # chunk statistics alone exceed the fixed array
    assert B.gs_spec_accept_workspace(N, Tq, V) > cap
    dummy = torch.zeros(16, dtype=torch.float32, device=DEV)
    L = B.lib()
    code = L.gs_spec_accept_static(dummy.data_ptr(), None, None, dummy.data_ptr(), None, dummy.data_ptr(), 1.0,
                                   N, Tq, V, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), None, None,
                                   None, None, None, 0.1, 0.5, 1e-3, 0.999, None, None)
    assert code == 4                             # GS_ERR_WORKSPACE, nothing launched
    torch.cuda.synchronize()
