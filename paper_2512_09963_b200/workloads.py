"""Seeded synthetic inputs for one verification round.

This module stands in for the parts of the system that are outside the
verification hot path: the draft servers (which would sample draft tokens from
their own small models and ship the tokens plus full draft distributions) and
the transformer stack below the attention layer and the LM head.  It produces
arrays with the shapes, dtypes and value distributions of the five workload
configurations and nothing else: it contains no verification arithmetic
(no acceptance test, no correction sampling, no estimator, no scheduler) and it
is imported by neither the CUDA binding nor the CPU oracle.  Tests and the
benchmark call it once and hand the same arrays to both sides.

Draft-server simulation: the draft model is "the target plus noise".  The draft
logits of server i are (H W) + sigma_i * eps with eps ~ N(0,1), computed here
with a library fp32 matmul; the draft distribution is their softmax and the
draft tokens are drawn from it by inverse CDF with their own seeded uniforms.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field, replace
from typing import Callable, Optional, Sequence

import numpy as np
import torch

MASTER_SEED = 20251209


@dataclass(frozen=True)
class VerifyConfig:
    """Shape and distribution parameters of one workload configuration."""
    name: str
    N: int                      # draft servers
    d: int                      # model width
    Hq: int
    Hkv: int
    hd: int
    V: int
    dtype: str                  # "f32" or "bf16" for Q/K/V/H/W
    tau: float
    gamma_mode: str             # "list" | "uniform" | "alloc"
    gamma_list: Sequence[int] = ()
    gamma_lo: int = 1
    gamma_hi: int = 8
    C: int = 0                  # token budget (alloc mode / closed loop)
    prefix_mode: str = "fixed"  # "fixed" | "uniform" | "lognormal"
    prefix_lo: int = 2048
    prefix_hi: int = 2048
    prefix_median: int = 1024
    prefix_sigma_ln: float = 0.75
    sigma_list: Sequence[float] = ()
    sigma_lo: float = 0.2
    sigma_hi: float = 1.5
    seed_tag: str = ""


CONFIGS = {
    # Tiny fp32 step; also run with tau = 0 (greedy target).
    "cfg1": VerifyConfig("cfg1", N=4, d=256, Hq=4, Hkv=2, hd=64, V=1024, dtype="f32", tau=1.0,
                         gamma_mode="list", gamma_list=(1, 2, 3, 4),
                         prefix_mode="uniform", prefix_lo=64, prefix_hi=128,
                         sigma_list=(0.1, 0.5, 1.0, 2.0)),
    # Qwen3-32B-shaped layer and vocabulary.
    "cfg2": VerifyConfig("cfg2", N=8, d=5120, Hq=64, Hkv=8, hd=128, V=151936, dtype="bf16", tau=0.7,
                         gamma_mode="uniform", gamma_lo=1, gamma_hi=8,
                         prefix_mode="fixed", prefix_lo=2048, prefix_hi=2048,
                         sigma_lo=0.2, sigma_hi=1.5),
    # Heterogeneous large fan-in: gamma from a budgeted allocation, lognormal prefixes.
    "cfg3": VerifyConfig("cfg3", N=32, d=5120, Hq=64, Hkv=8, hd=128, V=151936, dtype="bf16", tau=1.0,
                         gamma_mode="alloc", gamma_lo=1, gamma_hi=16, C=256,
                         prefix_mode="lognormal", prefix_lo=128, prefix_hi=8192, prefix_median=1024,
                         sigma_lo=0.1, sigma_hi=2.0),
    # Llama-3-70B-shaped layer and vocabulary.
    "cfg4": VerifyConfig("cfg4", N=16, d=8192, Hq=64, Hkv=8, hd=128, V=128256, dtype="bf16", tau=1.0,
                         gamma_mode="uniform", gamma_lo=2, gamma_hi=8,
                         prefix_mode="fixed", prefix_lo=4096, prefix_hi=4096,
                         sigma_lo=0.2, sigma_hi=1.0),
    # Closed-loop scheduling at cfg2 layer shapes; gamma comes from the scheduler each round.
    "cfg5": VerifyConfig("cfg5", N=16, d=5120, Hq=64, Hkv=8, hd=128, V=151936, dtype="bf16", tau=0.7,
                         gamma_mode="given", C=128,
                         prefix_mode="fixed", prefix_lo=2048, prefix_hi=2048),
    # The paper's own deployment scale (Sec. V: 8 clients, token budget C = 20, up to 150 generated
    # tokens per prompt) on a 14B-class layer: 40 query heads over 8 KV heads (a group of 5, which
    # does not divide the 128 rows of a score tile), short ragged prefixes, small drafts.
    "cfg6": VerifyConfig("cfg6", N=8, d=5120, Hq=40, Hkv=8, hd=128, V=151936, dtype="bf16", tau=1.0,
                         gamma_mode="alloc", gamma_lo=1, gamma_hi=8, C=20,
                         prefix_mode="uniform", prefix_lo=200, prefix_hi=1200,
                         sigma_lo=0.2, sigma_hi=1.5),
}


def shrink(cfg: VerifyConfig, *, d=None, V=None, prefix_scale=None, N=None, name=None) -> VerifyConfig:
    """Same structure, smaller sizes (for cases the CPU oracle finishes in seconds)."""
    kw = {}
    if d is not None:
        kw["d"] = d
    if V is not None:
        kw["V"] = V
    if N is not None:
        kw["N"] = N
    if prefix_scale is not None:
        kw["prefix_lo"] = max(1, int(cfg.prefix_lo * prefix_scale))
        kw["prefix_hi"] = max(1, int(cfg.prefix_hi * prefix_scale))
        kw["prefix_median"] = max(1, int(cfg.prefix_median * prefix_scale))
    kw["name"] = name or (cfg.name + "_small")
    return replace(cfg, **kw)


def _seed(cfg: VerifyConfig, tensor: str, round_idx: int = 0) -> int:
    h = hashlib.sha256(f"{MASTER_SEED}/{cfg.name}{cfg.seed_tag}/{tensor}/{round_idx}".encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def _rng(cfg, tensor, round_idx=0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(_seed(cfg, tensor, round_idx)))


def _tgen(cfg, tensor, round_idx, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(cfg, tensor, round_idx))
    return g


def _normal(cfg, tensor, round_idx, shape, std, dtype, device):
    """N(0, std^2) array.  Small arrays come from numpy's PCG64 (stable across
    machines); arrays above 2^22 elements come from torch's generator on `device`."""
    n = int(np.prod(shape))
    if n <= (1 << 22):
        x = torch.from_numpy(_rng(cfg, tensor, round_idx).standard_normal(n, dtype=np.float32))
        x = x.reshape(shape).to(device)
    else:
        x = torch.randn(shape, generator=_tgen(cfg, tensor, round_idx, device),
                        device=device, dtype=torch.float32)
    return (x * std).to(dtype)


def open_uniform(rng: np.random.Generator, n: int) -> np.ndarray:
    """fp32 uniforms on the open interval: (k + 0.5) / 2^24, k in [0, 2^24)."""
    k = rng.integers(0, 1 << 24, size=n, dtype=np.int64)
    return ((k.astype(np.float64) + 0.5) / float(1 << 24)).astype(np.float32)


def draw_gamma(cfg: VerifyConfig, round_idx=0, allocator: Optional[Callable] = None) -> np.ndarray:
    """Draft lengths gamma_i.  In "alloc" mode the lengths are a budgeted allocation
    computed by `allocator(X, alpha_hat, C, s_min, s_max)` (passed in by the caller,
    so that this module holds no scheduler) on seeded estimator values."""
    if cfg.gamma_mode == "list":
        return np.asarray(cfg.gamma_list, dtype=np.int64)
    rng = _rng(cfg, "gamma", round_idx)
    if cfg.gamma_mode == "uniform":
        return rng.integers(cfg.gamma_lo, cfg.gamma_hi + 1, size=cfg.N, dtype=np.int64)
    if cfg.gamma_mode == "alloc":
        if allocator is None:
            raise ValueError("alloc mode needs an allocator callable")
        alpha_hat = rng.uniform(0.3, 0.95, size=cfg.N)
        X = rng.uniform(1.0, 6.0, size=cfg.N)
        s_min = np.full(cfg.N, cfg.gamma_lo, np.int32)
        s_max = np.full(cfg.N, cfg.gamma_hi, np.int32)
        return np.asarray(allocator(X, alpha_hat, cfg.C, s_min, s_max), dtype=np.int64)
    raise ValueError("gamma must be given for mode " + cfg.gamma_mode)


def draw_prefix(cfg: VerifyConfig, round_idx=0) -> np.ndarray:
    rng = _rng(cfg, "prefix", round_idx)
    if cfg.prefix_mode == "fixed":
        return np.full(cfg.N, cfg.prefix_lo, np.int64)
    if cfg.prefix_mode == "uniform":
        return rng.integers(cfg.prefix_lo, cfg.prefix_hi + 1, size=cfg.N, dtype=np.int64)
    z = rng.standard_normal(cfg.N)
    L = np.rint(cfg.prefix_median * np.exp(cfg.prefix_sigma_ln * z))
    return np.clip(L, cfg.prefix_lo, cfg.prefix_hi).astype(np.int64)


def draw_sigma(cfg: VerifyConfig, round_idx=0) -> np.ndarray:
    if len(cfg.sigma_list):
        return np.asarray(cfg.sigma_list, dtype=np.float64)
    return _rng(cfg, "sigma", round_idx).uniform(cfg.sigma_lo, cfg.sigma_hi, size=cfg.N)


def torch_dtype(cfg: VerifyConfig):
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def make_layer(cfg: VerifyConfig, device="cpu"):
    """The fixed tensors of the layer: LM-head weight W [d, V] ~ N(0, 1/d)."""
    return {"W": _normal(cfg, "W", 0, (cfg.d, cfg.V), cfg.d ** -0.5, torch_dtype(cfg), device)}


def make_w4_layer(cfg: VerifyConfig, group: int = 128, device="cpu"):
    """A synthetic 4-bit head weight in the library's storage format (include/goodspeed.h): random
    codes (every bit of every word drawn uniformly), per-group scales around 1 / (4.6 sqrt(d)) (so
    that the dequantised weight has about the variance 1/d of the bf16 layer) and zero points in
    6..9.  Returns qweight [d/8, V] int32, scales [d/group, V] bf16, zeros [d/group, V] uint8."""
    g = _tgen(cfg, "w4", 0, device)
    qweight = torch.randint(-(1 << 31), (1 << 31), (cfg.d // 8, cfg.V), generator=g, device=device, dtype=torch.int64).to(torch.int32)
    u = torch.rand((cfg.d // group, cfg.V), generator=g, device=device, dtype=torch.float32)
    scales = ((0.75 + 0.5 * u) / (4.6 * cfg.d ** 0.5)).to(torch.bfloat16)
    zeros = torch.randint(6, 10, (cfg.d // group, cfg.V), generator=g, device=device, dtype=torch.int64).to(torch.uint8)
    return {"qweight": qweight.contiguous(), "scales": scales.contiguous(), "zeros": zeros.contiguous(), "group": group}


def make_attention_inputs(cfg: VerifyConfig, gamma, prefix, round_idx=0, device="cpu"):
    """Q [T_q,H_q,hd], K/V [sum L_kv,H_kv,hd] ~ N(0,1) and the ragged offsets.
    L_kv,i = prefix_i + gamma_i + 1: the new positions' K/V are already appended."""
    gamma = np.asarray(gamma, np.int64)
    prefix = np.asarray(prefix, np.int64)
    n_new = gamma + 1
    cu_q = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    cu_kv = np.concatenate([[0], np.cumsum(prefix + n_new)]).astype(np.int32)
    Tq, Lkv = int(cu_q[-1]), int(cu_kv[-1])
    dt = torch_dtype(cfg)
    return {
        "Q": _normal(cfg, "Q", round_idx, (Tq, cfg.Hq, cfg.hd), 1.0, dt, device),
        "K": _normal(cfg, "K", round_idx, (Lkv, cfg.Hkv, cfg.hd), 1.0, dt, device),
        "V": _normal(cfg, "V", round_idx, (Lkv, cfg.Hkv, cfg.hd), 1.0, dt, device),
        "cu_q": torch.from_numpy(cu_q).to(device),
        "cu_kv": torch.from_numpy(cu_kv).to(device),
    }


def make_hidden(cfg: VerifyConfig, Tq: int, round_idx=0, device="cpu"):
    return _normal(cfg, "H", round_idx, (Tq, cfg.d), 1.0, torch_dtype(cfg), device)


def simulate_drafts(cfg: VerifyConfig, target_logits: torch.Tensor, cu_q, sigma, tau,
                    round_idx=0, greedy_draft=False):
    """Draft distributions and draft tokens from noisy copies of the target logits.

    target_logits [T_q, V] fp32 (any device).  Draft position j (1-based) of server i is
    conditioned like logits row cu_q[i]+j-1, so its draft distribution is
    softmax((row + sigma_i * eps) / tau_d); tau_d = tau, or 1 when tau == 0.
    Tokens are drawn by inverse CDF with seeded uniforms, or are argmax q when
    greedy_draft is set.  Returns q_probs [Gamma, V] fp32 and draft_tok [Gamma] int32.
    """
    dev = target_logits.device
    cu_q = np.asarray(cu_q.cpu() if hasattr(cu_q, "cpu") else cu_q, np.int64)
    N = len(cu_q) - 1
    V = target_logits.shape[1]
    rows, sig = [], []
    for i in range(N):
        gamma = int(cu_q[i + 1] - cu_q[i] - 1)
        rows += list(range(cu_q[i], cu_q[i] + gamma))
        sig += [float(sigma[i])] * gamma
    Gamma = len(rows)
    if Gamma == 0:
        return (torch.zeros((0, V), dtype=torch.float32, device=dev),
                torch.zeros((0,), dtype=torch.int32, device=dev))
    rows_t = torch.tensor(rows, dtype=torch.long, device=dev)
    sig_t = torch.tensor(sig, dtype=torch.float32, device=dev).unsqueeze(1)
    eps = torch.randn((Gamma, V), generator=_tgen(cfg, "draft_noise", round_idx, dev),
                      device=dev, dtype=torch.float32)
    tau_d = tau if tau > 0 else 1.0
    noisy = (target_logits.index_select(0, rows_t) + sig_t * eps) / tau_d
    del eps
    q = torch.softmax(noisy, dim=1)
    del noisy
    if greedy_draft:
        tok = torch.argmax(q, dim=1)
    else:
        u = torch.from_numpy(open_uniform(_rng(cfg, "draft_u", round_idx), Gamma)).to(dev)
        cdf = torch.cumsum(q.double(), dim=1)
        thr = (u.double() * cdf[:, -1]).unsqueeze(1)
        tok = torch.clamp((cdf <= thr).sum(dim=1), max=V - 1)
        del cdf
    return q.contiguous(), tok.to(torch.int32)


def library_logits(H: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """fp32 H @ W by the library matmul: only the draft-server simulator uses it."""
    return torch.matmul(H.float(), W.float())


def make_step(cfg: VerifyConfig, round_idx=0, device="cpu", gamma=None, sigma=None, tau=None,
              allocator=None, layer=None, synthetic_logits=False):
    """All inputs of one verification round as torch tensors on `device`.

    Returns a dict with Q, K, V, cu_q, cu_kv, H, W, q_probs, draft_tok, u_accept,
    u_sample, tau, gamma, prefix, sigma (+ target_logits_f32, the simulator's own
    fp32 product, kept so that per-kernel tests can feed identical logits to both
    sides).  synthetic_logits=True skips H @ W and draws the target logits
    directly from N(0,1) (for acceptance-kernel tests at sizes where the head
    product on the CPU would dominate the test time).
    """
    tau = cfg.tau if tau is None else tau
    gamma = draw_gamma(cfg, round_idx, allocator) if gamma is None else np.asarray(gamma, np.int64)
    prefix = draw_prefix(cfg, round_idx)
    sigma = draw_sigma(cfg, round_idx) if sigma is None else np.asarray(sigma, np.float64)
    out = make_attention_inputs(cfg, gamma, prefix, round_idx, device)
    Tq = int(out["cu_q"][-1])
    if layer is None and not synthetic_logits:
        layer = make_layer(cfg, device)
    if synthetic_logits:
        out["H"], out["W"] = None, None
        logits = _normal(cfg, "logits", round_idx, (Tq, cfg.V), 1.0, torch.float32, device)
    else:
        out["W"] = layer["W"]
        out["H"] = make_hidden(cfg, Tq, round_idx, device)
        logits = library_logits(out["H"], out["W"])
    out["target_logits_f32"] = logits
    q, tok = simulate_drafts(cfg, logits, out["cu_q"], sigma, tau, round_idx,
                             greedy_draft=(tau == 0))
    out["q_probs"], out["draft_tok"] = q, tok
    Gamma = int(gamma.sum())
    out["u_accept"] = torch.from_numpy(open_uniform(_rng(cfg, "u_accept", round_idx), Gamma)).to(device)
    out["u_sample"] = torch.from_numpy(open_uniform(_rng(cfg, "u_sample", round_idx), cfg.N)).to(device)
    out["tau"] = float(tau)
    out["gamma"], out["prefix"], out["sigma"] = gamma, prefix, sigma
    return out


# ----------------------------- closed loop (cfg5) --------------------------- #
def draw_true_alpha(cfg: VerifyConfig, epoch: int) -> np.ndarray:
    """True acceptance rates alpha_i ~ Beta(4, 2), redrawn i.i.d. at every epoch
    (an epoch is 100 rounds): piecewise-constant drift."""
    return _rng(cfg, "true_alpha", epoch).beta(4.0, 2.0, size=cfg.N)


def overlap_table(V: int, tau: float, sigmas: Sequence[float], rows: int = 8, seed_tag="calib"):
    """Mean overlap sum_v min(p, q) between p = softmax(l / tau) and
    q = softmax((l + sigma eps) / tau), l ~ N(0,1)^V, for each sigma: the acceptance
    probability a draft with that noise level would see.  Monte-Carlo, seeded."""
    g = torch.Generator().manual_seed(_seed(CONFIGS["cfg5"], f"{seed_tag}/{V}/{tau}", 0))
    l = torch.randn((rows, V), generator=g, dtype=torch.float64)
    eps = torch.randn((rows, V), generator=g, dtype=torch.float64)
    p = torch.softmax(l / tau, dim=1)
    vals = []
    for s in sigmas:
        q = torch.softmax((l + s * eps) / tau, dim=1)
        vals.append(float(torch.minimum(p, q).sum(dim=1).mean()))
    return np.asarray(vals)


def calibrate_sigma(alpha_true: np.ndarray, V: int, tau: float) -> np.ndarray:
    """Noise level whose overlap equals the wanted acceptance rate (monotone table lookup)."""
    grid = np.concatenate([[0.0], np.geomspace(0.02, 6.0, 40)])
    ov = overlap_table(V, tau, grid)
    order = np.argsort(ov)
    return np.interp(np.clip(alpha_true, ov.min(), ov.max()), ov[order], grid[order])
