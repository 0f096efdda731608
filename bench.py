#!/usr/bin/env python
"""Benchmark of one GoodSpeed verification round on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config cfg2]

A step is one pass of the whole hot path (verify attention, LM head, acceptance + estimator
update, next allocation) over one batch of synthetic drafts.  The default workload is the
Qwen3-32B-shaped configuration (8 servers, prefix 2048, d=5120, V=151936, bf16).  Rank 0 prints
one JSON line.  `--impl reference` times the fp64 CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import contextlib
import dataclasses
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2512_09963_b200 import workloads as wl  # noqa: E402

METRIC = "verified tokens/sec per verify step"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
ETA, BETA = 0.1, 0.5

# DRAM traffic of the LM-head kernel from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum
# per launch), keyed by the sha256 of the kernel's sources (lm_head_pair.cuh and the PTX wrappers it uses)
# as they were when it was taken; a changed kernel reports null.
# cfg2's full launch is within ncu's single-pass size rule only for the launch list, so the counters
# were taken on a smaller vocabulary and scale with the units processed (see profiles/).
# small case (V = 32768), the kernel with the statistics epilogue: 336.082 MB read + 3.510 MB written
# per launch (part of the logits was still in L2 when the capture ended), times 151936/32768
NCU_TRAFFIC = {"76d66cc5d5348fec": {"cfg2": 1574592297}}


def _kernel_hash():
    h = hashlib.sha256()
    for f in ("lm_head_pair.cuh", "sm100_ptx.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2512_09963_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured", p
    return FALLBACK_HBM_GBS, "fallback", {}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.samples = []
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [s for t, s in self.samples if t0 - 0.05 <= t <= t1 + 0.15] or [s for _, s in self.samples]
        sm, mx, reasons, power = [], [], set(), []
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def subset_servers(inp, n_srv):
    """The first n_srv servers of a step's inputs (host tensors): a bounded sample for the CPU oracle."""
    cu_q, cu_kv = inp["cu_q"].numpy(), inp["cu_kv"].numpy()
    q1, k1 = int(cu_q[n_srv]), int(cu_kv[n_srv])
    g1 = q1 - n_srv
    out = dict(inp)
    out.update(Q=inp["Q"][:q1], H=inp["H"][:q1], K=inp["K"][:k1], V=inp["V"][:k1],
               cu_q=inp["cu_q"][:n_srv + 1], cu_kv=inp["cu_kv"][:n_srv + 1],
               q_probs=inp["q_probs"][:g1], draft_tok=inp["draft_tok"][:g1], u_accept=inp["u_accept"][:g1],
               u_sample=inp["u_sample"][:n_srv], gamma=inp["gamma"][:n_srv])
    return out


def oracle_round(inp, N, C):
    from oracle import goodspeed_oracle as orc
    host = dict(inp)
    host["tau"] = float(np.float32(inp["tau"]))
    return orc.ref_verify_round(host, np.full(N, 0.5), np.ones(N), ETA, BETA, C)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info()]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def library_allocator(device):
    """Budgeted allocation for workloads whose draft lengths come from a scheduler run: the
    library's own gs_schedule (bit-identical to the oracle's greedy, see the GPU tests)."""
    def alloc(X, alpha_hat, C, s_min, s_max):
        from paper_2512_09963_b200 import binding as B
        t = lambda a, dt: torch.as_tensor(np.asarray(a), dtype=dt, device=device)
        S = torch.empty(len(X), dtype=torch.int32, device=device)
        B.gs_schedule(t(X, torch.float64), t(alpha_hat, torch.float64), C, S, t(s_min, torch.int32),
                      t(s_max, torch.int32))
        torch.cuda.synchronize()
        return S.cpu().numpy()
    return alloc


def make_host_inputs(cfg, device):
    alloc = library_allocator(device) if cfg.gamma_mode == "alloc" else None
    dev_inp = wl.make_step(cfg, device=device, allocator=alloc)
    host = {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in dev_inp.items()}
    return dev_inp, host


# ------------------------------------------------------------------------------------------------
def config_dict(cfg, inp, n_gpus):
    """What the workload is: the same keys and values in both arms."""
    N = cfg.N
    Tq = int(inp["cu_q"][-1])
    return {"workload": cfg.name, "servers_per_gpu": N, "draft_tokens_per_gpu": int(inp["gamma"].sum()),
            "verify_positions": Tq, "prefix": int(inp["prefix"][0]) if cfg.prefix_mode == "fixed" else
            f"{int(inp['prefix'].min())}..{int(inp['prefix'].max())}", "d": cfg.d, "V": cfg.V,
            "heads": f"{cfg.Hq}q/{cfg.Hkv}kv x {cfg.hd}", "temperature": float(inp["tau"]),
            "parallelism": f"dp{n_gpus} over draft servers",
            "l2": "inputs larger than L2: the head weight (1.5-2.1 GB) streams through L2 every step and evicts "
                  "the KV cache and logits"}


def run_reference(args, cfg, rank, world):
    """The CPU oracle as it stands, on a bounded sample of the same workload."""
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    _, host = make_host_inputs(cfg, dev)
    if dev == "cuda":
        torch.cuda.empty_cache()
    C = cfg.C if cfg.C else 8 * cfg.N
    t0 = time.time()
    oracle_round(subset_servers(host, 1), 1, 8)            # calibration: one server
    t1 = time.time() - t0
    budget = 150.0 / max(1, args.steps + args.warmup)      # seconds per step
    n_srv = int(max(1, min(cfg.N, budget // max(t1, 1e-3))))
    sample = subset_servers(host, n_srv)
    gamma = int(sample["gamma"].sum())
    for _ in range(args.warmup):
        oracle_round(sample, n_srv, C)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_round(sample, n_srv, C)
    dt = (time.time() - t0) / max(1, args.steps)
    val = gamma / dt
    cores = blas_threads()
    desc = f"servers 0..{n_srv - 1} of {cfg.N} ({gamma} draft tokens): their attention, LM-head rows against the full W, acceptance, estimators, schedule"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(cfg, host, args.gpus),
            "arm": "fp64 CPU oracle on host cores, bounded sample of the workload (see cpu_baseline.sample)",
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
def head_roofline(T, d, V, es, us, peak_hbm, peaks):
    """The LM head against the roofline that binds it: time / max(t_HBM, t_tensor), with both raw
    fractions.  Tensor peak: the measured bf16 burst figure (the kernel is timed alone, for tens of
    milliseconds); the sustained figure is quoted beside it."""
    by = d * V * es + T * V * 4 + T * d * es
    fl = 2.0 * T * d * V
    tf_burst = float(peaks.get("bf16_tflops", 1590.0))
    tf_sust = float(peaks.get("bf16_tflops_sustained", 1400.0))
    t_hbm = by / (peak_hbm * 1e9) * 1e6              # us
    t_tc = fl / (tf_burst * 1e12) * 1e6
    gbs, tfs = by / us / 1e3, fl / us / 1e6
    tensor = t_tc > t_hbm
    return {"bound": "tensor" if tensor else "hbm",
            "achieved": tfs if tensor else gbs, "peak": tf_burst if tensor else peak_hbm,
            "unit": "TFLOP/s" if tensor else "GB/s", "frac": (tfs / tf_burst) if tensor else (gbs / peak_hbm),
            "frac_of_binding_roofline": max(t_hbm, t_tc) / us,
            "frac_hbm": gbs / peak_hbm, "frac_bf16_burst": tfs / tf_burst, "frac_bf16_sustained": tfs / tf_sust,
            "t_hbm_us": t_hbm, "t_tensor_us": t_tc, "duration_us": us, "algorithmic_bytes": by, "flops": fl,
            "gbs": gbs, "tensor_tflops": tfs}


def measure_config(args, cfg, rank, world, local_rank, steps, warmup, detail):
    """One workload on this rank's GPU: W warm-up steps, K timed steps, per-kernel durations.
    detail=True adds the end-to-end leg, the CPU baseline and the parity check (single GPU only)."""
    from paper_2512_09963_b200 import binding as B
    from paper_2512_09963_b200.runner import VerifyRound
    from paper_2512_09963_b200.sharded import ShardedScheduler, aggregate_throughput
    import torch.distributed as dist

    dev = torch.device("cuda", local_rank)
    cfg_r = dataclasses.replace(cfg, seed_tag=f"/rank{rank}") if world > 1 else cfg
    inp, host = make_host_inputs(cfg_r, dev)
    N, Tq = cfg.N, int(inp["cu_q"][-1])
    Gamma = int(inp["gamma"].sum())
    C = cfg.C if cfg.C else 8 * N
    rnd = VerifyRound.for_inputs(inp, C=C, eta=ETA, beta=BETA)
    s_min = torch.ones(N * world, dtype=torch.int32, device=dev)
    s_max = torch.full((N * world,), max(8, cfg.gamma_hi), dtype=torch.int32, device=dev)
    # multi-GPU: servers are sharded over ranks; only the scheduler couples them, through an
    # all-gather of the estimator state (16 bytes per server) before every rank runs the same greedy.
    sharded = ShardedScheduler(N, rank, world, C * world, dev, s_min, s_max) if world > 1 else None

    def reset_state():
        rnd.alpha_hat.fill_(0.5)
        rnd.X.fill_(1.0)

    # Does this shape have the LM head that writes the softmax statistics in its epilogue (then the
    # acceptance step does not read the logits a second time)?
    fused = False
    if not args.no_fused_stats:
        fused = rnd.head_accept_fused(inp["H"], inp["W"], inp["q_probs"], inp["draft_tok"], inp["cu_q"],
                                      inp["u_accept"], inp["u_sample"], inp["tau"], update=False)
        torch.cuda.synchronize()
    n_chunk_fused = None

    def head_call():
        nonlocal n_chunk_fused
        if fused:
            n_chunk_fused = B.gs_lm_head_logits_stats(inp["H"], inp["W"], rnd.logits, inp["tau"], rnd.stats, rnd.ws_head,
                                                      rnd.d_status)
        else:
            rnd.head(inp["H"], inp["W"])

    def accept_call():
        if fused:
            ok = B.gs_spec_accept_prestats(rnd.logits, inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"],
                                           inp["u_sample"], inp["tau"], rnd.accepted, rnd.out_tok, rnd.n_out, rnd.ratio,
                                           rnd.p_tok, rnd.stats, n_chunk_fused, rnd.margin, rnd.alpha_hat, rnd.X,
                                           rnd.eta, rnd.beta, rnd.alpha_min, rnd.alpha_max, ws=rnd.ws_acc,
                                           d_status=rnd.d_status)
            assert ok
        else:
            rnd.accept(inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"], inp["u_sample"], inp["tau"])

    def step():
        rnd.attn(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
        head_call()
        accept_call()
        if world == 1:
            rnd.schedule(s_min, s_max)
        else:
            sharded.step(rnd.alpha_hat, rnd.X, rnd.S_next, rnd.d_status)

    # ---- launches per step and a first (eager) run
    reset_state()
    c0 = B.gs_launch_count()
    step()
    torch.cuda.synchronize()
    launches_per_step = B.gs_launch_count() - c0
    assert int(rnd.d_status.item()) == 0, "device status after the first step"
    first = {k: getattr(rnd, k).clone() for k in ("accepted", "out_tok", "n_out", "S_next")}

    # ---- CUDA graph of one step (single GPU only)
    graph = None
    if world == 1 and not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
    run_step = graph.replay if graph is not None else step

    # ---- timed region: W warm-up steps, then exactly K steps between barriers/synchronisations
    for _ in range(warmup):
        run_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t_wall0 = time.time()
    e0.record()
    for _ in range(steps):
        run_step()
    e1.record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms_total, gamma_all = aggregate_throughput(e0.elapsed_time(e1), Gamma, dev)
    ms_step = ms_total / steps
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None

    # ---- per-kernel durations.  The LM head is long enough to be timed eagerly with events around
    # the call inside a running step sequence.  The short calls are timed as CUDA-graph replays of
    # [L2 flush; call] minus replays of [L2 flush] alone, so that neither the host's launch cost nor a
    # warm L2 enters the figure.
    n_k = min(steps, 30)
    calls = {
        "verify_attn": lambda: rnd.attn(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"]),
        "lm_head_logits": head_call,
        "spec_accept": accept_call,
        "gs_schedule": lambda: rnd.schedule(s_min[:N], s_max[:N]),
    }
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_k)]
    for i in range(n_k):
        calls["verify_attn"]()
        evs[i][0].record(); calls["lm_head_logits"](); evs[i][1].record()
        calls["spec_accept"](); calls["gs_schedule"]()
    torch.cuda.synchronize()
    k_us = {"lm_head_logits": float(np.mean([e[0].elapsed_time(e[1]) for e in evs])) * 1e3}
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    flush_sink = torch.zeros((), dtype=torch.int64, device=dev)

    def flush():
        # read 256 MB: L2 ends up full of clean lines (a write flush would leave dirty lines whose
        # write-back the next kernel pays for)
        flush_sink.copy_(flush_buf.view(torch.int64).sum())

    def graph_of(fn):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            flush()
            if fn is not None:
                fn()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            flush()
            if fn is not None:
                fn()
        return g

    def replay_us(g, n=20):
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / n

    base_us = replay_us(graph_of(None))
    for nme in ("verify_attn", "spec_accept", "gs_schedule"):
        k_us[nme] = max(replay_us(graph_of(calls[nme])) - base_us, 0.0)
    del flush_buf, flush_sink

    # ---- rooflines
    peak, peak_kind, peaks = _peaks()
    d, V = cfg.d, cfg.V
    es = 2 if cfg.dtype == "bf16" else 4
    total_kv = int(inp["K"].shape[0])
    bytes_attn = 2 * total_kv * cfg.Hkv * cfg.hd * es + 2 * Tq * cfg.Hq * cfg.hd * es
    # with the statistics from the LM head's epilogue the pass over all logits is gone
    bytes_acc = N * V * 8 if fused else Tq * V * 4 + N * V * 8
    bytes_acc_two_pass = Tq * V * 4 + N * V * 8
    head = head_roofline(Tq, d, V, es, k_us["lm_head_logits"], peak, peaks)
    khash = _kernel_hash()
    roofline = {"kernel": ("lm_head_pair_kernel with the statistics epilogue" if fused else "lm_head_pair_kernel"),
                "bound": head["bound"], "achieved": head["achieved"], "peak": head["peak"], "unit": head["unit"],
                "frac": head["frac"],
                "peak_source": (f"{peak_kind} (MEASURED_PEAKS.json " + ("bf16_tflops, burst" if head["bound"] == "tensor" else "hbm_gbs") + ")")
                if peak_kind == "measured" else "fallback 6650 GB/s / 1590 TFLOP/s",
                "traffic": NCU_TRAFFIC.get(khash, {}).get(cfg.name),
                "algorithmic_bytes": head["algorithmic_bytes"], "duration_us": head["duration_us"],
                "frac_of_binding_roofline": head["frac_of_binding_roofline"], "frac_hbm": head["frac_hbm"],
                "frac_bf16_burst": head["frac_bf16_burst"], "frac_bf16_sustained": head["frac_bf16_sustained"],
                "t_hbm_us": head["t_hbm_us"], "t_tensor_us": head["t_tensor_us"], "tensor_tflops": head["tensor_tflops"]}
    kernels = {
        "verify_attn": {"us": k_us["verify_attn"], "algorithmic_bytes": bytes_attn,
                        "gbs": bytes_attn / k_us["verify_attn"] / 1e3, "frac_hbm": bytes_attn / k_us["verify_attn"] / 1e3 / peak},
        "lm_head_logits": {"us": k_us["lm_head_logits"], "algorithmic_bytes": head["algorithmic_bytes"], "gbs": head["gbs"],
                           "bound": head["bound"], "frac_of_binding_roofline": head["frac_of_binding_roofline"],
                           "frac_hbm": head["frac_hbm"], "frac_bf16_burst": head["frac_bf16_burst"],
                           "frac_bf16_sustained": head["frac_bf16_sustained"]},
        "spec_accept": {"us": k_us["spec_accept"], "algorithmic_bytes": bytes_acc,
                        "gbs": bytes_acc / k_us["spec_accept"] / 1e3, "frac_hbm": bytes_acc / k_us["spec_accept"] / 1e3 / peak,
                        "two_pass_bytes": bytes_acc_two_pass,
                        "frac_hbm_on_two_pass_bytes": bytes_acc_two_pass / k_us["spec_accept"] / 1e3 / peak},
        "gs_schedule": {"us": k_us["gs_schedule"]},
    }
    # ---- the same head on a 4-bit weight (codes + per-group scales and zero points), timed alone: the
    # weight stream is a quarter of the bf16 one
    w4 = None
    if detail and world == 1 and cfg.dtype == "bf16" and d % 128 == 0 and V % 16 == 0 and not args.profile_small:
        layer = wl.make_w4_layer(cfg, 128, dev)
        lg = torch.empty((min(Tq, 256), V), dtype=torch.float32, device=dev)
        Hs = inp["H"][:min(Tq, 256)].contiguous()
        f4 = lambda: B.gs_lm_head_logits_w4(Hs, layer["qweight"], layer["scales"], layer["zeros"], 128, lg, rnd.d_status)
        for _ in range(3):
            f4()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(20):                       # 390 MB of packed weights per launch: the inputs are cold
            f4()
        b.record()
        torch.cuda.synchronize()
        us4 = a.elapsed_time(b) * 1e3 / 20
        Tw = lg.shape[0]
        by4 = d * V // 2 + (d // 128) * V * 3 + Tw * V * 4 + Tw * d * 2
        w4 = {"entry_point": "gs_lm_head_logits_w4", "rows": Tw, "group": 128, "us": us4, "algorithmic_bytes": by4,
              "gbs": by4 / us4 / 1e3, "frac_hbm": by4 / us4 / 1e3 / peak, "bf16_head_us": k_us["lm_head_logits"],
              "speedup_over_bf16_head": k_us["lm_head_logits"] / us4}
        # ... and the whole step with that head: attention, 4-bit head, acceptance (statistics pass + finish on
        # its logits), scheduler, as a CUDA-graph replay like the headline.  The synthetic codes are unrelated
        # to the drafts, so nearly every first draft is rejected; the metric counts verified drafts per second.
        if not args.no_graph:
            lg_full = torch.empty((Tq, V), dtype=torch.float32, device=dev)

            def step4():
                rnd.attn(inp["Q"], inp["K"], inp["V"], inp["cu_q"], inp["cu_kv"])
                B.gs_lm_head_logits_w4(inp["H"], layer["qweight"], layer["scales"], layer["zeros"], 128, lg_full, rnd.d_status)
                rnd.accept(inp["q_probs"], inp["draft_tok"], inp["cu_q"], inp["u_accept"], inp["u_sample"], inp["tau"],
                           logits=lg_full, update=False)
                rnd.schedule(s_min, s_max)

            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step4()
            torch.cuda.current_stream().wait_stream(side)
            g4 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g4):
                step4()
            for _ in range(5):
                g4.replay()
            torch.cuda.synchronize()
            n4 = 200
            a.record()
            for _ in range(n4):
                g4.replay()
            b.record()
            torch.cuda.synchronize()
            assert int(rnd.d_status.item()) == 0, "device status after the steps with the 4-bit head"
            step4_us = a.elapsed_time(b) * 1e3 / n4
            w4["step_us"] = step4_us
            w4["step_verified_tokens_per_s"] = Gamma / (step4_us * 1e-6)
            w4["step_speedup_over_bf16_step"] = ms_step * 1e3 / step4_us
            del lg_full, g4
        del layer, lg, Hs
    out = {"cfg": cfg, "inp": inp, "host": host, "rnd": rnd, "first": first, "N": N, "Tq": Tq, "Gamma": Gamma, "C": C, "w4": w4,
           "ms_step": ms_step, "gamma_all": gamma_all, "clocks": clocks, "kernels": kernels, "roofline": roofline,
           "fused": fused, "graph": graph is not None, "launches_per_step": int(launches_per_step), "khash": khash,
           "s_min": s_min, "s_max": s_max, "step": step, "reset_state": reset_state, "total_kv": total_kv,
           "e2e": None, "cpu": None, "parity": None}
    if not detail or world > 1:
        return out

    # ---- end to end through the host-buffer entry point (pinned inputs, results read back each step)
    if not args.profile_small:
        desc = B.RoundDesc(N=N, Tq=Tq, total_kv=total_kv, max_kv_len=rnd.max_kv_len, Hq=cfg.Hq, Hkv=cfg.Hkv,
                           hd=cfg.hd, d=d, V=V, C=C, dt=B.GS_BF16 if cfg.dtype == "bf16" else B.GS_F32,
                           scale=cfg.hd ** -0.5, temperature=float(inp["tau"]), eta=ETA, beta=BETA,
                           alpha_min=1e-3, alpha_max=0.999)
        ws = torch.empty(B.gs_verify_round_workspace(desc), dtype=torch.uint8, device=dev)
        pin = {k: host[k].contiguous().pin_memory() for k in
               ("Q", "H", "q_probs", "draft_tok", "u_accept", "u_sample", "cu_q", "cu_kv")}
        outs = {k: torch.empty(n, dtype=torch.int32).pin_memory() for k, n in
                (("accepted", N), ("out_tok", Tq), ("n_out", N), ("S_next", N), ("status", 1))}
        # Bytes that cross the bus host -> device per step.  Pinned draft distributions are not copied:
        # the acceptance kernels read q(s_j) of each drafted token (a 32-byte sector each) and at most one
        # row per server where they lie; everything else is staged with copies.
        in_place = B.gs_verify_round_reads_in_place(pin["q_probs"])
        staged = sum(t.numel() * t.element_size() for k, t in pin.items() if not (in_place and k == "q_probs"))
        pulled = (N * V * 4 + 32 * Gamma) if in_place else 0
        if in_place:        # ... and the first rows of every server, which the copy engine brings over meanwhile
            near = B.gs_verify_round_near_rows(desc)
            staged += int(np.minimum(np.asarray(host["gamma"]), near).sum()) * V * 4
        h2d = staged + pulled
        d2h = sum(t.numel() * t.element_size() for t in outs.values())

        def e2e_step():
            B.gs_verify_round_host(desc, pin["Q"], pin["H"], pin["q_probs"], pin["draft_tok"], pin["u_accept"],
                                   pin["u_sample"], pin["cu_q"], pin["cu_kv"], inp["K"], inp["V"], inp["W"],
                                   rnd.alpha_hat, rnd.X, s_min, s_max, ws, outs["accepted"], outs["out_tok"],
                                   outs["n_out"], outs["S_next"], outs["status"])
            torch.cuda.current_stream().synchronize()

        reset_state()
        e2e_step()
        e2e_ok = (int(outs["status"][0]) == 0 and torch.equal(outs["accepted"], first["accepted"].cpu())
                  and torch.equal(outs["out_tok"], first["out_tok"].cpu()))
        n_e = min(steps, 30)
        for _ in range(3):
            e2e_step()
        t0 = time.time()
        for _ in range(n_e):
            e2e_step()
        dt = (time.time() - t0) / n_e
        out["e2e"] = {"value": Gamma / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "ms_per_step": dt * 1e3, "matches_device_path": bool(e2e_ok),
                      "h2d_detail": {"copied": staged, "read_in_place_by_kernels_at_most": pulled,
                                     "draft_distributions_bytes": pin["q_probs"].numel() * 4,
                                     "draft_distributions": "read in place (pinned host memory)" if in_place else "copied"}}
        if in_place:        # the same with the distributions staged by a copy, for comparison
            B.gs_verify_round_configure(False)
            try:
                for _ in range(3):
                    e2e_step()
                t0 = time.time()
                for _ in range(n_e):
                    e2e_step()
                out["e2e"]["ms_per_step_with_distributions_copied"] = (time.time() - t0) / n_e * 1e3
            finally:
                B.gs_verify_round_configure(True)
        del ws

    # ---- CPU baseline = the oracle on the host cores, and a parity check of this launch configuration
    if not args.skip_cpu_baseline:
        import parity_utils as pu
        t0 = time.time()
        ref = oracle_round(host, N, C)
        dt = time.time() - t0
        out["cpu"] = {"value": Gamma / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "seconds": dt,
                      "sample": f"the whole {cfg.name} step once ({Gamma} draft tokens, {Tq} verify positions)"}
        got = {k: first[k].cpu().numpy() for k in ("accepted", "out_tok", "n_out")}
        reset_state()
        step()
        torch.cuda.synchronize()
        got.update(ratio=rnd.ratio.cpu().numpy(), p_tok=rnd.p_tok.cpu().numpy())
        tau = float(np.float32(inp["tau"]))
        try:
            pu.assert_close_rel(rnd.O, ref["O"], "attention")
            pu.assert_close_rel(rnd.logits, ref["logits"], "logits")
            slack = pu.chain_slack(rnd.logits, ref["logits"], tau)
            with contextlib.redirect_stdout(sys.stderr):       # the near-tie lines go to stderr; stdout carries the JSON line only
                log = pu.compare_accept(got, ref, ref["logits"], host["q_probs"], host["cu_q"].numpy(),
                                        host["u_sample"], tau, V, slack=slack)
            out["parity"] = {"status": "ok", "near_tie_band": pu.NEAR_TIE + slack, **pu.log_for_json(log)}
        except AssertionError as ex:
            out["parity"] = {"status": "FAILED", "detail": str(ex)[:300]}
    return out


def run_ours(args, cfg, rank, world, local_rank):
    from paper_2512_09963_b200 import binding as B
    from paper_2512_09963_b200 import build as gs_build
    import torch.distributed as dist

    if rank == 0:
        gs_build.build()
    if world > 1:
        dist.barrier()
    B.lib()
    B.gs_set_dependent_launch(not args.no_dependent_launch)
    m = measure_config(args, cfg, rank, world, local_rank, args.steps, args.warmup, detail=True)
    ms_step, first, inp = m["ms_step"], m["first"], m["inp"]
    goodput = float(first["n_out"].sum().item()) * world / (ms_step * 1e-3)
    config = config_dict(cfg, m["host"], world)
    launch_info = {"launch": "CUDA graph replay of the four calls" if m["graph"] else "eager, four calls per step",
                   "softmax_statistics": "LM-head epilogue (gs_lm_head_logits_stats + gs_spec_accept_prestats)" if m["fused"]
                   else "statistics pass of gs_spec_accept"}
    # ---- the other single-GPU workloads, on the same box in the same run: step time and per-kernel rooflines
    others = {}
    extra = [] if (world > 1 or args.profile_small or args.only_headline) else [c for c in ("cfg3", "cfg4") if c != cfg.name]
    del m["inp"], m["host"], m["rnd"], m["step"], m["reset_state"]
    inp = None
    for name in extra:
        torch.cuda.empty_cache()
        c2 = wl.CONFIGS[name]
        k = min(args.steps, 300)
        m2 = measure_config(args, c2, rank, world, local_rank, k, args.warmup, detail=False)
        others[name] = {"config": config_dict(c2, m2["host"], 1), "steps": k, "ms_per_step": m2["ms_step"],
                        "value": m2["gamma_all"] / (m2["ms_step"] * 1e-3), "unit": UNIT,
                        "goodput_tokens_per_s": float(m2["first"]["n_out"].sum().item()) / (m2["ms_step"] * 1e-3),
                        "kernels": m2["kernels"], "lm_head_roofline": m2["roofline"], "clocks": m2["clocks"],
                        "softmax_statistics": "LM-head epilogue" if m2["fused"] else "statistics pass of gs_spec_accept",
                        "launches_per_step": m2["launches_per_step"]}
        del m2
    if rank != 0:
        return
    line = {
        "metric": METRIC, "value": m["gamma_all"] / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": config, "launch_info": launch_info,
        "goodput_tokens_per_s": goodput,
        "roofline": m["roofline"], "kernels": m["kernels"], "cpu_baseline": m["cpu"], "e2e": m["e2e"],
        "gpu_launches": m["launches_per_step"] * args.steps, "launches_per_step": m["launches_per_step"],
        "clocks": m["clocks"], "parity_vs_oracle": m["parity"], "kernel_source_hash": m["khash"],
        "lm_head_w4": m["w4"],
        "configs": others,
    }
    print(json.dumps(line), flush=True)


def run_rank_check(args, rank, world):
    """`--rank-check`: the rank plumbing without the GPU work.  Every rank joins the process group
    (gloo on host tensors when there is no CUDA device), runs the estimator exchange of
    paper_2512_09963_b200.sharded on seeded estimates and rank 0 prints what it saw."""
    import torch.distributed as dist
    from paper_2512_09963_b200 import build as gs_build
    from paper_2512_09963_b200.sharded import ShardedScheduler
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if world > 1:
        dist.init_process_group("nccl" if use_cuda else "gloo", rank=rank, world_size=world)
    if rank == 0:
        gs_build.build()
    if world > 1:
        dist.barrier()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0"))) if use_cuda else torch.device("cpu")
    n, C = 8, 64
    r = np.random.default_rng(7 + rank)
    alpha = torch.from_numpy(r.uniform(0.3, 0.95, n)).to(dev)
    X = torch.from_numpy(r.uniform(1.0, 6.0, n)).to(dev)
    sched = ShardedScheduler(n, rank, world, C * world, dev)
    mine = torch.empty(n, dtype=torch.int32, device=dev)
    S_all = sched.step(alpha, X, mine)
    seen = torch.zeros(world, dtype=torch.int64, device=dev)
    seen[rank] = 1
    if world > 1:
        dist.all_reduce(seen)
    if rank == 0:
        print(json.dumps({"rank_check": True, "n_gpus": args.gpus, "world_size": world, "backend": "nccl" if use_cuda else "gloo",
                          "ranks_seen": [i for i in range(world) if int(seen[i]) == 1], "servers_per_rank": n,
                          "budget_total": C * world, "allocation": S_all.cpu().tolist(),
                          "allocation_sum": int(S_all.sum().item())}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def spawn_ranks(n):
    """`--gpus N` without a launcher around it: start N ranks of this very command under torch's
    launcher on this node and hand their exit code back."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def run_head_sweep(args, cfg, local_rank):
    """LM head alone over a range of row counts at the workload's d and V: where it is bound by HBM
    (few rows) and where by the tensor pipe (many rows), against the measured peaks of both."""
    from paper_2512_09963_b200 import binding as B
    from paper_2512_09963_b200 import build as gs_build
    gs_build.build()
    B.lib()
    dev = torch.device("cuda", local_rank)
    peak_hbm, kind, peaks = _peaks()
    tf_burst = float(peaks.get("bf16_tflops", 1590.0))
    tf_sust = float(peaks.get("bf16_tflops_sustained", 1400.0))
    W = wl.make_layer(cfg, dev)["W"]
    d, V = cfg.d, cfg.V
    rows_out = []
    w4_layer = None
    for T in (16, 46, 96, 144, 256, 288, 512, 1024, 2048):
        H = wl.make_hidden(cfg, T, 0, dev)
        logits = torch.empty((T, V), dtype=torch.float32, device=dev)
        ws = torch.empty(max(256, B.gs_lm_head_workspace(T, d, V, B.GS_BF16)), dtype=torch.uint8, device=dev)
        for _ in range(3):
            B.gs_lm_head_logits(H, W, logits, ws)
        n = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n):                       # W (1.5 GB) streams through L2 every launch: inputs are cold
            B.gs_lm_head_logits(H, W, logits, ws)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        by = d * V * 2 + T * V * 4 + T * d * 2
        fl = 2.0 * T * d * V
        gbs, tfs = by / us / 1e3, fl / us / 1e6
        row = {"rows": T, "us": us, "GBps": gbs, "frac_hbm": gbs / peak_hbm, "TFLOPs": tfs,
               "frac_bf16_burst": tfs / tf_burst, "frac_bf16_sustained": tfs / tf_sust,
               "bound": "hbm" if by / peak_hbm / 1e3 > fl / tf_burst / 1e6 else "tensor"}
        if T <= 256 and d % 128 == 0 and V % 16 == 0:      # the same rows on a 4-bit weight
            if w4_layer is None:
                w4_layer = wl.make_w4_layer(cfg, 128, dev)
            f4 = lambda: B.gs_lm_head_logits_w4(H, w4_layer["qweight"], w4_layer["scales"], w4_layer["zeros"], 128, logits)
            for _ in range(3):
                f4()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n):
                f4()
            e1.record()
            torch.cuda.synchronize()
            us4 = e0.elapsed_time(e1) * 1e3 / n
            by4 = d * V // 2 + (d // 128) * V * 3 + T * V * 4 + T * d * 2
            row.update(w4_us=us4, w4_GBps=by4 / us4 / 1e3, w4_frac_hbm=by4 / us4 / 1e3 / peak_hbm)
        rows_out.append(row)
        del H, logits, ws
    print(json.dumps({"head_sweep": rows_out, "d": d, "V": V, "peaks": {"hbm_gbs": peak_hbm, "bf16_tflops": tf_burst,
                                                                      "bf16_tflops_sustained": tf_sust, "source": kind}}), flush=True)


def run_attn_sweep(args, local_rank):
    """gs_verify_attn alone on every workload's attention inputs, per kernel choice: automatic, the
    persistent kernel, one CTA per group, clusters of 2 / 4 / 8.  Timed as CUDA-graph replays of [read 256 MB; call] minus
    replays of [read 256 MB] alone (cold L2, no host launch cost), best of three."""
    from paper_2512_09963_b200 import binding as B
    from paper_2512_09963_b200 import build as gs_build
    gs_build.build()
    B.lib()
    dev = torch.device("cuda", local_rank)
    peak, kind, _ = _peaks()
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    sink = torch.zeros((), dtype=torch.int64, device=dev)

    def graph_of(fn):
        def body():
            sink.copy_(flush_buf.view(torch.int64).sum())
            if fn is not None:
                fn()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            body()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            body()
        return g

    def replay_us(g, n=30):
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / n

    base = replay_us(graph_of(None))
    rows = []
    for name in ("cfg2", "cfg6", "cfg5", "cfg3", "cfg4"):
        cfg = wl.CONFIGS[name]
        if name == "cfg5":                      # one round of the closed loop at its first allocation, C / N drafts each
            cfg = dataclasses.replace(cfg, gamma_mode="uniform", gamma_lo=cfg.C // cfg.N, gamma_hi=cfg.C // cfg.N)
        alloc = library_allocator(dev) if cfg.gamma_mode == "alloc" else None
        inp = wl.make_attention_inputs(cfg, wl.draw_gamma(cfg, allocator=alloc), wl.draw_prefix(cfg), device=dev)
        Tq, Hq, hd = inp["Q"].shape
        total_kv, Hkv, _ = inp["K"].shape
        cu = inp["cu_kv"].cpu()
        max_len, N = int((cu[1:] - cu[:-1]).max()), cu.numel() - 1
        by = 2 * total_kv * Hkv * hd * 2 + 2 * Tq * Hq * hd * 2
        O = torch.empty_like(inp["Q"])
        st = torch.zeros(1, dtype=torch.int32, device=dev)
        for variant in (0, 1, 3, 2, 4, 8):
            B.gs_verify_attn_select(variant)
            ws = torch.empty(max(256, B.gs_verify_attn_workspace(N, Tq, total_kv, max_len, Hq, Hkv, hd, B.GS_BF16)),
                             dtype=torch.uint8, device=dev)
            call = lambda: B.gs_verify_attn(inp["Q"], inp["K"], inp["V"], O, inp["cu_q"], inp["cu_kv"], max_len, hd ** -0.5, ws, st)
            c0 = B.gs_launch_count()
            call()
            torch.cuda.synchronize()
            launches = B.gs_launch_count() - c0
            assert int(st.item()) == 0
            us = min(replay_us(graph_of(call)) - base for _ in range(3))
            rows.append({"workload": name, "kernel": {0: "automatic", 1: "persistent", 3: "one CTA per group", 2: "clusters of 2",
                                                      4: "clusters of 4", 8: "clusters of 8"}[variant], "launches": int(launches), "us": us,
                         "algorithmic_bytes": by, "GBps": by / us / 1e3, "frac_hbm": by / us / 1e3 / peak})
        B.gs_verify_attn_select(0)
    print(json.dumps({"attn_sweep": rows, "peak_hbm_gbs": peak, "peak_source": kind}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default 2000; 20 for --impl reference, whose steps are CPU-seconds long)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2", choices=["cfg2", "cfg3", "cfg4", "cfg5", "cfg6"])
    ap.add_argument("--rounds", type=int, default=1000, help="rounds of the closed loop (--config cfg5)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--no-fused-stats", action="store_true",
                    help="plain gs_lm_head_logits + gs_spec_accept even where the LM head could write the softmax statistics")
    ap.add_argument("--head-sweep", action="store_true",
                    help="time gs_lm_head_logits alone for 16..2048 rows at the workload's d and V")
    ap.add_argument("--attn-sweep", action="store_true",
                    help="time gs_verify_attn alone on every workload's attention inputs, per kernel choice")
    ap.add_argument("--no-dependent-launch", action="store_true",
                    help="launch the kernels without the programmatic-dependent-launch attribute")
    ap.add_argument("--only-headline", action="store_true",
                    help="time the named workload only (the default run also times cfg3 and cfg4 at --gpus 1)")
    ap.add_argument("--rank-check", action="store_true",
                    help="start the ranks, run the estimator exchange of the sharded path on seeded estimates and "
                         "print what rank 0 saw; no GPU work (gloo on host tensors when there is no CUDA device)")
    ap.add_argument("--profile-small", action="store_true",
                    help="profiling case: vocabulary cut to 32768 (W = 336 MB, still larger than L2), eager "
                         "launches, no CPU baseline and no end-to-end leg; for ncu --set full captures")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 2000 if args.impl == "ours" else 20
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.rank_check):
        sys.exit(spawn_ranks(args.gpus))             # no launcher around this process: start the ranks here
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.rank_check:
        run_rank_check(args, rank, world)
        return
    cfg = wl.CONFIGS[args.config]
    if args.profile_small:
        cfg = wl.shrink(cfg, V=32768, name=cfg.name + "_V32768")
        args.no_graph = args.skip_cpu_baseline = True
    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    if args.head_sweep:
        if rank == 0:
            run_head_sweep(args, cfg, local_rank)
        return
    if args.attn_sweep:
        if rank == 0:
            run_attn_sweep(args, local_rank)
        return
    if args.config == "cfg5":
        # closed-loop scheduling: Algorithm 1 for --rounds rounds with gs_schedule in the loop
        if rank == 0:
            from paper_2512_09963_b200 import build as gs_build
            from paper_2512_09963_b200.closed_loop import run_closed_loop
            gs_build.build()
            rep = run_closed_loop(cfg, args.rounds, device=f"cuda:{local_rank}", curve_every=max(1, args.rounds // 20))
            # the paper's two baselines on the same simulated servers (Sec. V): Fixed-S and Random-S
            rep["baseline_policies"] = {}
            for pol in ("fixed", "random"):
                r2 = run_closed_loop(cfg, args.rounds, device=f"cuda:{local_rank}", policy=pol,
                                     curve_every=max(1, args.rounds // 20))
                rep["baseline_policies"][pol] = {k: r2[k] for k in ("utility_sum_log", "jain", "goodput_tokens_per_s",
                                                                     "verified_tokens_per_s", "gpu_ms_per_round",
                                                                     "utility_curve")}
            rep.update(metric=METRIC, unit=UNIT, value=rep["verified_tokens_per_s"], n_gpus=1, dtype=cfg.dtype,
                       data="synthetic", config={"workload": "cfg5", "servers": cfg.N, "budget_C": cfg.C,
                                                 "drift": "true alpha ~ Beta(4,2) redrawn every 100 rounds",
                                                 "timing": "GPU time of the four library calls per round (CUDA events); "
                                                           "input generation between rounds is untimed"})
            print(json.dumps(rep), flush=True)
        return
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, cfg, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
