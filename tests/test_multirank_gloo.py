"""The N > 1 path on CPU: two gloo ranks shard the draft servers and run the package's own exchange
(paper_2512_09963_b200.sharded.ShardedScheduler: all-gather of the estimator state, the global
allocation by gs_schedule_host, the rank's slice) and its throughput aggregation.  The expected
allocation is the oracle's greedy on the concatenated estimates.  A second test starts
`bench.py --gpus 2` without any launcher and checks that it brings up two ranks by itself."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
N_LOCAL, C_LOCAL = 8, 64


def _estimates(rank):
    r = np.random.default_rng(100 + rank)
    return r.uniform(0.3, 0.95, N_LOCAL), r.uniform(1.0, 6.0, N_LOCAL)


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from paper_2512_09963_b200 import build as gs_build
    from paper_2512_09963_b200.sharded import ShardedScheduler, aggregate_throughput
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    if rank == 0:
        gs_build.build()
    dist.barrier()
    alpha, X = _estimates(rank)
    s_min = torch.ones(N_LOCAL * world, dtype=torch.int32)
    s_max = torch.full((N_LOCAL * world,), 8, dtype=torch.int32)
    sched = ShardedScheduler(N_LOCAL, rank, world, C_LOCAL * world, "cpu", s_min, s_max)
    mine = torch.empty(N_LOCAL, dtype=torch.int32)
    for _ in range(2):                                   # buffers are reused from round to round
        S_all = sched.step(torch.from_numpy(alpha), torch.from_numpy(X), mine)
    np.save(os.path.join(out_dir, f"S_all_{rank}.npy"), S_all.numpy())
    np.save(os.path.join(out_dir, f"mine_{rank}.npy"), mine.numpy())
    ms, units = aggregate_throughput(1.0 + rank, 10 * (rank + 1), "cpu")
    np.save(os.path.join(out_dir, f"agg_{rank}.npy"), np.array([ms, units]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_estimator_exchange_and_allocation(tmp_path):
    sys.path.insert(0, ROOT)
    from oracle import goodspeed_oracle as orc
    world, port = 2, 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    S0, S1 = np.load(tmp_path / "S_all_0.npy"), np.load(tmp_path / "S_all_1.npy")
    assert np.array_equal(S0, S1)                                   # every rank derives the same allocation
    est = [_estimates(r) for r in range(world)]
    a_all = np.concatenate([e[0] for e in est])
    X_all = np.concatenate([e[1] for e in est])
    want = orc.ref_schedule_greedy(X_all, a_all, 128, np.ones(16, np.int32), np.full(16, 8, np.int32))
    assert np.array_equal(S0, want)                                 # gather layout is rank-major, alpha before X
    assert S0.sum() <= 128 and S0.min() >= 1 and S0.max() <= 8
    for r in range(world):
        assert np.array_equal(np.load(tmp_path / f"mine_{r}.npy"), want[r * 8:(r + 1) * 8])
        agg = np.load(tmp_path / f"agg_{r}.npy")
        assert agg[0] == 2.0 and agg[1] == 30                       # max over ranks, sum of the units
    # the budget couples the ranks: the global optimum is at least as good as two independent per-rank solves
    local = np.concatenate([orc.ref_schedule_greedy(est[r][1], est[r][0], 64, np.ones(8, np.int32),
                                                    np.full(8, 8, np.int32)) for r in range(world)])
    assert orc.ref_sched_objective(X_all, a_all, want) >= orc.ref_sched_objective(X_all, a_all, local) - 1e-12


def test_bench_starts_its_own_ranks(tmp_path):
    """`python bench.py --gpus 2` with no launcher around it (WORLD_SIZE unset) starts two ranks.  The
    rank check replaces the GPU work by the estimator exchange on host tensors (gloo), so it runs here."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                          # rank 0 alone prints
    rep = lines[0]
    assert rep["rank_check"] and rep["n_gpus"] == 2 and rep["world_size"] == 2
    assert rep["ranks_seen"] == [0, 1]
    assert rep["allocation_sum"] <= rep["budget_total"] and len(rep["allocation"]) == 2 * rep["servers_per_rank"]
