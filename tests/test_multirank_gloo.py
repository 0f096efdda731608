"""The N > 1 path on CPU: two gloo ranks shard the draft servers, exchange only the estimator state
(alpha_hat, X) with an all-gather, run the same deterministic allocation and keep their slice.
The allocation itself is the oracle's greedy here (the GPU test shows gs_schedule is bit-identical
to it); what this test covers is the host logic bench.py uses for --gpus N: gather layout, budget
scaling, slicing, and that every rank derives the same global allocation."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import goodspeed_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, C = 8, 64
    r = np.random.default_rng(100 + rank)
    alpha = torch.from_numpy(r.uniform(0.3, 0.95, N))
    X = torch.from_numpy(r.uniform(1.0, 6.0, N))
    # same packing as bench.py: [alpha_hat | X] per rank, gathered rank-major
    est_local = torch.cat([alpha, X])
    est_all = torch.empty(2 * N * world, dtype=torch.float64)
    dist.all_gather_into_tensor(est_all, est_local)
    g = est_all.view(world, 2, N)
    a_all, X_all = g[:, 0, :].reshape(-1), g[:, 1, :].reshape(-1)
    s_min, s_max = np.ones(N * world, np.int32), np.full(N * world, 8, np.int32)
    S_all = orc.ref_schedule_greedy(X_all.numpy(), a_all.numpy(), C * world, s_min, s_max)
    mine = S_all[rank * N:(rank + 1) * N]
    np.save(os.path.join(out_dir, f"S_all_{rank}.npy"), S_all)
    np.save(os.path.join(out_dir, f"mine_{rank}.npy"), mine)
    np.save(os.path.join(out_dir, f"est_{rank}.npy"), np.stack([alpha.numpy(), X.numpy()]))
    # throughput aggregation as in bench.py: MAX of the per-rank times, SUM of the tokens
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tok = torch.tensor([10 * (rank + 1)], dtype=torch.int64)
    dist.all_reduce(tok)
    np.save(os.path.join(out_dir, f"agg_{rank}.npy"), np.array([t.item(), tok.item()]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_estimator_exchange_and_allocation(tmp_path):
    sys.path.insert(0, ROOT)
    from oracle import goodspeed_oracle as orc
    world, port = 2, 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    S0, S1 = np.load(tmp_path / "S_all_0.npy"), np.load(tmp_path / "S_all_1.npy")
    assert np.array_equal(S0, S1)                                   # every rank derives the same allocation
    est = [np.load(tmp_path / f"est_{r}.npy") for r in range(world)]
    a_all = np.concatenate([e[0] for e in est])
    X_all = np.concatenate([e[1] for e in est])
    want = orc.ref_schedule_greedy(X_all, a_all, 128, np.ones(16, np.int32), np.full(16, 8, np.int32))
    assert np.array_equal(S0, want)                                 # gather layout is rank-major, alpha before X
    assert S0.sum() <= 128 and S0.min() >= 1 and S0.max() <= 8
    for r in range(world):
        assert np.array_equal(np.load(tmp_path / f"mine_{r}.npy"), want[r * 8:(r + 1) * 8])
        agg = np.load(tmp_path / f"agg_{r}.npy")
        assert agg[0] == 2.0 and agg[1] == 30                       # max over ranks, sum of tokens
    # the budget couples the ranks: the global optimum differs from two independent per-rank solves
    local = np.concatenate([orc.ref_schedule_greedy(est[r][1], est[r][0], 64, np.ones(8, np.int32),
                                                    np.full(8, 8, np.int32)) for r in range(world)])
    assert orc.ref_sched_objective(X_all, a_all, want) >= orc.ref_sched_objective(X_all, a_all, local) - 1e-12
