"""gs_schedule_host (the scheduler on host arrays, no CUDA call) through the C ABI against the oracle's
greedy: allocations must be identical, bit for bit, on the cases the device kernels are tested on."""
import numpy as np
import pytest
import torch

from oracle import goodspeed_oracle as orc
from paper_2512_09963_b200 import binding as B
from paper_2512_09963_b200 import build as gs_build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gs_build.build()
    return B.lib()


def host_schedule(X, al, C, lo=None, hi=None):
    S = torch.full((len(X),), -5, dtype=torch.int32)
    t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt)
    B.gs_schedule_host(t(X, torch.float64), t(al, torch.float64), C, S, t(lo, torch.int32), t(hi, torch.int32))
    return S.numpy()


@pytest.mark.parametrize("N,C", [(1, 5), (4, 10), (8, 64), (16, 128), (32, 256), (32, 600), (33, 64), (100, 300),
                                 (1024, 512), (8, 0)])
def test_host_schedule_bit_exact(N, C):
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
        got = host_schedule(X, al, C, lo, hi)
        want = orc.ref_schedule_greedy(X, al, C, lo, hi)
        assert np.array_equal(got, want), (N, C, trial)
        assert got.sum() <= C


def test_host_schedule_matches_brute_force_on_tiny_instances():
    r = np.random.default_rng(11)
    for _ in range(20):
        N, C = int(r.integers(1, 5)), int(r.integers(0, 9))
        X, al = r.uniform(0.5, 4.0, N), r.uniform(0.05, 0.95, N)
        S = host_schedule(X, al, C)
        _, best = orc.ref_schedule_bruteforce(X, al, C)
        assert abs(orc.ref_sched_objective(X, al, S) - best) <= 1e-12 * abs(best)


def test_host_schedule_argument_errors():
    L = B.lib()
    assert L.gs_schedule_host(None, None, -1, 4, None, None, None) == 1
    assert L.gs_schedule_host(None, None, 3, 4, None, None, None) == 1
    assert L.gs_schedule_host(None, None, 0, 4, None, None, None) == 0
    # floors above the budget: returned as they are, with GS_ERR_SHAPE
    X = torch.ones(4, dtype=torch.float64)
    al = torch.full((4,), 0.5, dtype=torch.float64)
    lo = torch.full((4,), 2, dtype=torch.int32)
    S = torch.zeros(4, dtype=torch.int32)
    with pytest.raises(B.GoodSpeedError) as e:
        B.gs_schedule_host(X, al, 3, S, lo, None)
    assert e.value.code == 2 and S.tolist() == [2, 2, 2, 2]
