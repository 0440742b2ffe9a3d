"""IO-Adaptive Offloading Admission against brute force and the properties the paper states
(Sec. 4.3): Eq. 1, m >= 1 gives the normal batch at least half the weight, m = ceil(t_io/t_layer),
interpolation on the profiled grid, and the two pruning rules losing nothing."""
import itertools
import math

import numpy as np
import pytest

from paper_2609_34555_b200.ioaa import OverlapDepthGrid, admit_fcfs, ioaa_admit, overlap_depth, throughput_model


def test_throughput_model_and_overlap_depth():
    assert throughput_model(1, 10, 10) == 10
    assert throughput_model(3, 8, 4) == pytest.approx(0.75 * 8 + 0.25 * 4)
    for m in (1, 1.5, 2, 7):                               # m >= 1: the normal batch weighs at least one half
        assert m / (m + 1) >= 0.5
        assert throughput_model(m, 11, 10) - throughput_model(m, 10, 10) >= throughput_model(m, 10, 11) - throughput_model(m, 10, 10)
    assert throughput_model(0.2, 6, 2) == throughput_model(1, 6, 2)        # never below one layer of overlap
    assert overlap_depth(1.0, 3.0) == 1 and overlap_depth(3.0, 3.0) == 1 and overlap_depth(3.1, 3.0) == 2
    assert overlap_depth(10.0, 3.0) == math.ceil(10 / 3)


def test_grid_interpolation():
    g = OverlapDepthGrid([0, 8, 16], [0, 32], [[1, 1], [3, 2], [7, 5]])
    assert g(8, 0) == 3 and g(16, 32) == 5 and g(0, 10) == 1
    assert g(12, 0) == pytest.approx(5.0) and g(8, 16) == pytest.approx(2.5)
    assert g(12, 16) == pytest.approx((3 + 2 + 7 + 5) / 4)
    assert g(100, 100) == 5 and g(-5, -5) == 1                             # clamped
    t = OverlapDepthGrid.from_timings([4], [8], [[1.0, 2.5, 7.0]], [2.0])
    assert t.m[0][0] == pytest.approx((1 + 2 + 4) / 3)                     # mean over layers of ceil(t_io/t_layer)


def _brute(lengths, budget, off_tokens, depth, rn=0, ro=0):
    best = None
    for mask in itertools.product((0, 1), repeat=len(lengths)):             # 1 = offload
        mem = sum(off_tokens if o else L for o, L in zip(mask, lengths))
        if mem > budget:
            continue
        b_o, b_n = ro + sum(mask), rn + len(mask) - sum(mask)
        thr = throughput_model(depth(b_o, b_n), b_n, b_o)
        if best is None or thr > best + 1e-12:
            best = thr
    return best


@pytest.mark.parametrize("seed", range(12))
def test_pruned_search_equals_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 12))
    lengths = [int(x) for x in np.exp(rng.normal(9.5, 1.0, n)).clip(512, 131072)]
    off_tokens = 2048
    budget = int(rng.uniform(0.2, 1.2) * sum(lengths))
    grid = OverlapDepthGrid([0, 4, 8, 16, 32], [0, 16, 64],
                            [[1, 1, 1], [1.5, 1.2, 1.0], [3, 2.5, 2], [6, 5, 4], [13, 11, 9]])
    got = ioaa_admit(lengths, budget, off_tokens, grid, running_normal=3, running_offload=1)
    want = _brute(lengths, budget, off_tokens, grid, 3, 1)
    if want is None:
        assert got is None
        return
    assert got is not None and got.throughput == pytest.approx(want)
    assert sorted(got.normal + got.offload) == list(range(n))
    assert sum(off_tokens if i in got.offload else lengths[i] for i in range(n)) <= budget
    # threshold structure: every offloaded request is at least as long as every normal one
    if got.offload and got.normal:
        assert min(lengths[i] for i in got.offload) >= max(lengths[i] for i in got.normal)
    assert got.nodes_visited <= 2 * n + 2


def test_few_nodes_visited_when_memory_is_the_constraint():
    rng = np.random.default_rng(5)
    grid = OverlapDepthGrid([0, 64], [0, 64], [[1, 1], [9, 7]])
    visited = []
    for _ in range(50):
        lengths = [int(x) for x in np.exp(rng.normal(9.7, 1.0, 30)).clip(512, 131072)]
        a = admit_fcfs(lengths, memory_budget=int(0.15 * sum(lengths)), offload_budget_tokens=2048, depth=grid)
        visited.append(a.nodes_visited)
        assert a.normal or a.offload
    assert np.mean(visited) < 62                     # at most two nodes per level, far from 2^30
