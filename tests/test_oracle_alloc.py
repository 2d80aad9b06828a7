"""Pins for the oracle's allocators (Algorithm 1 and Algorithm 2 on the proxy loss).

The exhaustive search and the knapsack DP below are written here, independent of
the oracle.  Algorithm 2's exact trajectory is a reading of the paper, so it is
pinned only through invariants and bounds (budget never exceeded, proxy loss
never above the warm start, never below the exhaustive optimum, special budgets).
"""
import itertools

import numpy as np
import pytest

from oracle import sbo
from paper_2602_17698_b200 import synth

M = 128 * 128


def exhaustive_optimum(err, bits, sizes, cap):
    """min sum_i E[i][l_i] s.t. sum_i M_i b_{l_i} <= cap, by trying every assignment."""
    N, L = err.shape
    best = None
    for lv in itertools.product(range(L), repeat=N):
        cost = sum(sizes[i] * bits[l] for i, l in enumerate(lv))
        if cost > cap:
            continue
        val = sum(err[i, l] for i, l in enumerate(lv))
        if best is None or val < best:
            best = val
    return best


def knapsack_dp(err, bits, cap_units):
    """Multiple-choice knapsack by DP over integer bit units (uniform block size)."""
    N, L = err.shape
    INF = float("inf")
    dp = [INF] * (cap_units + 1)
    dp[0] = 0.0
    for i in range(N):
        nd = [INF] * (cap_units + 1)
        for u in range(cap_units + 1):
            if dp[u] == INF:
                continue
            for l in range(L):
                v = u + bits[l]
                if v <= cap_units and dp[u] + err[i, l] < nd[v]:
                    nd[v] = dp[u] + err[i, l]
        dp = nd
    return min(dp)


def convex_table(N, L, rng):
    """Strictly decreasing, strictly convex rows: E[l] = A * r^l with r in (0, 1)."""
    A = rng.uniform(0.5, 50.0, size=(N, 1))
    r = rng.uniform(0.2, 0.6, size=(N, 1))
    return A * r ** np.arange(L)[None, :]


def random_table(N, L, rng):
    """Decreasing on average but neither monotone nor convex everywhere."""
    base = rng.uniform(1, 30, size=(N, 1)) * 0.4 ** np.arange(L)[None, :]
    return base * rng.uniform(0.5, 1.8, size=(N, L))


@pytest.mark.parametrize("seed", range(6))
def test_greedy_is_optimal_on_convex_unit_step_tables(seed):
    """Marginal allocation on convex separable costs with unit steps is optimal
    whenever the budget is spent exactly."""
    rng = np.random.default_rng(seed)
    N, bits = 7, [1, 2, 3, 4]
    err = convex_table(N, len(bits), rng)
    for extra in range(0, 3 * N + 1, 4):
        cap_units = N * bits[0] + extra
        budget = cap_units / N
        st, lv, rep = sbo.allocate_greedy(err, bits, budget, uniform_block_elems=M)
        assert st == sbo.OK
        assert rep["used_bits"] == cap_units * M == rep["cap_bits"]
        opt = knapsack_dp(err, bits, cap_units)
        assert rep["proxy_loss_final"] == pytest.approx(opt, rel=1e-12)
        assert rep["proxy_loss_final"] == pytest.approx(err[np.arange(N), lv].sum(), rel=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_greedy_bounds_on_general_tables(seed):
    rng = np.random.default_rng(100 + seed)
    N, bits = 6, [2, 3, 4, 8]
    err = random_table(N, len(bits), rng)
    sizes = [M] * N
    for budget in (2.0, 2.4, 3.0, 3.7, 5.0, 8.0):
        st, lv, rep = sbo.allocate_greedy(err, bits, budget, uniform_block_elems=M)
        assert st == sbo.OK
        cap = int(np.floor(budget * N * M))
        used = sum(M * bits[l] for l in lv)
        assert used == rep["used_bits"] <= cap == rep["cap_bits"]
        val = err[np.arange(N), lv].sum()
        assert val == pytest.approx(rep["proxy_loss_final"], rel=1e-12)
        opt = exhaustive_optimum(err, bits, sizes, cap)
        assert val >= opt * (1 - 1e-12)
        assert val <= err[:, 0].sum() * (1 + 1e-12)
        # every step taken lies on the block's lower convex hull: no level of higher error
        assert np.all(err[np.arange(N), lv] <= err[:, 0])
        st2, lv2, rep2 = sbo.allocate_greedy(err, bits, budget, uniform_block_elems=M, heap=True)
        assert st2 == sbo.OK and np.array_equal(lv, lv2) and rep2["used_bits"] == rep["used_bits"]


def test_greedy_stops_at_first_step_that_does_not_fit():
    """Two blocks, bits {2, 4}: the best step costs 2 units; with 1 unit left nothing is taken."""
    err = np.array([[10.0, 1.0], [5.0, 4.0]])
    st, lv, rep = sbo.allocate_greedy(err, [2, 4], 2.5, uniform_block_elems=M)
    assert st == sbo.OK and list(lv) == [0, 0] and rep["used_bits"] == 4 * M
    st, lv, rep = sbo.allocate_greedy(err, [2, 4], 3.0, uniform_block_elems=M)
    assert list(lv) == [1, 0] and rep["used_bits"] == 6 * M
    st, lv, _ = sbo.allocate_greedy(err, [2, 4], 1.9, uniform_block_elems=M)
    assert st == sbo.ERR_BUDGET


def test_greedy_literal_equals_heap_on_medium_instance():
    rng = np.random.default_rng(3)
    err = random_table(600, 4, rng)
    sizes = rng.choice([32 * 32, 64 * 64, 128 * 128], size=600).astype(np.int64)
    for budget in (2.3, 3.1, 4.5):
        a = sbo.allocate_greedy(err, [2, 3, 4, 8], budget, block_elems=sizes)
        b = sbo.allocate_greedy(err, [2, 3, 4, 8], budget, block_elems=sizes, heap=True)
        assert a[0] == b[0] == sbo.OK
        assert np.array_equal(a[1], b[1]) and a[2]["used_bits"] == b[2]["used_bits"]
        assert a[2]["used_bits"] <= a[2]["cap_bits"] == int(np.floor(budget * sizes.sum()))


@pytest.mark.parametrize("seed", range(5))
def test_scalebits_invariants_tiny(seed):
    rng = np.random.default_rng(200 + seed)
    N, bits = 7, [2, 3, 4]
    err = random_table(N, 3, rng) if seed % 2 else convex_table(N, 3, rng)
    sizes = [M] * N
    for budget in (2.0, 2.3, 2.5, 3.0, 3.4, 4.0, 4.5):
        st, lv, rep = sbo.allocate_scalebits(err, bits, budget, 0.3, 0.15, uniform_block_elems=M)
        assert st == sbo.OK
        cap = int(np.floor(budget * N * M))
        used = sum(M * bits[l] for l in lv)
        assert used == rep["used_bits"] <= cap == rep["cap_bits"]
        val = err[np.arange(N), lv].sum()
        assert val == pytest.approx(rep["proxy_loss_final"], rel=1e-12)
        warm = max(l for l, b in enumerate(bits) if b <= budget)
        assert rep["proxy_loss_init"] == pytest.approx(err[:, warm].sum(), rel=1e-12)
        assert val <= rep["proxy_loss_init"] * (1 + 1e-12)
        assert val >= exhaustive_optimum(err, bits, sizes, cap) * (1 - 1e-12)
        assert rep["iterations"] == rep["expansions"] + rep["accepted"] + rep["rejected"]


def test_scalebits_special_budgets():
    rng = np.random.default_rng(7)
    N, bits = 40, [2, 3, 4]
    err = convex_table(N, 3, rng)
    st, lv, rep = sbo.allocate_scalebits(err, bits, 9.0, uniform_block_elems=M)      # B >= max
    assert st == sbo.OK and np.all(lv == 2)
    st, lv, rep = sbo.allocate_scalebits(err, bits, 1.5, uniform_block_elems=M)      # B < min
    assert st == sbo.ERR_BUDGET
    # identical rows at a candidate budget: an exchange gains dU = E1-E2 < dD = E0-E1, rejected
    same = np.tile(np.array([[8.0, 2.0, 0.5]]), (N, 1))
    st, lv, rep = sbo.allocate_scalebits(same, bits, 3.0, uniform_block_elems=M)
    assert st == sbo.OK and np.all(lv == 1) and rep["accepted"] == 0 and rep["rejected"] >= 1
    st, lv, rep = sbo.allocate_scalebits(same, bits, 2.0, uniform_block_elems=M)     # B = min
    assert st == sbo.OK and np.all(lv == 0)


def test_scalebits_expansion_matches_greedy_between_candidates():
    """With a static convex table and a budget strictly between two candidates, the
    expansion stage raises exactly the blocks classic greedy would raise from the warm start."""
    rng = np.random.default_rng(11)
    N, bits = 400, [2, 3, 4]
    err = convex_table(N, 3, rng)
    # make level 0 -> 1 always the steepest step so greedy from the bottom passes the warm start
    err[:, 0] = err[:, 1] + 10 * (err[:, 1] - err[:, 2]) + 100.0
    st, lv, rep = sbo.allocate_scalebits(err, bits, 3.25, 0.05, 0.02, uniform_block_elems=M)
    stg, lvg, repg = sbo.allocate_greedy(err, bits, 3.25, uniform_block_elems=M)
    assert st == stg == sbo.OK
    assert rep["used_bits"] == repg["used_bits"] == rep["cap_bits"]
    assert rep["expansions"] == 5                       # 100 blocks to raise, 20 per batch
    assert np.array_equal(lv, lvg)


def test_scalebits_iteration_count_is_in_the_papers_range():
    """Table 3 quotes 16 - 36 search iterations in the 3-4 bit regime (plausibility only)."""
    W = synth.make_weight(1024, 1024, 5)
    X = synth.make_activations(1024, 1024, 6)
    c = sbo.calib_moments(X, 1.0 / 1024)
    bits = [1, 2, 3, 4, 5, 6, 7, 8]
    err, _ = sbo.block_scores(W, c, bits, 64, 128, 128)
    its = []
    for budget in (3.25, 3.5, 3.75):
        st, lv, rep = sbo.allocate_scalebits(err, bits, budget, 0.05, 0.02, uniform_block_elems=64 * 128)
        assert st == sbo.OK and rep["used_bits"] <= rep["cap_bits"]
        its.append(rep["iterations"])
    assert 5 <= min(its) and max(its) <= 60, its


def test_nonuniform_block_sizes_budget_accounting():
    rng = np.random.default_rng(13)
    N, bits = 300, [2, 3, 4, 8]
    err = random_table(N, 4, rng)
    sizes = rng.choice([1024, 4096, 16384], size=N).astype(np.int64)
    for budget in (2.5, 3.0, 3.6):
        st, lv, rep = sbo.allocate_scalebits(err, bits, budget, block_elems=sizes)
        assert st == sbo.OK
        used = int((sizes * np.array(bits)[lv]).sum())
        assert used == rep["used_bits"] <= rep["cap_bits"] == int(np.floor(budget * sizes.sum()))
        assert sum(rep["level_hist"]) == N
        assert rep["level_hist"][:4] == np.bincount(lv, minlength=4).tolist()
