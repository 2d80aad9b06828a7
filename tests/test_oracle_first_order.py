"""Pins for the oracle's first-order statistics (Appendix E.3: s_up, s_down from a caller's
gradient) and for one iteration of Algorithm 2 on caller-supplied scores.

The statistics are pinned by closed forms (on-grid weights, constant gradients), by
linearity and sign symmetries, by an explicit permutation and by plain Python loops over a
tiny matrix; the iteration is pinned to the (separately pinned) whole-loop allocator: driven
with scores taken from a static table and the strict-decrease acceptance rule it must walk the
same trajectory, and a plain Python selection on tiny instances must agree with it."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth


def _bf16(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def _f64(t: torch.Tensor) -> np.ndarray:
    return t.double().numpy()


def _grad(R, C, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn((R, C), generator=g) * 1e-3).to(torch.bfloat16)


# ---- first-order statistics ----------------------------------------------------------------
def test_on_grid_weights_have_no_up_gain_and_a_closed_form_down_score():
    bits, br, bc, g = [2, 3], 4, 32, 32
    R, C = 8, 64
    rng = np.random.default_rng(0)
    # every group holds exactly the 4 levels {0, 1, 2, 3} * 0.25 - 0.5 of a 2-bit grid
    codes = rng.integers(0, 4, size=(R, C))
    codes[:, 0::32] = 0
    codes[:, 1::32] = 3
    W = _bf16(codes * 0.25 - 0.5)
    G = _grad(R, C, 1)
    level = np.zeros(4, dtype=np.uint8)
    up, down, l1 = sbo.first_order_scores(W, G, bits, level, br, bc, g)
    assert np.all(up == 0.0) and np.all(l1 == 0.0)
    ref = np.abs(_f64(G) * _f64(W)).reshape(2, br, 2, bc).sum(axis=(1, 3)).reshape(-1) / 4.0
    assert np.allclose(down, ref, rtol=1e-13, atol=0)


@pytest.mark.parametrize("b", [2, 4, 8])
def test_constant_gradient_reduces_to_sums_of_the_pinned_quantizer(b):
    R, C, br, bc, g = 16, 128, 8, 64, 32
    W = synth.make_weight(R, C, 3)
    G = _bf16(np.full((R, C), 0.5))
    level = np.zeros((R // br) * (C // bc), dtype=np.uint8)
    up, down, l1 = sbo.first_order_scores(W, G, [b], level, br, bc, g)
    Wd = _f64(W)
    vh = np.empty_like(Wd)
    for r in range(R):
        for c0 in range(0, C, g):
            _, vh[r, c0:c0 + g], _, _ = sbo.quantize_group(Wd[r, c0:c0 + g], b)
    blk = lambda x: x.reshape(R // br, br, C // bc, bc).sum(axis=(1, 3)).reshape(-1)
    assert np.allclose(up, -0.5 * blk(Wd - vh), rtol=1e-12, atol=1e-18)
    assert np.allclose(l1, 0.5 * blk(np.abs(Wd - vh)), rtol=1e-12)
    assert np.allclose(down, 0.5 * blk(np.abs(vh)) / 2 ** b, rtol=1e-12)


def test_linearity_signs_and_bounds():
    R, C, br, bc, g = 32, 128, 16, 64, 64
    bits = [2, 3, 4, 8]
    W = synth.make_weight(R, C, 5)
    G = _grad(R, C, 7)
    rng = np.random.default_rng(1)
    level = rng.integers(0, 4, size=(R // br) * (C // bc)).astype(np.uint8)
    up, down, l1 = sbo.first_order_scores(W, G, bits, level, br, bc, g)
    up2, down2, l12 = sbo.first_order_scores(W, _bf16(_f64(G) * 2), bits, level, br, bc, g)
    upn, downn, l1n = sbo.first_order_scores(W, _bf16(-_f64(G)), bits, level, br, bc, g)
    assert np.array_equal(up2, 2 * up) and np.array_equal(down2, 2 * down) and np.array_equal(l12, 2 * l1)
    assert np.array_equal(upn, -up) and np.array_equal(downn, down) and np.array_equal(l1n, l1)
    assert np.all(l1 >= np.abs(up) - 1e-18) and np.all(down >= 0)
    # |w - Q(w)| <= half a grid step of its group: the l1 score is bounded by sum |G| step / 2
    Wd, Gd = _f64(W), _f64(G)
    nbc = C // bc
    for blk in range(level.size):
        bi, bj = divmod(blk, nbc)
        b = bits[level[blk]]
        bound = 0.0
        for r in range(bi * br, (bi + 1) * br):
            for c0 in range(bj * bc, (bj + 1) * bc, g):
                v = Wd[r, c0:c0 + g]
                step = (v.max() - v.min()) / (2 ** b - 1)
                bound += np.abs(Gd[r, c0:c0 + g]).sum() * step / 2
        assert l1[blk] <= bound * (1 + 1e-12)


def test_plain_loops_on_a_tiny_matrix_with_mixed_levels():
    R, C, br, bc, g = 8, 64, 4, 32, 16
    bits = [1, 2, 3, 5]
    W = synth.make_weight(R, C, 9)
    G = _grad(R, C, 11)
    level = np.array([0, 3, 2, 1], dtype=np.uint8)
    up, down, l1 = sbo.first_order_scores(W, G, bits, level, br, bc, g)
    Wd, Gd = _f64(W), _f64(G)
    nbc = C // bc
    for blk in range(4):
        bi, bj = divmod(blk, nbc)
        b = bits[level[blk]]
        qmax = 2 ** b - 1
        s_up = s_dn = s_abs = 0.0
        for r in range(bi * br, (bi + 1) * br):
            for c0 in range(bj * bc, (bj + 1) * bc, g):
                v = [float(x) for x in Wd[r, c0:c0 + g]]
                lo, hi = min(v), max(v)
                for k, x in enumerate(v):
                    if hi == lo:
                        xh = lo
                    else:
                        q = round((x - lo) * (qmax / (hi - lo)))      # Python rounds half to even
                        xh = lo + q * ((hi - lo) / qmax)
                    gk = float(Gd[r, c0 + k])
                    s_up -= gk * (x - xh)
                    s_abs += abs(gk * (x - xh))
                    s_dn += abs(gk * xh)
        assert up[blk] == pytest.approx(s_up, rel=1e-12, abs=1e-20)
        assert l1[blk] == pytest.approx(s_abs, rel=1e-12)
        assert down[blk] == pytest.approx(s_dn / 2 ** b, rel=1e-12)


def test_permutations_equal_an_explicitly_permuted_matrix():
    R, C, br, bc, g = 16, 64, 8, 32, 32
    bits = [2, 4]
    W = synth.make_weight(R, C, 13)
    G = _grad(R, C, 15)
    rng = np.random.default_rng(3)
    pr, pc = rng.permutation(R).astype(np.int32), rng.permutation(C).astype(np.int32)
    level = rng.integers(0, 2, size=4).astype(np.uint8)
    a = sbo.first_order_scores(W, G, bits, level, br, bc, g, row_perm=pr, col_perm=pc)
    Wp = W[torch.from_numpy(pr).long()][:, torch.from_numpy(pc).long()].contiguous()
    Gp = G[torch.from_numpy(pr).long()][:, torch.from_numpy(pc).long()].contiguous()
    b = sbo.first_order_scores(Wp, Gp, bits, level, br, bc, g)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


# ---- channel sums of the p = 1 sensitivity ------------------------------------------------------------
def test_first_order_channel_scores_agree_with_the_block_sums_and_plain_loops():
    R, C, g, b = 32, 128, 32, 3
    W = synth.make_weight(R, C, 17)
    G = _grad(R, C, 19)
    rs, cs = sbo.reorder_scores_first_order(W, G, b, g)
    # the same element sensitivities summed three ways: by row, by column, by block
    _, _, l1 = sbo.first_order_scores(W, G, [b], np.zeros(8, dtype=np.uint8), 16, 32, g)
    assert rs.sum() == pytest.approx(cs.sum(), rel=1e-13)
    assert rs.sum() == pytest.approx(l1.sum(), rel=1e-13)
    assert rs[:16].sum() == pytest.approx(l1[:4].sum(), rel=1e-13)            # first block row
    assert cs[32:64].sum() == pytest.approx(l1[1] + l1[5], rel=1e-13)        # second block column
    # plain loops for two rows and two columns, through the pinned group quantizer
    Wd, Gd = _f64(W), _f64(G)
    sig = np.empty_like(Wd)
    for r in range(R):
        for c0 in range(0, C, g):
            _, vh, _, _ = sbo.quantize_group(Wd[r, c0:c0 + g], b)
            sig[r, c0:c0 + g] = np.abs(Gd[r, c0:c0 + g] * (Wd[r, c0:c0 + g] - vh))
    assert np.allclose(rs, sig.sum(axis=1), rtol=1e-13) and np.allclose(cs, sig.sum(axis=0), rtol=1e-13)
    # accumulation over coupled matrices
    rs2, cs2 = sbo.reorder_scores_first_order(W, G, b, g, row_score=rs.copy(), col_score=cs.copy(),
                                              accumulate=True)
    assert np.allclose(rs2, 2 * rs, rtol=1e-15) and np.allclose(cs2, 2 * cs, rtol=1e-15)
    # a gradient that vanishes on a channel makes that channel's score vanish
    G0 = G.clone()
    G0[:, 7] = 0
    G0[5, :] = 0
    rs0, cs0 = sbo.reorder_scores_first_order(W, G0, b, g)
    assert cs0[7] == 0.0 and rs0[5] == 0.0


# ---- one iteration of Algorithm 2 on given scores -------------------------------------------------
def _table(N, L, seed, ragged):
    rng = np.random.default_rng(seed)
    A = rng.uniform(0.5, 50.0, size=(N, 1))
    r = rng.uniform(0.2, 0.6, size=(N, 1))
    E = A * r ** np.arange(L)[None, :]
    if ragged:
        E *= rng.uniform(0.7, 1.3, size=E.shape)
    return E


def _drive(E, bits, budget, gamma0, gammaT, M):
    """Algorithm 2 as a host loop around sbo.exchange_step: scores from the static table at the
    current levels, expansion steps taken as they come, exchange steps kept iff the proxy loss
    strictly falls, else k halves."""
    N, L = E.shape
    l0 = max(l for l in range(L) if bits[l] <= budget)
    level = np.full(N, l0, dtype=np.uint8)
    k = max(1, int(np.floor(gamma0 * N)))
    kT = max(1, int(np.floor(gammaT * N)))
    k = max(k, kT)
    idx = np.arange(N)
    iters = 0
    while k >= kT:
        iters += 1
        lv = level.astype(np.int64)
        s_up = np.where(lv + 1 < L, E[idx, lv] - E[idx, np.minimum(lv + 1, L - 1)], 0.0)
        s_dn = np.where(lv > 0, E[idx, np.maximum(lv - 1, 0)] - E[idx, lv], 0.0)
        st, out, rep = sbo.exchange_step(s_up, s_dn, level, bits, budget, k, uniform_block_elems=M)
        assert st == sbo.OK
        assert rep["used_out"] <= rep["cap_bits"] or rep["used_out"] <= rep["used_in"]
        assert np.all(np.abs(out.astype(int) - level.astype(int)) <= 1)
        if rep["moved"] and (rep["expansion"] or rep["sum_up"] > rep["sum_down"]):
            level = out
        else:
            k //= 2
    return level, iters


@pytest.mark.parametrize("ragged", [False, True])
@pytest.mark.parametrize("N,bits,budget", [(40, [2, 3, 4], 3.0), (300, [2, 3, 4, 8], 2.5),
                                           (257, [1, 2, 3, 4, 5, 6, 8], 3.3), (64, [2, 3, 4, 8], 2.0)])
def test_stepwise_loop_walks_the_same_trajectory_as_the_whole_loop_allocator(N, bits, budget, ragged):
    E = _table(N, len(bits), N + int(budget * 10), ragged)
    M = 64
    st, want, rep = sbo.allocate_scalebits(E, bits, budget, 0.1, 0.01, M)
    assert st == sbo.OK
    got, iters = _drive(E, bits, budget, 0.1, 0.01, M)
    if rep["min_margin"] >= 1e-9:
        assert np.array_equal(got, want)
        assert iters == rep["iterations"]


def test_step_against_a_plain_python_selection_on_tiny_instances():
    rng = np.random.default_rng(5)
    bits = [2, 3, 4, 8]
    L = len(bits)
    for trial in range(200):
        N = int(rng.integers(3, 9))
        sizes = rng.integers(1, 4, size=N).astype(np.int64) * 8
        level = rng.integers(0, L, size=N).astype(np.uint8)
        s_up = rng.choice([0.0, 1.0, 2.0, 3.5, -1.0], size=N)          # ties and non-positive gains
        s_dn = rng.choice([0.5, 1.0, 2.0, 4.0], size=N)
        used = int(sum(sizes[i] * bits[level[i]] for i in range(N)))
        budget = (used + int(rng.integers(0, 3)) * 8) / sizes.sum()
        k = int(rng.integers(1, 5))
        st, out, rep = sbo.exchange_step(s_up, s_dn, level, bits, budget, k, block_elems=sizes)
        assert st == sbo.OK
        cap = int(np.floor(budget * sizes.sum()))
        # plain selection
        ups = sorted((i for i in range(N) if level[i] + 1 < L and s_up[i] > 0),
                     key=lambda i: (-s_up[i] / ((bits[level[i] + 1] - bits[level[i]]) * sizes[i]), i))
        want = level.copy()
        moved = False
        if used < cap:
            cum = 0
            for i in ups[:k]:
                c = sizes[i] * (bits[level[i] + 1] - bits[level[i]])
                if cum + c > cap - used:
                    break
                cum += c
                want[i] += 1
                moved = True
        if not moved:
            h = max(1, k // 2)
            u0 = ups[:h]
            dns = sorted((i for i in range(N) if level[i] > 0 and i not in u0),
                         key=lambda i: (s_dn[i] / ((bits[level[i]] - bits[level[i] - 1]) * sizes[i]), i))[:h]
            freed = sum(sizes[i] * (bits[level[i]] - bits[level[i] - 1]) for i in dns)
            take, cum = [], 0
            for i in u0:
                c = sizes[i] * (bits[level[i] + 1] - bits[level[i]])
                if cum + c > cap - used + freed:
                    break
                cum += c
                take.append(i)
            if take and dns:
                for i in take:
                    want[i] += 1
                for i in dns:
                    want[i] -= 1
                moved = True
        assert np.array_equal(out, want), (trial, level, s_up, s_dn, k, budget)
        assert bool(rep["moved"]) == moved
        new_used = int(sum(sizes[i] * bits[out[i]] for i in range(N)))
        assert rep["used_out"] == new_used
        assert new_used <= max(cap, used)
