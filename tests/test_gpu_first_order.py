"""First-order mode on the GPU against the oracle: block statistics from a caller's gradient
(Appendix E.3) and single iterations of Algorithm 2 on given scores, alone and as a host loop
that must walk the same trajectory as the oracle's."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests.helpers import REL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    from paper_2602_17698_b200.binding import Context
    torch.cuda.set_device(0)
    c = Context()
    yield c
    c.close()


def _grad(R, C, seed, dev=DEV):
    g = torch.Generator(device=dev).manual_seed(seed)
    return (torch.randn((R, C), generator=g, device=dev) * 1e-3).to(torch.bfloat16)


@pytest.mark.parametrize("R,C,br,bc,g,bits", [
    (512, 1024, 128, 128, 128, [2, 3, 4, 8]),
    (256, 512, 32, 32, 32, [1, 2, 3, 4, 5, 6, 8]),
    (256, 512, 64, 64, 16, [2, 3, 4, 8]),
    (512, 512, 256, 128, 64, [3, 4]),
    (256, 768, 128, 256, 128, [2, 4, 8]),
    (96, 640, 48, 128, 128, [2, 3, 4, 5, 6]),
])
@pytest.mark.parametrize("perm", [False, True])
def test_first_order_scores(ctx, R, C, br, bc, g, bits, perm):
    W = synth.make_weight(R, C, 21 + R + C, DEV)
    G = _grad(R, C, 23 + R)
    rng = np.random.default_rng(R + bc)
    nb = (R // br) * (C // bc)
    level = torch.from_numpy(rng.integers(0, len(bits), size=nb).astype(np.uint8)).to(DEV)
    pr = torch.from_numpy(rng.permutation(R).astype(np.int32)).to(DEV) if perm else None
    pc = torch.from_numpy(rng.permutation(C).astype(np.int32)).to(DEV) if perm else None
    up, down, l1 = ctx.first_order_scores(W, G, bits, level, br, bc, g, row_perm=pr, col_perm=pc)
    ctx.sync()
    oup, odown, ol1 = sbo.first_order_scores(W.cpu(), G.cpu(), bits, level.cpu().numpy(), br, bc, g,
                                             row_perm=None if pr is None else pr.cpu().numpy(),
                                             col_perm=None if pc is None else pc.cpu().numpy())
    up, down, l1 = (t.cpu().double().numpy() for t in (up, down, l1))
    # the signed sum cancels: it is compared at the scale of the absolute sum
    assert np.all(np.abs(up - oup) <= REL * ol1 + 1e-30), np.abs(up - oup).max()
    assert np.all(np.abs(l1 - ol1) <= REL * ol1 + 1e-30)
    assert np.all(np.abs(down - odown) <= REL * odown + 1e-30)
    # deterministic
    up2, down2, l12 = ctx.first_order_scores(W, G, bits, level, br, bc, g, row_perm=pr, col_perm=pc)
    ctx.sync()
    assert np.array_equal(up2.cpu().double().numpy(), up) and np.array_equal(down2.cpu().double().numpy(), down)


def test_first_order_scores_on_grid_weights_and_constant_groups(ctx):
    R, C, br, bc, g = 128, 256, 64, 128, 32
    rng = np.random.default_rng(4)
    codes = rng.integers(0, 4, size=(R, C))
    codes[:, 0::32] = 0
    codes[:, 1::32] = 3
    codes[5, 64:96] = 2                               # a constant group
    W = torch.from_numpy((codes * 0.25 - 0.5).astype(np.float32)).to(torch.bfloat16).to(DEV)
    G = _grad(R, C, 3)
    level = torch.zeros(4, dtype=torch.uint8, device=DEV)
    up, down, l1 = ctx.first_order_scores(W, G, [2, 3], level, br, bc, g)
    ctx.sync()
    ref = (G.double() * W.double()).abs().reshape(2, br, 2, bc).sum(dim=(1, 3)).reshape(-1) / 4.0
    scale = ref.cpu().numpy()
    assert np.all(np.abs(up.cpu().numpy()) <= 1e-6 * scale)          # on the grid: no gain
    assert np.all(np.abs(l1.cpu().numpy()) <= 1e-6 * scale)
    assert np.allclose(down.cpu().double().numpy(), scale, rtol=1e-5)


def _scores(rng, N, L, level):
    s_up = rng.choice([0.0, 1.0, 2.0, 3.5, -1.0, 0.25], size=N).astype(np.float32) * \
        rng.uniform(0.5, 2.0, size=N).astype(np.float32)
    s_dn = rng.uniform(0.1, 4.0, size=N).astype(np.float32)
    ties = rng.random(N) < 0.2                       # exact ties in both lists
    s_up[ties] = 1.5
    s_dn[ties] = 0.75
    return s_up, s_dn


@pytest.mark.parametrize("N,bits,k", [(7, [2, 3, 4], 2), (300, [2, 3, 4, 8], 15), (5000, [1, 2, 3, 4, 5, 6, 8], 250),
                                      (70000, [2, 3, 4, 8], 3500), (300, [2, 3, 4, 8], 1)])
@pytest.mark.parametrize("slack_blocks", [0, 3, 10 ** 9])
def test_exchange_step_matches_the_oracle(ctx, N, bits, k, slack_blocks):
    rng = np.random.default_rng(N + k)
    L = len(bits)
    M = 64
    level = rng.integers(0, L, size=N).astype(np.uint8)
    s_up, s_dn = _scores(rng, N, L, level)
    used = int(sum(M * bits[l] for l in level))
    budget = min(float(max(bits)), (used + min(slack_blocks, 4 * N) * M) / (N * M))
    st, want, orep = sbo.exchange_step(s_up, s_dn, level, bits, budget, k, uniform_block_elems=M)
    assert st == sbo.OK
    got, rep = ctx.exchange_step(torch.from_numpy(s_up).to(DEV), torch.from_numpy(s_dn).to(DEV),
                                 torch.from_numpy(level).to(DEV), bits, budget, k, uniform_block_elems=M)
    assert np.array_equal(got.cpu().numpy(), want)
    for key in ("cap_bits", "used_in", "used_out", "expansion", "moved", "n_up", "n_down"):
        assert rep[key] == orep[key], key
    assert rep["sum_up"] == pytest.approx(orep["sum_up"], rel=1e-12, abs=1e-30)
    assert rep["sum_down"] == pytest.approx(orep["sum_down"], rel=1e-12, abs=1e-30)


def test_exchange_step_nonuniform_blocks_and_in_place(ctx):
    rng = np.random.default_rng(9)
    N, bits, k = 2000, [2, 3, 4, 8], 100
    sizes = (rng.integers(1, 5, size=N) * 1024).astype(np.int64)
    level = rng.integers(0, 4, size=N).astype(np.uint8)
    s_up, s_dn = _scores(rng, N, 4, level)
    used = int((sizes * np.array(bits)[level]).sum())
    budget = (used + 5 * 1024) / sizes.sum()
    st, want, orep = sbo.exchange_step(s_up, s_dn, level, bits, budget, k, block_elems=sizes)
    lv = torch.from_numpy(level).to(DEV)
    got, rep = ctx.exchange_step(torch.from_numpy(s_up).to(DEV), torch.from_numpy(s_dn).to(DEV), lv, bits,
                                 budget, k, block_elems=torch.from_numpy(sizes).to(DEV), level_out=lv)
    assert got.data_ptr() == lv.data_ptr()
    assert np.array_equal(got.cpu().numpy(), want)
    assert rep["used_out"] == orep["used_out"] and rep["n_up"] == orep["n_up"] and rep["n_down"] == orep["n_down"]


def test_first_order_loop_on_a_layer_walks_the_oracle_trajectory(ctx):
    """Algorithm 2 as the paper runs it, on one matrix: scores refreshed from (W, G) at the
    current levels every iteration, the caller's loss stood in for by the first-order prediction;
    the oracle's step is fed the GPU's scores (hand-off) and must move the same blocks.  The
    synthetic gradient points along the 3-bit quantisation residual plus noise, so that both
    expansion and exchange steps are taken."""
    R, C, br, bc, g = 1024, 512, 64, 128, 128
    bits, budget = [2, 3, 4, 8], 3.25
    W = synth.make_weight(R, C, 41, DEV)
    Wg = W.float().reshape(R, C // g, g)
    lo, hi = Wg.amin(dim=2, keepdim=True), Wg.amax(dim=2, keepdim=True)
    step = (hi - lo) / 7
    resid = (Wg - (lo + torch.round((Wg - lo) / step) * step)).reshape(R, C)
    G = (-0.05 * resid + _grad(R, C, 43).float() * 0.02).to(torch.bfloat16)
    nb = (R // br) * (C // bc)
    level = torch.full((nb,), 1, dtype=torch.uint8, device=DEV)
    k, kT = max(1, nb // 10), 1
    expansions = exchanges = 0
    for it in range(60):
        if k < kT:
            break
        up, down, _ = ctx.first_order_scores(W, G, bits, level, br, bc, g, want_l1=False)
        cand, rep = ctx.exchange_step(up, down, level, bits, budget, k, uniform_block_elems=br * bc)
        st, ocand, orep = sbo.exchange_step(up.cpu().numpy(), down.cpu().numpy(), level.cpu().numpy(), bits,
                                            budget, k, uniform_block_elems=br * bc)
        assert st == sbo.OK and np.array_equal(cand.cpu().numpy(), ocand), it
        assert rep["expansion"] == orep["expansion"] and rep["n_up"] == orep["n_up"]
        assert rep["used_out"] <= rep["cap_bits"]
        if rep["moved"] and (rep["expansion"] or rep["sum_up"] > rep["sum_down"]):
            level = cand
            expansions += rep["expansion"]
            exchanges += 1 - rep["expansion"]
        else:
            k //= 2
    assert expansions > 0 and exchanges > 0, (expansions, exchanges)
    used = int((torch.tensor(bits, device=DEV)[level.long()] * (br * bc)).sum())
    assert used <= int(budget * R * C)


@pytest.mark.parametrize("R,C,g,bits", [(2048, 2048, 128, 3), (200, 384, 64, 2), (130, 272, 16, 4),
                                        (1024, 512, 32, 8)])
def test_first_order_reorder_scores_and_sort(ctx, R, C, g, bits):
    W = synth.make_weight(R, C, 7 + R, DEV)
    G = _grad(R, C, 9 + C)
    rs = torch.empty(R, dtype=torch.float32, device=DEV)
    cs = torch.empty(C, dtype=torch.float32, device=DEV)
    pr = torch.empty(R, dtype=torch.int32, device=DEV)
    pc = torch.empty(C, dtype=torch.int32, device=DEV)
    ctx.reorder_channels_first_order(W, G, bits, g, row_score=rs, col_score=cs, row_segment=R,
                                     col_segment=C, row_perm=pr, col_perm=pc)
    ctx.sync()
    ors, ocs = sbo.reorder_scores_first_order(W.cpu(), G.cpu(), ref_bits=bits, group=g)
    assert np.allclose(rs.cpu().numpy(), ors, rtol=REL, atol=0)
    assert np.allclose(cs.cpu().numpy(), ocs, rtol=REL, atol=0)
    # hand-off: the oracle's sort of the GPU's scores must equal the GPU's permutation exactly
    assert np.array_equal(pr.cpu().numpy(), sbo.argsort_desc_segments(rs.cpu().double().numpy()))
    assert np.array_equal(pc.cpu().numpy(), sbo.argsort_desc_segments(cs.cpu().double().numpy()))
    # accumulation over coupled matrices
    rs2 = rs.clone()
    ctx.reorder_channels_first_order(W, G, bits, g, row_score=rs2, col_score=cs, accumulate_row=True)
    ctx.sync()
    assert np.allclose(rs2.cpu().numpy(), 2 * ors, rtol=REL)
    assert np.allclose(cs.cpu().numpy(), ocs, rtol=REL)
