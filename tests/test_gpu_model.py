"""Several decoder layers searched as one model: the residual-stream permutation is shared by
all layers and the allocation is global over the blocks of all layers.  Stage-wise against the
oracle with hand-off of the GPU's integer outputs."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests import helpers
from tests.helpers import REL, REL_MOMENT, assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_tiny_model_global_allocation_stagewise():
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import COUPLING, SearchConfig, search_model
    torch.cuda.set_device(0)
    shape, n_layers, tokens = synth.LLAMA_TINY, 3, 512
    bits, br, bc, g = [2, 3, 4, 8], 128, 128, 128
    budgets = [2.25, 2.5, 3.0]                        # warm starts 2, 2 and 3: two sweeps
    cfg = SearchConfig(bits=bits, block_rows=br, block_cols=bc, group=g, gamma0=0.1, gammaT=0.02)

    def make_weights(layer):
        W = synth.make_layer_weights(shape, 3, layer, DEV)
        if layer == 1:                                # a 50-sigma "super weight"
            synth.inject_super_weights(W["down_proj"], 11, 1)
        return W

    def make_acts(layer):
        return synth.make_layer_activations(shape, tokens, 3, layer, DEV)

    ctx = Context()
    res = search_model(ctx, shape, n_layers, cfg, budgets, make_weights, make_acts, DEV)
    lin = {l.name: l for l in shape.linears}
    Wh = [{n: w.cpu() for n, w in make_weights(layer).items()} for layer in range(n_layers)]

    # a1: moments of every layer
    gm = []
    for layer in range(n_layers):
        X = make_acts(layer)
        for n, x in X.items():
            ref = sbo.calib_moments(x.cpu(), 1.0 / x.shape[0])
            assert_close(res.moments[layer][n].cpu().numpy(), ref, REL_MOMENT, what=f"moments {layer} {n}")
        gm.append({n: res.moments[layer][n].cpu().double().numpy() for n in X})

    assert sorted(res.tables) == [2, 3]
    for rb in (2, 3):
        sc, pm = res.scores[rb], res.perms[rb]
        # a2: hidden scores summed over ALL layers, the other sets per layer
        osc = [helpers.oracle_layer_scores(shape, Wh[layer], gm[layer], rb, g) for layer in range(n_layers)]
        assert_close(sc["hidden"].cpu().numpy(), sum(o["hidden"] for o in osc), REL, what="hidden")
        for layer in range(n_layers):
            assert_close(sc["intermediate"][layer].cpu().numpy(), osc[layer]["intermediate"], REL)
            assert_close(sc["v_heads"][layer].cpu().numpy(), osc[layer]["v_heads"], REL)
        # a3: permutations given the GPU's scores: exact
        operm = []
        for layer in range(n_layers):
            gsc = {"hidden": sc["hidden"].cpu().double().numpy(),
                   "intermediate": sc["intermediate"][layer].cpu().double().numpy(),
                   "v_heads": sc["v_heads"][layer].cpu().double().numpy()}
            op = helpers.oracle_layer_perms(shape, gsc)
            operm.append(op)
            assert np.array_equal(pm["hidden"].cpu().numpy(), op["hidden"])
            for key in ("intermediate", "v_heads", "o_heads"):
                assert np.array_equal(pm[(key, layer)].cpu().numpy(), op[key]), (key, layer)
        # a4: the global table, matrix by matrix
        table = res.tables[rb].cpu().numpy()
        for layer in range(n_layers):
            for name, l in lin.items():
                rp, cp = COUPLING[name]
                oerr, _ = sbo.block_scores(Wh[layer][name], gm[layer][l.act], bits, br, bc, g,
                                           row_perm=None if rp is None else operm[layer][rp],
                                           col_perm=None if cp is None else operm[layer][cp])
                s = res.block_start[(layer, name)]
                assert_close(table[s:s + oerr.shape[0]], oerr, REL, what=f"err {layer} {name}")
        assert res.n_blocks == table.shape[0] == n_layers * sum(
            (l.rows // br) * (l.cols // bc) for l in shape.linears)

    # a5: global allocation given the GPU's table: exact, budget by budget
    for b in budgets:
        rb = max(x for x in bits if x <= b)
        table = res.tables[rb].cpu().double().numpy()
        st, olv, orep = sbo.allocate_scalebits(table, bits, b, cfg.gamma0, cfg.gammaT, br * bc)
        assert st == sbo.OK
        rep = res.reports[b]
        assert rep["cap_bits"] == int(np.floor(b * n_layers * shape.n_weights))
        assert rep["used_bits"] <= rep["cap_bits"]
        if orep["min_margin"] >= 1e-9:
            assert np.array_equal(res.levels[b].cpu().numpy(), olv), b
            assert rep["used_bits"] == orep["used_bits"]
            assert rep["iterations"] == orep["iterations"]
    assert set(res.ms) >= {"moments", "stats@2", "sort@2", "scores@2", "allocate@2.5", "allocate@3"}
    ctx.close()


def test_llama3_8b_full_model_allocation_matches_oracle():
    """configs[2]: 32 layers of the 8B shape (N = 425,984 blocks), four injected super weights,
    global allocation for several budgets.  The oracle allocates on the GPU's table (exact
    levels); permutations are exact given the GPU's scores; sampled blocks of two layers are
    re-scored by the oracle."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import COUPLING, SearchConfig, search_model
    torch.cuda.set_device(0)
    shape, n_layers, tokens = synth.LLAMA3_8B, 32, 8192
    bits, br, bc, g = [2, 3, 4, 8], 128, 128, 128
    budgets = [2.0, 2.5, 3.25]
    cfg = SearchConfig(bits=bits, block_rows=br, block_cols=bc, group=g)
    super_layers = {3: 101, 12: 102, 20: 103, 29: 104}

    def make_weights(layer):
        W = synth.make_layer_weights(shape, 0, layer, DEV)
        if layer in super_layers:
            synth.inject_super_weights(W["down_proj"], super_layers[layer], 1)
        return W

    def make_acts(layer):
        return synth.make_layer_activations(shape, tokens, 0, layer, DEV)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ctx = Context()
        res = search_model(ctx, shape, n_layers, cfg, budgets, make_weights, make_acts, DEV)
    torch.cuda.synchronize()
    assert res.n_blocks == 425984
    lin = {l.name: l for l in shape.linears}
    rng = np.random.default_rng(1)

    for rb in (2, 3):
        sc, pm = res.scores[rb], res.perms[rb]
        hid = sc["hidden"].cpu().double().numpy()
        assert np.array_equal(pm["hidden"].cpu().numpy(), sbo.argsort_desc_segments(hid))
        for layer in (5, 29):
            gsc = {"hidden": hid, "intermediate": sc["intermediate"][layer].cpu().double().numpy(),
                   "v_heads": sc["v_heads"][layer].cpu().double().numpy()}
            op = helpers.oracle_layer_perms(shape, gsc)
            for key in ("intermediate", "v_heads", "o_heads"):
                assert np.array_equal(pm[(key, layer)].cpu().numpy(), op[key]), (key, layer)
            if rb != 2:
                continue
            # sampled blocks of the table (the layer with a super weight included)
            W = make_weights(layer)
            gm = {n: res.moments[layer][n].cpu().double().numpy() for n in shape.act_dims}
            table = res.tables[rb]
            for name, l in lin.items():
                rp, cp = COUPLING[name]
                pr = op[rp] if rp else np.arange(l.rows)
                pc = op[cp] if cp else np.arange(l.cols)
                nbc = l.cols // bc
                nb = (l.rows // br) * nbc
                s0 = res.block_start[(layer, name)]
                Wn = W[name]
                for blk in rng.choice(nb, 3, replace=False):
                    bi, bj = divmod(int(blk), nbc)
                    rows = torch.from_numpy(pr[bi * br:(bi + 1) * br].astype(np.int64)).to(DEV)
                    cols = pc[bj * bc:(bj + 1) * bc]
                    tile = Wn[rows][:, torch.from_numpy(cols.astype(np.int64)).to(DEV)].contiguous().cpu()
                    oerr, _ = sbo.block_scores(tile, gm[l.act][cols], bits, br, bc, g)
                    assert_close(table[s0 + blk:s0 + blk + 1].cpu().numpy(), oerr, REL,
                                 what=f"err layer {layer} {name} block {blk}")
            del W

    for b in budgets:
        rb = max(x for x in bits if x <= b)
        table = res.tables[rb].cpu().double().numpy()
        st, olv, orep = sbo.allocate_scalebits(table, bits, b, cfg.gamma0, cfg.gammaT, br * bc)
        assert st == sbo.OK
        rep = res.reports[b]
        assert rep["cap_bits"] == int(np.floor(b * n_layers * shape.n_weights))
        assert rep["used_bits"] <= rep["cap_bits"]
        if orep["min_margin"] >= 1e-9:
            assert np.array_equal(res.levels[b].cpu().numpy(), olv), b
            assert rep["used_bits"] == orep["used_bits"]
            assert rep["iterations"] == orep["iterations"]
    ctx.close()


def test_llama3_70b_streamed_allocation_matches_oracle():
    """configs[3]: 80 layers of the 70B shape (N = 4,177,920 blocks of 128 x 128), bits {2,3,4},
    budget 2.25, weights regenerated from their seeds in each sweep (never resident).  The oracle
    allocates on the GPU's table; sampled blocks of one layer are re-scored."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import COUPLING, SearchConfig, search_model
    torch.cuda.set_device(0)
    shape, n_layers, tokens = synth.LLAMA3_70B, 80, 2048
    bits, br, bc, g = [2, 3, 4], 128, 128, 128
    budget = 2.25
    cfg = SearchConfig(bits=bits, block_rows=br, block_cols=bc, group=g)

    def make_weights(layer):
        return synth.make_layer_weights(shape, 0, layer, DEV)

    def make_acts(layer):
        return synth.make_layer_activations(shape, tokens, 0, layer, DEV)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ctx = Context()
        res = search_model(ctx, shape, n_layers, cfg, [budget], make_weights, make_acts, DEV,
                           keep_weights=False)
    torch.cuda.synchronize()
    assert res.n_blocks == 4177920
    lin = {l.name: l for l in shape.linears}
    rng = np.random.default_rng(2)
    sc, pm = res.scores[2], res.perms[2]
    hid = sc["hidden"].cpu().double().numpy()
    assert np.array_equal(pm["hidden"].cpu().numpy(), sbo.argsort_desc_segments(hid))
    layer = 41
    gsc = {"hidden": hid, "intermediate": sc["intermediate"][layer].cpu().double().numpy(),
           "v_heads": sc["v_heads"][layer].cpu().double().numpy()}
    op = helpers.oracle_layer_perms(shape, gsc)
    for key in ("intermediate", "v_heads", "o_heads"):
        assert np.array_equal(pm[(key, layer)].cpu().numpy(), op[key]), key
    W = make_weights(layer)
    gm = {n: res.moments[layer][n].cpu().double().numpy() for n in shape.act_dims}
    table = res.tables[2]
    for name, l in lin.items():
        rp, cp = COUPLING[name]
        pr = op[rp] if rp else np.arange(l.rows)
        pc = op[cp] if cp else np.arange(l.cols)
        nbc = l.cols // bc
        nb = (l.rows // br) * nbc
        s0 = res.block_start[(layer, name)]
        for blk in rng.choice(nb, 3, replace=False):
            bi, bj = divmod(int(blk), nbc)
            rows = torch.from_numpy(pr[bi * br:(bi + 1) * br].astype(np.int64)).to(DEV)
            cols = pc[bj * bc:(bj + 1) * bc]
            tile = W[name][rows][:, torch.from_numpy(cols.astype(np.int64)).to(DEV)].contiguous().cpu()
            oerr, _ = sbo.block_scores(tile, gm[l.act][cols], bits, br, bc, g)
            assert_close(table[s0 + blk:s0 + blk + 1].cpu().numpy(), oerr, REL, what=f"err {name} block {blk}")
    del W
    th = table.cpu().double().numpy()
    st, olv, orep = sbo.allocate_scalebits(th, bits, budget, cfg.gamma0, cfg.gammaT, br * bc)
    assert st == sbo.OK
    rep = res.reports[budget]
    assert rep["cap_bits"] == int(np.floor(budget * n_layers * shape.n_weights))
    assert rep["used_bits"] <= rep["cap_bits"]
    if orep["min_margin"] >= 1e-9:
        assert np.array_equal(res.levels[budget].cpu().numpy(), olv)
        assert rep["used_bits"] == orep["used_bits"]
        assert rep["iterations"] == orep["iterations"]
    ctx.close()


def test_second_context_gives_the_same_model_result():
    """The independent calls of a layer dealt to two and to seven contexts on streams of their own: tables,
    permutations, levels and reports are those of the one-context run, bit for bit."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import SearchConfig, search_model
    torch.cuda.set_device(0)
    shape, n_layers, tokens = synth.LLAMA_TINY, 3, 384
    budgets = [2.5, 3.25]
    cfg = SearchConfig(bits=[2, 3, 4, 8])

    def make_weights(layer):
        return synth.make_layer_weights(shape, 5, layer, DEV)

    def make_acts(layer):
        return synth.make_layer_activations(shape, tokens, 5, layer, DEV)

    ctx = Context()
    ctx2 = Context(stream=torch.cuda.Stream(device=DEV))
    one = search_model(ctx, shape, n_layers, cfg, budgets, make_weights, make_acts, DEV)
    two = search_model(ctx, shape, n_layers, cfg, budgets, make_weights, make_acts, DEV, ctx2=ctx2)
    more = [ctx2] + [Context(stream=torch.cuda.Stream(device=DEV)) for _ in range(5)]
    seven = search_model(ctx, shape, n_layers, cfg, budgets, make_weights, make_acts, DEV, ctx2=more)
    torch.cuda.synchronize()
    for other in (two, seven):
        assert sorted(one.tables) == sorted(other.tables)
        for rb in one.tables:
            assert torch.equal(one.tables[rb], other.tables[rb]), rb
            for k in one.perms[rb]:
                assert torch.equal(one.perms[rb][k], other.perms[rb][k]), (rb, k)
        for b in budgets:
            assert torch.equal(one.levels[b], other.levels[b]), b
            for k in ("used_bits", "iterations", "cap_bits"):
                assert one.reports[b][k] == other.reports[b][k], (b, k)
    for c in more:
        assert c.kernel_launches() > 0
        c.close()
    ctx.close()
