"""The benchmark's workload at full size (one Llama-3-8B-shaped layer, 65536 tokens) in the
launch configuration bench.py times (non-default stream, the whole step as one CUDA graph with
the enqueue-only allocation, block scores and pack shared between seven contexts), and the
corners of the stress sweep (block shapes, group sizes, seven candidates) on the same layer,
checked on sampled outputs the oracle can compute one by one, plus the exact stages
(permutations given scores, levels given the table, budget accounting)."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests import helpers
from tests.helpers import REL, REL_MOMENT, assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


STRESS_BITS = [1, 2, 3, 4, 5, 6, 8]


@pytest.mark.parametrize("bits,br,bc,g,budget,tokens", [
    ([2, 3, 4, 8], 128, 128, 128, 2.5, 65536),        # configs[1], as bench.py times it
    (STRESS_BITS, 32, 32, 32, 1.75, 4096),            # configs[4]: the stress sweep's corners
    (STRESS_BITS, 64, 64, 64, 2.5, 4096),
    (STRESS_BITS, 256, 128, 128, 3.5, 4096),
    ([2, 3, 4], 128, 128, 64, 3.0, 4096),
    (STRESS_BITS, 128, 128, 32, 2.75, 4096),          # seven candidates, four groups per block width
])
def test_llama3_8b_layer_full_size_sampled_parity(bits, br, bc, g, budget, tokens):
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import COUPLING, LayerWorkspace, SearchConfig, StageGraphs, search_layer
    torch.cuda.set_device(0)
    shape = synth.LLAMA3_8B
    cfg = SearchConfig(bits=bits, budget=budget, block_rows=br, block_cols=bc, group=g)
    W = synth.make_layer_weights(shape, 0, 0, DEV)
    X = synth.make_layer_activations(shape, tokens, 0, 0, DEV)
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        ctx = Context()
        ctx2 = [Context(stream=torch.cuda.Stream()) for _ in range(6)]       # seven streams, as bench.py
        ws = LayerWorkspace(shape, cfg, DEV)
        graphs = StageGraphs(ctx, ctx2, whole=True)
        search_layer(ctx, W, X, ws, graphs=graphs, ctx2=ctx2)            # eager once, captures, replays
        res = search_layer(ctx, W, X, ws, graphs=graphs, ctx2=ctx2)      # replays
        ctx.sync()
        for c in ctx2:
            c.sync()
        res.read_report()
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    lin = {l.name: l for l in shape.linears}

    # a1: moments on sampled columns of every input
    for name, x in X.items():
        cols = np.sort(rng.choice(x.shape[1], 48, replace=False))
        ref = sbo.calib_moments(x[:, torch.from_numpy(cols).to(DEV)].contiguous().cpu(), 1.0 / x.shape[0])
        assert_close(res.moments[name].cpu().numpy()[cols], ref, REL_MOMENT, what=f"moments {name}")
    gm = {n: res.moments[n].cpu().double().numpy() for n in X}

    # a2: channel scores of the coupled sets, whole vectors (oracle fed the GPU's moments)
    Wh = {n: w.cpu() for n, w in W.items()}
    osc = helpers.oracle_layer_scores(shape, Wh, gm, cfg.ref_bits, g)
    for n in ("hidden", "intermediate", "v_heads"):
        assert_close(res.scores[n].cpu().numpy(), osc[n], REL, what=f"scores {n}")
    # a3: permutations given the GPU's scores: exact
    gsc = {n: res.scores[n].cpu().double().numpy() for n in ("hidden", "intermediate", "v_heads")}
    operm = helpers.oracle_layer_perms(shape, gsc)
    for n, p in operm.items():
        assert np.array_equal(res.perms[n].cpu().numpy(), p), n

    # a4: sampled blocks of every matrix; the permuted copy is exact on the sampled tiles
    for name, l in lin.items():
        rp, cp = COUPLING[name]
        pr = operm[rp] if rp else np.arange(l.rows, dtype=np.int32)
        pc = operm[cp] if cp else np.arange(l.cols, dtype=np.int32)
        nbc = l.cols // bc
        nb = (l.rows // br) * nbc
        s0 = res.block_start[name]
        err = res.err[s0:s0 + nb].cpu().numpy()
        for blk in rng.choice(nb, 12, replace=False):
            bi, bj = divmod(int(blk), nbc)
            rows, cols = pr[bi * br:(bi + 1) * br], pc[bj * bc:(bj + 1) * bc]
            tile = Wh[name][torch.from_numpy(rows).long()][:, torch.from_numpy(cols).long()].contiguous()
            got = ws.w_perm[name][bi * br:(bi + 1) * br, bj * bc:(bj + 1) * bc].cpu()
            assert torch.equal(got, tile), f"permuted copy {name} block {blk}"
            oerr, _ = sbo.block_scores(tile, gm[l.act][cols], bits, br, bc, g)
            assert_close(err[blk:blk + 1], oerr, REL, what=f"err {name} block {blk}")

    # a5: allocation given the GPU's table: exact
    table = res.err.cpu().double().numpy()
    st, olv, orep = sbo.allocate_scalebits(table, bits, cfg.budget, cfg.gamma0, cfg.gammaT, br * bc)
    assert st == sbo.OK
    lv = res.level.cpu().numpy()
    if orep["min_margin"] >= 1e-9:
        assert np.array_equal(lv, olv)
        assert res.report["used_bits"] == orep["used_bits"]
        assert res.report["iterations"] == orep["iterations"]
    assert res.report["used_bits"] <= res.report["cap_bits"] == int(np.floor(budget * shape.n_weights))

    # a6: sampled blocks of the packed stream and their metadata; exact budget accounting
    total_words = 0
    for name, l in lin.items():
        rp, cp = COUPLING[name]
        pr = operm[rp] if rp else np.arange(l.rows, dtype=np.int32)
        pc = operm[cp] if cp else np.arange(l.cols, dtype=np.int32)
        nbc = l.cols // bc
        nb = (l.rows // br) * nbc
        s0 = res.block_start[name]
        packed, off, meta = res.packed[name]
        off_h = off.cpu().numpy()
        sizes = np.array(bits)[lv[s0:s0 + nb]] * (br * bc // 32)
        assert off_h[0] == 0 and np.array_equal(np.diff(off_h), sizes)
        total_words += int(off_h[-1])
        meta_h = meta.cpu().numpy().reshape(l.rows, l.cols // g, 2)
        for blk in rng.choice(nb, 6, replace=False):
            bi, bj = divmod(int(blk), nbc)
            rows, cols = pr[bi * br:(bi + 1) * br], pc[bj * bc:(bj + 1) * bc]
            tile = Wh[name][torch.from_numpy(rows).long()][:, torch.from_numpy(cols).long()].contiguous()
            op, _, ometa = sbo.pack_blocks(tile, bits, lv[s0 + blk:s0 + blk + 1], br, bc, g)
            got = packed[int(off_h[blk]):int(off_h[blk + 1])].cpu().numpy().view(np.uint32)
            assert np.array_equal(got, op), f"packed {name} block {blk}"
            gpb = bc // g                                # quantisation groups across one block
            got_meta = np.ascontiguousarray(meta_h[bi * br:(bi + 1) * br, bj * gpb:(bj + 1) * gpb])
            assert np.array_equal(got_meta.view(np.uint32).reshape(-1),
                                  ometa.view(np.uint32).reshape(-1)), f"meta {name} block {blk}"
    assert total_words * 32 == res.report["used_bits"]
    for c in ctx2:
        c.close()
    ctx.close()
