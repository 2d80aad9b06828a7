"""One Llama-shaped decoder layer through the whole path, stage-wise against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests import helpers
from tests.helpers import REL, REL_MOMENT, assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("bits,budget,br,bc,g", [([2, 3, 4, 8], 2.5, 128, 128, 128),
                                                 ([2, 3, 4], 3.0, 64, 128, 64)])
def test_tiny_layer_stagewise(bits, budget, br, bc, g):
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import COUPLING, LayerWorkspace, SearchConfig, search_layer
    torch.cuda.set_device(0)
    shape = synth.LLAMA_TINY
    W = synth.make_layer_weights(shape, 0, 0, DEV)
    X = synth.make_layer_activations(shape, 1024, 0, 0, DEV)
    cfg = SearchConfig(bits=bits, budget=budget, block_rows=br, block_cols=bc, group=g,
                       gamma0=0.2, gammaT=0.05)
    ctx = Context()
    ws = LayerWorkspace(shape, cfg, DEV)
    res = search_layer(ctx, W, X, ws)
    ctx.sync()
    Wh = {n: w.cpu() for n, w in W.items()}
    lin = {l.name: l for l in shape.linears}

    # a1 moments
    mom = {n: sbo.calib_moments(x.cpu(), 1.0 / x.shape[0]) for n, x in X.items()}
    for n in mom:
        assert_close(res.moments[n].cpu().numpy(), mom[n], REL_MOMENT, what=f"moments {n}")
    gm = {n: res.moments[n].cpu().double().numpy() for n in mom}      # hand-off: GPU moments

    # a2 coupled channel scores (oracle fed the GPU's moments)
    osc = helpers.oracle_layer_scores(shape, Wh, gm, cfg.ref_bits, g)
    for n in ("hidden", "intermediate", "v_heads"):
        assert_close(res.scores[n].cpu().numpy(), osc[n], REL, what=f"scores {n}")

    # a3 permutations (oracle sorts the GPU's scores): exact
    gsc = {n: res.scores[n].cpu().double().numpy() for n in ("hidden", "intermediate", "v_heads")}
    operm = helpers.oracle_layer_perms(shape, gsc)
    for n, p in operm.items():
        assert np.array_equal(res.perms[n].cpu().numpy(), p), n
        assert sorted(p.tolist()) == list(range(p.size))

    # a4 block table (oracle fed the GPU's permutations and moments)
    L = len(bits)
    for name, l in lin.items():
        rp, cp = COUPLING[name]
        oerr, _ = sbo.block_scores(Wh[name], gm[l.act], bits, br, bc, g,
                                   row_perm=None if rp is None else operm[rp],
                                   col_perm=None if cp is None else operm[cp])
        s = res.block_start[name]
        assert_close(res.err[s:s + oerr.shape[0]].cpu().numpy(), oerr, REL, what=f"err {name}")

    # a5 allocation (oracle fed the GPU's table): exact
    table = res.err.cpu().double().numpy()
    st, olv, orep = sbo.allocate_scalebits(table, bits, budget, cfg.gamma0, cfg.gammaT, br * bc)
    assert st == sbo.OK
    if orep["min_margin"] >= 1e-9:
        assert np.array_equal(res.level.cpu().numpy(), olv)
        assert res.report["used_bits"] == orep["used_bits"]
        assert res.report["iterations"] == orep["iterations"]
    assert res.report["used_bits"] <= res.report["cap_bits"]

    # a6 pack (oracle fed the GPU's permutations and levels): exact
    lv = res.level.cpu().numpy()
    total_words = 0
    for name, l in lin.items():
        rp, cp = COUPLING[name]
        nb = (l.rows // br) * (l.cols // bc)
        s = res.block_start[name]
        op, ooff, ometa = sbo.pack_blocks(Wh[name], bits, lv[s:s + nb], br, bc, g,
                                          row_perm=None if rp is None else operm[rp],
                                          col_perm=None if cp is None else operm[cp])
        packed, off, meta = res.packed[name]
        assert np.array_equal(off.cpu().numpy(), ooff)
        assert np.array_equal(packed.cpu().numpy().view(np.uint32)[: int(ooff[-1])], op)
        assert np.array_equal(meta.cpu().numpy().view(np.uint32), ometa.view(np.uint32))
        total_words += int(ooff[-1])
    assert total_words * 32 == res.report["used_bits"]          # exact budget accounting
    ctx.close()


def test_two_contexts_give_the_same_layer_result():
    """search_layer with a second context (the independent calls of the stages dealt to two streams, eager and
    from CUDA graphs) against the one-context run: every output identical."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import LayerWorkspace, SearchConfig, StageGraphs, search_layer
    torch.cuda.set_device(0)
    shape = synth.LLAMA_TINY
    cfg = SearchConfig(bits=[2, 3, 4, 8], budget=2.75)
    W = synth.make_layer_weights(shape, 5, 0, DEV)
    X = synth.make_layer_activations(shape, 1024, 5, 0, DEV)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s1):
        ctx = Context()
        ctx2 = Context(stream=s2)
        ws_a, ws_b, ws_c = (LayerWorkspace(shape, cfg, DEV) for _ in range(3))
        ref = search_layer(ctx, W, X, ws_a)
        ctx.sync()
        eager = search_layer(ctx, W, X, ws_b, ctx2=ctx2)
        ctx.sync(); ctx2.sync()
        graphs = StageGraphs(ctx, ctx2)
        search_layer(ctx, W, X, ws_c, graphs=graphs, ctx2=ctx2)           # captures
        replay = search_layer(ctx, W, X, ws_c, graphs=graphs, ctx2=ctx2)  # replays
        ctx.sync(); ctx2.sync()
    torch.cuda.synchronize()
    assert ctx2.kernel_launches() > 0
    for got in (eager, replay):
        assert torch.equal(got.err, ref.err) and torch.equal(got.level, ref.level)
        assert got.report == ref.report
        for name in ref.packed:
            for a, b in zip(got.packed[name], ref.packed[name]):
                n = int(ref.packed[name][1][-1].item()) if a.dtype == torch.int32 else a.numel()
                assert torch.equal(a.reshape(-1)[:n], b.reshape(-1)[:n]), name
    ctx2.close()
    ctx.close()


def test_whole_step_graph_gives_the_same_layer_result():
    """The step as ONE CUDA graph (allocation enqueued, report on the device) against the eager
    step with the synchronous allocation: identical levels, report and packed words, on one
    context and on two."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import LayerWorkspace, SearchConfig, StageGraphs, search_layer
    torch.cuda.set_device(0)
    shape = synth.LLAMA_TINY
    cfg = SearchConfig(bits=[2, 3, 4, 8], budget=2.75)
    W = synth.make_layer_weights(shape, 21, 0, DEV)
    X = synth.make_layer_activations(shape, 640, 21, 0, DEV)
    stream = torch.cuda.Stream(device=DEV)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        ctx = Context()
        ctx2 = Context(stream=torch.cuda.Stream(device=DEV))
        ws_ref = LayerWorkspace(shape, cfg, DEV)
        ref = search_layer(ctx, W, X, ws_ref)
        torch.cuda.synchronize()
        more = [Context(stream=torch.cuda.Stream(device=DEV)) for _ in range(6)]
        for second in (None, ctx2, more):                        # one, two and seven streams
            ws = LayerWorkspace(shape, cfg, DEV)
            graphs = StageGraphs(ctx, second, whole=True)
            for _ in range(3):                                   # eager + capture + replay, then two replays
                got = search_layer(ctx, W, X, ws, graphs=graphs, ctx2=second)
            ctx.sync()
            for c in ([] if second is None else [second] if second is ctx2 else second):
                c.sync()
                assert c.kernel_launches() > 0
            assert got.report is None and got.read_report() == ref.report
            assert torch.equal(got.level, ref.level)
            assert torch.equal(ws.err, ws_ref.err)
            for name in ref.packed:
                off = ref.packed[name][1]
                n = int(off[-1].item())
                assert torch.equal(got.packed[name][1], off), name
                assert torch.equal(got.packed[name][0][:n], ref.packed[name][0][:n]), name
                assert torch.equal(got.packed[name][2], ref.packed[name][2]), name
        for c in more:
            c.close()
        ctx2.close()
        ctx.close()
