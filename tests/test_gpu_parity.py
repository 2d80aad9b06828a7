"""Parity of the CUDA library (through its C ABI) against the fp64 CPU oracle.

Stage-wise with hand-off: each stage is checked against the oracle stage fed the GPU's
integer outputs of the previous stage (permutations, levels), so a tolerated near-tie
upstream cannot cascade.  Integer outputs (permutations given scores, levels given the
table, codes, offsets, used bits) must be bit-exact; floating-point outputs agree to
1e-4 relative (fp32 accumulation against fp64), moments to 1e-5.
"""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests.helpers import REL, REL_MOMENT, assert_close, unpack_block

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    from paper_2602_17698_b200.binding import Context
    torch.cuda.set_device(0)
    c = Context()
    yield c
    c.sync()
    c.close()


def _host_moments(X):
    return sbo.calib_moments(X.cpu(), 1.0 / max(X.shape[0], 1))


# ---- a1 moments ------------------------------------------------------------------------
@pytest.mark.parametrize("T,K", [(1, 8), (7, 264), (64, 256), (1000, 520), (8192, 2048), (4099, 1032)])
def test_moments(ctx, T, K):
    X = synth.make_activations(T, K, 100 + T, DEV)
    c = ctx.calib_moments(X)
    ctx.sync()
    assert_close(c.cpu().numpy(), _host_moments(X), REL_MOMENT, what="moments")


def test_moments_accumulate_strided_and_deterministic(ctx):
    X = synth.make_activations(3000, 512, 5, DEV)
    out = ctx.calib_moments(X[:1111], scale=1.0)
    ctx.calib_moments(X[1111:], out, accumulate=True, scale=1.0)
    ref = sbo.calib_moments(X.cpu(), 1.0)
    assert_close(out.cpu().numpy(), ref, REL_MOMENT, what="accumulated moments")
    # a column slice has ldx > K
    c = ctx.calib_moments(X[:, 128:384])
    assert_close(c.cpu().numpy(), _host_moments(X[:, 128:384].contiguous()), REL_MOMENT)
    a = ctx.calib_moments(X).clone()
    b = ctx.calib_moments(X)
    ctx.sync()
    assert torch.equal(a, b)                      # fixed summation order: bit-identical reruns
    # no tokens: zero sums
    z = ctx.calib_moments(X[:0], scale=1.0)
    ctx.sync()
    assert torch.count_nonzero(z) == 0


# ---- a2 / a3 reorder ---------------------------------------------------------------------
@pytest.mark.parametrize("R,C,g,bits,roww", [(2048, 2048, 128, 3, False), (200, 384, 64, 2, True),
                                             (130, 272, 16, 4, False), (1024, 512, 32, 8, True)])
def test_reorder_scores_and_sort(ctx, R, C, g, bits, roww):
    W = synth.make_weight(R, C, 7 + R, DEV)
    X = synth.make_activations(512, C, 9 + C, DEV)
    c = ctx.calib_moments(X)
    a = (torch.rand(R, device=DEV) + 0.25) if roww else None
    rs = torch.empty(R, dtype=torch.float32, device=DEV)
    cs = torch.empty(C, dtype=torch.float32, device=DEV)
    pr = torch.empty(R, dtype=torch.int32, device=DEV)
    pc = torch.empty(C, dtype=torch.int32, device=DEV)
    ctx.reorder_channels(W, c, bits, g, row_score=rs, col_score=cs, row_segment=R, col_segment=C,
                         row_perm=pr, col_perm=pc, row_weight=a)
    ctx.sync()
    ch = c.cpu().double().numpy()
    ors, ocs = sbo.reorder_scores(W.cpu(), ch, a=None if a is None else a.cpu().double().numpy(),
                                  ref_bits=bits, group=g)
    assert_close(rs.cpu().numpy(), ors, REL, what="row scores")
    assert_close(cs.cpu().numpy(), ocs, REL, what="col scores")
    # hand-off: the oracle's sort of the GPU's scores must equal the GPU's permutation exactly
    assert np.array_equal(pr.cpu().numpy(), sbo.argsort_desc_segments(rs.cpu().double().numpy()))
    assert np.array_equal(pc.cpu().numpy(), sbo.argsort_desc_segments(cs.cpu().double().numpy()))
    # accumulation over coupled matrices and overwrite semantics
    rs2 = rs.clone()
    ctx.reorder_channels(W, c, bits, g, row_score=rs2, col_score=cs, accumulate_row=True, row_weight=a)
    ctx.sync()
    assert_close(rs2.cpu().numpy(), 2 * ors, REL)
    assert_close(cs.cpu().numpy(), ocs, REL)


def test_segmented_sort_with_ties(ctx):
    K, seg = 1024, 128
    s = torch.randint(0, 5, (K,), device=DEV).float()
    p = torch.empty(K, dtype=torch.int32, device=DEV)
    ctx.reorder_channels(None, None, 2, 128, row_score=s, row_segment=seg, row_perm=p, shape=(K, 128))
    ctx.sync()
    assert np.array_equal(p.cpu().numpy(), sbo.argsort_desc_segments(s.cpu().double().numpy(), seg))
    # a long axis exercises the split counting path
    K = 28672
    s = torch.rand(K, device=DEV)
    s[::7] = s[3]
    p = torch.empty(K, dtype=torch.int32, device=DEV)
    ctx.reorder_channels(None, None, 2, 128, row_score=s, row_segment=K, row_perm=p, shape=(K, 128))
    ctx.sync()
    assert np.array_equal(p.cpu().numpy(), sbo.argsort_desc_segments(s.cpu().double().numpy()))


def test_fold_and_expand(ctx):
    seg, kv, reps = 128, 4, 4
    dst = torch.rand(kv * seg, device=DEV)
    src = torch.rand(kv * reps * seg, device=DEV)
    ref = dst.cpu().double().numpy().copy()
    sbo.fold_segment_scores(ref, src.cpu().double().numpy(), reps, seg)
    ctx.fold_segment_scores(dst, src, reps, seg)
    perm = torch.from_numpy(sbo.argsort_desc_segments(np.random.default_rng(0).random(kv * seg), seg)).to(DEV)
    out = ctx.expand_segment_perm(perm, reps, seg)
    ctx.sync()
    assert_close(dst.cpu().numpy(), ref, 1e-6)
    assert np.array_equal(out.cpu().numpy(), sbo.expand_segment_perm(perm.cpu().numpy(), reps, seg))


# ---- a4 block scores -------------------------------------------------------------------------
def _gain_close(gain, err_ref, bits, M, what):
    """Gains are differences of neighbouring errors: compare at the scale of those errors."""
    gain = gain.cpu().double().numpy()
    for l in range(len(bits) - 1):
        ref = (err_ref[:, l] - err_ref[:, l + 1]) / ((bits[l + 1] - bits[l]) * M)
        tol = REL * (np.abs(err_ref[:, l]) + np.abs(err_ref[:, l + 1])) / ((bits[l + 1] - bits[l]) * M)
        assert np.all(np.abs(gain[:, l] - ref) <= tol + 1e-300), what


@pytest.mark.parametrize("R,C,br,bc,g,bits", [
    (2048, 2048, 128, 128, 128, [2, 3, 4]),            # config 1
    (512, 1024, 128, 128, 128, [2, 3, 4, 8]),
    (256, 512, 32, 32, 32, [1, 2, 3, 4, 5, 6, 8]),
    (256, 512, 64, 64, 32, [2, 3, 4, 8]),
    (384, 256, 64, 128, 64, [1, 2, 3, 4, 5, 6, 7, 8]),
    (512, 512, 256, 128, 16, [3]),
    (256, 768, 128, 256, 128, [2, 4]),
    (96, 640, 48, 128, 128, [2, 3, 4, 5, 6]),          # ragged: block rows not a multiple of 32
])
def test_block_scores_identity(ctx, R, C, br, bc, g, bits):
    W = synth.make_weight(R, C, 11 + R + C, DEV)
    c = ctx.calib_moments(synth.make_activations(256, C, 13, DEV))
    err, gain = ctx.block_scores(W, c, bits, br, bc, g)
    ctx.sync()
    oerr, ogain = sbo.block_scores(W.cpu(), c.cpu().double().numpy(), bits, br, bc, g)
    assert_close(err.cpu().numpy(), oerr, REL, what=f"err {br}x{bc} g{g}")
    if len(bits) > 1:
        _gain_close(gain, oerr, bits, br * bc, "gain")
    e2, _ = ctx.block_scores(W, c, bits, br, bc, g)
    ctx.sync()
    assert torch.equal(err, e2)                      # deterministic


@pytest.mark.parametrize("roww", [False, True])
def test_block_scores_permuted(ctx, roww):
    R, C, bits = 512, 768, [2, 3, 4, 8]
    W = synth.make_weight(R, C, 17, DEV)
    c = ctx.calib_moments(synth.make_activations(256, C, 19, DEV))
    gen = torch.Generator(device="cpu").manual_seed(3)
    pr = torch.randperm(R, generator=gen).int().to(DEV)
    pc = torch.randperm(C, generator=gen).int().to(DEV)
    a = (torch.rand(R, device=DEV) * 3 + 0.1) if roww else None
    ch = c.cpu().double().numpy()
    ah = None if a is None else a.cpu().double().numpy()
    for rp, cp in [(pr, None), (None, pc), (pr, pc)]:
        wout = torch.empty_like(W)
        err, _ = ctx.block_scores(W, c, bits, 128, 128, 64, row_perm=rp, col_perm=cp, row_weight=a,
                                  W_perm_out=wout)
        ctx.sync()
        oerr, _ = sbo.block_scores(W.cpu(), ch, bits, 128, 128, 64,
                                   row_perm=None if rp is None else rp.cpu().numpy(),
                                   col_perm=None if cp is None else cp.cpu().numpy(), a=ah)
        assert_close(err.cpu().numpy(), oerr, REL, what="permuted err")
        ref = W
        if rp is not None:
            ref = ref[rp.long()]
        if cp is not None:
            ref = ref[:, cp.long()]
        assert torch.equal(wout, ref)               # the permuted copy is bit-exact
        e2, _ = ctx.block_scores(W, c, bits, 128, 128, 64, row_perm=rp, col_perm=cp, row_weight=a)
        ctx.sync()
        assert torch.equal(e2, err)                 # with and without the copy requested


def test_block_scores_degenerate_groups(ctx):
    """Constant groups, on-grid groups, a zero matrix and a non-finite weight."""
    R = C = 256
    W = synth.make_weight(R, C, 23, DEV)
    W[0:64] = 0.375                                  # constant rows: zero error
    q = torch.randint(0, 4, (64, C), device=DEV)
    q[:, 0::128] = 0
    q[:, 1::128] = 3
    W[64:128] = (q.float() * 0.25 - 1.0).to(torch.bfloat16)    # exactly on the 2-bit grid
    c = torch.ones(C, device=DEV)
    bits = [2, 4]
    err, _ = ctx.block_scores(W, c, bits, 64, 128, 128)
    ctx.sync()
    oerr, _ = sbo.block_scores(W.cpu(), np.ones(C), bits, 64, 128, 128)
    # on-grid data has zero error in exact arithmetic; fp32 leaves the rounding of the grid
    # step: floor 1e-12 * sum W^2 of a block (~3e3 here)
    assert_close(err.cpu().numpy(), oerr, REL, abs_floor=3e-9)
    assert torch.count_nonzero(err[:2]) == 0         # block row 0: constant groups
    assert float(err[2:4].max()) < 3e-9              # block row 1: on the 2- and 4-bit grids
    Wz = torch.zeros_like(W)
    ez, _ = ctx.block_scores(Wz, c, bits, 64, 128, 128)
    ctx.sync()
    assert torch.count_nonzero(ez) == 0
    from paper_2602_17698_b200.binding import SbError, SB_ERR_NONFINITE
    W[200, 5] = float("inf")
    ctx.block_scores(W, c, bits, 64, 128, 128)
    with pytest.raises(SbError) as ei:
        ctx.sync()
    assert ei.value.status == SB_ERR_NONFINITE
    ctx.sync()                                       # the latch is cleared by the failing sync


def test_argument_errors_touch_no_gpu(ctx):
    from paper_2602_17698_b200.binding import SbError, SB_ERR_SHAPE, SB_ERR_INVALID, SB_ERR_BUDGET
    W = synth.make_weight(256, 256, 1, DEV)
    c = torch.ones(256, device=DEV)
    n0 = ctx.kernel_launches()
    for kw, st in [(dict(bits=[4, 3]), SB_ERR_INVALID), (dict(bits=[0, 2]), SB_ERR_INVALID),
                   (dict(bits=[2], block_rows=100), SB_ERR_SHAPE),
                   (dict(bits=[2], block_cols=128, group=96), SB_ERR_SHAPE),
                   (dict(bits=[2], block_cols=64, group=128), SB_ERR_SHAPE)]:
        with pytest.raises(SbError) as ei:
            ctx.block_scores(W, c, **kw)
        assert ei.value.status == st
    err = torch.rand(64, 3, device=DEV)
    with pytest.raises(SbError) as ei:
        ctx.allocate_bits(err, [2, 3, 4], 1.5)
    assert ei.value.status == SB_ERR_BUDGET
    with pytest.raises(SbError) as ei:
        ctx.allocate_bits(err, [2, 3, 4], 3.0, gamma0=0.0)
    assert ei.value.status == SB_ERR_INVALID
    assert ctx.kernel_launches() == n0


# ---- a5 allocation -------------------------------------------------------------------------------
def _tables(N, L, seed, kind):
    rng = np.random.default_rng(seed)
    if kind == "convex":
        A = rng.uniform(0.5, 50.0, size=(N, 1))
        r = rng.uniform(0.2, 0.6, size=(N, 1))
        t = A * r ** np.arange(L)[None, :]
    elif kind == "ragged":      # neither monotone nor convex everywhere
        t = rng.uniform(1, 30, size=(N, 1)) * 0.4 ** np.arange(L)[None, :] * rng.uniform(0.5, 1.8, size=(N, L))
    else:                        # many exact ties
        t = np.tile(np.array([8.0, 2.0, 0.5, 0.125, 0.03, 0.01, 0.004, 0.001])[:L], (N, 1))
        t[::3] *= 2.0
    return t.astype(np.float32)


def _check_alloc(ctx, table, bits, budget, mode, g0=0.05, gT=0.02, sizes=None, M=128 * 128):
    from paper_2602_17698_b200.binding import SB_ALLOC_GREEDY
    err = torch.from_numpy(table).to(DEV)
    be = None if sizes is None else torch.from_numpy(sizes).to(DEV)
    level, rep = ctx.allocate_bits(err, bits, budget, mode, g0, gT, uniform_block_elems=M, block_elems=be)
    t64 = table.astype(np.float64)
    if mode == SB_ALLOC_GREEDY:
        N = table.shape[0]
        st, olv, orep = sbo.allocate_greedy(t64, bits, budget, M, sizes, heap=N > 2000)
    else:
        st, olv, orep = sbo.allocate_scalebits(t64, bits, budget, g0, gT, M, sizes)
    assert st == sbo.OK
    lv = level.cpu().numpy()
    if mode != SB_ALLOC_GREEDY and orep["min_margin"] < 1e-9:
        # an accept decision sat on a rounding-level tie of the two fp64 sums: only the
        # invariants are comparable
        assert rep["used_bits"] <= rep["cap_bits"]
        return lv, rep
    assert np.array_equal(lv, olv), (np.flatnonzero(lv != olv)[:10], rep, orep)
    assert rep["used_bits"] == orep["used_bits"] and rep["cap_bits"] == orep["cap_bits"]
    assert rep["used_bits"] <= rep["cap_bits"]
    assert rep["proxy_loss_final"] == pytest.approx(orep["proxy_loss_final"], rel=1e-9)
    assert rep["proxy_loss_init"] == pytest.approx(orep["proxy_loss_init"], rel=1e-9)
    assert rep["level_hist"] == orep["level_hist"]
    if mode != SB_ALLOC_GREEDY:
        for k in ("iterations", "accepted", "rejected", "expansions"):
            assert rep[k] == orep[k], (k, rep, orep)
    else:
        assert rep["iterations"] == orep["iterations"]
    return lv, rep


@pytest.mark.parametrize("kind", ["convex", "ragged", "ties"])
@pytest.mark.parametrize("N,bits", [(7, [2, 3, 4]), (300, [2, 3, 4, 8]), (5000, [1, 2, 3, 4, 5, 6, 8]),
                                    (13312, [2, 3, 4, 8]),
                                    # step lists of 7500, 65535 and 65538 keys: a two-CTA cluster sort, the
                                    # largest one, and the first size of the multi-launch sort
                                    (2500, [2, 3, 4, 8]), (21845, [2, 3, 4, 8]), (21846, [2, 3, 4, 8])])
def test_allocate_scalebits(ctx, kind, N, bits):
    from paper_2602_17698_b200.binding import SB_ALLOC_SCALEBITS
    table = _tables(N, len(bits), N, kind)
    for budget in (bits[0], bits[0] + 0.25, 2.5, 3.0, 3.3, bits[-1], bits[-1] + 1.0):
        if budget < bits[0]:
            continue
        _check_alloc(ctx, table, bits, budget, SB_ALLOC_SCALEBITS)
    _check_alloc(ctx, table, bits, 2.75, SB_ALLOC_SCALEBITS, g0=0.3, gT=0.01)


@pytest.mark.parametrize("kind", ["convex", "ragged", "ties"])
@pytest.mark.parametrize("N,bits", [(7, [2, 3, 4]), (300, [2, 3, 4, 8]), (5000, [1, 2, 3, 4, 5, 6, 8])])
def test_allocate_greedy(ctx, kind, N, bits):
    from paper_2602_17698_b200.binding import SB_ALLOC_GREEDY
    table = _tables(N, len(bits), 50 + N, kind)
    for budget in (bits[0], bits[0] + 0.25, 2.5, 3.0, 3.3, bits[-1], bits[-1] + 1.0):
        if budget < bits[0]:
            continue
        _check_alloc(ctx, table, bits, budget, SB_ALLOC_GREEDY)


def test_allocate_scalebits_walks_the_handworked_trajectories(ctx):
    """The instances of tests/golden/alg2_handworked.txt (derived by hand from Algorithm 2's
    text): final levels and every counter, straight against the file."""
    from paper_2602_17698_b200.binding import SB_ALLOC_SCALEBITS
    from tests.test_oracle_alg2_handworked import CASES
    for case in CASES:
        err = torch.tensor(case["table"], dtype=torch.float32, device=DEV)
        be = torch.tensor(case["block_elems"], dtype=torch.int64, device=DEV)
        level, rep = ctx.allocate_bits(err, case["bits"], case["budget"], SB_ALLOC_SCALEBITS,
                                       case["gamma0"], case["gammaT"], uniform_block_elems=0, block_elems=be)
        fin = case["final"]
        assert level.cpu().tolist() == case["trace"][-1], case["name"]
        for key in ("iterations", "expansions", "accepted", "rejected", "used_bits", "cap_bits"):
            assert rep[key] == int(fin[key]), (case["name"], key, rep)
        assert rep["proxy_loss_init"] == fin["loss_init"] and rep["proxy_loss_final"] == fin["loss_final"]


def test_lookback_wait_runs_out_and_the_context_stays_usable(ctx):
    """The one device-side wait of the path (a scan tile waiting for its predecessor) is bounded:
    with the test hook tile 0 of the cost prefix sum publishes nothing, tile 1 waits 1 ms, gives
    up, latches SB_ERR_TIMEOUT and the kernel returns.  Nothing hangs or traps; the context works
    afterwards."""
    from paper_2602_17698_b200.binding import SB_ALLOC_GREEDY, SB_ERR_TIMEOUT, SbError
    N, bits = 20000, [2, 3, 4, 8]                       # <= 60000 steps: one-launch sort, a scan of many tiles
    table = _tables(N, len(bits), 5, "convex")
    err = torch.from_numpy(table).to(DEV)
    ctx.debug_lookback(wait_ns=1_000_000, mute_tile=0)
    try:
        with pytest.raises(SbError) as ei:
            ctx.allocate_bits(err, bits, 2.5, SB_ALLOC_GREEDY)
        assert ei.value.status == SB_ERR_TIMEOUT
    finally:
        ctx.debug_lookback()                            # defaults: 250 ms, no muted tile
    _check_alloc(ctx, table, bits, 2.5, SB_ALLOC_GREEDY)    # exact again, the status was cleared


def test_allocate_enqueue_only_form_and_its_latched_errors(ctx):
    """sb_allocate_bits_async: same levels and report as the synchronous call (which is checked
    against the oracle above), eager and replayed from a CUDA graph; a greedy budget below the
    smallest candidate is latched and comes back from the next sync."""
    from paper_2602_17698_b200.binding import (Context, SB_ALLOC_GREEDY, SB_ALLOC_SCALEBITS, SB_ERR_BUDGET,
                                               SbError)
    rng = np.random.default_rng(8)
    N, bits = 3000, [2, 3, 4, 8]
    table = _tables(N, 4, 78, "ragged")
    err = torch.from_numpy(table).to(DEV)
    sizes = torch.from_numpy(rng.choice([1024, 4096, 16384], size=N).astype(np.int64)).to(DEV)
    for mode in (SB_ALLOC_SCALEBITS, SB_ALLOC_GREEDY):
        for be in (None, sizes):
            lv_ref, rep_ref = ctx.allocate_bits(err, bits, 2.6, mode, block_elems=be)
            lv, rep = ctx.allocate_bits_async(err, bits, 2.6, mode, block_elems=be)
            n0 = ctx.kernel_launches()
            ctx.sync()
            assert ctx.kernel_launches() == n0
            assert torch.equal(lv, lv_ref) and Context.read_report(rep) == rep_ref
    # degenerate tables: a single candidate (no steps at all), a single block
    for tab, bb, budget in ((table[:, :1].copy(), [4], 4.0), (table[:1].copy(), bits, 3.0)):
        e1 = torch.from_numpy(tab).to(DEV)
        for mode in (SB_ALLOC_SCALEBITS, SB_ALLOC_GREEDY):
            lv_ref, rep_ref = ctx.allocate_bits(e1, bb, budget, mode)
            lv, rep = ctx.allocate_bits_async(e1, bb, budget, mode)
            ctx.sync()
            assert torch.equal(lv, lv_ref) and Context.read_report(rep) == rep_ref
            assert rep_ref["used_bits"] <= rep_ref["cap_bits"]
    # captured once, replayed on a changed table: the graph holds no value of the first run
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        c2 = Context()
        e2 = err.clone()
        lv, rep = c2.allocate_bits_async(e2, bits, 2.6)          # eager once: scratch growth
        c2.sync()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            c2.allocate_bits_async(e2, bits, 2.6, level=lv, report=rep)
        table2 = _tables(N, 4, 79, "convex")
        e2.copy_(torch.from_numpy(table2).to(DEV))
        g.replay()
        c2.sync()
        lv_ref, rep_ref = c2.allocate_bits(e2, bits, 2.6)
        assert torch.equal(lv, lv_ref) and Context.read_report(rep) == rep_ref
        c2.close()
    torch.cuda.synchronize()
    _check_alloc(ctx, table2, bits, 2.6, SB_ALLOC_SCALEBITS)
    # greedy below the smallest candidate: the synchronous call and the next sync report it
    with pytest.raises(SbError) as ei:
        ctx.allocate_bits(err, bits, 1.5, SB_ALLOC_GREEDY)
    assert ei.value.status == SB_ERR_BUDGET
    lv, rep = ctx.allocate_bits_async(err, bits, 1.5, SB_ALLOC_GREEDY)
    with pytest.raises(SbError) as ei:
        ctx.sync()
    assert ei.value.status == SB_ERR_BUDGET
    assert int(lv.max().item()) == 0                            # no step was applied
    ctx.sync()                                                  # the latch is cleared


def test_allocate_nonuniform_block_sizes(ctx):
    from paper_2602_17698_b200.binding import SB_ALLOC_GREEDY, SB_ALLOC_SCALEBITS
    rng = np.random.default_rng(4)
    N, bits = 3000, [2, 3, 4, 8]
    table = _tables(N, 4, 77, "ragged")
    sizes = rng.choice([1024, 4096, 16384, 32768], size=N).astype(np.int64)
    for budget in (2.5, 3.1, 5.0):
        _check_alloc(ctx, table, bits, budget, SB_ALLOC_SCALEBITS, sizes=sizes)
        _check_alloc(ctx, table, bits, budget, SB_ALLOC_GREEDY, sizes=sizes)


def test_allocate_large_table_spans_many_scan_tiles(ctx):
    from paper_2602_17698_b200.binding import SB_ALLOC_SCALEBITS, SB_ALLOC_GREEDY
    N, bits = 425_984, [2, 3, 4, 8]                  # the 8B-shaped model's block count
    table = _tables(N, 4, 99, "ragged")
    _check_alloc(ctx, table, bits, 2.5, SB_ALLOC_SCALEBITS)
    _check_alloc(ctx, table, bits, 3.0, SB_ALLOC_SCALEBITS)
    _check_alloc(ctx, table, bits, 2.5, SB_ALLOC_GREEDY)


# ---- a6 pack ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("br,bc,g", [(128, 128, 128), (64, 128, 64), (32, 32, 32), (64, 64, 16),
                                     (256, 128, 128), (128, 256, 128)])
def test_pack(ctx, br, bc, g):
    R, C = 512, 512
    bits = [1, 2, 3, 4, 5, 6, 8]
    W = synth.make_weight(R, C, 31 + br, DEV)
    W[3, 0:128] = 0.5                                # a constant group
    rng = np.random.default_rng(br + bc)
    nb = (R // br) * (C // bc)
    level = torch.from_numpy(rng.integers(0, len(bits), size=nb).astype(np.uint8)).to(DEV)
    pr = torch.from_numpy(rng.permutation(R).astype(np.int32)).to(DEV)
    pc = torch.from_numpy(rng.permutation(C).astype(np.int32)).to(DEV)
    for rp, cp in [(None, None), (pr, pc)]:
        packed, off, meta = ctx.pack_blocks(W, bits, level, br, bc, g, row_perm=rp, col_perm=cp)
        ctx.sync()
        op, ooff, ometa = sbo.pack_blocks(W.cpu(), bits, level.cpu().numpy(), br, bc, g,
                                          row_perm=None if rp is None else rp.cpu().numpy(),
                                          col_perm=None if cp is None else cp.cpu().numpy())
        assert np.array_equal(off.cpu().numpy(), ooff)
        n = int(ooff[-1])
        assert np.array_equal(packed.cpu().numpy().view(np.uint32)[:n], op)
        assert np.array_equal(meta.cpu().numpy().view(np.uint32), ometa.view(np.uint32))
    # a spot check that the stream really decodes to codes in range
    b = bits[int(level[0])]
    codes = unpack_block(packed.cpu().numpy().view(np.uint32)[: int(ooff[1])], br * bc, b)
    assert codes.max() <= 2 ** b - 1


def test_pack_many_blocks_offsets_span_several_scan_tiles(ctx):
    R, C, br, bc, g = 2048, 4096, 32, 32, 32          # 8192 blocks x 2 = 16384 > one CTA's scan
    bits = [2, 3, 4]
    W = synth.make_weight(2 * R, C, 77, DEV)
    nb = (2 * R // br) * (C // bc)
    rng = np.random.default_rng(5)
    level = torch.from_numpy(rng.integers(0, len(bits), size=nb).astype(np.uint8)).to(DEV)
    packed, off, meta = ctx.pack_blocks(W, bits, level, br, bc, g)
    ctx.sync()
    sizes = np.array(bits)[level.cpu().numpy()] * (br * bc // 32)
    off_h = off.cpu().numpy()
    assert off_h[0] == 0 and np.array_equal(np.diff(off_h), sizes)
    # sampled blocks against the oracle
    Wh = W.cpu()
    nbc = C // bc
    for blk in rng.choice(nb, 16, replace=False):
        bi, bj = divmod(int(blk), nbc)
        tile = Wh[bi * br:(bi + 1) * br, bj * bc:(bj + 1) * bc].contiguous()
        op, _, ometa = sbo.pack_blocks(tile, bits, level[blk:blk + 1].cpu().numpy(), br, bc, g)
        got = packed[int(off_h[blk]):int(off_h[blk + 1])].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, op)


def test_pack_capacity_is_enforced(ctx):
    from paper_2602_17698_b200.binding import SbError, SB_ERR_SCRATCH
    W = synth.make_weight(256, 256, 3, DEV)
    level = torch.full((4,), 2, dtype=torch.uint8, device=DEV)
    small = torch.zeros(100, dtype=torch.int32, device=DEV)
    ctx.pack_blocks(W, [2, 3, 4], level, 128, 128, 128, packed=small)
    with pytest.raises(SbError) as ei:
        ctx.sync()
    assert ei.value.status == SB_ERR_SCRATCH


def test_sum_scores_adds_left_to_right(ctx):
    """sb_sum_scores: fp32 adds in source order, with and without the destination as first term
    (bit-exact against the same adds in numpy float32)."""
    from paper_2602_17698_b200.binding import SbError, SB_ERR_INVALID
    rng = np.random.default_rng(3)
    n = 5000
    srcs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-3, 4)).astype(np.float32) for _ in range(8)]
    d0 = rng.standard_normal(n).astype(np.float32)
    for k in (1, 3, 8):
        for acc in (False, True):
            want = d0.copy() if acc else np.zeros(n, np.float32)
            start = 0
            if not acc:
                want = srcs[0].copy(); start = 1
            for s_ in srcs[start:k]:
                want = (want + s_).astype(np.float32)
            dst = torch.from_numpy(d0.copy()).to(DEV)
            ctx.sum_scores(dst, [torch.from_numpy(s_).to(DEV) for s_ in srcs[:k]], accumulate=acc)
            ctx.sync()
            assert np.array_equal(dst.cpu().numpy().view(np.uint32), want.view(np.uint32)), (k, acc)
    with pytest.raises(AssertionError):
        ctx.sum_scores(dst, [])
