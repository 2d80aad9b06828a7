"""Full second-moment matrix H = X^T X / T on the tensor cores against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    from paper_2602_17698_b200.binding import Context
    torch.cuda.set_device(0)
    c = Context()
    yield c
    c.close()


def _check(H, ref):
    """bf16 products are exact in fp32; the sum over tokens is accumulated in fp32: entries are
    compared at the scale sqrt(H_ii H_jj) of their row and column (off-diagonal sums cancel)."""
    d = np.sqrt(np.diag(ref))
    scale = np.outer(d, d) + 1e-300
    err = np.abs(H - ref) / scale
    assert err.max() <= 5e-6, (err.max(), np.unravel_index(err.argmax(), err.shape))


@pytest.mark.parametrize("T,K", [(256, 128), (64, 128), (256, 256), (1000, 384), (100, 200), (4096, 520),
                                 (8192, 1024)])
def test_gram_matrix(ctx, T, K):
    X = synth.make_activations(T, K, 3 + T + K, DEV)
    H = ctx.calib_gram(X)
    ctx.sync()
    Hh = H.cpu().double().numpy()
    assert np.array_equal(Hh, Hh.T)                       # both triangles written, mirror images
    ref = sbo.calib_gram(X.cpu())
    _check(Hh, ref)
    # the diagonal is what sb_calib_moments returns
    c = ctx.calib_moments(X)
    ctx.sync()
    assert np.allclose(np.diag(Hh), c.cpu().double().numpy(), rtol=2e-5)


def test_gram_matrix_at_the_calibration_token_count(ctx):
    """65536 tokens = 128 accumulator drains of 512 tokens each: the regime in which a single
    tensor-core accumulator was seen to drift."""
    T, K = 65536, 256
    X = synth.make_activations(T, K, 77, DEV)
    H = ctx.calib_gram(X)
    ctx.sync()
    _check(H.cpu().double().numpy(), sbo.calib_gram(X.cpu()))


def test_gram_accumulate_strided_and_deterministic(ctx):
    T, K = 512, 256
    big = synth.make_activations(T, K + 64, 9, DEV)
    X = big[:, :K]                                        # leading dimension K + 64
    H1 = ctx.calib_gram(X, scale=1.0)
    H2 = ctx.calib_gram(X, scale=1.0)
    ctx.sync()
    assert torch.equal(H1, H2)
    ctx.calib_gram(X, H=H2, accumulate=True, scale=1.0)
    ctx.sync()
    assert torch.allclose(H2, 2 * H1, rtol=1e-6)
    ref = sbo.calib_gram(X.contiguous().cpu(), scale=1.0)
    _check(H1.cpu().double().numpy(), ref)


# ---- block error table with the full second-moment matrix -------------------------------------------
@pytest.mark.parametrize("R,C,g,bits,perm", [(128, 128, 128, [2, 3, 4, 8], False), (256, 256, 128, [2, 3, 4, 8], False),
                                             (512, 384, 64, [2, 3, 4], True), (384, 512, 16, [1, 2, 3, 4, 5, 6, 8], True),
                                             (2048, 1024, 32, [3, 4], False)])
def test_block_scores_with_the_full_second_moment_matrix(ctx, R, C, g, bits, perm):
    from tests.helpers import REL
    W = synth.make_weight(R, C, 51 + R + C, DEV)
    X = synth.make_activations(2048, C, 53 + C, DEV)
    H = ctx.calib_gram(X)
    rng = np.random.default_rng(R + C)
    pr = torch.from_numpy(rng.permutation(R).astype(np.int32)).to(DEV) if perm else None
    pc = torch.from_numpy(rng.permutation(C).astype(np.int32)).to(DEV) if perm else None
    err, gain = ctx.block_scores_full(W, H, bits, 128, 128, g, row_perm=pr, col_perm=pc)
    ctx.sync()
    # hand-off: the oracle is fed the GPU's matrix
    ref = sbo.block_scores_full(W.cpu(), H.cpu().double().numpy(), bits, 128, 128, g,
                                row_perm=None if pr is None else pr.cpu().numpy(),
                                col_perm=None if pc is None else pc.cpu().numpy())
    got = err.cpu().double().numpy()
    assert np.all(np.abs(got - ref) <= REL * np.abs(ref)), np.max(np.abs(got - ref) / np.abs(ref))
    if len(bits) > 1:
        gref = (ref[:, :-1] - ref[:, 1:]) / (np.diff(bits)[None, :] * 128 * 128)
        tol = REL * (np.abs(ref[:, :-1]) + np.abs(ref[:, 1:])) / (np.diff(bits)[None, :] * 128 * 128)
        assert np.all(np.abs(gain.cpu().double().numpy() - gref) <= tol)
    e2, _ = ctx.block_scores_full(W, H, bits, 128, 128, g, row_perm=pr, col_perm=pc)
    ctx.sync()
    assert torch.equal(err, e2)                       # deterministic


@pytest.mark.parametrize("R,C,g,bits", [(2560, 2048, 128, [2, 3, 4, 8]),     # 320 blocks, 20 per block column
                                        (640, 8192, 64, [2, 3, 4])])        # 320 blocks, 5 per block column
def test_full_scores_when_a_cta_walks_several_blocks_and_block_columns(ctx, R, C, g, bits):
    """More blocks than CTAs: every CTA walks a stretch of two or three blocks of the
    column-major block sequence, most stretches of the second shape cross a block-column
    boundary (a new H tile), and the operand ring carries over from block to block."""
    from tests.helpers import REL
    W = synth.make_weight(R, C, 71 + R, DEV)
    X = synth.make_activations(1024, C, 73 + C, DEV)
    H = ctx.calib_gram(X)
    rng = np.random.default_rng(R + C)
    pc = torch.from_numpy(rng.permutation(C).astype(np.int32)).to(DEV)
    err, _ = ctx.block_scores_full(W, H, bits, 128, 128, g, col_perm=pc)
    ctx.sync()
    assert err.shape[0] == (R // 128) * (C // 128) > 2 * 148
    ref = sbo.block_scores_full(W.cpu(), H.cpu().double().numpy(), bits, 128, 128, g,
                                col_perm=pc.cpu().numpy())
    got = err.cpu().double().numpy()
    assert np.all(np.abs(got - ref) <= REL * np.abs(ref)), np.max(np.abs(got - ref) / np.abs(ref))


def test_full_scores_sampled_blocks_of_a_layer_sized_matrix(ctx):
    """The matrix bench.py times (14336 x 4096, four candidates, 3584 blocks on 148 CTAs):
    sampled blocks against the oracle, which is fed the GPU's H and the block's own rows and
    columns (a block's error depends on nothing else)."""
    from tests.helpers import REL
    R, C, g, bits = 14336, 4096, 128, [2, 3, 4, 8]
    W = synth.make_weight(R, C, 81, DEV)
    X = synth.make_activations(4096, C, 83, DEV)
    H = ctx.calib_gram(X)
    err, _ = ctx.block_scores_full(W, H, bits, 128, 128, g)
    ctx.sync()
    got = err.cpu().double().numpy()
    rng = np.random.default_rng(5)
    nbc = C // 128
    picks = list(rng.choice(got.shape[0], 10, replace=False)) + [0, got.shape[0] - 1]
    for blk in picks:
        bi, bj = divmod(int(blk), nbc)
        tile = W[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128].contiguous().cpu()
        Hjj = H[bj * 128:(bj + 1) * 128, bj * 128:(bj + 1) * 128].cpu().double().numpy()
        ref = sbo.block_scores_full(tile, np.ascontiguousarray(Hjj), bits, 128, 128, g)
        assert np.all(np.abs(got[blk:blk + 1] - ref) <= REL * np.abs(ref)), (blk, got[blk], ref)


@pytest.mark.parametrize("R,C,br,bc,g,bits,weights,perm", [
    (512, 384, 64, 128, 128, [2, 3, 4, 8], False, False),     # the paper's default partition, 64 x 128
    (1024, 256, 64, 128, 32, [2, 3, 4], True, True),
    (1024, 384, 256, 128, 64, [2, 3, 4, 8], False, True),     # 256 x 128: two contraction units per block
    (512, 256, 256, 128, 128, [3, 4], True, False),
    (512, 512, 128, 128, 128, [2, 3, 4, 8], True, True),      # row weights on the 128 x 128 form
    (512, 384, 64, 64, 64, [2, 3, 4, 8], False, False),       # 64-column blocks: two side by side in a unit
    (512, 256, 128, 64, 32, [2, 3, 4], True, True),
    (1024, 384, 256, 64, 64, [2, 4, 8], False, True),
    (1280, 4096, 64, 64, 16, [3, 4], True, False),            # more units than CTAs
])
def test_full_scores_block_shapes_and_row_weights(ctx, R, C, br, bc, g, bits, weights, perm):
    from tests.helpers import REL
    W = synth.make_weight(R, C, 91 + R + br, DEV)
    X = synth.make_activations(1024, C, 93 + C, DEV)
    H = ctx.calib_gram(X)
    rng = np.random.default_rng(R + C + br)
    pr = torch.from_numpy(rng.permutation(R).astype(np.int32)).to(DEV) if perm else None
    pc = torch.from_numpy(rng.permutation(C).astype(np.int32)).to(DEV) if perm else None
    a = (torch.rand(R, device=DEV) * 3 + 0.1) if weights else None
    err, gain = ctx.block_scores_full(W, H, bits, br, bc, g, row_perm=pr, col_perm=pc, row_weight=a)
    ctx.sync()
    ref = sbo.block_scores_full(W.cpu(), H.cpu().double().numpy(), bits, br, bc, g,
                                row_perm=None if pr is None else pr.cpu().numpy(),
                                col_perm=None if pc is None else pc.cpu().numpy(),
                                a=None if a is None else a.cpu().double().numpy())
    got = err.cpu().double().numpy()
    assert got.shape == ref.shape == ((R // br) * (C // bc), len(bits))
    assert np.all(np.abs(got - ref) <= REL * np.abs(ref)), np.max(np.abs(got - ref) / np.abs(ref))
    gref = (ref[:, :-1] - ref[:, 1:]) / (np.diff(bits)[None, :] * br * bc)
    tol = REL * (np.abs(ref[:, :-1]) + np.abs(ref[:, 1:])) / (np.diff(bits)[None, :] * br * bc)
    assert np.all(np.abs(gain.cpu().double().numpy() - gref) <= tol)
    e2, _ = ctx.block_scores_full(W, H, bits, br, bc, g, row_perm=pr, col_perm=pc, row_weight=a)
    ctx.sync()
    assert torch.equal(err, e2)                       # deterministic


def test_full_scores_with_a_diagonal_matrix_equal_the_diagonal_path(ctx):
    from tests.helpers import REL
    R, C, g, bits = 256, 384, 128, [2, 3, 4, 8]
    W = synth.make_weight(R, C, 61, DEV)
    c = torch.rand(C, device=DEV) + 0.25
    e_full, _ = ctx.block_scores_full(W, torch.diag(c).contiguous(), bits, 128, 128, g)
    e_diag, _ = ctx.block_scores(W, c, bits, 128, 128, g)
    ctx.sync()
    assert torch.allclose(e_full, e_diag, rtol=REL, atol=0)
