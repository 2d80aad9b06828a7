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


def test_full_scores_with_a_diagonal_matrix_equal_the_diagonal_path(ctx):
    from tests.helpers import REL
    R, C, g, bits = 256, 384, 128, [2, 3, 4, 8]
    W = synth.make_weight(R, C, 61, DEV)
    c = torch.rand(C, device=DEV) + 0.25
    e_full, _ = ctx.block_scores_full(W, torch.diag(c).contiguous(), bits, 128, 128, g)
    e_diag, _ = ctx.block_scores(W, c, bits, 128, 128, g)
    ctx.sync()
    assert torch.allclose(e_full, e_diag, rtol=REL, atol=0)
