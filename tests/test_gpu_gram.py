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
