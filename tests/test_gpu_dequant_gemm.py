"""Fused dequantisation + matrix product on the packed format (Section 5.3, Table 4) against
the fp64 oracle.  The packed input comes from the ORACLE's pack (the CUDA pack is checked
bit for bit against it elsewhere), so this file tests the product alone."""
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


def _tolerance(X, meta, level, bits, R, Cc, br=128):
    """The kernel contracts the integer codes exactly (bf16 x bf16 products are exact in fp32) and
    rounds only in fp32 sums: the tensor cores' accumulation over a block, scale * acc + lo * colsum
    per block, and the sum over blocks.  Each is within a few 2^-24 of the magnitudes it adds, which
    are bounded by sum_j (sum_{c in j} |x_c|) (|lo_rj| + scale_rj qmax_j): 2e-6 of that bound."""
    nbc = Cc // 128
    qmax = np.array([2 ** bits[l] - 1 for l in level], dtype=np.float64).reshape(R // br, nbc)
    qmax = np.repeat(qmax, br, axis=0)                                    # [R][nbc]
    m = meta.reshape(R, nbc, 2).astype(np.float64)
    bound_w = np.abs(m[:, :, 1]) + m[:, :, 0] * qmax                      # [R][nbc]
    xabs = X.double().abs().reshape(X.shape[0], nbc, 128).sum(-1).numpy() # [T][nbc]
    return 2e-6 * xabs @ bound_w.T + 1e-30


def _run(ctx, R, Cc, T, bits, seed, ldx=None, ldy=None, br=128):
    W = synth.make_weight(R, Cc, 300 + seed)
    X = synth.make_activations(T, Cc, 400 + seed)
    rng = np.random.default_rng(seed)
    level = rng.integers(0, len(bits), (R // br) * (Cc // 128)).astype(np.uint8)
    packed, off, meta = sbo.pack_blocks(W, bits, level, br, 128, 128)
    ref = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, bits, br, 128, 128)
    Xg = X.to(DEV)
    if ldx:
        buf = torch.zeros(T, ldx, dtype=torch.bfloat16, device=DEV)
        buf[:, :Cc] = Xg
        Xg = buf[:, :Cc]
    Y = None
    if ldy:
        Y = torch.full((T, ldy), float("nan"), dtype=torch.float32, device=DEV)[:, :R]
    out = ctx.dequant_gemm(Xg, torch.from_numpy(packed.view(np.int32)).to(DEV), torch.from_numpy(off).to(DEV),
                           torch.from_numpy(meta).to(DEV), torch.from_numpy(level).to(DEV), R, Cc, bits,
                           block_rows=br, Y=Y)
    ctx.sync()
    got = out.cpu().double().numpy()
    tol = _tolerance(X, meta, level, bits, R, Cc, br)
    err = np.abs(got - ref)
    assert np.all(err <= tol), (float((err / tol).max()), np.unravel_index((err / tol).argmax(), err.shape))
    return got, ref


@pytest.mark.parametrize("R,Cc,T", [(128, 128, 16), (256, 384, 16), (256, 384, 32), (384, 1024, 32),
                                    (1024, 2048, 16)])
def test_table_4_mix_of_2_4_8_bits(ctx, R, Cc, T):
    _run(ctx, R, Cc, T, [2, 4, 8], seed=R + Cc + T)


@pytest.mark.parametrize("T", [1, 5, 8, 9, 17, 40, 64])
def test_any_number_of_tokens(ctx, T):
    """Padding to 8, 16 or 32 tokens, and slices of 32."""
    _run(ctx, 256, 512, T, [2, 4, 8], seed=T)


@pytest.mark.parametrize("R,Cc,T,bits", [(64, 128, 16, [4]), (192, 384, 32, [2, 4, 8]), (448, 1024, 7, [2, 4, 8]),
                                         (1024, 2048, 32, [1, 2, 3, 4, 5, 6, 7, 8])])
def test_blocks_of_64_rows(ctx, R, Cc, T, bits):
    """The paper's own partition (Section 5 "Implementation": 64 x 128 blocks, group 128)."""
    _run(ctx, R, Cc, T, bits, seed=R + T, br=64)


def test_every_bitwidth(ctx):
    """1, 2, 4 through the mask-per-pair unpacking, 8 as two nibbles, 3, 5, 6, 7 cut out code by code."""
    _run(ctx, 512, 1024, 16, [1, 2, 3, 4, 5, 6, 7, 8], seed=11)
    for b in range(1, 9):
        _run(ctx, 128, 256, 16, [b], seed=20 + b)


def test_strided_input_and_output(ctx):
    _run(ctx, 256, 256, 16, [2, 4, 8], seed=5, ldx=256 + 64, ldy=256 + 8)


def test_many_column_segments_and_a_ragged_last_one(ctx):
    """Few row tiles: the columns are cut into many segments (one with fewer blocks) whose
    partial sums are added in order."""
    _run(ctx, 128, 128 * 37, 32, [2, 4, 8], seed=7)
    _run(ctx, 128, 128 * 70, 16, [4], seed=8)


@pytest.mark.parametrize("R,Cc,T,br", [(4096, 1024, 32, 128),      # 32 row tiles x 8 segments of one block: clusters of 8
                                        (8192, 1024, 16, 64),       # 128 row tiles of 64 rows x 4 segments
                                        (2048, 2560, 8, 128)])      # 16 x 18 CTAs: 20 blocks in segments of 2, partial sums
def test_segments_added_inside_a_cluster_and_by_the_second_kernel(ctx, R, Cc, T, br):
    """With 2 to 8 column segments the segments of a row tile are one cluster and are added through
    shared memory; with more they go through partial sums and a second kernel."""
    _run(ctx, R, Cc, T, [2, 4, 8], seed=R + Cc + br, br=br)


def test_deterministic(ctx):
    a, _ = _run(ctx, 256, 1024, 32, [2, 4, 8], seed=3)
    b, _ = _run(ctx, 256, 1024, 32, [2, 4, 8], seed=3)
    assert np.array_equal(a, b)


def test_rejects_other_block_shapes(ctx):
    from paper_2602_17698_b200.binding import SbError
    X = torch.zeros(16, 256, dtype=torch.bfloat16, device=DEV)
    z32 = torch.zeros(1024, dtype=torch.int32, device=DEV)
    off = torch.zeros(9, dtype=torch.int64, device=DEV)
    meta = torch.zeros((256 * 256 // 64, 2), dtype=torch.float32, device=DEV)
    lvl = torch.zeros(8, dtype=torch.uint8, device=DEV)
    with pytest.raises(SbError):
        ctx.dequant_gemm(X, z32, off, meta, lvl, 256, 256, [4], 64, 128, 64)


def test_table_4_size(ctx):
    """8192 x 8192 at 40 / 40 / 20 % of 2 / 4 / 8 bits (4 bits on average), 32 tokens: every
    output against the oracle."""
    R = Cc = 8192
    T = 32
    bits = [2, 4, 8]
    W = synth.make_weight(R, Cc, 900)
    X = synth.make_activations(T, Cc, 901)
    level = synth.table4_levels((R // 128) * (Cc // 128), 902)
    packed, off, meta = sbo.pack_blocks(W, bits, level, 128, 128, 128)
    ref = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, bits, 128, 128, 128)
    out = ctx.dequant_gemm(X.to(DEV), torch.from_numpy(packed.view(np.int32)).to(DEV), torch.from_numpy(off).to(DEV),
                           torch.from_numpy(meta).to(DEV), torch.from_numpy(level).to(DEV), R, Cc, bits)
    ctx.sync()
    err = np.abs(out.cpu().double().numpy() - ref)
    tol = _tolerance(X, meta, level, bits, R, Cc)
    assert np.all(err <= tol), float((err / tol).max())
