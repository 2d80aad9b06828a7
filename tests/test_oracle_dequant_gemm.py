"""Pins for the oracle's fused dequantisation + matrix product on the packed format
(Section 5.3, Table 4)."""
import numpy as np
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth

BITS = [2, 3, 4, 8]


def _case(R=256, Cc=384, T=5, br=128, bc=128, group=64, seed=3):
    W = synth.make_weight(R, Cc, 40 + seed)
    X = synth.make_activations(T, Cc, 50 + seed)
    rng = np.random.default_rng(seed)
    level = rng.integers(0, len(BITS), (R // br) * (Cc // bc)).astype(np.uint8)
    packed, off, meta = sbo.pack_blocks(W, BITS, level, br, bc, group)
    return W, X, level, packed, off, meta


def _fake_quant_matrix(W, level, br, bc, group):
    """Round-to-nearest fake quantisation of every block at its bitwidth, group by group through
    the oracle's (separately pinned) group quantiser: exact ties round as in the packed codes."""
    R, Cc = W.shape
    Wd = W.double().numpy()
    out = np.empty_like(Wd)
    nbc = Cc // bc
    for r in range(R):
        for g0 in range(0, Cc, group):
            b = BITS[level[(r // br) * nbc + g0 // bc]]
            out[r, g0:g0 + group] = sbo.quantize_group(Wd[r, g0:g0 + group], b)[1]
    return torch.from_numpy(out)


def test_equals_activations_times_the_fake_quantised_matrix():
    """Packing then dequantising is the round-to-nearest fake quantisation of every block at its
    bitwidth, so the product is X What^T (a library matrix product) with What from the group
    quantiser; the only difference is the fp32 rounding of the stored scale and minimum."""
    br, bc, group = 128, 128, 64
    W, X, level, packed, off, meta = _case(br=br, bc=bc, group=group)
    R, Cc = W.shape
    Y = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, BITS, br, bc, group)
    What = _fake_quant_matrix(W, level, br, bc, group)
    ref = (X.double() @ What.T).numpy()
    # two fp32 roundings per weight (minimum, scale), each at most 2^-24 of the largest weight or range
    bound = X.double().abs().sum(1, keepdim=True).numpy() * 3 * 2.0 ** -24 * float(W.double().abs().max())
    assert np.all(np.abs(Y - ref) <= bound), np.abs(Y - ref).max()


def test_bit_stream_is_read_as_written_on_a_tiny_case():
    """Decode the little-endian b-bit stream by hand (Python integers) for every block of a tiny
    matrix and form the product with plain loops."""
    br, bc, group = 4, 16, 16
    R, Cc, T = 8, 32, 3
    W = synth.make_weight(R, Cc, 77)
    X = synth.make_activations(T, Cc, 78)
    bits = [1, 3, 5, 8]
    level = np.array([0, 1, 2, 3], dtype=np.uint8)
    packed, off, meta = sbo.pack_blocks(W, bits, level, br, bc, group)
    Y = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, bits, br, bc, group)
    Xd = X.double().numpy()
    nbc = Cc // bc
    What = np.zeros((R, Cc))
    for blk in range(len(level)):
        b = bits[level[blk]]
        stream = 0
        words = packed[off[blk]:off[blk + 1]]
        for k, w in enumerate(words):
            stream |= int(w) << (32 * k)
        bi, bj = divmod(blk, nbc)
        for rr in range(br):
            for cc in range(bc):
                q = (stream >> ((rr * bc + cc) * b)) & ((1 << b) - 1)
                r, j = bi * br + rr, bj * bc + cc
                scale, lo = meta[r * (Cc // group) + j // group]
                What[r, j] = float(lo) + float(scale) * q
    ref = np.zeros((T, R))
    for t in range(T):
        for r in range(R):
            ref[t, r] = sum(Xd[t, j] * What[r, j] for j in range(Cc))
    assert np.allclose(Y, ref, rtol=1e-13, atol=1e-13)
    # and the decoded matrix is within half a grid step of W wherever the group is not constant
    Wd = W.double().numpy()
    for r in range(R):
        for j in range(Cc):
            scale = float(meta[r * (Cc // group) + j // group][0])
            assert abs(What[r, j] - Wd[r, j]) <= 0.5 * scale * (1 + 1e-6) + 1e-7 * abs(Wd[r, j])


def test_identity_activations_return_the_dequantised_rows():
    br, bc, group = 128, 128, 128
    W, _, level, packed, off, meta = _case(R=128, Cc=256, br=br, bc=bc, group=group, seed=5)
    R, Cc = W.shape
    X = torch.eye(Cc, dtype=torch.bfloat16)
    Y = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, BITS, br, bc, group)     # [Cc][R] = What^T
    What = _fake_quant_matrix(W, level, br, bc, group).numpy()
    # the stored minimum and scale are fp32: each is off by at most 2^-24 of values no larger than the
    # group's extreme weight (minimum) and range (scale times the code)
    assert np.all(np.abs(Y.T - What) <= 3 * 2.0 ** -24 * np.abs(W.double().numpy()).max())


def test_linear_in_the_activations_and_zero_for_zero():
    br, bc, group = 128, 128, 32
    W, X, level, packed, off, meta = _case(br=br, bc=bc, group=group, seed=9)
    R, Cc = W.shape
    X2 = synth.make_activations(X.shape[0], Cc, 99)
    # 2 X and X + X2 must stay bf16-exact for the test to be about linearity only
    Xa, Xb = (X.float() * 2).to(torch.bfloat16), X2
    Ya = sbo.dequant_gemm(Xa, packed, off, meta, level, R, Cc, BITS, br, bc, group)
    Y1 = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, BITS, br, bc, group)
    Yb = sbo.dequant_gemm(Xb, packed, off, meta, level, R, Cc, BITS, br, bc, group)
    assert np.allclose(Ya, 2 * Y1, rtol=1e-14, atol=0)
    Xs = torch.cat([X, Xb])                                   # rows are independent
    Ys = sbo.dequant_gemm(Xs, packed, off, meta, level, R, Cc, BITS, br, bc, group)
    assert np.array_equal(Ys[:X.shape[0]], Y1) and np.array_equal(Ys[X.shape[0]:], Yb)
    Z = sbo.dequant_gemm(torch.zeros_like(X), packed, off, meta, level, R, Cc, BITS, br, bc, group)
    assert np.all(Z == 0)


def test_eight_bits_everywhere_is_close_to_the_unquantised_product():
    """At 8 bits the reconstruction error per weight is at most half a step = range / 510."""
    br, bc, group = 128, 128, 128
    R, Cc, T = 128, 256, 4
    W = synth.make_weight(R, Cc, 11)
    X = synth.make_activations(T, Cc, 12)
    level = np.zeros((R // br) * (Cc // bc), dtype=np.uint8)
    packed, off, meta = sbo.pack_blocks(W, [8], level, br, bc, group)
    Y = sbo.dequant_gemm(X, packed, off, meta, level, R, Cc, [8], br, bc, group)
    Wd, Xd = W.double(), X.double()
    rng_ = (Wd.reshape(R, Cc // group, group).amax(-1) - Wd.reshape(R, Cc // group, group).amin(-1))
    half_step = (rng_ / 510).repeat_interleave(group, dim=1)          # [R][Cc]
    bound = (Xd.abs() @ half_step.T).numpy() * (1 + 1e-5) + 1e-9
    assert np.all(np.abs(Y - (Xd @ Wd.T).numpy()) <= bound)
