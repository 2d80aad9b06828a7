"""Pins for the oracle's packer: round trip, offsets, dequantisation error bound."""
import numpy as np
import pytest

from oracle import sbo
from paper_2602_17698_b200 import synth


def unpack_block(words: np.ndarray, n: int, b: int) -> np.ndarray:
    """Read n codes of b bits from a little-endian stream of 32-bit words (written here,
    bit by bit, independently of the packer)."""
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")
    return (bits[: n * b].reshape(n, b).astype(np.int64) << np.arange(b)).sum(1)


@pytest.mark.parametrize("br,bc,g", [(128, 128, 128), (64, 128, 64), (32, 32, 32), (256, 128, 128)])
def test_pack_round_trip_and_offsets(br, bc, g):
    R, Cc = 256, 256
    bits = [1, 2, 3, 4, 5, 6, 8]
    W = synth.make_weight(R, Cc, 31)
    rng = np.random.default_rng(2)
    nb = (R // br) * (Cc // bc)
    level = rng.integers(0, len(bits), size=nb).astype(np.uint8)
    pr = rng.permutation(R).astype(np.int32)
    pc = rng.permutation(Cc).astype(np.int32)
    packed, off, meta = sbo.pack_blocks(W, bits, level, br, bc, g, row_perm=pr, col_perm=pc)
    sizes = np.array([br * bc * bits[l] // 32 for l in level])
    assert off[0] == 0 and np.array_equal(np.diff(off), sizes)
    assert packed.size == off[-1] == sum(br * bc * bits[l] for l in level) // 32
    Wp = W.double().numpy()[pr][:, pc]
    nbc = Cc // bc
    for blk in range(nb):
        b = bits[level[blk]]
        bi, bj = divmod(blk, nbc)
        codes = unpack_block(packed[off[blk]:off[blk + 1]], br * bc, b).reshape(br, bc)
        tile = Wp[bi * br:(bi + 1) * br, bj * bc:(bj + 1) * bc]
        for rr in range(0, br, max(1, br // 4)):
            for g0 in range(0, bc, g):
                ref_codes, _, scale, lo = sbo.quantize_group(tile[rr, g0:g0 + g], b)
                assert np.array_equal(codes[rr, g0:g0 + g], ref_codes)
                gi = (bi * br + rr) * (Cc // g) + (bj * bc + g0) // g
                assert meta[gi, 0] == np.float32(scale) and meta[gi, 1] == np.float32(lo)
        # dequantised values are within half a step of the weights
        scale = meta[:, 0].reshape(R, Cc // g)[bi * br:(bi + 1) * br, bj * bc // g:(bj + 1) * bc // g]
        lo = meta[:, 1].reshape(R, Cc // g)[bi * br:(bi + 1) * br, bj * bc // g:(bj + 1) * bc // g]
        deq = np.repeat(lo, g, axis=1).astype(np.float64) + codes * np.repeat(scale, g, axis=1).astype(np.float64)
        # half a step, plus the fp32 rounding of the stored scale (times the code) and offset
        bound = (np.repeat(scale, g, axis=1) * (0.5 + 1.2e-7 * (2 ** b - 1))
                 + 1.2e-7 * np.abs(np.repeat(lo, g, axis=1)))
        assert np.all(np.abs(deq - tile) <= bound)
        assert codes.min() >= 0 and codes.max() <= 2 ** b - 1


def test_pack_used_bits_matches_allocation():
    R = Cc = 256
    bits = [2, 3, 4, 8]
    W = synth.make_weight(R, Cc, 32)
    X = synth.make_activations(256, Cc, 33)
    c = sbo.calib_moments(X, 1 / 256)
    err, _ = sbo.block_scores(W, c, bits, 64, 64, 64)
    st, level, rep = sbo.allocate_scalebits(err, bits, 2.75, 0.2, 0.1, uniform_block_elems=64 * 64)
    assert st == sbo.OK
    packed, off, _ = sbo.pack_blocks(W, bits, level, 64, 64, 64)
    assert off[-1] * 32 == rep["used_bits"]
