"""Pins for the oracle's decode, quantizer and calibration moments.

None of these re-type the oracle's formula: each checks a fact that the paper or
the mathematics fixes (error bound of a uniform grid, on-grid inputs, textbook
limits, an independent formulation through the step size instead of its
reciprocal).
"""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth


def test_bf16_decode_exhaustive():
    """All 65,536 bit patterns against torch's own bf16 -> fp64 conversion."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    vec = sbo.bf16_array_to_f64(bits)
    finite = np.isfinite(ref)
    assert np.array_equal(vec[finite], ref[finite])
    assert np.array_equal(np.isnan(vec), np.isnan(ref))
    for h in list(range(0, 65536, 97)) + [0, 1, 0x7F7F, 0x8000, 0xFF7F, 0x3F80, 0xBF80]:
        r = ref[h]
        o = sbo.bf16_to_f64(h)
        assert (np.isnan(r) and np.isnan(o)) or r == o


def _bf16_rand(n, seed, outliers=True):
    w = synth.make_weight(1, n, seed, outliers=outliers)
    return w.double().numpy().ravel()


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 6, 8])
def test_error_bound_and_range_ends(bits):
    """|v - vhat| <= scale/2; the group's min and max sit on the grid (codes 0, qmax)."""
    qmax = 2 ** bits - 1
    for seed in range(8):
        v = _bf16_rand(128, 100 + seed)
        code, vhat, scale, lo = sbo.quantize_group(v, bits)
        assert lo == v.min()
        assert scale == (v.max() - v.min()) / qmax
        assert np.all(np.abs(v - vhat) <= scale / 2 * (1 + 1e-12))
        assert code.min() == 0 and code.max() == qmax
        assert code[np.argmin(v)] == 0 and code[np.argmax(v)] == qmax
        assert abs(vhat[np.argmin(v)] - v.min()) == 0.0
        assert abs(vhat[np.argmax(v)] - v.max()) <= 1e-15 * abs(v.max())
        # codes are monotone in the value
        order = np.argsort(v, kind="stable")
        assert np.all(np.diff(code[order]) >= 0)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_on_grid_input_has_zero_error(bits):
    """v = lo + q * s with s a power of two and both range ends present: exact."""
    rng = np.random.default_rng(bits)
    qmax = 2 ** bits - 1
    for s in (2.0 ** -7, 2.0 ** -3, 1.0):
        q = rng.integers(0, qmax + 1, size=128)
        q[0], q[1] = 0, qmax
        lo = -3.0 * s * qmax
        v = lo + q * s
        code, vhat, scale, lo_o = sbo.quantize_group(v, bits)
        assert np.array_equal(code, q)
        assert np.array_equal(vhat, v)
        assert scale == s and lo_o == lo


def test_constant_group_and_full_8bit_grid():
    code, vhat, scale, lo = sbo.quantize_group(np.full(128, 0.375), 3)
    assert scale == 0.0 and lo == 0.375 and np.all(code == 0) and np.all(vhat == 0.375)
    v = np.arange(256, dtype=np.float64) * 0.5 - 17.0     # 256 evenly spaced values, 8 bits
    code, vhat, scale, lo = sbo.quantize_group(v, 8)
    assert np.array_equal(code, np.arange(256)) and np.array_equal(vhat, v)


def test_ties_round_half_to_even():
    """Range [0, 3] at 2 bits has step 1: the mid-points .5, 1.5, 2.5 go to 0, 2, 2."""
    v = np.array([0.0, 3.0, 0.5, 1.5, 2.5, 1.0, 2.0, 0.25])
    code, vhat, scale, lo = sbo.quantize_group(v, 2)
    assert list(code) == [0, 3, 0, 2, 2, 1, 2, 0]
    assert scale == 1.0


def test_power_of_two_equivariance():
    """E(2^k W) = 4^k E(W) bit for bit (scaling by a power of two is exact)."""
    v = _bf16_rand(128, 7)
    for bits in (2, 3, 4):
        c0, vh0, s0, l0 = sbo.quantize_group(v, bits)
        for k in (-5, 3):
            c1, vh1, s1, l1 = sbo.quantize_group(v * 2.0 ** k, bits)
            assert np.array_equal(c0, c1)
            assert np.array_equal(vh1, vh0 * 2.0 ** k)
            assert s1 == s0 * 2.0 ** k


def test_uniform_noise_limit():
    """Outlier-free data: mean squared error -> scale^2 / 12 and
    E(b)/E(b+1) -> ((2^(b+1)-1)/(2^b-1))^2 for b >= 2 (uniform-quantiser theory)."""
    groups = [_bf16_rand(128, 1000 + s, outliers=False) for s in range(400)]
    mse = {}
    for bits in (2, 3, 4, 5):
        num, den = 0.0, 0.0
        for v in groups:
            _, vhat, scale, _ = sbo.quantize_group(v, bits)
            num += np.sum((v - vhat) ** 2)
            den += 128 * scale ** 2 / 12.0
        mse[bits] = num
        if bits >= 4:
            assert abs(num / den - 1.0) < 0.05, (bits, num / den)
    for b in (3, 4):
        expect = ((2 ** (b + 1) - 1) / (2 ** b - 1)) ** 2
        assert abs(mse[b] / mse[b + 1] / expect - 1.0) < 0.05


def _independent_fake_quant(v: torch.Tensor, bits: int):
    """A different route to the same grid: divide by the step, torch.round (half-even)."""
    lo = v.amin(-1, keepdim=True)
    hi = v.amax(-1, keepdim=True)
    qmax = 2 ** bits - 1
    step = (hi - lo) / qmax
    t = torch.where(step > 0, (v - lo) / torch.where(step > 0, step, torch.ones_like(step)),
                    torch.zeros_like(v))
    q = torch.round(t).clamp_(0, qmax)
    return lo + q * step, q, t


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_against_independent_formulation(bits):
    w = synth.make_weight(64, 512, 5).double()
    g = w.reshape(-1, 128)
    vh_ref, q_ref, t = _independent_fake_quant(g, bits)
    frac = (t - torch.floor(t) - 0.5).abs()
    n_checked = 0
    for r in range(g.shape[0]):
        code, vhat, _, _ = sbo.quantize_group(g[r].numpy(), bits)
        not_tie = (frac[r] > 1e-9).numpy()
        assert np.array_equal(code[not_tie], q_ref[r].numpy().astype(np.int32)[not_tie])
        # squared errors agree everywhere (the error is continuous across a tie)
        e0 = (g[r].numpy() - vhat) ** 2
        e1 = ((g[r] - vh_ref[r]) ** 2).numpy()
        assert np.allclose(e0, e1, rtol=1e-9, atol=1e-22)
        n_checked += int(not_tie.sum())
    assert n_checked > 0.99 * g.numel()


# ---- calibration moments -------------------------------------------------------

def test_moments_closed_forms():
    T, K = 64, 24
    ones = torch.ones(T, K, dtype=torch.bfloat16)
    assert np.array_equal(sbo.calib_moments(ones, 1.0 / T), np.ones(K))
    # one-hot rows: channel j is 1 on count[j] tokens
    x = torch.zeros(T, K, dtype=torch.bfloat16)
    hot = torch.arange(T) % 5
    x[torch.arange(T), hot] = 1.0
    c = sbo.calib_moments(x, 1.0 / T)
    cnt = np.bincount(hot.numpy(), minlength=K)
    assert np.allclose(c, cnt / T, rtol=0, atol=1e-15)


def test_moments_against_numpy_and_accumulate():
    x = synth.make_activations(512, 96, 3)
    xd = x.double().numpy()
    c = sbo.calib_moments(x, 1.0 / 512)
    assert np.allclose(c, (xd ** 2).mean(0), rtol=1e-12)
    # two chunks accumulate to the same sums
    out = sbo.calib_moments(x[:200], 1.0)
    out = sbo.calib_moments(x[200:], 1.0, out=out)
    assert np.allclose(out, (xd ** 2).sum(0), rtol=1e-12)


def test_moments_recover_channel_std():
    T, K, seed = 8192, 64, 11
    x = synth.make_activations(T, K, seed)
    s = synth.expected_channel_std(K, seed).double().numpy()
    c = sbo.calib_moments(x, 1.0 / T)
    # chi-square spread 3*sqrt(2/T) plus bf16 rounding of x (rel 2^-9 per element, averaged)
    assert np.all(np.abs(c / s ** 2 - 1.0) < 3 * np.sqrt(2.0 / T) + 4e-3)
