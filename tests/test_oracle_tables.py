"""Pins for the oracle's reorder statistics, permutations and block error table."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth


def _fake_quant(v: torch.Tensor, bits: int):
    """Independent route (divide by the step) used only to build expected values here."""
    lo = v.amin(-1, keepdim=True)
    hi = v.amax(-1, keepdim=True)
    step = (hi - lo) / (2 ** bits - 1)
    safe = torch.where(step > 0, step, torch.ones_like(step))
    q = torch.round((v - lo) / safe).clamp_(0, 2 ** bits - 1)
    return lo + q * step


def _setup(R=256, Cc=384, T=512, seed=0):
    W = synth.make_weight(R, Cc, synth.tensor_seed(seed, 0, 0))
    X = synth.make_activations(T, Cc, synth.tensor_seed(seed, 0, 16))
    c = sbo.calib_moments(X, 1.0 / T)
    return W, X, c


def test_block_error_is_activation_weighted_output_error():
    """With one active input channel per token X^T X is diagonal, and then
    E = (1/T) || X_J dW_{R,J}^T ||_F^2 exactly (the quantity the column factor stands for)."""
    R, Cc, T = 128, 256, 1024
    W = synth.make_weight(R, Cc, 21)
    rng = np.random.default_rng(0)
    X = torch.zeros(T, Cc, dtype=torch.bfloat16)
    X[torch.arange(T), torch.from_numpy(rng.integers(0, Cc, T))] = \
        torch.from_numpy(rng.normal(size=T)).to(torch.bfloat16)
    c = sbo.calib_moments(X, 1.0 / T)
    bits = [2, 3, 4]
    err, gain = sbo.block_scores(W, c, bits, 128, 128, 128)
    Wd, Xd = W.double(), X.double()
    for l, b in enumerate(bits):
        dW = Wd - _fake_quant(Wd.reshape(R, Cc // 128, 128), b).reshape(R, Cc)
        for bj in range(Cc // 128):
            J = slice(bj * 128, (bj + 1) * 128)
            ref = float(((Xd[:, J] @ dW[:, J].T) ** 2).sum() / T)
            assert err[bj, l] == pytest.approx(ref, rel=1e-9)
    M = 128 * 128
    assert np.allclose(gain[:, 0], (err[:, 0] - err[:, 1]) / M, rtol=1e-15)
    assert np.allclose(gain[:, 1], (err[:, 1] - err[:, 2]) / M, rtol=1e-15)


def test_gain_divides_by_bit_distance():
    W, X, c = _setup(128, 128)
    err, gain = sbo.block_scores(W, c, [2, 4, 8], 128, 128, 128)
    M = 128 * 128
    assert gain[0, 0] == pytest.approx((err[0, 0] - err[0, 1]) / (2 * M), rel=1e-15)
    assert gain[0, 1] == pytest.approx((err[0, 1] - err[0, 2]) / (4 * M), rel=1e-15)


def test_linearity_in_column_and_row_factors():
    W, X, c = _setup()
    R = W.shape[0]
    bits = [2, 3]
    e0, _ = sbo.block_scores(W, c, bits, 64, 128, 64)
    e1, _ = sbo.block_scores(W, 4.0 * c, bits, 64, 128, 64)
    assert np.array_equal(e1, 4.0 * e0)                       # power of two: exact
    a = np.full(R, 0.25)
    e2, _ = sbo.block_scores(W, c, bits, 64, 128, 64, a=a)
    assert np.array_equal(e2, 0.25 * e0)
    c_a, c_b = c.copy(), c.copy()
    c_a[::2] = 0.0
    c_b[1::2] = 0.0
    ea, _ = sbo.block_scores(W, c_a, bits, 64, 128, 64)
    eb, _ = sbo.block_scores(W, c_b, bits, 64, 128, 64)
    assert np.allclose(ea + eb, e0, rtol=1e-12)
    # a row factor that is zero outside block-row 1 leaves only that block-row
    a = np.zeros(R)
    a[64:128] = 1.0
    e3, _ = sbo.block_scores(W, c, bits, 64, 128, 64, a=a)
    nbc = W.shape[1] // 128
    assert np.allclose(e3[nbc:2 * nbc], e0[nbc:2 * nbc], rtol=1e-12)
    assert np.all(e3[:nbc] == 0) and np.all(e3[2 * nbc:] == 0)


def test_reorder_scores_against_direct_sums_and_block_table():
    W, X, c = _setup()
    R, Cc = W.shape
    rs, cs = sbo.reorder_scores(W, c, ref_bits=3, group=128)
    Wd = W.double()
    dW2 = (Wd - _fake_quant(Wd.reshape(R, Cc // 128, 128), 3).reshape(R, Cc)) ** 2
    sig = dW2 * torch.from_numpy(c)[None, :]
    assert np.allclose(rs, sig.sum(1).numpy(), rtol=1e-9)
    assert np.allclose(cs, sig.sum(0).numpy(), rtol=1e-9)
    # identity permutations: the table at ref_bits sums to the same total
    err, _ = sbo.block_scores(W, c, [3], 128, 128, 128)
    assert err.sum() == pytest.approx(rs.sum(), rel=1e-12)
    assert err.sum() == pytest.approx(cs.sum(), rel=1e-12)
    # accumulation over coupled matrices adds
    rs2, cs2 = sbo.reorder_scores(W, c, ref_bits=3, group=128, row_score=rs.copy(),
                                  col_score=cs.copy(), accumulate=True)
    assert np.allclose(rs2, 2 * rs, rtol=1e-15) and np.allclose(cs2, 2 * cs, rtol=1e-15)


def test_argsort_is_stable_descending_permutation():
    rng = np.random.default_rng(1)
    s = rng.integers(0, 6, size=512).astype(np.float64)       # many ties
    p = sbo.argsort_desc_segments(s)
    assert sorted(p.tolist()) == list(range(512))
    assert np.all(np.diff(s[p]) <= 0)
    same = np.diff(s[p]) == 0
    assert np.all(np.diff(p)[same] > 0)                        # ties keep the lower index first
    assert np.array_equal(p, np.argsort(-s, kind="stable"))
    # segments sort independently and stay inside their segment
    ps = sbo.argsort_desc_segments(s, 128)
    for h in range(4):
        seg = ps[h * 128:(h + 1) * 128]
        assert sorted(seg.tolist()) == list(range(h * 128, (h + 1) * 128))
        assert np.array_equal(seg, h * 128 + np.argsort(-s[h * 128:(h + 1) * 128], kind="stable"))


def test_planted_hot_channels_come_first():
    """Sensitive rows and columns move to the top-left (Section 4.1)."""
    R, Cc, T = 256, 256, 256
    W = synth.make_weight(R, Cc, 3, outliers=False)
    c = np.ones(Cc)
    hot_cols = [200, 17, 90]
    c[hot_cols] = [400.0, 300.0, 200.0]
    a = np.ones(R)
    hot_rows = [255, 3]
    a[hot_rows] = [500.0, 250.0]
    rs, _ = sbo.reorder_scores(W, c, a=a, ref_bits=2, group=128)
    _, cs = sbo.reorder_scores(W, c, ref_bits=2, group=128)
    pr = sbo.argsort_desc_segments(rs)
    pc = sbo.argsort_desc_segments(cs)
    assert pr[:2].tolist() == hot_rows
    assert pc[:3].tolist() == hot_cols


def test_block_error_invariances_under_permutation():
    W, X, c = _setup(256, 256)
    R, Cc = W.shape
    bits = [2, 4]
    rng = np.random.default_rng(5)
    e0, _ = sbo.block_scores(W, c, bits, 128, 128, 64)
    # rows shuffled inside each block-row, columns inside each 64-group: same table
    pr = np.concatenate([rng.permutation(128) + 128 * i for i in range(R // 128)]).astype(np.int32)
    pc = np.concatenate([rng.permutation(64) + 64 * i for i in range(Cc // 64)]).astype(np.int32)
    e1, _ = sbo.block_scores(W, c, bits, 128, 128, 64, row_perm=pr, col_perm=pc)
    assert np.allclose(e1, e0, rtol=1e-12)
    # an arbitrary row permutation keeps every group intact: the column-block totals stay
    pr = rng.permutation(R).astype(np.int32)
    e2, _ = sbo.block_scores(W, c, bits, 128, 128, 64, row_perm=pr)
    nbc = Cc // 128
    assert np.allclose(e2.reshape(-1, nbc, 2).sum(0), e0.reshape(-1, nbc, 2).sum(0), rtol=1e-12)
    # explicit permuted copy + identity == permutation arguments
    pc = rng.permutation(Cc).astype(np.int32)
    Wp = W[torch.from_numpy(pr).long()][:, torch.from_numpy(pc).long()].contiguous()
    e3, _ = sbo.block_scores(W, c, bits, 128, 128, 64, row_perm=pr, col_perm=pc)
    e4, _ = sbo.block_scores(Wp, c[pc], bits, 128, 128, 64)
    assert np.array_equal(e3, e4)


def test_fold_and_expand_for_grouped_query_heads():
    seg, kv, reps = 4, 3, 2
    dst = np.zeros(kv * seg)
    src = np.arange(kv * reps * seg, dtype=np.float64)
    sbo.fold_segment_scores(dst, src, reps, seg)
    assert np.array_equal(dst, src.reshape(kv, reps, seg).sum(1).ravel())
    perm = np.array([3, 1, 0, 2, 4, 7, 6, 5, 9, 8, 11, 10], dtype=np.int32)
    out = sbo.expand_segment_perm(perm, reps, seg)
    for h in range(kv):
        local = perm[h * seg:(h + 1) * seg] - h * seg
        for u in range(reps):
            q = h * reps + u
            assert np.array_equal(out[q * seg:(q + 1) * seg], q * seg + local)


def test_outlier_free_tables_are_monotone_and_convex():
    """Monotone, diminishing-returns tables (Appendix B) hold on outlier-free data."""
    W = synth.make_weight(256, 256, 9, outliers=False)
    c = np.ones(256)
    bits = [2, 3, 4, 5, 6]
    err, gain = sbo.block_scores(W, c, bits, 128, 128, 128)
    assert np.all(np.diff(err, axis=1) < 0)
    assert np.all(np.diff(gain, axis=1) < 0)


def test_block_counts_quoted_by_the_paper():
    rows = {}
    with open(__file__.rsplit("/", 1)[0] + "/golden/paper_counts.txt") as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val, tol, _ = line.split(None, 3)
            rows[name] = (float(val), float(tol))
    v, tol = rows["gemma2_9b_blocks_64x64"]
    assert abs(rows["gemma2_9b_weights"][0] / rows["gemma2_9b_block_elems"][0] / v - 1) <= tol
    # Llama-3-8B linear weights at 64 x 128 blocks, times the 3-4 one-bit steps from zero bits
    n_blocks = 32 * synth.LLAMA3_8B.n_weights / (64 * 128)
    v, tol = rows["llama3_8b_classic_greedy_iterations"]
    assert abs(n_blocks * 3.5 / v - 1) <= tol
    assert synth.LLAMA3_8B.n_weights == 218_103_808


def test_gram_matrix_pins():
    """Diagonal = the pinned second moments; symmetric; positive semi-definite; equal to a
    float64 matrix product; closed form for one-hot rows."""
    import torch
    X = synth.make_activations(300, 40, 5)
    H = sbo.calib_gram(X)
    assert np.array_equal(H, H.T)
    assert np.allclose(np.diag(H), sbo.calib_moments(X, 1.0 / 300), rtol=1e-13)
    Xd = X.double().numpy()
    assert np.allclose(H, Xd.T @ Xd / 300, rtol=1e-12, atol=1e-14)
    assert np.linalg.eigvalsh(H).min() >= -1e-9 * np.abs(H).max()
    # one-hot rows: H = diag(counts) * value^2 / T
    idx = np.arange(64) % 8
    onehot = torch.zeros(64, 8)
    onehot[np.arange(64), idx] = 3.0
    Ho = sbo.calib_gram(onehot.to(torch.bfloat16))
    assert np.allclose(Ho, np.eye(8) * 9.0 * 8 / 64, rtol=0, atol=1e-15)


def test_full_second_moment_block_scores_pins():
    """Diagonal H reduces to the pinned block table; H = u u^T gives sum_r (d_r . u)^2; a
    positive semi-definite H gives non-negative errors; permutations equal an explicitly
    permuted problem."""
    import torch
    R, C, br, bc, g = 64, 128, 32, 64, 32
    bits = [2, 3, 4]
    W = synth.make_weight(R, C, 21)
    rng = np.random.default_rng(2)
    c = rng.uniform(0.1, 2.0, size=C)
    e_diag = sbo.block_scores_full(W, np.diag(c), bits, br, bc, g)
    e_ref, _ = sbo.block_scores(W, c, bits, br, bc, g)
    assert np.allclose(e_diag, e_ref, rtol=1e-12)
    # rank one: E = sum over rows of (d_r . u_J)^2, through the pinned group quantizer
    u = rng.normal(size=C)
    e_rank1 = sbo.block_scores_full(W, np.outer(u, u), bits, br, bc, g)
    Wd = W.double().numpy()
    for l, b in enumerate(bits):
        D = np.empty_like(Wd)
        for r in range(R):
            for c0 in range(0, C, g):
                _, vh, _, _ = sbo.quantize_group(Wd[r, c0:c0 + g], b)
                D[r, c0:c0 + g] = Wd[r, c0:c0 + g] - vh
        for blk in range((R // br) * (C // bc)):
            bi, bj = divmod(blk, C // bc)
            proj = D[bi * br:(bi + 1) * br, bj * bc:(bj + 1) * bc] @ u[bj * bc:(bj + 1) * bc]
            assert e_rank1[blk, l] == pytest.approx((proj ** 2).sum(), rel=1e-11)
    # a Gram matrix is positive semi-definite: errors are non-negative and fall with the bits
    X = synth.make_activations(256, C, 5)
    H = sbo.calib_gram(X)
    e_full = sbo.block_scores_full(W, H, bits, br, bc, g)
    assert np.all(e_full >= 0)
    # permutations
    pr, pc = rng.permutation(R).astype(np.int32), rng.permutation(C).astype(np.int32)
    e_perm = sbo.block_scores_full(W, H, bits, br, bc, g, row_perm=pr, col_perm=pc)
    Wp = W[torch.from_numpy(pr).long()][:, torch.from_numpy(pc).long()].contiguous()
    Hp = H[np.ix_(pc, pc)]
    assert np.allclose(e_perm, sbo.block_scores_full(Wp, Hp, bits, br, bc, g), rtol=1e-12)
    # row weights a_r (the row factor of Section 3.2), indexed by ORIGINAL row: with a diagonal H the
    # weighted form is the pinned weighted block table; with the rank-one H it is sum_r a_r (d_r . u)^2
    # (rows of a block-row written out here); it is linear in a
    a = rng.uniform(0.2, 3.0, size=R)
    e_wd = sbo.block_scores_full(W, np.diag(c), bits, br, bc, g, a=a)
    e_wref, _ = sbo.block_scores(W, c, bits, br, bc, g, a=a)
    assert np.allclose(e_wd, e_wref, rtol=1e-12)
    e_w1 = sbo.block_scores_full(W, np.outer(u, u), bits, br, bc, g, a=a)
    for l, b in enumerate(bits):
        D = np.empty_like(Wd)
        for r in range(R):
            for c0 in range(0, C, g):
                _, vh, _, _ = sbo.quantize_group(Wd[r, c0:c0 + g], b)
                D[r, c0:c0 + g] = Wd[r, c0:c0 + g] - vh
        for blk in range((R // br) * (C // bc)):
            bi, bj = divmod(blk, C // bc)
            proj = D[bi * br:(bi + 1) * br, bj * bc:(bj + 1) * bc] @ u[bj * bc:(bj + 1) * bc]
            assert e_w1[blk, l] == pytest.approx((a[bi * br:(bi + 1) * br] * proj ** 2).sum(), rel=1e-11)
    assert np.allclose(sbo.block_scores_full(W, H, bits, br, bc, g, a=2.5 * a),
                       2.5 * sbo.block_scores_full(W, H, bits, br, bc, g, a=a), rtol=1e-12)
    # with a row permutation the weight follows the ORIGINAL row
    e_wp = sbo.block_scores_full(W, H, bits, br, bc, g, row_perm=pr, col_perm=pc, a=a)
    assert np.allclose(e_wp, sbo.block_scores_full(Wp, Hp, bits, br, bc, g, a=a[pr]), rtol=1e-12)
