"""Algorithm 2 as the paper runs it (scores refreshed from the gradient at the current quantized
model, acceptance by the model's loss), driven through `dynamic.search_layer_dynamic` on a tiny
Llama-shaped layer with a synthetic quadratic model whose gradient is analytic:

    L(b) = 1/2 sum_m sum_ij d_ij (Q_b(W)_ij - W_ij)^2,    dL/dQ(W) = d (Q_b(W) - W)

The oracle follows the same loop on the host: every iteration's step is checked by hand-off (the
oracle's selection on the GPU's scores must move exactly the same blocks, its own fp64 scores
must agree with the GPU's), the channel permutations must be the oracle's sort of the GPU's
first-order statistics, and an independent oracle-side run of the whole loop must end on the
same allocation."""
import numpy as np
import pytest
import torch

from oracle import sbo
from paper_2602_17698_b200 import synth
from tests.helpers import REL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class QuadraticModel:
    """The stand-in for the network: fake-quantizes the permuted matrices block by block in fp64
    (asymmetric min-max round-to-nearest, groups along the input axis) and returns loss and
    gradient in the original layout.  Test scaffolding, not the checker."""

    def __init__(self, shape, W, d, bits, br, bc, g, coupling, names):
        self.shape, self.W, self.d, self.bits = shape, W, d, bits
        self.br, self.bc, self.g, self.cp, self.names = br, bc, g, coupling, names
        self.calls = {"grad": 0, "loss": 0}

    def _quantized(self, level, perms):
        out, s = {}, 0
        for nm in self.names:
            W = self.W[nm].double()
            R, C = W.shape
            rs, cs = self.cp.linears[nm]
            pr = perms[rs].long() if rs and perms.get(rs) is not None else torch.arange(R, device=W.device)
            pc = perms[cs].long() if cs and perms.get(cs) is not None else torch.arange(C, device=W.device)
            Wp = W[pr][:, pc]
            nbr, nbc = R // self.br, C // self.bc
            lv = level[s:s + nbr * nbc].long().reshape(nbr, nbc)
            b = torch.tensor(self.bits, device=W.device)[lv]                     # bits per block
            qmax = (2.0 ** b.double() - 1).repeat_interleave(self.br, 0).repeat_interleave(self.bc // self.g, 1)
            Wg = Wp.reshape(R, C // self.g, self.g)
            lo, hi = Wg.amin(2, keepdim=True), Wg.amax(2, keepdim=True)
            rng = hi - lo
            q = torch.round((Wg - lo) * (qmax[..., None] / rng.clamp_min(1e-300)))
            Wq = torch.where(rng > 0, lo + q * (rng / qmax[..., None]), lo.expand_as(Wg)).reshape(R, C)
            back = torch.empty_like(Wq)
            back[pr[:, None], pc[None, :]] = Wq
            out[nm] = back
            s += nbr * nbc
        return out

    def grad(self, level, perms):
        self.calls["grad"] += 1
        Q = self._quantized(level, perms)
        return {nm: (self.d[nm] * (Q[nm] - self.W[nm].double())).to(torch.bfloat16) for nm in self.names}

    def loss(self, level, perms):
        self.calls["loss"] += 1
        Q = self._quantized(level, perms)
        return float(sum(0.5 * (self.d[nm] * (Q[nm] - self.W[nm].double()) ** 2).sum() for nm in self.names))


def _setup(budget, bits, seed=0):
    from paper_2602_17698_b200.dynamic import COUPLING_TABLES
    from paper_2602_17698_b200.pipeline import SearchConfig
    shape = synth.LLAMA_TINY
    names = [l.name for l in shape.linears]
    W = synth.make_layer_weights(shape, seed, 0, DEV)
    gen = torch.Generator(device=DEV).manual_seed(17 + seed)
    d = {}
    for nm in names:
        R, C = W[nm].shape
        a = torch.exp(0.8 * torch.randn(R, device=DEV, generator=gen, dtype=torch.float64))
        c = torch.exp(0.8 * torch.randn(C, device=DEV, generator=gen, dtype=torch.float64))
        d[nm] = a[:, None] * c[None, :]
    cfg = SearchConfig(bits=bits, budget=budget, block_rows=64, block_cols=128, group=128, gamma0=0.1, gammaT=0.02)
    model = QuadraticModel(shape, W, d, list(bits), 64, 128, 128, COUPLING_TABLES["llama"], names)
    return shape, names, W, cfg, model


@pytest.mark.parametrize("budget,bits", [(3.25, (2, 3, 4, 8)),      # expansion steps, then rejected exchanges
                                         (3.0, (2, 3, 4))])          # budget active from the start: exchanges
def test_dynamic_loop_walks_the_oracle_trajectory(budget, bits):
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.dynamic import COUPLING_TABLES, search_layer_dynamic
    torch.cuda.set_device(0)
    shape, names, W, cfg, model = _setup(budget, bits)
    cp = COUPLING_TABLES["llama"]
    ctx = Context()
    Wh = {nm: W[nm].cpu() for nm in names}
    seen = []

    def observer(it, level, s_up, s_down, cand, rep, kept):
        lv, up, dn = level.cpu().numpy(), s_up.cpu().double().numpy(), s_down.cpu().double().numpy()
        # the step on the GPU's scores: exactly the oracle's selection
        st, ocand, orep = sbo.exchange_step(up, dn, lv, list(bits), budget, seen_k[0], uniform_block_elems=64 * 128)
        assert st == sbo.OK and np.array_equal(cand.cpu().numpy(), ocand), it
        for key in ("expansion", "moved", "n_up", "n_down", "used_out", "cap_bits"):
            assert rep[key] == orep[key], (it, key)
        seen.append((lv.copy(), kept, bool(rep["expansion"])))

    # the observer needs the batch size of the iteration: mirror the loop's k from its history
    seen_k = [max(1, int(cfg.gamma0 * 288))]

    def tracking_observer(*a):
        observer(*a)
        if not a[-1]:
            seen_k[0] //= 2

    res = search_layer_dynamic(ctx, shape, W, model.grad, model.loss, cfg, observer=tracking_observer)
    ctx.sync()
    assert res.n_blocks == 288 and res.iterations == len(seen) == len(res.history)
    if budget == 3.0:
        assert res.expansions == 0 and res.accepted > 0 and res.rejected > 0, res.history
    else:
        assert res.expansions > 0 and res.rejected > 0, res.history
    assert res.used_bits <= res.cap_bits == int(np.floor(budget * shape.n_weights))
    used = sum(64 * 128 * bits[l] for l in res.level.cpu().tolist())
    assert used == res.used_bits

    # permutations: the oracle's sort of ITS first-order statistics equals the library's permutation
    # wherever the scores are not tied; checked as "scores along the permutation do not increase"
    perms_none = {k: None for k in res.perms}
    G0 = model.grad(torch.full((288,), max(i for i, b in enumerate(bits) if b <= budget), dtype=torch.uint8,
                               device=DEV), perms_none)
    ref_b = max(b for b in bits if b <= budget)
    hid = np.zeros(shape.hidden)
    for nm in names:
        rs, cs = cp.linears[nm]
        ors, ocs = sbo.reorder_scores_first_order(Wh[nm], G0[nm].cpu(), ref_bits=ref_b, group=128)
        if rs == "hidden":
            hid += ors
        if cs == "hidden":
            hid += ocs
    p = res.perms["hidden"].cpu().numpy()
    assert sorted(p.tolist()) == list(range(shape.hidden))
    along = hid[p]
    assert np.all(along[:-1] >= along[1:] * (1 - 1e-4))
    # v / o coupling: the o permutation is the v permutation repeated for the query heads of a group
    pv, po = res.perms["v_heads"].cpu().numpy(), res.perms["o_heads"].cpu().numpy()
    assert np.array_equal(po, sbo.expand_segment_perm(pv, shape.n_heads // shape.n_kv_heads, shape.head_dim))

    # the oracle's own scores at three points of the trajectory agree with the GPU's
    perms_h = {k: (None if v is None else v.cpu().numpy()) for k, v in res.perms.items()}
    for idx in sorted({0, len(seen) // 2, len(seen) - 1}):
        lv = seen[idx][0]
        G = model.grad(torch.from_numpy(lv).to(DEV), res.perms)
        s = 0
        for nm in names:
            R, C = W[nm].shape
            nb = (R // 64) * (C // 128)
            rs, cs = cp.linears[nm]
            oup, odn, ol1 = sbo.first_order_scores(Wh[nm], G[nm].cpu(), list(bits), lv[s:s + nb], 64, 128, 128,
                                                   row_perm=perms_h[rs] if rs else None,
                                                   col_perm=perms_h[cs] if cs else None)
            gup, gdn, _ = ctx.first_order_scores(W[nm], G[nm], list(bits), torch.from_numpy(lv[s:s + nb]).to(DEV), 64,
                                                 128, 128, row_perm=res.perms[rs] if rs else None,
                                                 col_perm=res.perms[cs] if cs else None, want_l1=False)
            assert np.all(np.abs(gup.cpu().double().numpy() - oup) <= REL * ol1 + 1e-30)
            assert np.allclose(gdn.cpu().double().numpy(), odn, rtol=REL, atol=0)
            s += nb

    # an independent oracle-side run of the loop (fp64 scores, the same model and permutations)
    level = np.full(288, max(i for i, b in enumerate(bits) if b <= budget), dtype=np.uint8)
    k, kT = max(1, int(cfg.gamma0 * 288)), max(1, int(cfg.gammaT * 288))
    it = 0
    while k >= kT:
        it += 1
        lt = torch.from_numpy(level).to(DEV)
        G = model.grad(lt, res.perms)
        up, dn, s = np.zeros(288), np.zeros(288), 0
        for nm in names:
            R, C = W[nm].shape
            nb = (R // 64) * (C // 128)
            rs, cs = cp.linears[nm]
            up[s:s + nb], dn[s:s + nb], _ = sbo.first_order_scores(
                Wh[nm], G[nm].cpu(), list(bits), level[s:s + nb], 64, 128, 128,
                row_perm=perms_h[rs] if rs else None, col_perm=perms_h[cs] if cs else None)
            s += nb
        # the library's scores are fp32: the oracle ranks on the same precision
        up, dn = up.astype(np.float32).astype(np.float64), dn.astype(np.float32).astype(np.float64)
        st, cand, rep = sbo.exchange_step(up, dn, level, list(bits), budget, k, uniform_block_elems=64 * 128)
        assert st == sbo.OK
        if rep["moved"] and (rep["expansion"] or
                             model.loss(torch.from_numpy(cand).to(DEV), res.perms) < model.loss(lt, res.perms)):
            level = cand
        else:
            k //= 2
    same = float(np.mean(level == res.level.cpu().numpy()))
    assert it == res.iterations and same >= 0.98, (it, res.iterations, same)
    ctx.close()


def test_outside_tensors_follow_the_residual_stream_permutation():
    """Appendix D: the embedding and the language-model head are shuffled with the hidden
    dimension, norm weights too (coupling tables as data, three architectures)."""
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.dynamic import COUPLING_TABLES, permute_outside
    torch.cuda.set_device(0)
    ctx = Context()
    hidden, vocab = 512, 1000
    perm = torch.randperm(hidden, device=DEV).int()
    emb = synth.make_weight(vocab, hidden, 5, DEV)
    norm = torch.randn(hidden, device=DEV)
    for arch, has_head in (("llama", True), ("gemma2", False), ("mha", True)):
        cp = COUPLING_TABLES[arch]
        assert ("lm_head" in cp.outside) == has_head
        assert cp.linears["q_proj"][0] is None and cp.linears["k_proj"][0] is None     # q / k output order kept
        tensors = {"embed_tokens": emb, "final_norm": norm}
        if has_head:
            tensors["lm_head"] = emb
        out = permute_outside(ctx, cp, {"hidden": perm}, tensors)
        ctx.sync()
        assert torch.equal(out["embed_tokens"], emb[:, perm.long()])
        assert torch.equal(out["final_norm"], norm[perm.long()])
    assert set(COUPLING_TABLES["gemma2"].vectors) >= {"pre_feedforward_layernorm", "post_feedforward_layernorm"}
    ctx.close()
