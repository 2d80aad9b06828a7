"""Algorithm 2 as the paper runs it: the dynamic search loop around a caller's model.

The static path (`pipeline.search_layer`) scores every candidate once and allocates on the
table.  The paper's own loop refreshes the sensitivities in every iteration from the gradient at
the CURRENT quantized model (Algorithm 2, lines 4-5; Appendix E.1) and asks the model for the
loss of the proposed allocation (line 11).  This module sequences that loop on the library's
kernels; the model stays with the caller, behind two callbacks:

    grad_fn(level, perms)  -> {matrix name: bf16 gradient dL/dW (original layout) at the model
                              quantized with `level`}, on a freshly drawn mini-batch
    loss_fn(level, perms)  -> float, the loss of the model quantized with `level` on that mini-batch

`level` is the uint8 device vector over all blocks, matrices in `names` order, blocks of a matrix
row-major over the grid of its PERMUTED layout; `perms` maps the coupled channel sets to their
permutations (perm[new] = old; all None in the very first call, which quantizes the original
layout: the one-time reordering is computed from that gradient).  Every number the search uses comes from the
library (`sb_reorder_channels_first_order`, `sb_first_order_scores`, `sb_exchange_step`); this
file only keeps the books: which matrices share a channel permutation (the coupling tables below,
Appendix D) and where a matrix's blocks start.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import torch

from .binding import Context


# ---- coupling tables (Appendix D) as data ---------------------------------------------------------
@dataclass(frozen=True)
class Coupling:
    """Which axes of which tensors move together.

    linears: matrix name -> (row set, column set), a set name or None (axis kept).
    sets: set name -> (size attribute, segment attribute or None for "the whole axis").
          A segmented set is sorted inside each segment (attention heads).
    expand: set name -> (source set, repetitions attribute): the set is not sorted itself, its
          permutation is the source's, repeated for every member of a group (the query heads
          that read one key/value head under grouped-query attention); its scores are folded
          into the source's before the sort.
    vectors: per-channel vectors (norm weights, biases) that move with a set.
    outside: matrices outside the decoder layers that are moved, not scored: name -> (row set,
          column set).  The residual-stream permutation shuffles the columns of the embedding and
          of the language-model head.
    """
    linears: Dict[str, Tuple[Optional[str], Optional[str]]]
    sets: Dict[str, Tuple[str, Optional[str]]]
    expand: Dict[str, Tuple[str, str]]
    vectors: Dict[str, str] = field(default_factory=dict)
    outside: Dict[str, Tuple[Optional[str], Optional[str]]] = field(default_factory=dict)


_LINEARS = {
    # the output order of q and k is kept (rotary embedding, and q/k norms where a model has them)
    "q_proj": (None, "hidden"), "k_proj": (None, "hidden"), "v_proj": ("v_heads", "hidden"),
    "o_proj": ("hidden", "o_heads"), "gate_proj": ("intermediate", "hidden"),
    "up_proj": ("intermediate", "hidden"), "down_proj": ("hidden", "intermediate"),
}
_SETS = {"hidden": ("hidden", None), "intermediate": ("intermediate", None), "v_heads": ("kv_dim", "head_dim")}

COUPLING_TABLES: Dict[str, Coupling] = {
    # Llama 2 / 3: grouped-query attention, two norms per layer, separate language-model head
    "llama": Coupling(
        linears=_LINEARS, sets=_SETS, expand={"o_heads": ("v_heads", "q_per_kv")},
        vectors={"input_layernorm": "hidden", "post_attention_layernorm": "hidden", "final_norm": "hidden"},
        outside={"embed_tokens": (None, "hidden"), "lm_head": (None, "hidden")}),
    # Gemma 2: the same projections, four norms per layer (before and after attention and MLP), the
    # language-model head is the embedding itself (tied), so only one outside matrix moves
    "gemma2": Coupling(
        linears=_LINEARS, sets=_SETS, expand={"o_heads": ("v_heads", "q_per_kv")},
        vectors={"input_layernorm": "hidden", "post_attention_layernorm": "hidden",
                 "pre_feedforward_layernorm": "hidden", "post_feedforward_layernorm": "hidden",
                 "final_norm": "hidden"},
        outside={"embed_tokens": (None, "hidden")}),
    # plain multi-head attention (every query head has its own value head): same table, the
    # repetition count is one
    "mha": Coupling(
        linears=_LINEARS, sets=_SETS, expand={"o_heads": ("v_heads", "q_per_kv")},
        vectors={"input_layernorm": "hidden", "post_attention_layernorm": "hidden", "final_norm": "hidden"},
        outside={"embed_tokens": (None, "hidden"), "lm_head": (None, "hidden")}),
}


def _dims(shape) -> Dict[str, int]:
    return {"hidden": shape.hidden, "intermediate": shape.intermediate, "head_dim": shape.head_dim,
            "kv_dim": shape.n_kv_heads * shape.head_dim, "q_dim": shape.n_heads * shape.head_dim,
            "q_per_kv": shape.n_heads // shape.n_kv_heads}


def reorder_first_order(ctx: Context, shape, coupling: Coupling, W: Dict[str, torch.Tensor],
                        G: Dict[str, torch.Tensor], ref_bits: int, group: int) -> Dict[str, torch.Tensor]:
    """Channel permutations of one layer from first-order element sensitivities |G (W - Q(W))|
    (Section 3.2 with p = 1; l1 aggregation per channel, Section 4.1), summed over every matrix
    that shares the set, sorted descending inside each segment."""
    d = _dims(shape)
    dev = next(iter(W.values())).device
    f32 = dict(dtype=torch.float32, device=dev)
    size = {s: d[a] for s, (a, _) in coupling.sets.items()}
    for s, (src, _) in coupling.expand.items():
        size[s] = size[src] * d[coupling.expand[s][1]]
    score = {s: torch.empty(n, **f32) for s, n in size.items()}
    touched = set()
    for name, (rs, cs) in coupling.linears.items():
        kw = {}
        if rs is not None:
            kw.update(row_score=score[rs], accumulate_row=rs in touched)
        if cs is not None:
            kw.update(col_score=score[cs], accumulate_col=cs in touched)
        if kw:
            ctx.reorder_channels_first_order(W[name], G[name], ref_bits, group, **kw)
        touched.update(x for x in (rs, cs) if x is not None)
    perms: Dict[str, torch.Tensor] = {}
    for s, (src, reps_attr) in coupling.expand.items():
        ctx.fold_segment_scores(score[src], score[s], d[reps_attr], d[coupling.sets[src][1]])
    for s, (_, seg_attr) in coupling.sets.items():
        seg = d[seg_attr] if seg_attr else size[s]
        perms[s] = torch.empty(size[s], dtype=torch.int32, device=dev)
        ctx.reorder_channels(None, None, ref_bits, group, row_score=score[s], row_segment=seg,
                             row_perm=perms[s], shape=(size[s], group))
    for s, (src, reps_attr) in coupling.expand.items():
        perms[s] = ctx.expand_segment_perm(perms[src], d[reps_attr], d[coupling.sets[src][1]])
    return perms


def permute_outside(ctx: Context, coupling: Coupling, perms: Dict[str, torch.Tensor],
                    tensors: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
    """The tensors that are not quantised but must follow a permutation: outside matrices through
    the library's gather, per-channel vectors by index."""
    out = {}
    for name, t in tensors.items():
        if name in coupling.outside:
            rs, cs = coupling.outside[name]
            out[name] = ctx.permute_matrix(t, row_perm=perms[rs] if rs else None, col_perm=perms[cs] if cs else None)
        elif name in coupling.vectors:
            out[name] = t.index_select(0, perms[coupling.vectors[name]].long())
        else:
            raise KeyError(f"{name} is in neither table")
    return out


@dataclass
class DynamicResult:
    level: torch.Tensor
    perms: Dict[str, Optional[torch.Tensor]]
    block_start: Dict[str, int]
    n_blocks: int
    iterations: int = 0
    expansions: int = 0
    accepted: int = 0
    rejected: int = 0
    loss: Optional[float] = None
    used_bits: int = 0
    cap_bits: int = 0
    history: List[dict] = field(default_factory=list)


def search_layer_dynamic(ctx: Context, shape, W: Dict[str, torch.Tensor],
                         grad_fn: Callable[..., Dict[str, torch.Tensor]],
                         loss_fn: Callable[..., float], cfg,
                         coupling: str = "llama", names: Optional[Sequence[str]] = None,
                         max_iterations: int = 4096, observer=None) -> DynamicResult:
    """Algorithm 2 on one decoder layer with refreshed first-order scores.

    Line 2: warm start at the largest candidate <= budget, k = floor(gamma0 N).  One-time channel
    reordering from the gradient at the warm start (Section 4.1).  Then, while k >= floor(gammaT N):
    lines 4-5: G = grad_fn(level), s_up / s_down of every block at its current bitwidth
    (Appendix E.3); lines 6-10: one step (expansion while the budget is slack, else the balanced
    exchange); line 11: an exchange is kept only if loss_fn says the loss fell, otherwise it is
    undone and k is halved (line 12).  `observer(it, level, s_up, s_down, candidate, report,
    kept)`, if given, sees every iteration.
    """
    cp = COUPLING_TABLES[coupling]
    names = list(names) if names is not None else [l.name for l in shape.linears]
    dev = W[names[0]].device
    br, bc, g, bits = cfg.block_rows, cfg.block_cols, cfg.group, list(cfg.bits)
    block_start, n = {}, 0
    for nm in names:
        R, C = W[nm].shape
        block_start[nm] = n
        n += (R // br) * (C // bc)
    ok = [i for i, b in enumerate(bits) if b <= cfg.budget]
    if not ok:
        raise ValueError("budget below the smallest candidate")
    level = torch.full((n,), max(ok), dtype=torch.uint8, device=dev)
    k = max(1, int(cfg.gamma0 * n))
    kT = max(1, int(cfg.gammaT * n))
    k = max(k, kT)

    perms: Dict[str, Optional[torch.Tensor]] = {s: None for s in list(cp.sets) + list(cp.expand)}
    G = grad_fn(level, perms)
    fresh = True                                       # G belongs to (level, perms)
    if cfg.reorder:
        perms = reorder_first_order(ctx, shape, cp, W, G, bits[max(ok)], g)
        fresh = False                                  # the groups have moved: quantize again

    def perm_of(key):
        return perms[key] if key is not None else None

    f32 = dict(dtype=torch.float32, device=dev)
    s_up, s_down = torch.empty(n, **f32), torch.empty(n, **f32)
    res = DynamicResult(level=level, perms=perms, block_start=block_start, n_blocks=n)
    loss = None
    while k >= kT and res.iterations < max_iterations:
        res.iterations += 1
        if not fresh:
            G = grad_fn(level, perms)                  # lines 4-5: a new mini-batch every iteration
        fresh = False
        for nm in names:
            R, C = W[nm].shape
            s, nb = block_start[nm], (R // br) * (C // bc)
            rs, cs = cp.linears[nm]
            ctx.first_order_scores(W[nm], G[nm], bits, level[s:s + nb], br, bc, g, row_perm=perm_of(rs),
                                   col_perm=perm_of(cs), s_up=s_up[s:s + nb], s_down=s_down[s:s + nb],
                                   want_l1=False)
        cand, rep = ctx.exchange_step(s_up, s_down, level, bits, cfg.budget, k, uniform_block_elems=br * bc)
        kept = False
        if rep["moved"] and rep["expansion"]:
            kept = True
            res.expansions += 1
        elif rep["moved"]:
            # line 11: both allocations on the current mini-batch
            loss, new_loss = float(loss_fn(level, perms)), float(loss_fn(cand, perms))
            if new_loss < loss:
                kept, loss = True, new_loss
                res.accepted += 1
        if observer is not None:
            observer(res.iterations, level, s_up, s_down, cand, rep, kept)
        res.history.append({"k": k, "expansion": bool(rep["expansion"]), "moved": bool(rep["moved"]),
                            "kept": kept, "n_up": rep["n_up"], "n_down": rep["n_down"],
                            "used_bits": rep["used_out"] if kept else rep["used_in"]})
        if kept:
            level = cand
            if rep["expansion"]:
                loss = None                            # the loss of the new allocation is not known yet
        else:
            k //= 2
            res.rejected += 1
        res.used_bits = rep["used_out"] if kept else rep["used_in"]
        res.cap_bits = rep["cap_bits"]
    res.level, res.loss = level, loss
    return res
