"""Sequences the C-ABI calls for one Llama-shaped decoder layer (harness, not hot path).

Only bookkeeping lives here: which matrices share a channel permutation (Appendix D of
the paper) and where each matrix's rows of the global error table start.  Every number
is produced by the library's kernels.

Coupling (Appendix D):
  * residual stream: the columns of q/k/v/gate/up and the rows of o/down share one
    permutation of the hidden dimension (scores summed over all of them);
  * MLP: rows of gate/up and columns of down share one permutation of the intermediate
    dimension;
  * attention: only v (rows) and o (columns) are reordered, inside each head; with
    grouped-query attention the query heads that read one value head share its order;
    the output order of q and k is kept.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Sequence

import torch

from .binding import Context, SB_ALLOC_SCALEBITS
from .synth import LayerShape


@dataclass
class SearchConfig:
    bits: Sequence[int] = (2, 3, 4, 8)
    budget: float = 2.5
    block_rows: int = 128
    block_cols: int = 128
    group: int = 128
    gamma0: float = 0.05
    gammaT: float = 0.02
    mode: int = SB_ALLOC_SCALEBITS
    reorder: bool = True

    @property
    def ref_bits(self) -> int:
        """Reorder statistics are taken at the warm-start precision (Algorithm 2, line 2)."""
        ok = [b for b in self.bits if b <= self.budget]
        return max(ok) if ok else min(self.bits)


# (row permutation, column permutation) of each linear, by name of the coupled channel set
COUPLING = {
    "q_proj": (None, "hidden"), "k_proj": (None, "hidden"), "v_proj": ("v_heads", "hidden"),
    "o_proj": ("hidden", "o_heads"), "gate_proj": ("intermediate", "hidden"),
    "up_proj": ("intermediate", "hidden"), "down_proj": ("hidden", "intermediate"),
}


@dataclass
class LayerResult:
    moments: Dict[str, torch.Tensor]
    perms: Dict[str, Optional[torch.Tensor]]
    scores: Dict[str, torch.Tensor]
    err: torch.Tensor                 # [N, L] global table, matrices in shape.linears order
    gain: Optional[torch.Tensor]
    block_start: Dict[str, int]
    n_blocks: int
    level: Optional[torch.Tensor] = None
    report: Optional[dict] = None
    report_dev: Optional[torch.Tensor] = None        # the report on the device (whole-step graphs)
    packed: Dict[str, tuple] = field(default_factory=dict)

    def read_report(self) -> dict:
        """The allocation's report; after a whole-step graph it is still on the device and is
        copied here (the caller has synchronised, or is on the stream that wrote it)."""
        if self.report is None and self.report_dev is not None:
            self.report = Context.read_report(self.report_dev)
        return self.report

    def row_perm(self, name):
        return self.perms[COUPLING[name][0]] if COUPLING[name][0] else None

    def col_perm(self, name):
        return self.perms[COUPLING[name][1]] if COUPLING[name][1] else None


# Reorder statistics (Appendix D): which coupled score vector a matrix's row / column sums belong
# to, in the order in which the sums of a set are added.  "vo" and "o_cols" have one writer each.
STAT_SETS = {
    "q_proj": (None, "hidden"), "k_proj": (None, "hidden"), "v_proj": ("vo", "hidden"),
    "o_proj": ("hidden", "o_cols"), "gate_proj": ("intermediate", "hidden"),
    "up_proj": ("intermediate", "hidden"), "down_proj": ("hidden", "intermediate"),
}


def stat_part_buffers(shape: LayerShape, device) -> Dict[str, list]:
    """One private fp32 vector per (matrix, axis) that feeds a shared score vector:
    {"hidden": [(matrix, axis, buffer), ...], "intermediate": [...]} in adding order."""
    size = {"hidden": shape.hidden, "intermediate": shape.intermediate}
    parts = {"hidden": [], "intermediate": []}
    for name, (row_set, col_set) in STAT_SETS.items():
        for axis, key in (("row", row_set), ("col", col_set)):
            if key in parts:
                parts[key].append((name, axis, torch.empty(size[key], dtype=torch.float32, device=device)))
    return parts


def layer_statistics(cxs, W, c, rb, g, parts, vo_score, o_col_score, hid_score, mid_score, accumulate_hidden=False):
    """a2 for one layer: every matrix's statistics by a call of its own (dealt to the contexts
    `cxs`), then the shared vectors as fixed-order sums of the matrices' parts on cxs[0]:
    bit for bit what the calls would give accumulating into the shared vectors one by one."""
    own = {(name, axis): buf for key in parts for name, axis, buf in parts[key]}
    own[("v_proj", "row")] = vo_score
    own[("o_proj", "col")] = o_col_score

    def one(cx, name):
        cx.reorder_channels(W[name], c[name], rb, g, row_score=own.get((name, "row")),
                            col_score=own.get((name, "col")))

    _dealt(cxs, list(STAT_SETS), one)
    cxs[0].sum_scores(hid_score, [buf for _, _, buf in parts["hidden"]], accumulate=accumulate_hidden)
    cxs[0].sum_scores(mid_score, [buf for _, _, buf in parts["intermediate"]])


class LayerWorkspace:
    """Device buffers for one layer, allocated once so a timed step allocates nothing."""

    def __init__(self, shape: LayerShape, cfg: SearchConfig, device, keep_permuted: bool = True):
        self.shape, self.cfg = shape, cfg
        f32 = dict(dtype=torch.float32, device=device)
        i32 = dict(dtype=torch.int32, device=device)
        L = len(cfg.bits)
        kv = shape.n_kv_heads * shape.head_dim
        qd = shape.n_heads * shape.head_dim
        self.moments = {n: torch.empty(k, **f32) for n, k in shape.act_dims.items()}
        self.hid_score = torch.empty(shape.hidden, **f32)
        self.mid_score = torch.empty(shape.intermediate, **f32)
        self.vo_score = torch.empty(kv, **f32)
        self.o_col_score = torch.empty(qd, **f32)
        # reorder statistics of each matrix on its own (added per coupled set in a fixed order)
        self.stat_parts = stat_part_buffers(shape, device)
        self.p_hid = torch.empty(shape.hidden, **i32)
        self.p_mid = torch.empty(shape.intermediate, **i32)
        self.p_v = torch.empty(kv, **i32)
        self.p_o = torch.empty(qd, **i32)
        self.block_start, n = {}, 0
        for lin in shape.linears:
            self.block_start[lin.name] = n
            n += (lin.rows // cfg.block_rows) * (lin.cols // cfg.block_cols)
        self.n_blocks = n
        self.err = torch.empty((n, L), **f32)
        self.gain = torch.empty((n, max(L - 1, 1)), **f32)   # [N, L-1] per-bit marginal gains
        self.level = torch.empty(n, dtype=torch.uint8, device=device)
        self.report_dev = torch.zeros(128, dtype=torch.uint8, device=device)   # sb_alloc_report
        self.w_perm = ({lin.name: torch.empty((lin.rows, lin.cols), dtype=torch.bfloat16, device=device)
                        for lin in shape.linears} if keep_permuted else None)
        self.packed = {}
        for lin in shape.linears:
            nb = (lin.rows // cfg.block_rows) * (lin.cols // cfg.block_cols)
            self.packed[lin.name] = (
                torch.empty(lin.rows * lin.cols * max(cfg.bits) // 32, dtype=torch.int32, device=device),
                torch.empty(nb + 1, dtype=torch.int64, device=device),
                torch.empty((lin.rows * lin.cols // cfg.group, 2), **f32))


class _Timed:
    """Brackets one library call with CUDA events on the current stream (None: no timing)."""

    def __init__(self, timers, stage):
        self.timers, self.stage = timers, stage

    def __enter__(self):
        if self.timers is not None:
            self.a = torch.cuda.Event(enable_timing=True)
            self.b = torch.cuda.Event(enable_timing=True)
            self.a.record()

    def __exit__(self, *exc):
        if self.timers is not None:
            self.b.record()
            self.timers.setdefault(self.stage, []).append((self.a, self.b))


def contexts_of(ctx: Context, ctx2) -> list:
    """[ctx] plus the extra contexts: `ctx2` is None, one Context or a sequence of them."""
    if ctx2 is None:
        return [ctx]
    if isinstance(ctx2, Context):
        return [ctx, ctx2]
    return [ctx] + list(ctx2)


class StageGraphs:
    """CUDA graphs of the stages of one (workspace, weights, activations) binding.

    Every pointer a stage uses is fixed (the workspace and the input tensors), so the stage's
    library calls can be captured once on the context's stream and replayed: the kernels then
    run back to back without per-call host overhead.  With `whole=False` there is one graph per
    stage and the allocation stays eager (it reads its report back to the host); with `whole=True`
    `search_layer` captures the whole step, moments to pack, as ONE graph with the allocation in
    its enqueue-only form (the report stays on the device), so that a step is one launch and
    nothing waits for the host.  The context must live on a non-default stream.
    """

    def __init__(self, ctx: Context, ctx2=None, whole: bool = False):
        # ctx2: the extra context(s) of a multi-stream search_layer; their launches are captured (and
        # counted) with the first one's
        self.ctx, self.ctx2, self.graphs, self.kernels = ctx, ctx2, {}, {}
        self.whole = whole
        self.results = {}                  # what the captured function returned, per graph
        self.replayed_kernels = 0          # kernels launched through graph replays so far

    def _launches(self) -> int:
        return sum(c.kernel_launches() for c in contexts_of(self.ctx, self.ctx2))

    def run(self, stage: str, fn):
        g = self.graphs.get(stage)
        if g is None:
            fn()                                   # eager once: scratch growth, attributes
            self.ctx.stream.synchronize()
            g = torch.cuda.CUDAGraph()
            n0 = self._launches()
            with torch.cuda.graph(g, stream=self.ctx.stream):
                self.results[stage] = fn()
            self.kernels[stage] = self._launches() - n0
            self.graphs[stage] = g
        g.replay()
        self.replayed_kernels += self.kernels[stage]
        return self.results[stage]


def _dealt(cxs, names, fn):
    """fn(context, name) for every name, the names dealt to the contexts in turn; the extra
    contexts' streams fork from the first one's and join it again (graph edges under capture)."""
    if len(cxs) == 1:
        for n in names:
            fn(cxs[0], n)
        return
    fork = torch.cuda.Event()
    fork.record(cxs[0].stream)
    for c in cxs[1:]:
        c.stream.wait_event(fork)
    for i, n in enumerate(names):
        fn(cxs[i % len(cxs)], n)
    for c in cxs[1:]:
        join = torch.cuda.Event()
        join.record(c.stream)
        cxs[0].stream.wait_event(join)


def search_layer(ctx: Context, weights: Dict[str, torch.Tensor], acts: Dict[str, torch.Tensor],
                 ws: LayerWorkspace, allocate: bool = True, pack: bool = True,
                 timers: Optional[dict] = None, graphs: Optional[StageGraphs] = None,
                 ctx2=None) -> LayerResult:
    """moments -> reorder statistics -> permutations -> block scores -> allocation -> pack.

    `timers`, if given, maps the stage names moments / reorder_stats / sort / scores /
    allocate / pack to lists that receive one (start, end) CUDA event pair per stage.
    `graphs`, if given, replays each stage from a CUDA graph captured on first use, or the whole
    step from one graph (`StageGraphs(whole=True)`: `timers` then receives one pair under "step",
    the report stays on the device until `LayerResult.read_report()`, and device-side conditions
    are reported by the caller's next `ctx.sync()`).
    `ctx2`, if given, is one more context, or a sequence of them, each on a stream of its own: the
    stages whose matrices are independent of one another (block scores, pack) deal the matrices to
    the contexts in turn, forked from and joined back to the first context's stream, so that the
    kernels of different matrices run beside one another (measured on the 8B layer, one / two /
    seven contexts: scores 0.40 / 0.35 / 0.32 ms, pack 0.21 / 0.17 / 0.14 ms).  The moments of the
    distinct inputs, the sorts of the three channel sets and the reorder statistics of the seven
    matrices are dealt the same way; the statistics of a coupled channel set are written per
    matrix and added afterwards in a fixed order (`layer_statistics`).  Every output is the same
    as with one context, bit for bit: each call runs the same kernels on its own data.
    """
    if graphs is not None and graphs.whole:
        # the whole step as one graph: the stages run under capture with direct calls and the
        # enqueue-only allocation; replays return the same result object (all of it lives in `ws`)
        with _Timed(timers, "step"):
            res = graphs.run(f"step:{int(allocate)}{int(pack)}",
                             lambda: _layer_stages(ctx, weights, acts, ws, allocate, pack, None, None, ctx2,
                                                   enqueue_only=True))
        res.report = None                          # decoded on demand from the device copy
        return res
    return _layer_stages(ctx, weights, acts, ws, allocate, pack, timers, graphs, ctx2, enqueue_only=False)


def _layer_stages(ctx, weights, acts, ws, allocate, pack, timers, graphs, ctx2, enqueue_only) -> LayerResult:
    """The stages of `search_layer`, each eager or from its own graph; `enqueue_only` takes the
    allocation without the host round trip (its report stays in `ws.report_dev`)."""
    def stage(name, fn):
        with _Timed(timers, name):
            if graphs is not None:
                graphs.run(name, fn)
            else:
                fn()

    def dealt(names, fn):
        """fn(context, name) for every name: on ctx alone, or in turn on ctx and the extra contexts."""
        _dealt(contexts_of(ctx, ctx2), names, fn)

    shape, cfg = ws.shape, ws.cfg
    lin = {l.name: l for l in shape.linears}
    g, rb = cfg.group, cfg.ref_bits
    reps = shape.n_heads // shape.n_kv_heads
    hd = shape.head_dim
    W = weights

    # a1: calibration second moments, one per distinct linear input
    def do_moments():
        dealt(list(acts), lambda cx, name: cx.calib_moments(acts[name], ws.moments[name]))

    stage("moments", do_moments)
    c = {n: ws.moments[l.act] for n, l in lin.items()}

    perms = {"hidden": None, "intermediate": None, "v_heads": None, "o_heads": None}
    if cfg.reorder:
        # a2: reorder statistics, one call per matrix, added per coupled channel set in a fixed order
        def do_stats():
            layer_statistics(contexts_of(ctx, ctx2), W, c, rb, g, ws.stat_parts, ws.vo_score, ws.o_col_score,
                             ws.hid_score, ws.mid_score)

        # the three channel sets are sorted independently of one another: three chains of calls
        def sort_hidden(cx):
            cx.reorder_channels(None, None, rb, g, row_score=ws.hid_score, row_segment=shape.hidden,
                                row_perm=ws.p_hid, shape=(shape.hidden, g))

        def sort_intermediate(cx):
            cx.reorder_channels(None, None, rb, g, row_score=ws.mid_score,
                                row_segment=shape.intermediate, row_perm=ws.p_mid,
                                shape=(shape.intermediate, g))

        def sort_heads(cx):
            cx.fold_segment_scores(ws.vo_score, ws.o_col_score, reps, hd)
            cx.reorder_channels(None, None, rb, g, row_score=ws.vo_score, row_segment=hd,
                                row_perm=ws.p_v, shape=(ws.vo_score.numel(), g))
            cx.expand_segment_perm(ws.p_v, reps, hd, out=ws.p_o)

        def do_sort():
            dealt([sort_intermediate, sort_hidden, sort_heads], lambda cx, chain: chain(cx))

        stage("reorder_stats", do_stats)
        stage("sort", do_sort)
        perms = {"hidden": ws.p_hid, "intermediate": ws.p_mid, "v_heads": ws.p_v, "o_heads": ws.p_o}

    res = LayerResult(moments=ws.moments, perms=perms,
                      scores={"hidden": ws.hid_score, "intermediate": ws.mid_score,
                              "v_heads": ws.vo_score, "o_cols": ws.o_col_score},
                      err=ws.err, gain=ws.gain if len(cfg.bits) > 1 else None,
                      block_start=ws.block_start, n_blocks=ws.n_blocks)

    # a4: block scores of every matrix into its rows of the global table
    L = len(cfg.bits)

    def score_one(cx, name):
        l = lin[name]
        nb = (l.rows // cfg.block_rows) * (l.cols // cfg.block_cols)
        s = ws.block_start[name]
        cx.block_scores(W[name], c[name], cfg.bits, cfg.block_rows, cfg.block_cols, g,
                        row_perm=res.row_perm(name), col_perm=res.col_perm(name),
                        err=ws.err[s:s + nb], gain=ws.gain[s:s + nb] if L > 1 else None,
                        want_gain=L > 1,
                        W_perm_out=ws.w_perm[name] if ws.w_perm is not None else None)

    def do_scores():
        dealt(list(lin.keys()), score_one)

    stage("scores", do_scores)
    if not allocate:
        return res

    # a5: one global allocation over all blocks of the layer
    if enqueue_only:
        res.level, res.report_dev = ctx.allocate_bits_async(
            ws.err, cfg.bits, cfg.budget, cfg.mode, cfg.gamma0, cfg.gammaT,
            uniform_block_elems=cfg.block_rows * cfg.block_cols, level=ws.level, report=ws.report_dev)
    else:
        with _Timed(timers, "allocate"):
            res.level, res.report = ctx.allocate_bits(
                ws.err, cfg.bits, cfg.budget, cfg.mode, cfg.gamma0, cfg.gammaT,
                uniform_block_elems=cfg.block_rows * cfg.block_cols, level=ws.level)
    if not enqueue_only:
        # the allocation has just synchronised with the host and checked the first context's device
        # status; the extra contexts' (their share of the score kernels) is read here.  What their
        # pack kernels latch is seen at the next call, or by the caller's own sync() of them.
        for c in contexts_of(ctx, ctx2)[1:]:
            c.sync()
    if not pack:
        return res

    # a6: pack every matrix at its blocks' levels (from the permuted copy when it was kept)
    def pack_one(cx, name):
        l = lin[name]
        nb = (l.rows // cfg.block_rows) * (l.cols // cfg.block_cols)
        s = ws.block_start[name]
        packed, off, meta = ws.packed[name]
        if ws.w_perm is not None:
            cx.pack_blocks(ws.w_perm[name], cfg.bits, ws.level[s:s + nb], cfg.block_rows,
                           cfg.block_cols, g, packed=packed, block_off=off, meta=meta)
        else:
            cx.pack_blocks(W[name], cfg.bits, ws.level[s:s + nb], cfg.block_rows, cfg.block_cols,
                           g, row_perm=res.row_perm(name), col_perm=res.col_perm(name),
                           packed=packed, block_off=off, meta=meta)

    def do_pack():
        dealt(list(lin.keys()), pack_one)

    stage("pack", do_pack)
    res.packed = dict(ws.packed)
    return res


# ---- whole model: one global allocation over the blocks of all layers --------------------------------
@dataclass
class ModelResult:
    """Outputs of `search_model`; `tables[ref_bits]` is the [N, L] table the budgets of that
    warm-start precision were allocated on, blocks ordered layer by layer, matrices in
    `shape.linears` order inside a layer."""
    moments: list                                    # per layer: {input name: [K] fp32}
    block_start: Dict[tuple, int]                    # (layer, matrix name) -> first table row
    n_blocks: int
    tables: Dict[int, torch.Tensor] = field(default_factory=dict)
    perms: Dict[int, dict] = field(default_factory=dict)      # ref_bits -> {"hidden": p, (set, layer): p}
    scores: Dict[int, dict] = field(default_factory=dict)     # ref_bits -> the sorted score vectors
    levels: Dict[float, torch.Tensor] = field(default_factory=dict)
    reports: Dict[float, dict] = field(default_factory=dict)
    ms: Dict[str, float] = field(default_factory=dict)        # CUDA-event time of the library calls


class _Clock:
    """Sums CUDA-event time of bracketed regions per key (read after a synchronise)."""

    def __init__(self):
        self.pairs = {}

    def __call__(self, key):
        clock = self

        class _R:
            def __enter__(self_inner):
                self_inner.a = torch.cuda.Event(enable_timing=True)
                self_inner.b = torch.cuda.Event(enable_timing=True)
                self_inner.a.record()

            def __exit__(self_inner, *exc):
                self_inner.b.record()
                clock.pairs.setdefault(key, []).append((self_inner.a, self_inner.b))

        return _R()

    def totals(self):
        return {k: sum(a.elapsed_time(b) for a, b in v) for k, v in self.pairs.items()}


def search_model(ctx: Context, shape: LayerShape, n_layers: int, cfg: SearchConfig,
                 budgets: Sequence[float], make_weights, make_acts, device,
                 keep_tables: bool = True, keep_weights: bool = True,
                 alloc_repeats: int = 1, ctx2=None) -> ModelResult:
    """Two sweeps over a model of `n_layers` identical decoder layers, then one global
    allocation per budget (Eq. 1 over ALL blocks of the model).

    The residual-stream permutation is shared by every layer (Appendix D: the hidden dimension
    runs through the whole network), so its score vector is accumulated over all layers before
    it is sorted: sweep 1 takes moments and reorder statistics, sweep 2 scores the blocks of
    the permuted matrices.  Reorder statistics are taken at the warm-start precision of the
    budget, so budgets are grouped by that precision and the sweeps run once per group.

    `make_weights(layer)` / `make_acts(layer)` return the layer's tensors on `device`.
    Activations are dropped after their moments; weights stay resident, or with
    `keep_weights=False` are made again in every sweep (a model larger than the device's
    memory is streamed layer by layer: only moments, permutations and tables persist).  Only library calls are
    timed (`ModelResult.ms`, keys moments / stats@b / sort@b / scores@b / allocate@budget).
    The allocation is eager and paced by the host; `alloc_repeats` > 1 repeats each (deterministic)
    allocation call and keeps the fastest time, so that a host hiccup does not pass for GPU time.
    `ctx2`, if given, is one more context or a sequence of them, each on a stream of its own: the
    independent calls of a layer (moments, statistics, sorts, block scores) are dealt to the
    contexts in turn (as in `search_layer`).
    """
    f32 = dict(dtype=torch.float32, device=device)
    i32 = dict(dtype=torch.int32, device=device)
    lin = {l.name: l for l in shape.linears}
    g = cfg.group
    L = len(cfg.bits)
    reps = shape.n_heads // shape.n_kv_heads
    hd = shape.head_dim
    kv, qd = shape.n_kv_heads * hd, shape.n_heads * hd
    clock = _Clock()
    prev_stream = torch.cuda.current_stream()

    block_start, n = {}, 0
    for layer in range(n_layers):
        for l in shape.linears:
            block_start[(layer, l.name)] = n
            n += (l.rows // cfg.block_rows) * (l.cols // cfg.block_cols)
    res = ModelResult(moments=[], block_start=block_start, n_blocks=n)

    with torch.cuda.stream(ctx.stream):
        # a1 once: the moments do not depend on the budget
        weights = []
        for layer in range(n_layers):
            X = make_acts(layer)
            m = {name: torch.empty(k, **f32) for name, k in shape.act_dims.items()}
            with clock("moments"):
                _dealt(contexts_of(ctx, ctx2), list(X), lambda cx, name: cx.calib_moments(X[name], m[name]))
            ctx.stream.synchronize()               # X is dropped: its memory must not be reused early
            del X
            res.moments.append(m)
            if keep_weights:
                weights.append(make_weights(layer))

        def layer_weights(layer):
            return weights[layer] if keep_weights else make_weights(layer)

        groups = {}
        for b in budgets:
            ok = [x for x in cfg.bits if x <= b]
            groups.setdefault(max(ok) if ok else min(cfg.bits), []).append(b)

        for rb, bs in sorted(groups.items()):
            hid = torch.empty(shape.hidden, **f32)
            mid = [torch.empty(shape.intermediate, **f32) for _ in range(n_layers)]
            vo = [torch.empty(kv, **f32) for _ in range(n_layers)]
            ocol = [torch.empty(qd, **f32) for _ in range(n_layers)]
            stat_parts = stat_part_buffers(shape, device)
            # sweep 1: a2, hidden scores accumulated over all layers
            for layer in range(n_layers):
                W, m = layer_weights(layer), res.moments[layer]
                c = {nm: m[l.act] for nm, l in lin.items()}
                first = layer == 0
                with clock(f"stats@{rb}"):
                    layer_statistics(contexts_of(ctx, ctx2), W, c, rb, g, stat_parts, vo[layer], ocol[layer],
                                     hid, mid[layer], accumulate_hidden=not first)
            # a3: one sort of the residual stream, per-layer sorts of the other sets
            p_hid = torch.empty(shape.hidden, **i32)
            p_mid = [torch.empty(shape.intermediate, **i32) for _ in range(n_layers)]
            p_v = [torch.empty(kv, **i32) for _ in range(n_layers)]
            p_o = [torch.empty(qd, **i32) for _ in range(n_layers)]
            with clock(f"sort@{rb}"):
                if cfg.reorder:
                    # independent chains of calls: the residual stream once, two channel sets per layer
                    def sort_hidden(cx):
                        cx.reorder_channels(None, None, rb, g, row_score=hid, row_segment=shape.hidden,
                                            row_perm=p_hid, shape=(shape.hidden, g))

                    def sort_intermediate(layer):
                        return lambda cx: cx.reorder_channels(
                            None, None, rb, g, row_score=mid[layer], row_segment=shape.intermediate,
                            row_perm=p_mid[layer], shape=(shape.intermediate, g))

                    def sort_heads(layer):
                        def chain(cx):
                            cx.fold_segment_scores(vo[layer], ocol[layer], reps, hd)
                            cx.reorder_channels(None, None, rb, g, row_score=vo[layer], row_segment=hd,
                                                row_perm=p_v[layer], shape=(kv, g))
                            cx.expand_segment_perm(p_v[layer], reps, hd, out=p_o[layer])
                        return chain

                    chains = [sort_hidden]
                    for layer in range(n_layers):
                        chains += [sort_intermediate(layer), sort_heads(layer)]
                    _dealt(contexts_of(ctx, ctx2), chains, lambda cx, chain: chain(cx))
            perms = {"hidden": p_hid if cfg.reorder else None}
            for layer in range(n_layers):
                perms[("intermediate", layer)] = p_mid[layer] if cfg.reorder else None
                perms[("v_heads", layer)] = p_v[layer] if cfg.reorder else None
                perms[("o_heads", layer)] = p_o[layer] if cfg.reorder else None

            def perm_of(key, layer):
                if key is None:
                    return None
                return perms["hidden"] if key == "hidden" else perms[(key, layer)]

            # sweep 2: a4 into the global table
            err = torch.empty((n, L), **f32)
            for layer in range(n_layers):
                W, m = layer_weights(layer), res.moments[layer]
                with clock(f"scores@{rb}"):
                    def score_one(cx, nm):
                        l = lin[nm]
                        nb = (l.rows // cfg.block_rows) * (l.cols // cfg.block_cols)
                        s = block_start[(layer, nm)]
                        rp, cp = COUPLING[nm]
                        cx.block_scores(W[nm], m[l.act], cfg.bits, cfg.block_rows, cfg.block_cols, g,
                                        row_perm=perm_of(rp, layer), col_perm=perm_of(cp, layer),
                                        err=err[s:s + nb], want_gain=False)

                    _dealt(contexts_of(ctx, ctx2), list(lin), score_one)
            # a5: one global allocation per budget of the group
            for b in bs:
                for r in range(max(1, alloc_repeats)):
                    with clock(f"allocate@{b:g}#{r}"):
                        level, report = ctx.allocate_bits(err, cfg.bits, b, cfg.mode, cfg.gamma0, cfg.gammaT,
                                                          uniform_block_elems=cfg.block_rows * cfg.block_cols)
                res.levels[b], res.reports[b] = level, report
            if keep_tables:
                res.tables[rb] = err
                res.perms[rb] = perms
                res.scores[rb] = {"hidden": hid, "intermediate": mid, "v_heads": vo, "o_cols": ocol}
        ctx.stream.synchronize()
        for c in contexts_of(ctx, ctx2)[1:]:
            c.sync()                               # device status of the extra contexts' score kernels
    prev_stream.synchronize()
    totals = clock.totals()
    res.ms = {k: v for k, v in totals.items() if "#" not in k}
    for k, v in totals.items():
        if "#" in k:
            key = k.split("#")[0]
            res.ms[key] = min(res.ms.get(key, v), v)
    return res
