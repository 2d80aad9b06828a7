#!/usr/bin/env python
"""Benchmark of the bitwidth-search hot path on one Llama-3-8B-shaped decoder layer.

One step = one pass of the whole path over one layer of synthetic input: calibration
moments of the four linear inputs, reorder statistics + permutations, block scores of the
seven matrices at every candidate bitwidth, global allocation, packing.  Prints ONE JSON
line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "weight elements scored/s across all candidate bits"
UNIT = "elements/s"
TOKENS = 65536
BITS = (2, 3, 4, 8)
BUDGET = 2.5
SEED = 0
WORKLOAD = ("one Llama-3-8B-shaped decoder layer (q/o 4096x4096, k/v 1024x4096, gate/up 14336x4096, "
            "down 4096x14336; 218,103,808 bf16 weights), 65536 calibration tokens per input, "
            "blocks 128x128, group 128, bits {2,3,4,8}, budget 2.5")

# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of the dominant kernel, from one
# ncu capture of a 65536 x 4096 input (541.04 MB moved for 536.87 MB of activations); the kernel's
# traffic is proportional to T * K, so the ratio carries over to the launches of the step
NCU_TRAFFIC_RATIO = {"moments_partial_kernel": 1.0071}
NOMINAL_HBM_GBS = 8000.0      # the B200's nominal HBM3e bandwidth: the figure the 70 % target is stated on
STRESS_BITS = (1, 2, 3, 4, 5, 6, 8)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ---- clocks during the timed region ----------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.rows, self.proc, self.uuid = [], None, uuid

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.05] or [r for (_, r) in self.rows]
        sm, smax, reasons = [], None, set()
        for r in inside:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax = float(f[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- the CPU oracle on a bounded sample (cpu_baseline leg and --impl reference) ---------------
SAMPLE_DIV = 2   # the oracle is timed on 1/SAMPLE_DIV of the rows of every matrix and of the tokens
SAMPLE_TEXT = ("first half of the rows of each of the 7 matrices (109,051,904 weights) and 32768 of the "
               "65536 tokens of each of the 4 inputs, all five stages, per step")


def oracle_sample_inputs():
    """A row slice of every matrix of the layer and a token slice of every input (CPU tensors)."""
    from paper_2602_17698_b200 import synth
    shape = synth.LLAMA3_8B
    W = {l.name: synth.make_weight(l.rows // SAMPLE_DIV, l.cols, synth.tensor_seed(SEED, 0, l.tensor_id))
         for l in shape.linears}
    X = {n: synth.make_activations(TOKENS // SAMPLE_DIV, k, synth.tensor_seed(SEED, 0, synth.ACT_TENSOR_ID[n]))
         for n, k in shape.act_dims.items()}
    return shape, W, X


def oracle_step(shape, W, X):
    """The oracle's five stages, as they stand, on the sample; returns weight elements scored."""
    import numpy as np
    from oracle import sbo
    lin = {l.name: l for l in shape.linears}
    mom = {n: sbo.calib_moments(x, 1.0 / x.shape[0]) for n, x in X.items()}
    tables, n_elems = [], 0
    for name, w in W.items():
        c = mom[lin[name].act]
        rs, cs = sbo.reorder_scores(w, c, ref_bits=2, group=128)
        pr = sbo.argsort_desc_segments(rs)
        pc = sbo.argsort_desc_segments(cs)
        err, _ = sbo.block_scores(w, c, BITS, 128, 128, 128, row_perm=pr, col_perm=pc)
        tables.append((name, pr, pc, err))
        n_elems += w.shape[0] * w.shape[1]
    table = np.concatenate([t[3] for t in tables])
    st, level, rep = sbo.allocate_scalebits(table, BITS, BUDGET, 0.05, 0.02, 128 * 128)
    assert st == sbo.OK
    s = 0
    for name, pr, pc, err in tables:
        nb = err.shape[0]
        sbo.pack_blocks(W[name], BITS, level[s:s + nb], 128, 128, 128, row_perm=pr, col_perm=pc)
        s += nb
    return n_elems


def time_oracle(steps: int, warmup: int):
    from oracle import sbo
    sbo.build()
    shape, W, X = oracle_sample_inputs()
    for _ in range(warmup):
        oracle_step(shape, W, X)
    t0 = time.perf_counter()
    n = 0
    for _ in range(steps):
        n += oracle_step(shape, W, X)
    dt = time.perf_counter() - t0
    return n / dt, dt / steps, sbo.num_threads(), SAMPLE_TEXT


def oracle_full_matrix():
    """The oracle on ONE full-size matrix of the layer (q_proj, 4096 x 4096) with the full 65536-token
    input: moments, reorder statistics and sorts, block scores, allocation, pack, as they stand."""
    import numpy as np
    from oracle import sbo
    from paper_2602_17698_b200 import synth
    shape = synth.LLAMA3_8B
    l = next(x for x in shape.linears if x.name == "q_proj")
    w = synth.make_weight(l.rows, l.cols, synth.tensor_seed(SEED, 0, l.tensor_id))
    x = synth.make_activations(TOKENS, l.cols, synth.tensor_seed(SEED, 0, synth.ACT_TENSOR_ID[l.act]))
    t0 = time.perf_counter()
    c = sbo.calib_moments(x, 1.0 / x.shape[0])
    t1 = time.perf_counter()
    rs, cs = sbo.reorder_scores(w, c, ref_bits=2, group=128)
    pr, pc = sbo.argsort_desc_segments(rs), sbo.argsort_desc_segments(cs)
    err, _ = sbo.block_scores(w, c, BITS, 128, 128, 128, row_perm=pr, col_perm=pc)
    st, level, _ = sbo.allocate_scalebits(err, BITS, BUDGET, 0.05, 0.02, 128 * 128)
    assert st == sbo.OK
    sbo.pack_blocks(w, BITS, level, 128, 128, 128, row_perm=pr, col_perm=pc)
    t2 = time.perf_counter()
    n = l.rows * l.cols
    return {"matrix": "q_proj 4096 x 4096, 65536 tokens", "seconds_moments": t1 - t0,
            "seconds_weight_stages": t2 - t1, "value": n / (t2 - t0), "unit": UNIT}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 3))
    warm = 1 if args.warmup > 0 else 0
    value, sec, cores, sample = time_oracle(steps, warm)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample_per_step": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- multi-rank plumbing (replicas: every rank searches its own layer, no data-path collective) --
def max_over_ranks(x: float, world: int, device=None) -> float:
    """The slowest rank's time: what the whole job waits for."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's step time."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# ---- the CUDA path ------------------------------------------------------------------------------
STAGES = ("moments", "reorder_stats", "sort", "scores", "allocate", "pack")
FULL_MODEL_LAYERS = 32
FULL_MODEL_BUDGETS = tuple(2.0 + 0.25 * i for i in range(9))          # 2.0 ... 4.0
FULL_MODEL_SUPER = {3: 101, 12: 102, 20: 103, 29: 104}                # layer -> seed of its super weight


def measured_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), "measured cuBLAS bf16 burst"
    return 1590.0, "fallback"


def kernel_rooflines(ctx, W, X, moments, dev, peak_gbs, sm_mhz, sm_count):
    """The other kernels of the path, one library call at a time on 14336 x 4096 matrices (three
    different ones in rotation, 352 MB > L2, so every call streams from HBM), CUDA events on the
    context's stream.  HBM-bound kernels against the measured copy bandwidth; the score kernel
    against the FP32 pipe: SMs x 128 lanes x SM clock lane-operations per second, with
    4 L + 1 + (candidates of >= 6 bits) algorithmic lane-operations per weight.  The score kernel is
    timed for the bit sets of every config ({2,3,4,8}, {2,3,4}, {1,2,3,4,5,6,8}) and for the block
    shapes and group sizes at the corners of the stress sweep."""
    import torch
    mats = [W["gate_proj"], W["up_proj"], W["gate_proj"].clone()]
    c = moments["mlp_in"]
    R, Cc = mats[0].shape
    n = R * Cc
    nb = (R // 128) * (Cc // 128)
    f32 = dict(dtype=torch.float32, device=dev)
    rs, cs = torch.empty(R, **f32), torch.empty(Cc, **f32)
    err = torch.empty(nb, len(BITS), **f32)
    out = torch.empty_like(mats[0])
    gen = torch.Generator(device=dev).manual_seed(SEED)
    pr = torch.randperm(R, device=dev, generator=gen).int()
    pc = torch.randperm(Cc, device=dev, generator=gen).int()
    level = torch.randint(0, len(BITS), (nb,), device=dev, dtype=torch.uint8, generator=gen)
    packed = torch.empty(n * max(BITS) // 32, dtype=torch.int32, device=dev)
    off = torch.empty(nb + 1, dtype=torch.int64, device=dev)
    meta = torch.empty((n // 128, 2), **f32)

    def timed(fn, reps=9):
        for i in range(3):
            fn(mats[i % 3])
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(reps):
            fn(mats[i % 3])
        b.record()
        b.synchronize()
        return a.elapsed_time(b) / reps

    t_stats = timed(lambda m: ctx.reorder_channels(m, c, 2, 128, row_score=rs, col_score=cs))
    t_score = timed(lambda m: ctx.block_scores(m, c, BITS, 128, 128, 128, err=err, want_gain=False))
    score_variants = []
    for bits_v, br_v, bc_v, g_v in (((2, 3, 4), 128, 128, 128), (STRESS_BITS, 128, 128, 128),
                                    (STRESS_BITS, 128, 128, 32), (STRESS_BITS, 32, 32, 32),
                                    (STRESS_BITS, 64, 64, 64), (STRESS_BITS, 256, 128, 128)):
        err_v = torch.empty((R // br_v) * (Cc // bc_v), len(bits_v), **f32)
        t_v = timed(lambda m: ctx.block_scores(m, c, bits_v, br_v, bc_v, g_v, err=err_v, want_gain=False))
        score_variants.append((bits_v, br_v, bc_v, g_v, t_v))
        del err_v
    t_perm = timed(lambda m: ctx.block_scores(m, c, BITS, 128, 128, 128, row_perm=pr, col_perm=pc, err=err,
                                              want_gain=False, W_perm_out=out))
    t_pack = timed(lambda m: ctx.pack_blocks(m, BITS, level, 128, 128, 128, packed=packed, block_off=off,
                                             meta=meta))
    Gm = [(m.float() * 1e-2).to(torch.bfloat16) for m in mats[:2]]       # stand-in gradients
    Gm.append(Gm[0].clone())
    s_up, s_dn = torch.empty(nb, **f32), torch.empty(nb, **f32)
    idx = {id(m): i for i, m in enumerate(mats)}
    t_first = timed(lambda m: ctx.first_order_scores(m, Gm[idx[id(m)]], BITS, level, 128, 128, 128,
                                                     s_up=s_up, s_down=s_dn, want_l1=False))
    t_fstats = timed(lambda m: ctx.reorder_channels_first_order(m, Gm[idx[id(m)]], 2, 128, row_score=rs,
                                                                col_score=cs))
    t_gather = max(t_perm - t_score, 1e-6)
    avg_bits = sum(BITS) / len(BITS)
    # the one contraction: H = X^T X / T of the layer's MLP input (65536 x 4096) on the tensor cores
    Xg = X["mlp_in"]
    Tg, Kg = Xg.shape
    Hg = torch.empty((Kg, Kg), **f32)
    for _ in range(2):
        ctx.calib_gram(Xg, H=Hg)
    ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ga.record()
    for _ in range(5):
        ctx.calib_gram(Xg, H=Hg)
    gb.record()
    gb.synchronize()
    t_gram = ga.elapsed_time(gb) / 5
    nt = (Kg + 127) // 128
    gram_flops = 2.0 * Tg * 128 * 128 * (nt * (nt + 1) // 2)          # the upper-triangular tiles it computes
    tpeak, tkind = measured_tensor_peak()
    # block scores with the full matrix (same 14336 x 4096 matrices, H of their input)
    t_full = timed(lambda m: ctx.block_scores_full(m, Hg, BITS, 128, 128, 128, err=err, want_gain=False), reps=6)
    full_flops = nb * len(BITS) * 2 * 2.0 * 128 ** 3            # two 128^3 contractions per block and candidate
    del Hg

    def hbm(name, bytes_, ms, note):
        a = bytes_ / (ms * 1e-3) / 1e9
        return {"kernel": name, "bound": "hbm", "achieved": a, "peak": peak_gbs, "unit": "GB/s",
                "frac": a / peak_gbs, "frac_nominal": a / NOMINAL_HBM_GBS, "ms_per_call": ms,
                "algorithmic_bytes": bytes_, "note": note}

    alu_peak = sm_count * 128 * sm_mhz * 1e6 / 1e12

    def score_entry(bits_v, br_v, bc_v, g_v, ms):
        ops = 4 * len(bits_v) + 1 + sum(1 for b in bits_v if b >= 6)
        a_ops = n * ops / (ms * 1e-3) / 1e12
        gbs = 2 * n / (ms * 1e-3) / 1e9
        return {"kernel": "block_scores_kernel (+ scores_finish_kernel)", "bound": "alu", "achieved": a_ops,
                "peak": alu_peak, "unit": "T fp32 lane-ops/s", "frac": a_ops / alu_peak, "ms_per_call": ms,
                "bits": list(bits_v), "block": [br_v, bc_v], "group": g_v, "lane_ops_per_weight": ops,
                "hbm_gbs": gbs, "hbm_frac": gbs / peak_gbs, "hbm_frac_nominal": gbs / NOMINAL_HBM_GBS,
                "elements_per_s": n / (ms * 1e-3),
                "note": f"one call of sb_block_scores without permutations; peak = {sm_count} SMs x 128 lanes "
                        "x SM clock"}

    return [
        hbm("block_scores_kernel<StatsScorer> + stats_finish_kernel", 2 * n, t_stats,
            "one call of sb_reorder_channels (statistics only): the score kernel's slab walk with one candidate"),
        score_entry(BITS, 128, 128, 128, t_score),
    ] + [score_entry(*v) for v in score_variants] + [
        hbm("gather_cols_kernel", 4 * n, t_gather,
            "sb_block_scores with both permutations and W_perm_out minus the call without (2 B read + 2 B written)"),
        hbm("pack_offsets_small_kernel + pack_kernel", int(2 * n + n * avg_bits / 8 + n / 128 * 8), t_pack,
            "one call of sb_pack_blocks, uniformly random levels (2 B read + codes + metadata written)"),
        {"kernel": "gram_kernel (tcgen05, TMA)", "bound": "tensor", "achieved": gram_flops / (t_gram * 1e-3) / 1e12,
         "peak": tpeak, "unit": "TFLOP/s", "frac": gram_flops / (t_gram * 1e-3) / 1e12 / tpeak,
         "peak_source": tkind, "ms_per_call": t_gram,
         "effective_tflops_of_full_product": 2.0 * Tg * Kg * Kg / (t_gram * 1e-3) / 1e12,
         "note": f"one call of sb_calib_gram on the {Tg} x {Kg} MLP input (CTA pairs, tcgen05.mma.cta_group::2 on "
                 "256 x 256 tiles); flops of the upper-triangular 128 x 128 blocks (the mirror image is copied)"},
        {"kernel": "full_scores_kernel (tcgen05)", "bound": "tensor", "achieved": full_flops / (t_full * 1e-3) / 1e12,
         "peak": tpeak, "unit": "TFLOP/s", "frac": full_flops / (t_full * 1e-3) / 1e12 / tpeak,
         "peak_source": tkind, "ms_per_call": t_full,
         "note": "one call of sb_block_scores_full on a 14336 x 4096 matrix, 4 candidates; flops of the two "
                 "128 x 128 x 128 contractions per block and candidate; the quantisation arithmetic in front of "
                 "the tensor cores (binary64 code decisions) is what bounds it"},
        hbm("first_order_kernel", 4 * n, t_first,
            "one call of sb_first_order_scores, uniformly random levels (weights and gradient, 2 B each)"),
        hbm("reorder_stats_kernel (first-order form)", 4 * n, t_fstats,
            "one call of sb_reorder_channels_first_order (weights and gradient, 2 B each)"),
    ]


def dequant_gemm_times(ctx, dev, peak_gbs):
    """sb_dequant_gemm on the workload of the paper's kernel table (Table 4): an 8192 x 8192 matrix,
    16 and 32 tokens, all blocks at 4 bits and the 40 / 40 / 20 % mix of 2 / 4 / 8 bits (4 bits on
    average).  Six packed copies in rotation (216 MB > L2), so every call streams its codes from
    HBM; CUDA events on the context's stream around one CUDA graph of 12 calls."""
    import torch
    import numpy as np
    from paper_2602_17698_b200 import synth
    R = Cc = 8192
    nb = (R // 128) * (Cc // 128)
    bits = [2, 4, 8]
    W = synth.make_weight(R, Cc, 4242, dev)
    paper_us = {("int4", 16): 57.8, ("int4", 32): 65.0, ("mix", 16): 58.0, ("mix", 32): 65.9}
    out = []
    for kind in ("int4", "mix"):
        sets = []
        for k in range(6):
            lv = np.ones(nb, np.uint8) if kind == "int4" else synth.table4_levels(nb, 100 + k)
            level = torch.from_numpy(lv).to(dev)
            packed, off, meta = ctx.pack_blocks(W, bits, level, 128, 128, 128)
            ctx.sync()
            words = int(off[-1].item())
            sets.append((packed[:words + 4].clone(), off, meta, level, words))
            del packed
        for T in (16, 32):
            X = synth.make_activations(T, Cc, 77 + T, dev)
            Y = torch.empty((T, R), dtype=torch.float32, device=dev)
            def call(i):
                pk, off, meta, level, _ = sets[i % 6]
                ctx.dequant_gemm(X, pk, off, meta, level, R, Cc, bits, Y=Y)
            for i in range(6):
                call(i)
            ctx.stream.synchronize()
            # the 12 calls as one CUDA graph: three short launches per call would otherwise be paced
            # by the host
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=ctx.stream):
                for i in range(12):
                    call(i)
            g.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(ctx.stream):
                a.record()
                g.replay()
                b.record()
            b.synchronize()
            ms = a.elapsed_time(b) / 12
            del g
            bytes_ = sets[0][4] * 4 + R * (Cc // 128) * 8 + T * Cc * 2 + T * R * 4
            gbs = bytes_ / (ms * 1e-3) / 1e9
            out.append({"kernel": "dq_prepare_x_kernel + dequant_gemm_kernel (register-fragment tensor-core products, segments added inside a cluster)",
                        "bound": "hbm", "achieved": gbs, "peak": peak_gbs, "unit": "GB/s", "frac": gbs / peak_gbs,
                        "ms_per_call": ms, "us_per_call": ms * 1e3, "algorithmic_bytes": bytes_,
                        "workload": f"8192 x 8192, {T} tokens, " + ("all blocks 4 bits" if kind == "int4"
                                                                    else "40/40/20 % of 2/4/8 bits"),
                        "paper_table_4_us": paper_us[(kind, T)],
                        "note": "one call of sb_dequant_gemm (two launches); packed codes + scale / minimum "
                                "metadata + activations read, outputs written; the paper's figure is its own "
                                "kernel on its own GPU: context, not a comparison on equal hardware"})
        del sets
    return out


def full_model_times(ctx, dev, ctx2=None):
    """configs[2]: 32 layers of the 8B shape searched as ONE model (residual-stream permutation
    shared by all layers, one global allocation over N = 425,984 blocks per budget), budgets
    2.0 ... 4.0.  Returns the CUDA-event time of the library calls only (the synthetic layers
    are generated between them); weights stay resident (13.96 GB), activations are regenerated
    per layer."""
    from paper_2602_17698_b200 import synth
    from paper_2602_17698_b200.pipeline import SearchConfig, search_model
    shape = synth.LLAMA3_8B

    def make_weights(layer):
        W = synth.make_layer_weights(shape, SEED, layer, dev)
        if layer in FULL_MODEL_SUPER:
            synth.inject_super_weights(W["down_proj"], FULL_MODEL_SUPER[layer], 1)
        return W

    def make_acts(layer):
        return synth.make_layer_activations(shape, TOKENS, SEED, layer, dev)

    cfg = SearchConfig(bits=BITS)
    # untimed warm-up on four layers: grows the library's scratch arena to its steady-state size
    # and loads the kernels that only large tables use (the cooperative form of the loop kernel)
    search_model(ctx, shape, 4, cfg, (2.25,), make_weights, make_acts, dev, keep_tables=False, ctx2=ctx2)
    res = search_model(ctx, shape, FULL_MODEL_LAYERS, cfg, FULL_MODEL_BUDGETS, make_weights, make_acts, dev,
                       keep_tables=False, alloc_repeats=2, ctx2=ctx2)
    ms = res.ms
    sweeps = sorted({int(k.split("@")[1]) for k in ms if k.startswith("stats@")})
    first = FULL_MODEL_BUDGETS[0]
    rb0 = sweeps[0]
    alloc = {f"{b:g}": ms[f"allocate@{b:g}"] for b in FULL_MODEL_BUDGETS}
    one_budget = ms["moments"] + ms[f"stats@{rb0}"] + ms[f"sort@{rb0}"] + ms[f"scores@{rb0}"] + alloc[f"{first:g}"]
    for b in FULL_MODEL_BUDGETS:
        r = res.reports[b]
        assert r["used_bits"] <= r["cap_bits"], (b, r)
    return {"workload": f"{FULL_MODEL_LAYERS} layers of the 8B shape searched as one model, "
                        f"{TOKENS} tokens per input, {res.n_blocks} blocks, bits {list(BITS)}, "
                        f"4 injected super weights, budgets 2.0-4.0 step 0.25",
            "n_blocks": res.n_blocks, "weights": FULL_MODEL_LAYERS * shape.n_weights,
            "ms_first_budget_total": one_budget,
            "ms_moments": ms["moments"],
            "ms_per_warm_start": {str(rb): {"reorder_stats": ms[f"stats@{rb}"], "sort": ms[f"sort@{rb}"],
                                            "scores": ms[f"scores@{rb}"]} for rb in sweeps},
            "ms_allocate_per_budget": alloc,
            "iterations_per_budget": {f"{b:g}": res.reports[b]["iterations"] for b in FULL_MODEL_BUDGETS},
            "ms_all_budgets_total": sum(ms.values()),
            "timing": "sum of CUDA-event times around the library calls; each allocation call is "
                      "made twice and the faster one counted (it is eager and paced by the host)"}


def small_layer_times(ctx, dev):
    """configs[0]: one 2048 x 2048 layer, 8192 calibration tokens, blocks 128 x 128, bits {2,3,4},
    budget 3.0, no coupling (rows and columns sorted freely): the whole path per call, CUDA events,
    20 repetitions after 3 warm-up passes.  2048 x 2048 weights (8 MB) and 8192 x 2048 activations
    (33.5 MB) fit in L2, so a buffer larger than L2 is written between repetitions."""
    import torch
    from paper_2602_17698_b200 import synth
    R = Cc = 2048
    T, bits, budget = 8192, (2, 3, 4), 3.0
    W = synth.make_weight(R, Cc, synth.tensor_seed(SEED, 0, 1), dev)
    X = synth.make_activations(T, Cc, synth.tensor_seed(SEED, 0, 2), dev)
    f32 = dict(dtype=torch.float32, device=dev)
    nb = (R // 128) * (Cc // 128)
    c, rs, cs = torch.empty(Cc, **f32), torch.empty(R, **f32), torch.empty(Cc, **f32)
    pr = torch.empty(R, dtype=torch.int32, device=dev)
    pc = torch.empty(Cc, dtype=torch.int32, device=dev)
    err, wp = torch.empty(nb, len(bits), **f32), torch.empty_like(W)
    packed = torch.empty(R * Cc * max(bits) // 32, dtype=torch.int32, device=dev)
    off, meta = torch.empty(nb + 1, dtype=torch.int64, device=dev), torch.empty((R * Cc // 128, 2), **f32)
    flush = torch.empty(160 * 1024 * 1024, dtype=torch.uint8, device=dev)
    rep = {}

    def once():
        ctx.calib_moments(X, c)
        ctx.reorder_channels(W, c, 3, 128, row_score=rs, col_score=cs, row_segment=R, col_segment=Cc,
                             row_perm=pr, col_perm=pc)
        ctx.block_scores(W, c, bits, 128, 128, 128, row_perm=pr, col_perm=pc, err=err, want_gain=False,
                         W_perm_out=wp)
        level, r = ctx.allocate_bits(err, bits, budget, uniform_block_elems=128 * 128)
        ctx.pack_blocks(wp, bits, level, 128, 128, 128, packed=packed, block_off=off, meta=meta)
        rep.update(r)

    for _ in range(3):
        once()
    total = 0.0
    reps = 20
    for _ in range(reps):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        once()
        b.record()
        b.synchronize()
        total += a.elapsed_time(b)
    ms = total / reps
    return {"workload": "configs[0]: W 2048 x 2048, X 8192 x 2048, blocks 128 x 128, bits {2,3,4}, group 128, "
                        "budget 3.0, free row and column sort",
            "ms_per_pass": ms, "elements_per_s": R * Cc / (ms * 1e-3), "allocation": dict(rep),
            "timing": "CUDA events around the five library calls (eager launches, one host synchronisation in "
                      "the allocation), mean of 20 passes, L2 flushed between passes"}


def streamed_model_times(ctx, dev, ctx2=None):
    """configs[3]: 80 layers of the 70B shape (68.5 G weights, N = 4,177,920 blocks), bits {2,3,4},
    budget 2.25.  Weights and activations are made again from their seeds in every sweep (the
    model is never resident: 136.9 GB of weights); only moments, score vectors, permutations and
    the table persist.  CUDA-event time of the library calls only."""
    from paper_2602_17698_b200 import synth
    from paper_2602_17698_b200.pipeline import SearchConfig, search_model
    shape, n_layers, tokens, bits, budget = synth.LLAMA3_70B, 80, 16384, (2, 3, 4), 2.25
    cfg = SearchConfig(bits=bits)
    t0 = time.time()
    res = search_model(ctx, shape, n_layers, cfg, (budget,),
                       lambda layer: synth.make_layer_weights(shape, SEED, layer, dev),
                       lambda layer: synth.make_layer_activations(shape, tokens, SEED, layer, dev), dev,
                       keep_tables=False, keep_weights=False, alloc_repeats=2, ctx2=ctx2)
    wall = time.time() - t0
    ms = res.ms
    r = res.reports[budget]
    assert r["used_bits"] <= r["cap_bits"]
    n_w = n_layers * shape.n_weights
    return {"workload": f"configs[3]: {n_layers} layers of the 70B shape ({n_w} weights, {res.n_blocks} blocks), "
                        f"{tokens} tokens per input, bits {list(bits)}, budget {budget}, streamed layer by layer",
            "ms_library_calls_total": sum(ms.values()),
            "ms": {"moments": ms["moments"], "reorder_stats": ms["stats@2"], "sort": ms["sort@2"],
                   "scores": ms["scores@2"], "allocate": ms[f"allocate@{budget:g}"]},
            "iterations": r["iterations"], "used_bits": r["used_bits"], "cap_bits": r["cap_bits"],
            "scoring_elements_per_s": n_w / (ms["scores@2"] * 1e-3),
            "wall_seconds_including_regeneration": wall,
            "timing": "sum of CUDA-event times around the library calls; inside the timed calls: nothing but the "
                      "library; outside: the synthetic layers (weights made twice, once per sweep; activations "
                      "once) and their release"}


def full_model_e2e(ctx, dev, ctx2=None):
    """configs[2] end to end for one budget: the weights of every layer come from pinned host memory
    (13.96 GB, copied once, then resident for the second sweep), the activations of every layer are
    copied from pinned host buffers as well (3.49 GB per layer; one set of host buffers serves all
    layers, so the bytes are real and the values repeat), the levels go back to the host.  Wall
    clock around the whole search after a device synchronisation on both sides."""
    import torch
    from paper_2602_17698_b200 import synth
    from paper_2602_17698_b200.pipeline import SearchConfig, search_model
    shape = synth.LLAMA3_8B
    hW = []
    for layer in range(FULL_MODEL_LAYERS):
        W = synth.make_layer_weights(shape, SEED, layer, dev)
        hW.append({n: torch.empty(w.shape, dtype=w.dtype, pin_memory=True).copy_(w) for n, w in W.items()})
        del W
    X0 = synth.make_layer_activations(shape, TOKENS, SEED, 0, dev)
    hX = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for n, x in X0.items()}
    del X0
    torch.cuda.synchronize()
    h2d = sum(w.numel() * 2 for lw in hW for w in lw.values()) + FULL_MODEL_LAYERS * sum(x.numel() * 2 for x in hX.values())
    budget = 2.5

    def make_weights(layer):
        return {n: w.to(dev, non_blocking=True) for n, w in hW[layer].items()}

    def make_acts(layer):
        return {n: x.to(dev, non_blocking=True) for n, x in hX.items()}

    cfg = SearchConfig(bits=BITS)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    res = search_model(ctx, shape, FULL_MODEL_LAYERS, cfg, (budget,), make_weights, make_acts, dev,
                       keep_tables=False, ctx2=ctx2)
    level_h = res.levels[budget].cpu()
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    n_w = FULL_MODEL_LAYERS * shape.n_weights
    return {"value": n_w / sec, "unit": UNIT, "seconds": sec, "h2d_bytes": h2d, "d2h_bytes": level_h.numel(),
            "h2d_gbs": h2d / sec / 1e9,
            "note": "configs[2], one budget (2.5), weights and activations from pinned host memory, levels back "
                    "to the host; bound by the host-to-device copies"}


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2602_17698_b200 import synth
    from paper_2602_17698_b200.binding import Context
    from paper_2602_17698_b200.pipeline import LayerWorkspace, SearchConfig, StageGraphs, search_layer

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    shape = synth.LLAMA3_8B
    cfg = SearchConfig(bits=BITS, budget=BUDGET)
    # replicas: every rank searches its own layer (layer index = rank), no data-path collective
    W = synth.make_layer_weights(shape, SEED, rank, dev)
    X = synth.make_layer_activations(shape, TOKENS, SEED, rank, dev)
    # the library works on one non-default stream, so that its stages can be captured into
    # CUDA graphs (fixed pointers: the workspace and the inputs) and replayed without host gaps
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize()
    torch.cuda.set_stream(stream)
    ctx = Context()
    # more contexts, each on a stream of its own: the stages whose matrices are independent (block
    # scores, pack) deal them to the contexts in turn (pipeline.search_layer)
    n_extra = 0 if args.one_stream else max(args.streams, 1) - 1
    ctx2 = [Context(stream=torch.cuda.Stream(device=dev)) for _ in range(n_extra)] or None
    ws = LayerWorkspace(shape, cfg, dev)
    # the timed step is ONE CUDA graph (moments ... pack, the allocation in its enqueue-only form);
    # a second pass below replays one graph per stage for the per-stage times
    graphs = None if args.no_graphs else StageGraphs(ctx, ctx2, whole=not args.stage_graphs)
    n_weights = shape.n_weights
    in_bytes = sum(w.numel() * 2 for w in W.values()) + sum(x.numel() * 2 for x in X.values())

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step(timers=None):
        return search_layer(ctx, W, X, ws, timers=timers, graphs=graphs, ctx2=ctx2)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    sampler = None
    if rank == 0:
        sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid))
        sampler.start()
        time.sleep(0.15)
    timers = {s: [] for s in STAGES}
    def launched():
        return (ctx.kernel_launches() + sum(c.kernel_launches() for c in ctx2 or [])
                + (graphs.replayed_kernels if graphs else 0))

    l0 = launched()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    e0.record()
    for _ in range(args.steps):
        res = step(timers)
    e1.record()
    barrier()
    t_wall1 = time.time()
    launches = launched() - l0
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms = max_over_ranks(ms, world, dev)
    ms_per_step = ms / args.steps
    value = job_throughput(n_weights, world, ms_per_step)

    res.read_report()
    ctx.sync()                                       # device-side status of everything replayed so far
    for c in ctx2 or []:
        c.sync()
    stagewise_ms = None
    if graphs is not None and graphs.whole:
        # per-stage times: the same steps again, one graph per stage with events between the stages
        # (the allocation eager and synchronous); this pass also times the roofline kernel
        timers = {s: [] for s in STAGES}
        stage_graphs = StageGraphs(ctx, ctx2)
        for _ in range(3):
            search_layer(ctx, W, X, ws, graphs=stage_graphs, ctx2=ctx2)
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(args.steps):
            search_layer(ctx, W, X, ws, timers=timers, graphs=stage_graphs, ctx2=ctx2)
        s1.record()
        barrier()
        stagewise_ms = s0.elapsed_time(s1) / args.steps
    stage_ms = {s: sum(a.elapsed_time(b) for a, b in timers[s]) / args.steps for s in STAGES}
    stage_launch_ms = {s: (sum(a.elapsed_time(b) for a, b in timers[s]) / max(len(timers[s]), 1))
                       for s in STAGES}

    # ---- end to end: pinned host inputs -> device every step, result back to the host --------
    e2e = None
    hW = hX = None
    if not args.no_e2e:
        hW = {n: torch.empty(w.shape, dtype=w.dtype, pin_memory=True).copy_(w) for n, w in W.items()}
        hX = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for n, x in X.items()}
        h_level = torch.empty(ws.n_blocks, dtype=torch.uint8, pin_memory=True)
        h_packed = {n: tuple(torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in ws.packed[n])
                    for n in ws.packed}
        d2h = h_level.numel() + sum(t.numel() * t.element_size() for tup in h_packed.values() for t in tup)

        # Three streams: the inputs of step i + 1 arrive (into a second set of device buffers)
        # while step i computes and while the results of step i - 1 leave (PCIe carries both
        # directions at once).  A step's kernels wait for their inputs and until the previous
        # step's results have left the output buffers; a set of input buffers is refilled only
        # after the step that read it has finished.
        in_stream = torch.cuda.Stream(device=dev)
        out_stream = torch.cuda.Stream(device=dev)
        W2 = {n: torch.empty_like(w) for n, w in W.items()}
        X2 = {n: torch.empty_like(x) for n, x in X.items()}
        graphs2 = None if graphs is None else StageGraphs(ctx, ctx2, whole=graphs.whole)
        sets = [(W, X, graphs), (W2, X2, graphs2)]
        inputs_read = [None, None]
        results_left = [None]

        def e2e_step(i):
            Wk, Xk, gk = sets[i & 1]
            with torch.cuda.stream(in_stream):
                if inputs_read[i & 1] is not None:
                    in_stream.wait_event(inputs_read[i & 1])
                for n in Wk:
                    Wk[n].copy_(hW[n], non_blocking=True)
                for n in Xk:
                    Xk[n].copy_(hX[n], non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(in_stream)
            stream.wait_event(arrived)
            if results_left[0] is not None:
                stream.wait_event(results_left[0])
            r = search_layer(ctx, Wk, Xk, ws, graphs=gk, ctx2=ctx2)
            computed = torch.cuda.Event()
            computed.record(stream)
            inputs_read[i & 1] = computed
            out_stream.wait_event(computed)
            with torch.cuda.stream(out_stream):
                h_level.copy_(r.level, non_blocking=True)
                for n, tup in r.packed.items():
                    for dst, src in zip(h_packed[n], tup):
                        dst.copy_(src, non_blocking=True)
                results_left[0] = torch.cuda.Event()
                results_left[0].record(out_stream)

        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        e2e_step(0)
        e2e_step(1)                                  # both sets of buffers (and their graphs) are warm
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        in_stream.wait_event(a)                      # no input copy starts before the clock does
        for i in range(e2e_steps):
            e2e_step(i)
        stream.wait_event(results_left[0])           # the last step's results are on the host
        b.record()
        barrier()
        del sets, W2, X2, graphs2
        e2e_ms = max_over_ranks(a.elapsed_time(b), world, dev) / e2e_steps
        e2e = {"value": job_throughput(n_weights, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": d2h}

    if rank == 0:
        peak, peak_kind = measured_peaks()
        # dominant kernel by time: the calibration-moments reduction (3.49 GB read per step)
        mom_bytes = sum(x.numel() * 2 for x in X.values())
        mom_launches = len(X)          # one kernel per input; the stage's events bracket all four
        achieved = mom_bytes / (stage_ms["moments"] * 1e-3) / 1e9
        traffic = NCU_TRAFFIC_RATIO["moments_partial_kernel"] * mom_bytes / mom_launches
        roofline = {"kernel": "moments_partial_kernel", "bound": "hbm", "achieved": achieved, "peak": peak,
                    "unit": "GB/s", "frac": achieved / peak, "frac_nominal": achieved / NOMINAL_HBM_GBS,
                    "peak_source": peak_kind + " copy bandwidth",
                    "traffic": traffic, "algorithmic_bytes_per_launch": mom_bytes / mom_launches,
                    "launches_per_step": mom_launches, "avg_launch_ms": stage_ms["moments"] / mom_launches,
                    "timing": "CUDA events around the stage's %d launches (one per distinct input%s): stage bytes / "
                              "stage time" % (mom_launches, "" if ctx2 is None else
                                              ", dealt to %d streams, so consecutive launches overlap at their "
                                              "ends" % min(len(ctx2) + 1, mom_launches))}
        w_bytes = 2 * n_weights
        stage_gbs = {"moments": achieved,
                     "reorder_stats": w_bytes / (stage_ms["reorder_stats"] * 1e-3) / 1e9,
                     "scores": w_bytes / (stage_ms["scores"] * 1e-3) / 1e9,
                     "pack": w_bytes / (stage_ms["pack"] * 1e-3) / 1e9}
        sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
        sm_count = torch.cuda.get_device_properties(local).multi_processor_count
        kernels = kernel_rooflines(ctx, W, X, ws.moments, dev, peak, sm_mhz, sm_count)
        if world == 1:
            kernels += dequant_gemm_times(ctx, dev, peak)
        full_model = small_layer = streamed = None
        if world == 1 and not args.no_full_model:
            del hW, hX                                   # pinned copies of the layer, if any
            small_layer = small_layer_times(ctx, dev)
            del W, X                                     # the layer's tensors: the models need the room
            full_model = full_model_times(ctx, dev, ctx2)
            full_model["e2e"] = full_model_e2e(ctx, dev, ctx2)
            streamed = streamed_model_times(ctx, dev, ctx2)
        cpu = None
        if not args.no_cpu_baseline:
            v, sec, cores, sample = time_oracle(3, 0)
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                   "seconds": sec, "full_size_matrix": oracle_full_matrix()}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": WORKLOAD, "tokens": TOKENS, "bits": list(BITS), "budget": BUDGET,
                           "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                           "l2": "inputs (3.9 GB per step) larger than L2, no flush needed",
                           "hbm_target": "fractions of the measured copy bandwidth (frac) and of the nominal "
                                         "8000 GB/s (frac_nominal): the 70 % target is stated on the nominal figure",
                           "launch": ("eager" if graphs is None else
                                      "one CUDA graph per step (allocation enqueued, report left on the device)"
                                      if graphs.whole else "one CUDA graph per stage (allocation eager)")
                                     + ("" if ctx2 is None else
                                        "; the matrices of the block-score and pack stages dealt to %d streams"
                                        % (len(ctx2) + 1)),
                           "allocation": res.read_report()},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
                "roofline": roofline, "cpu_baseline": cpu,
                "stages_ms_per_step": stage_ms, "stages_algorithmic_gbs": stage_gbs,
                "stages_timing": ("CUDA events between the stages of the timed steps" if stagewise_ms is None else
                                  "a second timed pass of the same steps with one CUDA graph per stage, events "
                                  "between the stages and the synchronous allocation: %.4f ms per step; the "
                                  "roofline kernel's launch time is taken there" % stagewise_ms),
                "ms_per_step_stagewise": stagewise_ms,
                "scoring_elements_per_s": n_weights / (stage_ms["scores"] * 1e-3),
                "roofline_other_kernels": kernels, "small_layer": small_layer, "full_model": full_model,
                "streamed_model": streamed}
        print(json.dumps(line), flush=True)
    for c in ctx2 or []:
        c.sync()
        c.close()
    ctx.close()
    if world > 1:
        dist.barrier()              # rank 0 may still have been timing its extra legs
        dist.destroy_process_group()


def run_only(which: str):
    """A few calls of ONE library call on one input of the layer (for ncu captures: small, a
    few launches, larger than L2): moments on a 65536 x 4096 input, the others on a
    14336 x 4096 matrix."""
    import torch
    from paper_2602_17698_b200 import synth
    from paper_2602_17698_b200.binding import Context
    torch.cuda.set_device(0)
    torch.manual_seed(0)
    dev = "cuda:0"
    ctx = Context()
    R, Cc = 14336, 4096
    c = torch.rand(Cc, device=dev) + 0.5
    if which == "moments":
        X = synth.make_activations(TOKENS, 4096, 7, dev)
        for _ in range(3):
            ctx.calib_moments(X)
    elif which == "gram":
        X = synth.make_activations(32768, 2048, 7, dev)           # 134 MB, 136 tiles of 128 x 128
        H = torch.empty((2048, 2048), device=dev)
        for _ in range(3):
            ctx.calib_gram(X, H=H)
    else:
        W = synth.make_weight(R, Cc, 100, dev)
        nb = (R // 128) * (Cc // 128)
        if which == "scores":
            err = torch.empty(nb, len(BITS), device=dev)
            for _ in range(3):
                ctx.block_scores(W, c, BITS, 128, 128, 128, err=err, want_gain=False)
        elif which == "reorder_stats":
            rs, cs = torch.empty(R, device=dev), torch.empty(Cc, device=dev)
            for _ in range(3):
                ctx.reorder_channels(W, c, 2, 128, row_score=rs, col_score=cs)
        elif which == "reorder_stats_first_order":
            G = (W.float() * 1e-2).to(torch.bfloat16)
            rs, cs = torch.empty(R, device=dev), torch.empty(Cc, device=dev)
            for _ in range(3):
                ctx.reorder_channels_first_order(W, G, 2, 128, row_score=rs, col_score=cs)
        elif which == "gather":
            pr, pc = torch.randperm(R, device=dev).int(), torch.randperm(Cc, device=dev).int()
            err, out = torch.empty(nb, len(BITS), device=dev), torch.empty_like(W)
            for _ in range(3):
                ctx.block_scores(W, c, BITS, 128, 128, 128, row_perm=pr, col_perm=pc, err=err,
                                 want_gain=False, W_perm_out=out)
        elif which == "full_scores":
            Xs = synth.make_activations(8192, Cc, 7, dev)
            H = ctx.calib_gram(Xs)
            err = torch.empty(nb, len(BITS), device=dev)
            for _ in range(3):
                ctx.block_scores_full(W, H, BITS, 128, 128, 128, err=err, want_gain=False)
        elif which == "dequant_gemm":
            import numpy as np
            Rq = Cq = 8192
            nbq = (Rq // 128) * (Cq // 128)
            Wq = synth.make_weight(Rq, Cq, 4242, dev)
            sets = []
            for k in range(5):                           # 180 MB of packed copies: larger than L2
                lv = torch.from_numpy(synth.table4_levels(nbq, 100 + k)).to(dev)
                sets.append(ctx.pack_blocks(Wq, [2, 4, 8], lv, 128, 128, 128) + (lv,))
            Xq = synth.make_activations(32, Cq, 109, dev)
            for pk, off, meta, lv in sets:
                ctx.dequant_gemm(Xq, pk, off, meta, lv, Rq, Cq, [2, 4, 8])
        elif which == "pack":
            level = torch.randint(0, len(BITS), (nb,), device=dev, dtype=torch.uint8)
            for _ in range(3):
                ctx.pack_blocks(W, BITS, level, 128, 128, 128)
        elif which == "scores3":
            err = torch.empty(nb, 3, device=dev)
            for _ in range(3):
                ctx.block_scores(W, c, (2, 3, 4), 128, 128, 128, err=err, want_gain=False)
        elif which == "scores7":
            err = torch.empty(nb, 7, device=dev)
            for _ in range(3):
                ctx.block_scores(W, c, STRESS_BITS, 128, 128, 128, err=err, want_gain=False)
        elif which == "first_order":
            G = (W.float() * 1e-2).to(torch.bfloat16)
            level = torch.randint(0, len(BITS), (nb,), device=dev, dtype=torch.uint8)
            for _ in range(3):
                ctx.first_order_scores(W, G, BITS, level, 128, 128, 128, want_l1=False)
        elif which == "sort":
            score = torch.rand(R, device=dev)
            perm = torch.empty(R, dtype=torch.int32, device=dev)
            for _ in range(3):
                ctx.reorder_channels(None, None, 2, 128, row_score=score, row_segment=R, row_perm=perm,
                                     shape=(R, 128))
        elif which in ("allocate", "allocate_model"):
            # the layer's table (13,312 blocks: one cluster sort, the masked loop kernel) or the
            # model's (425,984 blocks: multi-launch sort, cooperative loop kernel)
            N = 13312 if which == "allocate" else 425984
            table = (torch.rand(N, 1, device=dev) * 30 + 1) * (0.4 ** torch.arange(len(BITS), device=dev))[None, :] \
                * (torch.rand(N, len(BITS), device=dev) * 1.3 + 0.5)
            table = table.float().contiguous()
            for _ in range(3):
                ctx.allocate_bits(table, BITS, BUDGET)
        else:
            raise SystemExit(f"unknown stage {which}")
    ctx.sync()
    ctx.close()
    print("done", which)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-full-model", action="store_true",
                    help="skip the 32-layer global-allocation timing (single GPU only)")
    ap.add_argument("--no-graphs", action="store_true", help="launch every library call eagerly")
    ap.add_argument("--stage-graphs", action="store_true",
                    help="time the step as one CUDA graph per stage with an eager, synchronous allocation "
                         "instead of one graph for the whole step")
    ap.add_argument("--streams", type=int, default=7,
                    help="contexts (streams) the independent matrices of the block-score and pack stages are "
                         "dealt to (default 7: one per matrix of the layer)")
    ap.add_argument("--one-stream", action="store_true",
                    help="one context only (no dealing of a stage's independent calls to extra streams)")
    ap.add_argument("--only", default=None,
                    help="three calls of one library call on one input, then exit (for ncu captures): "
                         "moments | gram | full_scores | dequant_gemm | reorder_stats | reorder_stats_first_order | scores | scores3 | scores7 | "
                         "gather | pack | first_order | sort | allocate | allocate_model")
    args = ap.parse_args()
    if args.only:
        run_only(args.only)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
