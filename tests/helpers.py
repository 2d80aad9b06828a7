"""Test helpers: the oracle-side sequence for one decoder layer and comparison utilities."""
from __future__ import annotations

import numpy as np

from oracle import sbo

REL = 1e-4          # per-block errors / gains / scores: fp32 accumulation vs fp64 (the benchmark spec)
REL_MOMENT = 1e-5   # calibration moments


def assert_close(gpu, ref, rel=REL, abs_floor=0.0, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    tol = rel * np.abs(ref) + abs_floor
    bad = np.abs(gpu - ref) > tol
    if bad.any():
        i = np.argmax(np.abs(gpu - ref) / (np.abs(ref) + abs_floor + 1e-300))
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} off; worst at {np.unravel_index(i, ref.shape)}: "
                             f"gpu {gpu.flat[i]!r} ref {ref.flat[i]!r}")


COUPLING = {
    "q_proj": (None, "hidden"), "k_proj": (None, "hidden"), "v_proj": ("v_heads", "hidden"),
    "o_proj": ("hidden", "o_heads"), "gate_proj": ("intermediate", "hidden"),
    "up_proj": ("intermediate", "hidden"), "down_proj": ("hidden", "intermediate"),
}


def oracle_layer_scores(shape, weights, moments, ref_bits, group):
    """Channel scores of each coupled set (Appendix D), from the oracle's per-matrix sums."""
    lin = {l.name: l for l in shape.linears}
    rs, cs = {}, {}
    for name, l in lin.items():
        rs[name], cs[name] = sbo.reorder_scores(weights[name], moments[l.act], ref_bits=ref_bits, group=group)
    hidden = (cs["q_proj"] + cs["k_proj"] + cs["v_proj"] + rs["o_proj"] + cs["gate_proj"]
              + cs["up_proj"] + rs["down_proj"])
    inter = rs["gate_proj"] + rs["up_proj"] + cs["down_proj"]
    v_heads = rs["v_proj"].copy()
    reps = shape.n_heads // shape.n_kv_heads
    sbo.fold_segment_scores(v_heads, cs["o_proj"], reps, shape.head_dim)
    return {"hidden": hidden, "intermediate": inter, "v_heads": v_heads, "o_cols": cs["o_proj"]}


def oracle_layer_perms(shape, scores):
    reps = shape.n_heads // shape.n_kv_heads
    p_v = sbo.argsort_desc_segments(scores["v_heads"], shape.head_dim)
    return {"hidden": sbo.argsort_desc_segments(scores["hidden"]),
            "intermediate": sbo.argsort_desc_segments(scores["intermediate"]),
            "v_heads": p_v, "o_heads": sbo.expand_segment_perm(p_v, reps, shape.head_dim)}


def unpack_block(words: np.ndarray, n: int, b: int) -> np.ndarray:
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")
    return (bits[: n * b].reshape(n, b).astype(np.int64) << np.arange(b)).sum(1)
