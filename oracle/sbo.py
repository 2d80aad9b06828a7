"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only tests/, the smoke check and the benchmark's cpu_baseline / reference legs
may import this module.  It compiles oracle/scalebits_oracle.c with gcc on first
use and exposes numpy-in / numpy-out wrappers with the oracle's own names.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scalebits_oracle.c")
_LIB = os.path.join(_HERE, "libsbo.so")

OK, ERR_INVALID, ERR_SHAPE, ERR_BUDGET, ERR_NOCONVERGE, ERR_NONFINITE = 0, 1, 2, 3, 6, 7


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, fp64, no contraction of a*b+c into an FMA)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class AllocReport(C.Structure):
    _fields_ = [("cap_bits", C.c_int64), ("used_bits", C.c_int64),
                ("iterations", C.c_int32), ("accepted", C.c_int32),
                ("rejected", C.c_int32), ("expansions", C.c_int32),
                ("proxy_loss_init", C.c_double), ("proxy_loss_final", C.c_double),
                ("level_hist", C.c_int64 * 8), ("min_margin", C.c_double)]

    def as_dict(self):
        return {"cap_bits": self.cap_bits, "used_bits": self.used_bits,
                "iterations": self.iterations, "accepted": self.accepted,
                "rejected": self.rejected, "expansions": self.expansions,
                "proxy_loss_init": self.proxy_loss_init,
                "proxy_loss_final": self.proxy_loss_final,
                "level_hist": list(self.level_hist), "min_margin": self.min_margin}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.sbo_bf16_to_f64.restype = C.c_double
        _lib.sbo_bf16_to_f64.argtypes = [C.c_uint16]
        _lib.sbo_num_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(x) -> np.ndarray:
    """bf16 bit patterns as a C-contiguous 2-D uint16 array (torch bf16 tensors accepted)."""
    if hasattr(x, "dtype") and str(x.dtype) == "torch.bfloat16":
        import torch
        x = x.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
    x = np.ascontiguousarray(x)
    assert x.dtype == np.uint16
    return x


def _f64(x, n=None) -> Optional[np.ndarray]:
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    x = np.ascontiguousarray(x, dtype=np.float64)
    if n is not None:
        assert x.size == n, (x.size, n)
    return x


def _i32(x) -> Optional[np.ndarray]:
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _bits(bits: Sequence[int]):
    arr = (C.c_int * len(bits))(*[int(b) for b in bits])
    return arr, len(bits)


def num_threads() -> int:
    return int(lib().sbo_num_threads())


def bf16_to_f64(h: int) -> float:
    return float(lib().sbo_bf16_to_f64(int(h)))


def bf16_array_to_f64(bits_u16: np.ndarray) -> np.ndarray:
    """Vectorised exact decode (numpy bit manipulation; pinned against sbo_bf16_to_f64)."""
    u = bits_u16.astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def calib_moments(X, scale: float = 1.0, out: Optional[np.ndarray] = None) -> np.ndarray:
    X = _u16(X)
    T, K = X.shape
    acc = out is not None
    if out is None:
        out = np.zeros(K, dtype=np.float64)
    lib().sbo_calib_moments(_p(X), C.c_int64(T), C.c_int64(K), C.c_int64(K),
                            C.c_double(scale), C.c_int(int(acc)), _p(out))
    return out


def quantize_group(v: np.ndarray, bits: int):
    """-> (codes int32[g], vhat f64[g], scale, lo)"""
    v = np.ascontiguousarray(v, dtype=np.float64)
    g = v.size
    code = np.zeros(g, dtype=np.int32)
    vhat = np.zeros(g, dtype=np.float64)
    scale = C.c_double(0)
    lo = C.c_double(0)
    st = lib().sbo_quantize_group(_p(v), C.c_int(g), C.c_int(bits), _p(code), _p(vhat),
                                  C.byref(scale), C.byref(lo))
    assert st == OK, st
    return code, vhat, scale.value, lo.value


def reorder_scores(W, c, a=None, ref_bits: int = 3, group: int = 128,
                   row_score: Optional[np.ndarray] = None, col_score: Optional[np.ndarray] = None,
                   accumulate: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    W = _u16(W)
    R, Cc = W.shape
    c = _f64(c, Cc)
    a = _f64(a, R) if a is not None else None
    if row_score is None:
        row_score = np.zeros(R, dtype=np.float64)
    if col_score is None:
        col_score = np.zeros(Cc, dtype=np.float64)
    st = lib().sbo_reorder_scores(_p(W), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc), _p(c), _p(a),
                                  C.c_int(ref_bits), C.c_int(group), _p(row_score), _p(col_score),
                                  C.c_int(int(accumulate)))
    assert st == OK, st
    return row_score, col_score


def argsort_desc_segments(score, segment: Optional[int] = None) -> np.ndarray:
    score = _f64(score)
    K = score.size
    seg = K if not segment else segment
    perm = np.zeros(K, dtype=np.int32)
    st = lib().sbo_argsort_desc_segments(_p(score), C.c_int64(K), C.c_int64(seg), _p(perm))
    assert st == OK, st
    return perm


def fold_segment_scores(dst: np.ndarray, src, reps: int, seg: int) -> np.ndarray:
    src = _f64(src)
    assert dst.dtype == np.float64 and dst.size * reps == src.size
    lib().sbo_fold_segment_scores(_p(dst), _p(src), C.c_int64(dst.size), C.c_int(reps), C.c_int64(seg))
    return dst


def expand_segment_perm(perm, reps: int, seg: int) -> np.ndarray:
    perm = _i32(perm)
    out = np.zeros(perm.size * reps, dtype=np.int32)
    lib().sbo_expand_segment_perm(_p(out), _p(perm), C.c_int64(perm.size), C.c_int(reps), C.c_int64(seg))
    return out


def block_scores(W, c, bits: Sequence[int], block_rows: int = 128, block_cols: int = 128,
                 group: int = 128, row_perm=None, col_perm=None, a=None):
    """-> (err f64[nb, L], gain f64[nb, L-1])"""
    W = _u16(W)
    R, Cc = W.shape
    c = _f64(c, Cc)
    a = _f64(a, R) if a is not None else None
    rp, cp = _i32(row_perm), _i32(col_perm)
    barr, L = _bits(bits)
    nb = (R // block_rows) * (Cc // block_cols)
    err = np.zeros((nb, L), dtype=np.float64)
    gain = np.zeros((nb, max(L - 1, 1)), dtype=np.float64)
    st = lib().sbo_block_scores(_p(W), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc), _p(rp), _p(cp),
                                _p(c), _p(a), C.c_int(block_rows), C.c_int(block_cols),
                                C.c_int(group), barr, C.c_int(L), _p(err), _p(gain))
    if st != OK:
        raise ValueError(f"sbo_block_scores status {st}")
    return err, gain[:, :L - 1]


def _alloc(fn, err, bits, budget, block_elems, uniform_block_elems, extra=(), tail=()):
    err = _f64(err)
    N, L = err.shape
    barr, Lb = _bits(bits)
    assert L == Lb
    be = None if block_elems is None else np.ascontiguousarray(block_elems, dtype=np.int64)
    level = np.zeros(N, dtype=np.uint8)
    rep = AllocReport()
    st = fn(_p(err), C.c_int64(N), _p(be), C.c_int64(uniform_block_elems), barr, C.c_int(L),
            C.c_double(budget), *extra, _p(level), C.byref(rep), *tail)
    return int(st), level, rep.as_dict()


def allocate_greedy(err, bits, budget, uniform_block_elems=128 * 128, block_elems=None, heap=False):
    fn = lib().sbo_allocate_greedy_heap if heap else lib().sbo_allocate_greedy
    return _alloc(fn, err, bits, budget, block_elems, uniform_block_elems)


def allocate_scalebits(err, bits, budget, gamma0=0.05, gammaT=0.02, uniform_block_elems=128 * 128,
                       block_elems=None):
    return _alloc(lib().sbo_allocate_scalebits, err, bits, budget, block_elems, uniform_block_elems,
                  extra=(C.c_double(gamma0), C.c_double(gammaT)))


def allocate_scalebits_trace(err, bits, budget, gamma0=0.05, gammaT=0.02, uniform_block_elems=128 * 128,
                             block_elems=None, max_iters=64):
    """allocate_scalebits plus the level vector after every iteration -> (status, level, report,
    trace[iterations][N])."""
    err = _f64(err)
    N = err.shape[0]
    trace = np.zeros((max_iters, N), dtype=np.uint8)
    st, level, rep = _alloc(lib().sbo_allocate_scalebits_trace, err, bits, budget, block_elems,
                            uniform_block_elems, extra=(C.c_double(gamma0), C.c_double(gammaT)),
                            tail=(_p(trace), C.c_int64(max_iters)))
    return st, level, rep, trace[:min(max_iters, rep["iterations"])]


def pack_blocks(W, bits: Sequence[int], level, block_rows=128, block_cols=128, group=128,
                row_perm=None, col_perm=None):
    """-> (packed uint32[words], block_off int64[nb+1], meta f32[R*C/group, 2])"""
    W = _u16(W)
    R, Cc = W.shape
    rp, cp = _i32(row_perm), _i32(col_perm)
    barr, L = _bits(bits)
    level = np.ascontiguousarray(level, dtype=np.uint8)
    nb = (R // block_rows) * (Cc // block_cols)
    assert level.size == nb
    cap = R * Cc * max(bits) // 32
    packed = np.zeros(cap, dtype=np.uint32)
    off = np.zeros(nb + 1, dtype=np.int64)
    meta = np.zeros((R * Cc // group, 2), dtype=np.float32)
    st = lib().sbo_pack_blocks(_p(W), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc), _p(rp), _p(cp),
                               C.c_int(block_rows), C.c_int(block_cols), C.c_int(group), barr,
                               C.c_int(L), _p(level), _p(packed), C.c_int64(cap), _p(off), _p(meta))
    if st != OK:
        raise ValueError(f"sbo_pack_blocks status {st}")
    return packed[:off[nb]].copy(), off, meta


def dequant_gemm(X, packed, block_off, meta, level, R, Cc, bits: Sequence[int], block_rows=128,
                 block_cols=128, group=128):
    """Y[t][r] = sum_c X[t][c] (lo + scale q)[r][c] on the packed layout (Section 5.3) -> f64 [T][R]."""
    X = _u16(X)
    T = X.shape[0]
    assert X.shape[1] == Cc
    barr, L = _bits(bits)
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    block_off = np.ascontiguousarray(block_off, dtype=np.int64)
    meta = np.ascontiguousarray(meta, dtype=np.float32)
    level = np.ascontiguousarray(level, dtype=np.uint8)
    Y = np.zeros((T, R), dtype=np.float64)
    st = lib().sbo_dequant_gemm(_p(X), C.c_int64(T), C.c_int64(Cc), _p(packed), _p(block_off), _p(meta),
                                _p(level), C.c_int64(R), C.c_int64(Cc), C.c_int(block_rows),
                                C.c_int(block_cols), C.c_int(group), barr, C.c_int(L), _p(Y))
    if st != OK:
        raise ValueError(f"sbo_dequant_gemm status {st}")
    return Y


class StepReport(C.Structure):
    _fields_ = [("cap_bits", C.c_int64), ("used_in", C.c_int64), ("used_out", C.c_int64),
                ("expansion", C.c_int32), ("moved", C.c_int32),
                ("n_up", C.c_int64), ("n_down", C.c_int64),
                ("sum_up", C.c_double), ("sum_down", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


def first_order_scores(W, G, bits: Sequence[int], level, block_rows=128, block_cols=128, group=128,
                       row_perm=None, col_perm=None):
    """-> (s_up[nb], s_down[nb], s_l1[nb]) of every block at its current level (Appendix E.3)."""
    W, G = _u16(W), _u16(G)
    assert W.shape == G.shape
    R, Cc = W.shape
    rp, cp = _i32(row_perm), _i32(col_perm)
    barr, L = _bits(bits)
    level = np.ascontiguousarray(level, dtype=np.uint8)
    nb = (R // block_rows) * (Cc // block_cols)
    assert level.size == nb
    up, down, l1 = (np.zeros(nb, dtype=np.float64) for _ in range(3))
    st = lib().sbo_first_order_scores(_p(W), _p(G), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc), C.c_int64(Cc),
                                      _p(rp), _p(cp), C.c_int(block_rows), C.c_int(block_cols),
                                      C.c_int(group), barr, C.c_int(L), _p(level), _p(up), _p(down), _p(l1))
    if st != OK:
        raise ValueError(f"sbo_first_order_scores status {st}")
    return up, down, l1


def exchange_step(s_up, s_down, level, bits: Sequence[int], budget: float, k: int,
                  uniform_block_elems=128 * 128, block_elems=None):
    """One iteration of Algorithm 2 on given scores -> (status, level_out, report dict)."""
    s_up, s_down = _f64(s_up), _f64(s_down)
    level = np.ascontiguousarray(level, dtype=np.uint8)
    N = level.size
    assert s_up.size == N and s_down.size == N
    barr, L = _bits(bits)
    be = None if block_elems is None else np.ascontiguousarray(block_elems, dtype=np.int64)
    out = np.zeros(N, dtype=np.uint8)
    rep = StepReport()
    st = lib().sbo_exchange_step(_p(s_up), _p(s_down), _p(level), C.c_int64(N), _p(be),
                                 C.c_int64(uniform_block_elems), barr, C.c_int(L), C.c_double(budget),
                                 C.c_int64(k), _p(out), C.byref(rep))
    return int(st), out, rep.as_dict()


def reorder_scores_first_order(W, G, ref_bits: int = 3, group: int = 128,
                               row_score: Optional[np.ndarray] = None, col_score: Optional[np.ndarray] = None,
                               accumulate: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Channel sums of |G (W - Q(W))| on the original layout (the p = 1 sensitivity)."""
    W, G = _u16(W), _u16(G)
    assert W.shape == G.shape
    R, Cc = W.shape
    if row_score is None:
        row_score = np.zeros(R, dtype=np.float64)
    if col_score is None:
        col_score = np.zeros(Cc, dtype=np.float64)
    st = lib().sbo_reorder_scores_first_order(_p(W), _p(G), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc),
                                              C.c_int64(Cc), C.c_int(ref_bits), C.c_int(group),
                                              _p(row_score), _p(col_score), C.c_int(int(accumulate)))
    assert st == OK, st
    return row_score, col_score


def calib_gram(X, scale: Optional[float] = None) -> np.ndarray:
    """H = scale * X^T X in fp64 (scale defaults to 1 / T); [K, K]."""
    X = _u16(X)
    T, K = X.shape
    H = np.zeros((K, K), dtype=np.float64)
    lib().sbo_calib_gram(_p(X), C.c_int64(T), C.c_int64(K), C.c_int64(K),
                         C.c_double(1.0 / max(T, 1) if scale is None else scale), _p(H))
    return H


def block_scores_full(W, H, bits: Sequence[int], block_rows=128, block_cols=128, group=128,
                      row_perm=None, col_perm=None, a=None) -> np.ndarray:
    """Block error table with the full second-moment matrix H [C, C] (original column order)."""
    W = _u16(W)
    R, Cc = W.shape
    H = np.ascontiguousarray(_f64(H).reshape(Cc, Cc))
    rp, cp = _i32(row_perm), _i32(col_perm)
    barr, L = _bits(bits)
    nb = (R // block_rows) * (Cc // block_cols)
    err = np.zeros((nb, L), dtype=np.float64)
    st = lib().sbo_block_scores_full(_p(W), C.c_int64(R), C.c_int64(Cc), C.c_int64(Cc), _p(rp), _p(cp),
                                     _p(H), C.c_int(block_rows), C.c_int(block_cols), C.c_int(group),
                                     barr, C.c_int(L), _p(err), _p(_f64(a, R)))
    if st != OK:
        raise ValueError(f"sbo_block_scores_full status {st}")
    return err
