"""Thin ctypes binding of the C-ABI library (`include/scalebits.h`), same names.

Argument marshalling only: tensors are torch CUDA tensors (device memory and streams are
torch's job), every step runs in the library's kernels.  There is no CPU path: loading
fails loudly when `libscalebits.so` has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# SCALEBITS_LIB selects another build of the same library (the bounds-checked one, for tests)
LIB_PATH = os.environ.get("SCALEBITS_LIB") or os.path.join(_PKG, "libscalebits.so")

SB_OK, SB_ERR_INVALID, SB_ERR_SHAPE, SB_ERR_BUDGET, SB_ERR_SCRATCH, SB_ERR_CUDA, \
    SB_ERR_NOCONVERGE, SB_ERR_NONFINITE, SB_ERR_TIMEOUT = range(9)
SB_ALLOC_SCALEBITS, SB_ALLOC_GREEDY = 0, 1
SB_ACC_ROW, SB_ACC_COL = 1, 2

EXPORTS = ["sb_create", "sb_destroy", "sb_sync", "sb_last_error", "sb_kernel_launches", "sb_debug_lookback",
           "sb_checked_build",
           "sb_calib_moments", "sb_reorder_channels", "sb_fold_segment_scores",
           "sb_expand_segment_perm", "sb_sum_scores", "sb_permute_matrix", "sb_block_scores", "sb_allocate_bits", "sb_allocate_bits_async",
           "sb_pack_blocks",
           "sb_calib_moments_noalloc", "sb_first_order_scores", "sb_exchange_step",
           "sb_reorder_channels_first_order", "sb_calib_gram",
           "sb_block_scores_full", "sb_dequant_gemm"]


class SbError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"scalebits status {status}: {msg}")
        self.status = status


class AllocReport(C.Structure):
    _fields_ = [("cap_bits", C.c_int64), ("used_bits", C.c_int64),
                ("iterations", C.c_int32), ("accepted", C.c_int32),
                ("rejected", C.c_int32), ("expansions", C.c_int32),
                ("proxy_loss_init", C.c_double), ("proxy_loss_final", C.c_double),
                ("level_hist", C.c_int64 * 8)]

    def as_dict(self):
        return {"cap_bits": self.cap_bits, "used_bits": self.used_bits,
                "iterations": self.iterations, "accepted": self.accepted,
                "rejected": self.rejected, "expansions": self.expansions,
                "proxy_loss_init": self.proxy_loss_init,
                "proxy_loss_final": self.proxy_loss_final,
                "level_hist": list(self.level_hist)}


class StepReport(C.Structure):
    _fields_ = [("cap_bits", C.c_int64), ("used_in", C.c_int64), ("used_out", C.c_int64),
                ("expansion", C.c_int32), ("moved", C.c_int32),
                ("n_up", C.c_int64), ("n_down", C.c_int64),
                ("sum_up", C.c_double), ("sum_down", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def lib() -> C.CDLL:
    """Loads libscalebits.so (built in-tree by `python -m paper_2602_17698_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2602_17698_b200.build` "
                "(nvcc, sm_100a). There is no CPU fallback.")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, f32, f64 = C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_double
        L.sb_create.argtypes = [C.POINTER(vp), i32, vp]
        L.sb_destroy.argtypes = [vp]
        L.sb_sync.argtypes = [vp]
        L.sb_debug_lookback.argtypes = [vp, i64, i64]
        L.sb_checked_build.argtypes = []
        L.sb_last_error.argtypes = [vp]
        L.sb_last_error.restype = C.c_char_p
        L.sb_kernel_launches.argtypes = [vp]
        L.sb_kernel_launches.restype = i64
        L.sb_calib_moments.argtypes = [vp, vp, i64, i64, i64, vp, i32, f32]
        L.sb_reorder_channels.argtypes = [vp, vp, i64, i64, i64, vp, vp, i32, i32, vp, vp, i32,
                                          i64, i64, vp, vp]
        L.sb_fold_segment_scores.argtypes = [vp, vp, vp, i64, i32, i64]
        L.sb_expand_segment_perm.argtypes = [vp, vp, vp, i64, i32, i64]
        L.sb_sum_scores.argtypes = [vp, vp, C.POINTER(C.c_void_p), i32, i64, i32]
        L.sb_permute_matrix.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
        L.sb_block_scores.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp, i32, i32, i32,
                                      C.POINTER(C.c_int), i32, vp, vp, vp]
        L.sb_allocate_bits.argtypes = [vp, vp, i64, vp, i64, C.POINTER(C.c_int), i32, f64, i32,
                                       f64, f64, vp, C.POINTER(AllocReport)]
        L.sb_allocate_bits_async.argtypes = [vp, vp, i64, vp, i64, C.POINTER(C.c_int), i32, f64, i32,
                                             f64, f64, vp, vp]
        L.sb_pack_blocks.argtypes = [vp, vp, i64, i64, i64, vp, vp, i32, i32, i32,
                                     C.POINTER(C.c_int), i32, vp, vp, i64, vp, vp]
        L.sb_first_order_scores.argtypes = [vp, vp, vp, i64, i64, i64, i64, vp, vp, i32, i32, i32,
                                            C.POINTER(C.c_int), i32, vp, vp, vp, vp]
        L.sb_exchange_step.argtypes = [vp, vp, vp, vp, i64, vp, i64, C.POINTER(C.c_int), i32, f64, i64,
                                       vp, C.POINTER(StepReport)]
        L.sb_calib_moments_noalloc.argtypes = [vp, vp, i64, i64, i64, vp, i32, f32]
        L.sb_calib_gram.argtypes = [vp, vp, i64, i64, i64, vp, i32, f32]
        L.sb_block_scores_full.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp, i32, i32, i32,
                                           C.POINTER(C.c_int), i32, vp, vp, vp]
        L.sb_dequant_gemm.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, i64, i64, i32, i32, i32,
                                      C.POINTER(C.c_int), i32, vp, i64]
        L.sb_reorder_channels_first_order.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, i32, vp, vp, i32,
                                                      i64, i64, vp, vp]
        for name in EXPORTS:
            if name not in ("sb_last_error", "sb_kernel_launches"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype=None, cuda=True):
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {t.dtype}")
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor (the library has no CPU path)")
    return C.c_void_p(t.data_ptr())


def _bits(bits: Sequence[int]):
    return (C.c_int * len(bits))(*[int(b) for b in bits]), len(bits)


def _mat(W: torch.Tensor):
    if W.dim() != 2 or W.dtype != torch.bfloat16 or W.stride(1) != 1:
        raise ValueError("expected a row-major 2-D bf16 tensor")
    return W.shape[0], W.shape[1], W.stride(0)


class Context:
    """One sb_ctx on the current torch device and stream."""

    def __init__(self, device: Optional[int] = None, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the scalebits library has no CPU fallback")
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.stream = torch.cuda.current_stream(self.device) if stream is None else stream
        h = C.c_void_p()
        st = lib().sb_create(C.byref(h), self.device, C.c_void_p(self.stream.cuda_stream))
        if st != SB_OK:
            raise SbError(st, "sb_create failed (needs an sm_100 device)")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().sb_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != SB_OK:
            raise SbError(st, lib().sb_last_error(self._h).decode())

    # ---- the C-ABI calls, one method each -------------------------------------------------
    def sync(self):
        self._check(lib().sb_sync(self._h))

    def kernel_launches(self) -> int:
        return int(lib().sb_kernel_launches(self._h))

    def calib_moments(self, X: torch.Tensor, sumsq: Optional[torch.Tensor] = None,
                      accumulate: bool = False, scale: Optional[float] = None) -> torch.Tensor:
        T, K, ldx = _mat(X)
        if sumsq is None:
            sumsq = torch.empty(K, dtype=torch.float32, device=X.device)
            accumulate = False
        if scale is None:
            scale = 1.0 / T
        self._check(lib().sb_calib_moments(self._h, _ptr(X), T, K, ldx, _ptr(sumsq, torch.float32),
                                           int(accumulate), float(scale)))
        return sumsq

    def calib_gram(self, X: torch.Tensor, H: Optional[torch.Tensor] = None, accumulate: bool = False,
                   scale: Optional[float] = None) -> torch.Tensor:
        T, K, ldx = _mat(X)
        if H is None:
            H = torch.empty((K, K), dtype=torch.float32, device=X.device)
            accumulate = False
        if scale is None:
            scale = 1.0 / max(T, 1)
        self._check(lib().sb_calib_gram(self._h, _ptr(X), T, K, ldx, _ptr(H, torch.float32), int(accumulate),
                                        float(scale)))
        return H

    def reorder_channels(self, W: Optional[torch.Tensor], col_moment: Optional[torch.Tensor],
                         ref_bits: int, group: int, row_score=None, col_score=None,
                         accumulate_row: bool = False, accumulate_col: bool = False,
                         row_segment: int = 0, col_segment: int = 0,
                         row_perm=None, col_perm=None, row_weight=None, shape=None):
        if W is not None:
            R, Cc, ldw = _mat(W)
        else:
            R, Cc = shape
            ldw = Cc
        self._check(lib().sb_reorder_channels(
            self._h, _ptr(W), R, Cc, ldw, _ptr(col_moment, torch.float32),
            _ptr(row_weight, torch.float32), int(ref_bits), int(group),
            _ptr(row_score, torch.float32), _ptr(col_score, torch.float32),
            (SB_ACC_ROW if accumulate_row else 0) | (SB_ACC_COL if accumulate_col else 0),
            int(row_segment), int(col_segment), _ptr(row_perm, torch.int32), _ptr(col_perm, torch.int32)))

    def fold_segment_scores(self, dst: torch.Tensor, src: torch.Tensor, reps: int, seg: int):
        assert dst.numel() * reps == src.numel()
        self._check(lib().sb_fold_segment_scores(self._h, _ptr(dst, torch.float32),
                                                 _ptr(src, torch.float32), dst.numel(), reps, seg))

    def sum_scores(self, dst: torch.Tensor, srcs: Sequence[torch.Tensor], accumulate: bool = False):
        """dst = (dst +) srcs[0] + srcs[1] + ... left to right in fp32 (the score vectors of the
        matrices of a coupled channel set, in the order a one-stream accumulation would take)."""
        n = dst.numel()
        assert 1 <= len(srcs) <= 8 and all(t.numel() == n and t.is_contiguous() for t in srcs)
        arr = (C.c_void_p * len(srcs))(*[_ptr(t, torch.float32).value for t in srcs])
        self._check(lib().sb_sum_scores(self._h, _ptr(dst, torch.float32), arr, len(srcs), n, int(accumulate)))
        return dst

    def expand_segment_perm(self, perm: torch.Tensor, reps: int, seg: int, out=None) -> torch.Tensor:
        if out is None:
            out = torch.empty(perm.numel() * reps, dtype=torch.int32, device=perm.device)
        assert out.numel() == perm.numel() * reps and out.dtype == torch.int32
        self._check(lib().sb_expand_segment_perm(self._h, _ptr(out), _ptr(perm, torch.int32),
                                                 perm.numel(), reps, seg))
        return out

    def debug_lookback(self, wait_ns: int = -1, mute_tile: int = -1):
        """Test hook: the time limit of a look-back wait and a tile that publishes nothing."""
        self._check(lib().sb_debug_lookback(self._h, int(wait_ns), int(mute_tile)))

    def permute_matrix(self, W: torch.Tensor, row_perm=None, col_perm=None, out=None) -> torch.Tensor:
        """out[r][j] = W[row_perm[r]][col_perm[j]] (a matrix that is moved along with a channel
        permutation but not scored: embedding, language-model head)."""
        R, Cc, ldw = _mat(W)
        if out is None:
            out = torch.empty((R, Cc), dtype=torch.bfloat16, device=W.device)
        self._check(lib().sb_permute_matrix(self._h, _ptr(W), R, Cc, ldw, _ptr(row_perm, torch.int32),
                                            _ptr(col_perm, torch.int32), _ptr(out)))
        return out

    def block_scores(self, W: torch.Tensor, col_moment: torch.Tensor, bits: Sequence[int],
                     block_rows: int = 128, block_cols: int = 128, group: int = 128,
                     row_perm=None, col_perm=None, row_weight=None, err=None, gain=None,
                     want_gain: bool = True, W_perm_out=None):
        R, Cc, ldw = _mat(W)
        barr, L = _bits(bits)
        nb = (R // block_rows) * (Cc // block_cols)
        if err is None:
            err = torch.empty((nb, L), dtype=torch.float32, device=W.device)
        if gain is None and want_gain and L > 1:
            gain = torch.empty((nb, L - 1), dtype=torch.float32, device=W.device)
        self._check(lib().sb_block_scores(
            self._h, _ptr(W), R, Cc, ldw, _ptr(row_perm, torch.int32), _ptr(col_perm, torch.int32),
            _ptr(col_moment, torch.float32), _ptr(row_weight, torch.float32),
            block_rows, block_cols, group, barr, L, _ptr(err, torch.float32),
            _ptr(gain, torch.float32), _ptr(W_perm_out, torch.bfloat16)))
        return err, gain

    def block_scores_full(self, W: torch.Tensor, H: torch.Tensor, bits: Sequence[int],
                          block_rows: int = 128, block_cols: int = 128, group: int = 128,
                          row_perm=None, col_perm=None, row_weight=None, err=None, gain=None,
                          want_gain: bool = True, W_perm_out=None):
        R, Cc, ldw = _mat(W)
        assert H.shape == (Cc, Cc) and H.is_contiguous()
        barr, L = _bits(bits)
        nb = (R // block_rows) * (Cc // block_cols)
        if err is None:
            err = torch.empty((nb, L), dtype=torch.float32, device=W.device)
        if gain is None and want_gain and L > 1:
            gain = torch.empty((nb, L - 1), dtype=torch.float32, device=W.device)
        self._check(lib().sb_block_scores_full(
            self._h, _ptr(W), R, Cc, ldw, _ptr(row_perm, torch.int32), _ptr(col_perm, torch.int32),
            _ptr(H, torch.float32), _ptr(row_weight, torch.float32), block_rows, block_cols, group, barr, L,
            _ptr(err, torch.float32), _ptr(gain, torch.float32), _ptr(W_perm_out, torch.bfloat16)))
        return err, gain

    def allocate_bits(self, err: torch.Tensor, bits: Sequence[int], budget: float,
                      mode: int = SB_ALLOC_SCALEBITS, gamma0: float = 0.05, gammaT: float = 0.02,
                      uniform_block_elems: int = 128 * 128, block_elems=None, level=None):
        N, L = err.shape
        barr, Lb = _bits(bits)
        assert L == Lb and err.is_contiguous()
        if level is None:
            level = torch.empty(N, dtype=torch.uint8, device=err.device)
        rep = AllocReport()
        st = lib().sb_allocate_bits(self._h, _ptr(err, torch.float32), N, _ptr(block_elems, torch.int64),
                                    int(uniform_block_elems), barr, L, float(budget), int(mode),
                                    float(gamma0), float(gammaT), _ptr(level, torch.uint8), C.byref(rep))
        self._check(st)
        return level, rep.as_dict()

    def allocate_bits_async(self, err: torch.Tensor, bits: Sequence[int], budget: float,
                            mode: int = SB_ALLOC_SCALEBITS, gamma0: float = 0.05, gammaT: float = 0.02,
                            uniform_block_elems: int = 128 * 128, block_elems=None, level=None,
                            report=None):
        """The allocation enqueued only (no host round trip; can be captured in a CUDA graph).
        Returns (level, report): `report` is a uint8 device tensor holding the report struct;
        `read_report(report)` decodes it after a synchronisation."""
        N, L = err.shape
        barr, Lb = _bits(bits)
        assert L == Lb and err.is_contiguous()
        if level is None:
            level = torch.empty(N, dtype=torch.uint8, device=err.device)
        if report is None:
            report = torch.zeros(C.sizeof(AllocReport), dtype=torch.uint8, device=err.device)
        assert report.dtype == torch.uint8 and report.numel() >= C.sizeof(AllocReport) and report.is_contiguous()
        st = lib().sb_allocate_bits_async(self._h, _ptr(err, torch.float32), N, _ptr(block_elems, torch.int64),
                                          int(uniform_block_elems), barr, L, float(budget), int(mode),
                                          float(gamma0), float(gammaT), _ptr(level, torch.uint8),
                                          _ptr(report, torch.uint8))
        self._check(st)
        return level, report

    @staticmethod
    def read_report(report: torch.Tensor) -> dict:
        """Decodes the device report of `allocate_bits_async` (copies it to the host: the
        stream that wrote it must have been synchronised, or be the current one)."""
        raw = bytes(report.cpu().numpy().tobytes()[:C.sizeof(AllocReport)])
        return AllocReport.from_buffer_copy(raw).as_dict()

    def reorder_channels_first_order(self, W: torch.Tensor, G: torch.Tensor, ref_bits: int, group: int,
                                     row_score=None, col_score=None, accumulate_row: bool = False,
                                     accumulate_col: bool = False, row_segment: int = 0, col_segment: int = 0,
                                     row_perm=None, col_perm=None):
        R, Cc, ldw = _mat(W)
        Rg, Cg, ldg = _mat(G)
        assert (R, Cc) == (Rg, Cg)
        acc = (SB_ACC_ROW if accumulate_row else 0) | (SB_ACC_COL if accumulate_col else 0)
        self._check(lib().sb_reorder_channels_first_order(
            self._h, _ptr(W), _ptr(G), R, Cc, ldw, ldg, int(ref_bits), int(group),
            _ptr(row_score, torch.float32), _ptr(col_score, torch.float32), acc, int(row_segment),
            int(col_segment), _ptr(row_perm, torch.int32), _ptr(col_perm, torch.int32)))
        return row_score, col_score

    def first_order_scores(self, W: torch.Tensor, G: torch.Tensor, bits: Sequence[int], level: torch.Tensor,
                           block_rows: int = 128, block_cols: int = 128, group: int = 128,
                           row_perm=None, col_perm=None, s_up=None, s_down=None, s_l1=None,
                           want_l1: bool = True):
        R, Cc, ldw = _mat(W)
        Rg, Cg, ldg = _mat(G)
        assert (R, Cc) == (Rg, Cg)
        barr, L = _bits(bits)
        nb = (R // block_rows) * (Cc // block_cols)
        f32 = dict(dtype=torch.float32, device=W.device)
        if s_up is None:
            s_up = torch.empty(nb, **f32)
        if s_down is None:
            s_down = torch.empty(nb, **f32)
        if s_l1 is None and want_l1:
            s_l1 = torch.empty(nb, **f32)
        self._check(lib().sb_first_order_scores(
            self._h, _ptr(W), _ptr(G), R, Cc, ldw, ldg, _ptr(row_perm, torch.int32),
            _ptr(col_perm, torch.int32), block_rows, block_cols, group, barr, L, _ptr(level, torch.uint8),
            _ptr(s_up, torch.float32), _ptr(s_down, torch.float32), _ptr(s_l1, torch.float32)))
        return s_up, s_down, s_l1

    def exchange_step(self, s_up: torch.Tensor, s_down: torch.Tensor, level: torch.Tensor,
                      bits: Sequence[int], budget: float, k: int, uniform_block_elems: int = 128 * 128,
                      block_elems=None, level_out=None):
        N = level.numel()
        barr, L = _bits(bits)
        if level_out is None:
            level_out = torch.empty_like(level)
        rep = StepReport()
        st = lib().sb_exchange_step(self._h, _ptr(s_up, torch.float32), _ptr(s_down, torch.float32),
                                    _ptr(level, torch.uint8), N, _ptr(block_elems, torch.int64),
                                    int(uniform_block_elems), barr, L, float(budget), int(k),
                                    _ptr(level_out, torch.uint8), C.byref(rep))
        self._check(st)
        return level_out, rep.as_dict()

    def pack_blocks(self, W: torch.Tensor, bits: Sequence[int], level: torch.Tensor,
                    block_rows: int = 128, block_cols: int = 128, group: int = 128,
                    row_perm=None, col_perm=None, packed=None, block_off=None, meta=None):
        R, Cc, ldw = _mat(W)
        barr, L = _bits(bits)
        nb = (R // block_rows) * (Cc // block_cols)
        if packed is None:
            packed = torch.empty(R * Cc * max(bits) // 32, dtype=torch.int32, device=W.device)
        if block_off is None:
            block_off = torch.empty(nb + 1, dtype=torch.int64, device=W.device)
        if meta is None:
            meta = torch.empty((R * Cc // group, 2), dtype=torch.float32, device=W.device)
        self._check(lib().sb_pack_blocks(
            self._h, _ptr(W), R, Cc, ldw, _ptr(row_perm, torch.int32), _ptr(col_perm, torch.int32),
            block_rows, block_cols, group, barr, L, _ptr(level, torch.uint8), _ptr(packed),
            packed.numel(), _ptr(block_off, torch.int64), _ptr(meta, torch.float32)))
        return packed, block_off, meta


    def dequant_gemm(self, X: torch.Tensor, packed: torch.Tensor, block_off: torch.Tensor, meta: torch.Tensor,
                     level: torch.Tensor, R: int, Cc: int, bits: Sequence[int], block_rows: int = 128,
                     block_cols: int = 128, group: int = 128, Y: Optional[torch.Tensor] = None):
        """Y[t][r] = sum_c X[t][c] (lo + scale q)[r][c] on the output of pack_blocks -> fp32 [T][R]."""
        T, Kx, ldx = _mat(X)
        if Kx != Cc:
            raise ValueError("X must have one column per packed column")
        barr, L = _bits(bits)
        if Y is None:
            Y = torch.empty((T, R), dtype=torch.float32, device=X.device)
        self._check(lib().sb_dequant_gemm(
            self._h, _ptr(X), T, ldx, _ptr(packed), _ptr(block_off, torch.int64), _ptr(meta, torch.float32),
            _ptr(level, torch.uint8), R, Cc, block_rows, block_cols, group, barr, L,
            _ptr(Y, torch.float32), Y.stride(0)))
        return Y


def checked_build() -> bool:
    """True if the loaded library is the bounds-checked build (-DSB_CHECKED)."""
    return bool(lib().sb_checked_build())


def calib_moments_noalloc(X: torch.Tensor, sumsq: Optional[torch.Tensor] = None,
                          accumulate: bool = False, scale: Optional[float] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """sb_calib_moments_noalloc: second moments without a context and without any device
    allocation inside the library (fixed in-library scratch, K <= 65536).

    For callers that cannot allocate when they need the moments (device memory fully handed
    out at start-up, code under a caching allocator, latency-critical loops).  X's device
    must be current.  Calls share the scratch: do not let two of them overlap on the GPU.
    """
    T, K, ldx = _mat(X)
    if sumsq is None:
        sumsq = torch.empty(K, dtype=torch.float32, device=X.device)
        accumulate = False
    if scale is None:
        scale = 1.0 / max(T, 1)
    s = torch.cuda.current_stream(X.device) if stream is None else stream
    fn = lib().sb_calib_moments_noalloc
    st = fn(C.c_void_p(s.cuda_stream), _ptr(X), T, K, ldx, _ptr(sumsq, torch.float32),
            int(accumulate), float(scale))
    if st != SB_OK:
        raise SbError(st, "sb_calib_moments_noalloc failed (see stderr)")
    return sumsq
