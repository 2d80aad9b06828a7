"""Seeded synthetic inputs: Llama-shaped weights and calibration activations.

This module only draws random tensors.  It holds none of the method's
arithmetic (no quantizer, no moments, no scores) and is the single piece of
code that both the CUDA path's tests and the CPU oracle's tests use.

The paper's real workloads (Llama / Gemma checkpoints, RedPajama calibration
text, Section 5 "Implementation") are replaced by tensors with the same
shapes and value structure:

* weights: W = 0.02 * z, z ~ N(0, 1); a Bernoulli(1e-3) mask of entries is
  replaced by 0.02 * 20 * t with t ~ Student-t(df = 3) (heavy-tailed
  outliers); optional "super-weight" entries of magnitude 50 sigma
  (cf. the single-weight sensitivity remarks in Section 1);
* activations: X[t, j] = s_j * z with s_j = exp(N(0, 1)) per channel, i.e.
  sensitivity concentrated in few input channels (Section 3.2).

Everything is cast to bf16.  A tensor is a function of (seed, layer,
tensor_id, shape, device type): the CPU and CUDA generators of torch give
different streams, so a test draws on one device and copies to the other.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Tuple

import torch

SIGMA_W = 0.02
OUTLIER_FRAC = 1e-3
OUTLIER_SCALE = 20.0
OUTLIER_DF = 3
SUPER_WEIGHT_SIGMAS = 50.0


def tensor_seed(seed: int, layer: int, tensor_id: int) -> int:
    """One 63-bit seed per (base seed, layer, tensor)."""
    return (seed * 1_000_003 + 1009 * layer + tensor_id) & 0x7FFF_FFFF_FFFF_FFFF


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_weight(rows: int, cols: int, seed: int, device="cpu", outliers: bool = True,
                chunk_rows: int = 2048) -> torch.Tensor:
    """bf16 [rows, cols] weight matrix, N(0, 0.02) plus heavy-tailed outliers."""
    g = _gen(device, seed)
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        shape = (r1 - r0, cols)
        w = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * SIGMA_W
        if outliers:
            mask = torch.rand(shape, generator=g, device=device) < OUTLIER_FRAC
            z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
            chi = torch.zeros(shape, device=device, dtype=torch.float32)
            for _ in range(OUTLIER_DF):
                chi += torch.randn(shape, generator=g, device=device, dtype=torch.float32) ** 2
            t = z / torch.sqrt(chi / OUTLIER_DF + 1e-30)
            w = torch.where(mask, SIGMA_W * OUTLIER_SCALE * t, w)
        out[r0:r1] = w.to(torch.bfloat16)
    return out


def make_activations(tokens: int, channels: int, seed: int, device="cpu",
                     chunk_rows: int = 8192) -> torch.Tensor:
    """bf16 [tokens, channels] activations with log-normal(0, 1) per-channel std."""
    g = _gen(device, seed)
    s = torch.exp(torch.randn((channels,), generator=g, device=device, dtype=torch.float32))
    out = torch.empty((tokens, channels), dtype=torch.bfloat16, device=device)
    for t0 in range(0, tokens, chunk_rows):
        t1 = min(tokens, t0 + chunk_rows)
        z = torch.randn((t1 - t0, channels), generator=g, device=device, dtype=torch.float32)
        out[t0:t1] = (z * s).to(torch.bfloat16)
    return out


def inject_super_weights(w: torch.Tensor, seed: int, count: int = 1) -> List[Tuple[int, int, float]]:
    """Set `count` entries of `w` (in place) to +-50 sigma; returns (row, col, value)."""
    g = _gen("cpu", seed)
    placed = []
    for _ in range(count):
        r = int(torch.randint(0, w.shape[0], (1,), generator=g))
        c = int(torch.randint(0, w.shape[1], (1,), generator=g))
        sign = 1.0 if int(torch.randint(0, 2, (1,), generator=g)) else -1.0
        val = sign * SUPER_WEIGHT_SIGMAS * SIGMA_W
        w[r, c] = val
        placed.append((r, c, val))
    return placed


@dataclass(frozen=True)
class LinearShape:
    name: str
    rows: int          # d_out  (output channels)
    cols: int          # d_in   (input channels)
    act: str           # which calibration input feeds its columns
    tensor_id: int


@dataclass(frozen=True)
class LayerShape:
    hidden: int
    intermediate: int
    n_heads: int
    n_kv_heads: int
    head_dim: int

    @property
    def linears(self) -> List[LinearShape]:
        h, m = self.hidden, self.intermediate
        q = self.n_heads * self.head_dim
        kv = self.n_kv_heads * self.head_dim
        return [
            LinearShape("q_proj", q, h, "attn_in", 0),
            LinearShape("k_proj", kv, h, "attn_in", 1),
            LinearShape("v_proj", kv, h, "attn_in", 2),
            LinearShape("o_proj", h, q, "o_in", 3),
            LinearShape("gate_proj", m, h, "mlp_in", 4),
            LinearShape("up_proj", m, h, "mlp_in", 5),
            LinearShape("down_proj", h, m, "down_in", 6),
        ]

    @property
    def act_dims(self) -> Dict[str, int]:
        return {"attn_in": self.hidden, "o_in": self.n_heads * self.head_dim,
                "mlp_in": self.hidden, "down_in": self.intermediate}

    @property
    def n_weights(self) -> int:
        return sum(l.rows * l.cols for l in self.linears)


LLAMA3_8B = LayerShape(hidden=4096, intermediate=14336, n_heads=32, n_kv_heads=8, head_dim=128)
LLAMA3_70B = LayerShape(hidden=8192, intermediate=28672, n_heads=64, n_kv_heads=8, head_dim=128)
# a scaled-down layer of the same structure (GQA 4:1, head_dim 128) for tests
LLAMA_TINY = LayerShape(hidden=512, intermediate=1024, n_heads=4, n_kv_heads=2, head_dim=128)

ACT_TENSOR_ID = {"attn_in": 16, "o_in": 17, "mlp_in": 18, "down_in": 19}


def make_layer_weights(shape: LayerShape, seed: int, layer: int, device="cpu") -> Dict[str, torch.Tensor]:
    return {l.name: make_weight(l.rows, l.cols, tensor_seed(seed, layer, l.tensor_id), device)
            for l in shape.linears}


def make_layer_activations(shape: LayerShape, tokens: int, seed: int, layer: int,
                           device="cpu") -> Dict[str, torch.Tensor]:
    return {name: make_activations(tokens, k, tensor_seed(seed, layer, ACT_TENSOR_ID[name]), device)
            for name, k in shape.act_dims.items()}


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view (host copy) of a bf16 tensor, for the CPU oracle."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")


def expected_channel_std(channels: int, seed: int, device="cpu") -> torch.Tensor:
    """The per-channel std s_j that make_activations(…, channels, seed) draws first."""
    g = _gen(device, seed)
    return torch.exp(torch.randn((channels,), generator=g, device=device, dtype=torch.float32))


def table4_levels(n_blocks: int, seed: int):
    """Block levels of the mixed-precision kernel benchmark (Table 4): 40 % / 40 % / 20 % of the
    blocks at the first / second / third candidate (2 / 4 / 8 bits: 4 bits on average), in a seeded
    random arrangement.  numpy uint8 [n_blocks]."""
    import numpy as np
    n0 = (2 * n_blocks) // 5
    n1 = (2 * n_blocks) // 5
    lv = np.concatenate([np.zeros(n0, np.uint8), np.ones(n1, np.uint8), np.full(n_blocks - n0 - n1, 2, np.uint8)])
    np.random.default_rng(seed).shuffle(lv)
    return lv


__all__ = [n for n in dir() if not n.startswith("_") and n not in ("math", "torch")]
