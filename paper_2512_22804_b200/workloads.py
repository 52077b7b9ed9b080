"""Seeded synthetic BF16 tensors shaped like the operands of a transformer's linear layers.

The method is applied to the activation, weight and gradient operands of the four linear
layers of a transformer block (Section 4 of the paper).  The paper's tensors are not
available, so the recipes below stand in for them: Gaussian weights with per-column
spread, heavy-tailed activations with a few outlier channels, and gradients whose
magnitudes span tens of binades and contain exact zeros.

This module draws numbers and rounds them to BF16; it contains none of the method's
arithmetic (no scaling, casting, error metric or selection).  Both the CPU oracle's tests
and the CUDA path's tests take their inputs from here, as raw BF16 bit patterns
(``numpy.uint16``, row-major): the bytes are the contract, not the random generator.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

# enum values of the C boundary (kept as plain integers here so that this module
# depends on neither the binding nor the oracle)
FMT_E4M3, FMT_E5M2, FMT_BF16 = 0, 1, 2
CRIT_TENSOR_MEAN_REL, CRIT_BLOCK_VS_E5M2, CRIT_BLOCK_MEAN_REL = 0, 1, 2


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round a float array to BF16 (nearest, ties to even) and return the bit patterns."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    """Exact float32 values of BF16 bit patterns (for inspection and plots only)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def gaussian_outlier_rows(rows=1024, cols=1024, n_outlier_rows=8, gain=1000.0, seed=0):
    """N(0,1) values; ``n_outlier_rows`` distinct rows, drawn after the values, times ``gain``."""
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((rows, cols))
    k = min(n_outlier_rows, rows)
    idx = rng.choice(rows, k, replace=False)
    a[idx, :] *= gain
    return to_bf16_bits(a)


def weight_like(rows=4096, cols=4096, sigma=0.02, seed=1):
    """N(0, sigma) values times a per-column factor 10**U(-1, 1)."""
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((rows, cols)) * sigma
    colscale = 10.0 ** rng.uniform(-1.0, 1.0, size=cols)
    a *= colscale[None, :]
    return to_bf16_bits(a)


def activation_like(rows=8192, cols=4096, nu=3.0, n_outlier_cols=16, gain=100.0, seed=2):
    """Student-t (nu) values; ``n_outlier_cols`` fixed columns (same for every token) times ``gain``."""
    rng = np.random.default_rng(seed)
    a = rng.standard_t(nu, size=(rows, cols))
    k = min(n_outlier_cols, cols)
    idx = rng.choice(cols, k, replace=False)
    a[:, idx] *= gain
    return to_bf16_bits(a)


def gradient_like(rows=8192, cols=14336, mu=-13.0, sd=5.67, lo=-30.0, hi=4.0, p_zero=0.05, seed=3):
    """sign * 2**clip(N(mu, sd), lo, hi), then a fraction ``p_zero`` of exact zeros."""
    rng = np.random.default_rng(seed)
    sign = np.where(rng.random((rows, cols)) < 0.5, -1.0, 1.0)
    expo = np.clip(rng.normal(mu, sd, size=(rows, cols)), lo, hi)
    a = sign * np.exp2(expo)
    a[rng.random((rows, cols)) < p_zero] = 0.0
    return to_bf16_bits(a)


def mixed_grid(rows=4096, cols=4096, tile=128, lo_spread=4.0, hi_spread=36.0, seed=11):
    """A tensor whose 128x128 tiles differ: one magnitude level per tile drawn from 2**U(-12, 0) and, inside a tile,
    magnitudes spread uniformly in the exponent over a per-tile number of binades between ``lo_spread`` and
    ``hi_spread``; random signs.  Narrow tiles suit E4M3, wide ones E5M2 or BF16, side by side."""
    rng = np.random.default_rng(seed)
    tr, tc = -(-rows // tile), -(-cols // tile)
    level = np.repeat(np.repeat(np.exp2(rng.uniform(-12, 0, (tr, tc))), tile, 0), tile, 1)[:rows, :cols]
    spread = np.repeat(np.repeat(rng.uniform(lo_spread, hi_spread, (tr, tc)), tile, 0), tile, 1)[:rows, :cols]
    a = level * np.exp2(rng.uniform(-1, 0, (rows, cols)) * spread) * rng.choice([-1.0, 1.0], (rows, cols))
    return to_bf16_bits(a)


@dataclass
class Case:
    """One tensor plus the recipe it is analysed with."""

    name: str
    bits: np.ndarray                      # uint16 [rows, cols]
    block: Tuple[int, int]                # (0, 0) = whole tensor, (1, 128), (128, 128)
    formats: List[int]                    # ordered, most to least aggressive
    criterion: int
    threshold: float = 0.045
    extra: dict = field(default_factory=dict)


def config_case(i: int, scale: int = 1) -> List[Case]:
    """The five benchmark configurations; ``scale`` divides both dimensions (1 = full size).

    0: 1024x1024 Gaussian + outlier rows, per tensor, [E4M3, BF16], tensor mean-relative error
    1: 4096x4096 weight-like, 128x128 blocks, [E4M3, BF16], block test against E5M2
    2: 8192x4096 activation-like, 1x128 blocks, [E4M3, BF16], block test against E5M2
    3: 8192x14336 gradient-like, 1x128 and 128x128, [E4M3, E5M2, BF16]
    4: all operands of one Llama-style layer (hidden 4096, FFN 14336, 8192 tokens)
    """
    s = max(1, int(scale))
    two, three = [FMT_E4M3, FMT_BF16], [FMT_E4M3, FMT_E5M2, FMT_BF16]
    if i == 0:
        return [Case("c1_gauss_outlier_rows", gaussian_outlier_rows(1024 // s, 1024 // s, seed=0),
                     (0, 0), two, CRIT_TENSOR_MEAN_REL)]
    if i == 1:
        return [Case("c2_weight_128x128", weight_like(4096 // s, 4096 // s, seed=1),
                     (128, 128), two, CRIT_BLOCK_VS_E5M2)]
    if i == 2:
        return [Case("c3_activation_1x128", activation_like(8192 // s, 4096 // s, seed=2),
                     (1, 128), two, CRIT_BLOCK_VS_E5M2)]
    if i == 3:
        g = gradient_like(8192 // s, 14336 // s, seed=3)
        return [Case("c4_gradient_1x128", g, (1, 128), three, CRIT_BLOCK_VS_E5M2),
                Case("c4_gradient_128x128", g, (128, 128), three, CRIT_BLOCK_VS_E5M2)]
    if i == 4:
        return llama_layer_cases(scale=s)
    raise ValueError("config index 0..4")


def llama_layer_shapes(hidden=4096, ffn=14336, tokens=8192, n_heads=32, n_kv_heads=32):
    """(name, kind, rows, cols) of the 14 operands of one layer; kind in {weight, act, grad}."""
    head = hidden // n_heads
    qkv = hidden + 2 * n_kv_heads * head
    return [
        ("w_qkv", "weight", qkv, hidden), ("w_o", "weight", hidden, hidden),
        ("w_gate", "weight", ffn, hidden), ("w_up", "weight", ffn, hidden),
        ("w_down", "weight", hidden, ffn),
        ("x_qkv", "act", tokens, hidden), ("x_o", "act", tokens, hidden),
        ("x_gate_up", "act", tokens, hidden), ("x_down", "act", tokens, ffn),
        ("dy_qkv", "grad", tokens, qkv), ("dy_o", "grad", tokens, hidden),
        ("dy_gate", "grad", tokens, ffn), ("dy_up", "grad", tokens, ffn),
        ("dy_down", "grad", tokens, hidden),
    ]


def llama_layer_cases(scale: int = 1, grad_dist: str = "activation") -> List[Case]:
    """Weights 128x128 (weight_like), activations and output gradients 1x128.

    ``grad_dist`` = "activation" draws gradients like activations, "gradient" like
    ``gradient_like``.  Seeds are 100 + index.
    """
    s = max(1, int(scale))
    two = [FMT_E4M3, FMT_BF16]
    out = []
    for i, (name, kind, r, c) in enumerate(llama_layer_shapes()):
        r, c, seed = max(1, r // s), max(1, c // s), 100 + i
        if kind == "weight":
            out.append(Case(name, weight_like(r, c, seed=seed), (128, 128), two, CRIT_BLOCK_VS_E5M2))
        elif kind == "act" or grad_dist == "activation":
            out.append(Case(name, activation_like(r, c, seed=seed), (1, 128), two, CRIT_BLOCK_VS_E5M2))
        else:
            out.append(Case(name, gradient_like(r, c, seed=seed), (1, 128), two, CRIT_BLOCK_VS_E5M2))
    return out
