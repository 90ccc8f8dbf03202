"""Seeded synthetic inputs for the Prox sparse-FFN path.

This module holds data generation only: random draws, the bf16 storage
rounding of those draws, and the table of workload shapes.  It contains none
of the method's arithmetic (no quantizer, no selection, no projection, no
budget rule), so both the CUDA path and the CPU checker may be fed from it.

The paper's weights and activations are real-model tensors that are not
available here; these generators stand in for them with the shapes of the
SwiGLU FFNs the paper evaluates (Table "Qwen3 configurations": Qwen3-8B is
4096 x 12288) and of the Llama-class FFNs named by the benchmark configs.

Everything is returned as bf16 *bit patterns* (numpy uint16), so that the
very same bytes are handed to every consumer.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Tuple

import numpy as np


# --------------------------------------------------------------------------
# bf16 storage helpers (data conversion only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); return the uint16 bits."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rnd = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# Workload table
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    """One synthetic FFN workload.

    `points` maps a target effective sparsity (percent) to the integer budget
    (k1 kept inputs, k2 kept channels).  The integers are stored as data so
    that the generator needs no budget arithmetic; the tests check them
    against the budget rule separately.
    """
    name: str
    d_model: int
    d_ff: int
    w_std: float
    n_tokens: int
    outlier_frac: float
    outlier_gain: float
    outlier_fixed_channels: bool
    points: Dict[int, Tuple[int, int]]
    proxies: Tuple[Tuple[int, int], ...]          # (bits, group_size); 0 = one group per row
    batches: Tuple[int, ...] = (1,)
    seed: int = 0
    extra: Dict[str, object] = field(default_factory=dict)


WORKLOADS: Dict[str, Workload] = {
    "toy": Workload(
        "toy", 512, 1536, 0.02, 32, 0.01, 20.0, False,
        {50: (461, 461)}, ((4, 0),)),
    "qwen3_0p6b": Workload(
        "qwen3_0p6b", 1024, 3072, 0.02, 256, 0.01, 20.0, True,
        {50: (922, 922), 70: (307, 717), 90: (307, 102)}, ((4, 0),)),
    "qwen3_8b": Workload(
        "qwen3_8b", 4096, 12288, 0.015, 512, 0.005, 30.0, True,
        {70: (1229, 2867)}, ((4, 128),)),
    "llama3_8b": Workload(
        "llama3_8b", 4096, 14336, 0.015, 64, 0.005, 30.0, True,
        {40: (4096, 5416), 70: (1229, 3345)}, ((8, 0), (4, 128)), (1, 4, 8)),
    "llama3_70b": Workload(
        "llama3_70b", 8192, 28672, 0.01, 32, 0.005, 30.0, True,
        {70: (2458, 6690)}, ((4, 0), (4, 128)), (1, 8),
        extra={"s1_sweep": ((8192, 2230), (7373, 2867), (6554, 3504), (5734, 4142),
                            (4915, 4779), (4096, 5416), (3277, 6053), (2458, 6690),
                            (1638, 7327), (819, 7964))}),
}


# --------------------------------------------------------------------------
# Generators
# --------------------------------------------------------------------------
def _normal_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    rows, cols = shape
    out = np.empty((rows, cols), dtype=np.uint16)
    step = max(1, (1 << 24) // cols)               # draw in slabs to bound memory
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        slab = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        slab *= np.float32(std)
        out[r0:r1] = f32_to_bf16_bits(slab)
    return out


def make_weights(d_model: int, d_ff: int, std: float, rng: np.random.Generator):
    """Draw W_gate [d_ff, d_model], W_up [d_ff, d_model], W_down [d_model, d_ff]
    (row-major, the `nn.Linear` storage convention), iid N(0, std^2), bf16 bits.
    Draw order is fixed: gate, up, down."""
    w_gate = _normal_bf16(rng, (d_ff, d_model), std)
    w_up = _normal_bf16(rng, (d_ff, d_model), std)
    w_down = _normal_bf16(rng, (d_model, d_ff), std)
    return w_gate, w_up, w_down


def make_tokens(n_tokens: int, d_model: int, outlier_frac: float, outlier_gain: float,
                fixed_channels: bool, rng: np.random.Generator) -> np.ndarray:
    """Decode-time FFN inputs: Laplace(0,1) entries with a few large outliers.

    fixed_channels=True : a fixed set of round(outlier_frac*d_model) channels is
                          multiplied by outlier_gain in every token (the
                          "massive activation" pattern of LLM hidden states).
    fixed_channels=False: each entry is multiplied independently with
                          probability outlier_frac.
    Returns bf16 bits [n_tokens, d_model]."""
    if fixed_channels:
        n_out = int(round(outlier_frac * d_model))
        chans = rng.choice(d_model, size=n_out, replace=False)
    x = rng.laplace(0.0, 1.0, size=(n_tokens, d_model))
    if fixed_channels:
        x[:, chans] *= outlier_gain
    else:
        hit = rng.random(size=(n_tokens, d_model)) < outlier_frac
        x[hit] *= outlier_gain
    return f32_to_bf16_bits(x.astype(np.float32))


def make_workload(name: str, seed: int | None = None, n_tokens: int | None = None):
    """Return (workload, w_gate, w_up, w_down, x) for a named workload.
    All arrays are bf16 bit patterns (uint16)."""
    wl = WORKLOADS[name]
    rng = np.random.default_rng(wl.seed if seed is None else seed)
    w_gate, w_up, w_down = make_weights(wl.d_model, wl.d_ff, wl.w_std, rng)
    x = make_tokens(wl.n_tokens if n_tokens is None else n_tokens, wl.d_model,
                    wl.outlier_frac, wl.outlier_gain, wl.outlier_fixed_channels, rng)
    return wl, w_gate, w_up, w_down, x


def make_small(d_model: int, d_ff: int, n_tokens: int, seed: int, std: float = 0.02,
               outlier_frac: float = 0.01, outlier_gain: float = 20.0):
    """Free-form small problem for unit tests; same distributions as above."""
    rng = np.random.default_rng(seed)
    w_gate, w_up, w_down = make_weights(d_model, d_ff, std, rng)
    x = make_tokens(n_tokens, d_model, outlier_frac, outlier_gain, False, rng)
    return w_gate, w_up, w_down, x
