"""Seeded synthetic workloads shaped like the paper's models.

This module only draws random numbers and rounds them to the storage type.
It holds none of the method's arithmetic, so both the CPU oracle's tests and
the CUDA path's tests/bench can take their inputs from here.

The paper restructures LLaMA-2-7B/13B-, LLaMA-3-8B- and Mixtral/Qwen-MoE-shaped
SwiGLU FFNs (Section 5.1) and feeds them transformer hidden states; neither the
trained weights nor the text corpora are available, so N(0,1) tokens,
N(0,0.02^2) weights and a seeded uniform random neuron partition stand in for
them with the same shapes.

Draw order for one layer (fixed, so a seed names one workload):
    x[T_max,d], W_gate[d_ff,d], W_up[d_ff,d], W_down[d,d_ff], perm[d_ff]
all from ``numpy.random.Generator(PCG64(seed))``; fp32 draws, rounded once
(round-to-nearest-even) to the storage type, and that rounded value is what
every consumer sees.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

WEIGHT_STD = 0.02


# --------------------------------------------------------------------------
# storage-type rounding (bf16 has no numpy dtype: carry it as uint16 bits)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array holding values exactly representable in ``dtype``."""
    if dtype == "fp32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(a))
    raise ValueError(f"unknown dtype {dtype!r}")


# --------------------------------------------------------------------------
# shapes
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerShape:
    """One restructured FFN: N experts of m = d_ff/N neurons, N_s shared,
    N_r = N - N_s routed, N_k routed experts selected per token."""
    d_model: int
    d_ff: int
    n_experts: int
    n_shared: int
    top_k: int
    dtype: str = "bf16"            # storage type of x, out and all weights

    @property
    def m(self) -> int:
        return self.d_ff // self.n_experts

    @property
    def n_routed(self) -> int:
        return self.n_experts - self.n_shared

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    # ---- algorithmic work of one forward (the method's own work) ----------
    def flops_per_token(self) -> int:
        """Expert contractions 6*d*m*(N_s+N_k) plus the router's 4*d*N_r."""
        return (6 * self.d_model * self.m * (self.n_shared + self.top_k)
                + 4 * self.d_model * self.n_routed)

    def dense_flops_per_token(self) -> int:
        return 6 * self.d_model * self.d_ff

    def expert_weight_bytes(self) -> int:
        return 3 * self.d_model * self.m * self.elem_bytes

    def algorithmic_bytes(self, n_tokens: int, routed_touched: int) -> int:
        """Weights of every touched expert once, router rows, x read, out write."""
        w = (self.n_shared + routed_touched) * self.expert_weight_bytes()
        io = 2 * n_tokens * self.d_model * self.elem_bytes
        return w + io


@dataclass(frozen=True)
class Workload:
    name: str
    shape: LayerShape
    tokens: Tuple[int, ...]        # T values this workload is run at
    seed: int
    n_outer: int = 0               # >0: hierarchical (an existing MoE layer)
    outer_top_k: int = 0
    zipf_s: float = 0.0            # >0: routed load skewed by the selection bias
    note: str = ""

    @property
    def t_max(self) -> int:
        return max(self.tokens)


WORKLOADS: Dict[str, Workload] = {
    "c1_tiny_fp32": Workload(
        "c1_tiny_fp32", LayerShape(256, 1024, 8, 2, 2, "fp32"), (64,), seed=0,
        note="tiny fp32 exactness case"),
    "c2_llama2_7b": Workload(
        "c2_llama2_7b", LayerShape(4096, 11008, 8, 2, 2, "bf16"),
        (1, 16, 64, 512, 4096), seed=2, note="LLaMA-2-7B-shaped FFN, S2A2E8"),
    "c3_llama3_8b": Workload(
        "c3_llama3_8b", LayerShape(4096, 14336, 32, 4, 4, "bf16"),
        (32, 8192), seed=3, note="LLaMA-3-8B-shaped FFN, S4A4E32"),
    "c4_hier_8x7b": Workload(
        "c4_hier_8x7b", LayerShape(4096, 14336, 8, 2, 2, "bf16"), (4096,),
        seed=4, n_outer=8, outer_top_k=2,
        note="Mixtral-8x7B-shaped MoE layer, every outer expert restructured S2A2E8"),
    "c5_skew_13b": Workload(
        "c5_skew_13b", LayerShape(5120, 13824, 16, 2, 4, "bf16"), (16384,),
        seed=5, zipf_s=1.2, note="LLaMA-2-13B-shaped FFN, S2A4E16, Zipf(1.2) load"),
}


def shrunk(w: Workload, *, d_model: int, tokens: Tuple[int, ...],
           m: Optional[int] = None, n_outer: Optional[int] = None) -> Workload:
    """Same expert structure (N, N_s, N_k and, unless overridden, the expert
    width m with its ragged tile tails) at a smaller d_model and T."""
    m = w.shape.m if m is None else m
    shape = replace(w.shape, d_model=d_model, d_ff=m * w.shape.n_experts)
    return replace(w, name=w.name + "_small", shape=shape, tokens=tokens,
                   n_outer=w.n_outer if n_outer is None else n_outer)


# --------------------------------------------------------------------------
# one layer's inputs
# --------------------------------------------------------------------------
@dataclass
class LayerInputs:
    shape: LayerShape
    w_gate: np.ndarray             # fp32 [d_ff, d]   row n = neuron n's gate vector
    w_up: np.ndarray               # fp32 [d_ff, d]
    w_down: np.ndarray             # fp32 [d, d_ff]   column n = neuron n's output vector
    neuron_perm: np.ndarray        # int32 [d_ff]     expert e owns perm[e*m:(e+1)*m]
    rep_idx: np.ndarray            # int32 [N_r]      original index of expert j's representative
    gate_scale_u: Optional[np.ndarray] = None   # fp32 [N_r]
    select_bias_b: Optional[np.ndarray] = None  # fp32 [N_r]


def _normal(rng: np.random.Generator, shape, std: float, dtype: str) -> np.ndarray:
    a = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return round_to_storage(a, dtype)


def draw_tokens(rng: np.random.Generator, n_tokens: int, shape: LayerShape) -> np.ndarray:
    return _normal(rng, (n_tokens, shape.d_model), 1.0, shape.dtype)


def draw_layer(rng: np.random.Generator, shape: LayerShape) -> LayerInputs:
    """W_gate, W_up, W_down, perm in that order; representative of routed
    expert j = first neuron of its slice."""
    if shape.d_ff % shape.n_experts:
        raise ValueError("d_ff must be a multiple of n_experts")
    w_gate = _normal(rng, (shape.d_ff, shape.d_model), WEIGHT_STD, shape.dtype)
    w_up = _normal(rng, (shape.d_ff, shape.d_model), WEIGHT_STD, shape.dtype)
    w_down = _normal(rng, (shape.d_model, shape.d_ff), WEIGHT_STD, shape.dtype)
    perm = rng.permutation(shape.d_ff).astype(np.int32)
    m = shape.m
    rep = perm[(shape.n_shared + np.arange(shape.n_routed)) * m].astype(np.int32)
    return LayerInputs(shape, w_gate, w_up, w_down, perm, rep)


@dataclass
class WorkloadInputs:
    workload: Workload
    x: np.ndarray                          # fp32 [T_max, d]; a run at T uses x[:T]
    layers: List[LayerInputs]              # 1 layer, or n_outer layers (hierarchical)
    w_router: Optional[np.ndarray] = None  # fp32 [n_outer, d] outer router (hierarchical)


def make_inputs(w: Workload) -> WorkloadInputs:
    rng = np.random.Generator(np.random.PCG64(w.seed))
    x = draw_tokens(rng, w.t_max, w.shape)
    if w.n_outer == 0:
        return WorkloadInputs(w, x, [draw_layer(rng, w.shape)])
    layers = [draw_layer(rng, w.shape) for _ in range(w.n_outer)]
    w_router = _normal(rng, (w.n_outer, w.shape.d_model), WEIGHT_STD, w.shape.dtype)
    return WorkloadInputs(w, x, layers, w_router)


# --------------------------------------------------------------------------
# skewed-load target (input preparation for the Zipf workload)
# --------------------------------------------------------------------------
def zipf_target_shares(n_routed: int, top_k: int, s: float) -> np.ndarray:
    """Share of the T*N_k routed rows each expert should receive: p_i ~ i^-s,
    clipped at 1/N_k (an expert can be picked at most once per token) with the
    excess spread over the rest in proportion (water-filling)."""
    p = np.arange(1, n_routed + 1, dtype=np.float64) ** (-s)
    p /= p.sum()
    cap = 1.0 / top_k
    fixed = np.zeros(n_routed, dtype=bool)
    for _ in range(n_routed):
        over = (p > cap + 1e-15) & ~fixed
        if not over.any():
            break
        fixed |= over
        p[fixed] = cap
        rest = ~fixed
        p[rest] *= (1.0 - cap * fixed.sum()) / p[rest].sum()
    return p
