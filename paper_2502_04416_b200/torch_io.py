"""Moves seeded workload arrays to the device and builds layers from them
(marshalling only: numpy fp32 arrays holding storage-exact values <-> CUDA tensors)."""
from __future__ import annotations

import numpy as np

from . import binding, workloads as wl


def to_device(a: np.ndarray, dtype: str):
    import torch
    if dtype == "bf16":
        bits = wl.f32_to_bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_host(t) -> np.ndarray:
    import torch
    if t.dtype == torch.bfloat16:
        return wl.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.cpu().numpy()


def layer_from_inputs(lay: wl.LayerInputs, max_tokens: int) -> binding.Layer:
    s = lay.shape
    return binding.Layer.create(
        to_device(lay.w_gate, s.dtype), to_device(lay.w_up, s.dtype), to_device(lay.w_down, s.dtype),
        lay.neuron_perm, lay.rep_idx, s.n_experts, s.n_shared, s.top_k, max_tokens,
        lay.gate_scale_u, lay.select_bias_b)


def layer_from_workload(inputs: wl.WorkloadInputs, max_tokens: int) -> binding.Layer:
    """A plain layer, or the hierarchical layer over the workload's outer experts."""
    w = inputs.workload
    if not w.n_outer:
        return layer_from_inputs(inputs.layers[0], max_tokens)
    inner = [layer_from_inputs(l, 8) for l in inputs.layers]
    return binding.Layer.create_hier(to_device(inputs.w_router, w.shape.dtype), inner,
                                     w.outer_top_k, max_tokens)
