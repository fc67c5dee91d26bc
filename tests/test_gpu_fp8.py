"""-m gpu: FP8 (E4M3, power-of-two scale per output channel) expert weights (Section 6 of the
paper: composability with post-training quantisation; the format is this library's reading).
The quantiser is integer work and is compared bit for bit with the oracle; the quantised
layer's forward is compared with the oracle's forward on the same dequantised weights at the
tolerances of the bf16 layer."""
import dataclasses

import numpy as np
import pytest

import bench
from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, torch_io, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


def _quantised(lay):
    s = lay.shape
    return oracle.quantise_expert_weights(lay.w_gate, lay.w_up, lay.w_down, lay.neuron_perm, s.n_experts, s.n_shared)


def test_quantise_rows_bit_exact():
    import torch
    rng = np.random.default_rng(31)
    w = rng.normal(scale=0.02, size=(300, 1000)).astype(np.float32)
    w[0] = 0.0                                                   # all-zero channel
    w[1, :6] = [448.0, -448.0, 1.0625, 1.1875, 2.0 ** -9, 2.0 ** -10]     # scale 1: ties and subnormal codes
    w[2] *= 2.0 ** 40
    w[3] *= 2.0 ** -60
    w[4, 5:] = 0.0
    w[5] = np.where(np.arange(1000) == 7, 1.0, w[5] * 2.0 ** -12)           # one large weight, the rest subnormal codes
    w = wl.round_to_storage(w, "bf16")
    codes, scale, deq = binding.quantise_rows_fp8(parity.to_device(w, "bf16"), want_dequantised=True)
    torch.cuda.synchronize()
    want_codes, want_e = oracle.quantise_rows_fp8(w)
    np.testing.assert_array_equal(scale.cpu().numpy(), np.ldexp(1.0, want_e).astype(np.float32))
    np.testing.assert_array_equal(codes.cpu().numpy(), want_codes)
    np.testing.assert_array_equal(parity.to_host(deq), oracle.dequantise_rows_fp8(want_codes, want_e).astype(np.float32))
    assert (want_codes[5] & 0x78 == 0).sum() > 100               # the subnormal range really is exercised
    odd = parity.to_device(w[:7, :333], "bf16").contiguous()     # odd column count
    codes, scale = binding.quantise_rows_fp8(odd)
    want_codes, want_e = oracle.quantise_rows_fp8(w[:7, :333])
    np.testing.assert_array_equal(codes.cpu().numpy(), want_codes)


SHAPES = [
    ("c2_llama2_7b", 256, None, (1, 2, 16, 64, 300)),    # decode sizes stream FP8, 300 rows read the bf16 copies
    ("c3_llama3_8b", 256, None, (32, 5)),
    ("c2_llama2_7b", 1024, 768, (1, 7, 64)),             # K split 2-4 ways per tile
    ("c5_skew_13b", 320, None, (40,)),
]


@pytest.mark.parametrize("name,d,m,tokens", SHAPES, ids=[f"{s[0]}-d{s[1]}-m{s[2]}" for s in SHAPES])
def test_quantised_layer_small(name, d, m, tokens):
    inp = wl.make_inputs(wl.shrunk(wl.WORKLOADS[name], d_model=d, tokens=tokens, m=m))
    lay = inp.layers[0]
    if wl.WORKLOADS[name].zipf_s:
        rng = np.random.default_rng(2)
        lay.gate_scale_u = rng.normal(scale=0.5, size=lay.shape.n_routed).astype(np.float32)
    layer = parity.gpu_layer(lay, max(tokens))
    before = {t: parity.to_host(layer.forward(parity.to_device(inp.x[:t], "bf16"))) for t in tokens}
    layer.quantise_fp8()
    layer.quantise_fp8()                                          # idempotent
    q = _quantised(lay)
    for t in tokens:
        st = parity.check_plain_layer(layer, lay, inp.x[:t], expert_weights=q)
        assert st["differing"] <= st["near_tie"]
        after = parity.to_host(layer.forward(parity.to_device(inp.x[:t], "bf16")))
        assert np.abs(after - before[t]).max() > 0                # the weights really changed
    layer.destroy()


def test_subnormal_codes_reach_the_output():
    """Every weight row holds one weight of 1 and otherwise multiples 1..7 of 2^-17 of it (subnormal
    E4M3 codes); the token is zero at the large weight's position, so the result is made of the
    subnormal codes alone and vanishes if the expansion to bf16 drops them."""
    shape = wl.LayerShape(256, 8 * 64, 8, 2, 2, "bf16")
    rng = np.random.Generator(np.random.PCG64(9))
    x = wl.draw_tokens(rng, 8, shape)
    lay = wl.draw_layer(rng, shape)
    x[:, 3] = 0.0
    for w_ in (lay.w_gate, lay.w_up):
        w_[:] = wl.round_to_storage(np.ldexp(np.sign(w_) * rng.integers(1, 8, size=w_.shape), -17).astype(np.float32), "bf16")
        w_[:, 3] = 1.0
    layer = parity.gpu_layer(lay, 8)
    layer.quantise_fp8()
    q = _quantised(lay)
    assert ((q["gate_codes"] & 0x78) == 0).mean() > 0.9
    st = parity.check_plain_layer(layer, lay, x, expert_weights=q)
    got = parity.to_host(layer.forward(parity.to_device(x, "bf16")))
    assert np.abs(got).max() > 0
    layer.destroy()


def test_quantised_hierarchical_layer():
    """FP8 weights under a top-level router (Section 4.4): every outer expert's blocks get their own scales;
    decode-sized batches (outer rows <= 64) stream the codes, larger ones read the dequantised bf16 copies."""
    inp = wl.make_inputs(wl.shrunk(wl.WORKLOADS["c4_hier_8x7b"], d_model=256, tokens=(150,), m=224))
    inners = [parity.gpu_layer(lay, 8) for lay in inp.layers]
    layer = binding.Layer.create_hier(parity.to_device(inp.w_router, "bf16"), inners, 2, 150)
    layer.quantise_fp8()
    q = [_quantised(lay) for lay in inp.layers]
    for t in (3, 20, 32, 150):
        st = parity.check_hier_layer(layer, inp, inp.x[:t], expert_weights=q)
        assert st["differing"] <= st["near_tie"]
    layer.destroy()


def test_quantise_refusals():
    inp = wl.make_inputs(wl.WORKLOADS["c1_tiny_fp32"])
    layer = parity.gpu_layer(inp.layers[0], 64)
    with pytest.raises(binding.CmoeError) as e:
        layer.quantise_fp8()                                      # fp32 layer
    assert e.value.status == -7
    layer.destroy()


@pytest.mark.parametrize("name,tokens", [("c2_llama2_7b", (1, 2, 16, 64)), ("c3_llama3_8b", (2, 32))])
def test_quantised_decode_full_size(name, tokens):
    inputs = bench.prepare_inputs(name)
    lay = inputs.layers[0]
    layer = torch_io.layer_from_workload(inputs, 64)
    layer.quantise_fp8()
    q = _quantised(lay)
    for t in tokens:
        st = parity.check_plain_layer(layer, lay, inputs.x[:t], expert_weights=q)
        assert st["differing"] <= st["near_tie"]
        print(name, t, {k: st[k] for k in ("near_tie", "differing", "max_rel", "mean_rel")})
    layer.destroy()
