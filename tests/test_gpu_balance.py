"""-m gpu: expert utilisation and the load-balancing bias update (Section 4.3) on the device,
against the oracle's bias_update on the counts of the same forward."""
import dataclasses

import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, torch_io, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


def _layer(name, d, m, tokens, seed=None):
    w = wl.shrunk(wl.WORKLOADS[name], d_model=d, tokens=(tokens,), m=m)
    if seed is not None:
        w = dataclasses.replace(w, seed=seed)
    return wl.make_inputs(w)


@pytest.mark.parametrize("name,target", [("c3_llama3_8b", None), ("c5_skew_13b", "zipf"), ("c2_llama2_7b", None)])
def test_bias_update_matches_oracle(name, target):
    import torch
    inp = _layer(name, 256, 64, 700)
    lay = inp.layers[0]
    s = lay.shape
    rng = np.random.default_rng(3)
    lay.select_bias_b = rng.normal(scale=0.02, size=s.n_routed).astype(np.float32)
    layer = parity.gpu_layer(lay, 700)
    layer.forward(torch_io.to_device(inp.x, "bf16"))
    torch.cuda.synchronize()
    counts = layer.routing(700, s.n_routed)["counts"]
    tgt = None if target is None else wl.zipf_target_shares(s.n_routed, s.top_k, 1.2).astype(np.float32)
    util = layer.update_bias(gamma=1e-3, target_share=tgt)
    _, b_new = layer.get_gate_params()
    np.testing.assert_allclose(util, counts / counts.sum(), rtol=1e-6)
    want = oracle.bias_update(lay.select_bias_b, counts, None if tgt is None else tgt.astype(np.float64), 1e-3)
    np.testing.assert_allclose(b_new, want, rtol=0, atol=2e-7)
    moved = np.abs(b_new - lay.select_bias_b)
    assert np.all((np.abs(moved - 1e-3) < 1e-6) | (moved == 0)) and moved.max() > 0
    # the updated bias is what the next forward routes with
    lay.select_bias_b = b_new
    parity.check_plain_layer(layer, lay, inp.x)
    layer.destroy()


def test_bias_update_hierarchical_is_per_outer_expert():
    import torch
    w = wl.shrunk(wl.WORKLOADS["c4_hier_8x7b"], d_model=256, tokens=(400,), m=64)
    inp = wl.make_inputs(w)
    nr = w.shape.n_routed
    inner = [parity.gpu_layer(l, 8) for l in inp.layers]
    layer = binding.Layer.create_hier(torch_io.to_device(inp.w_router, "bf16"), inner, 2, 400)
    layer.forward(torch_io.to_device(inp.x, "bf16"))
    torch.cuda.synchronize()
    counts = layer.routing(400, nr)["counts"].reshape(w.n_outer, nr)
    util = layer.update_bias(gamma=5e-3).reshape(w.n_outer, nr)
    _, b = layer.get_gate_params()
    for i in range(w.n_outer):
        np.testing.assert_allclose(util[i], counts[i] / counts[i].sum(), rtol=1e-6)
        np.testing.assert_allclose(b.reshape(w.n_outer, nr)[i], oracle.bias_update(np.zeros(nr), counts[i], None, 5e-3),
                                   rtol=0, atol=1e-7)
    layer.destroy()


def test_repeated_updates_balance_the_load():
    """Iterating forward + update drives the utilisation towards uniform (the paper's
    load-balancing figure, qualitatively, on synthetic tokens)."""
    import torch
    inp = _layer("c2_llama2_7b", 128, 32, 2048, seed=9)
    lay = inp.layers[0]
    nr = lay.shape.n_routed
    lay.select_bias_b = np.linspace(-0.05, 0.05, nr).astype(np.float32)      # start skewed
    layer = parity.gpu_layer(lay, 2048)
    x = torch_io.to_device(inp.x, "bf16")
    out = torch.empty_like(x)
    dev = []
    for it in range(200):
        layer.forward(x, out)
        util = layer.update_bias(gamma=1e-3)
        dev.append(float(np.abs(util - 1.0 / nr).max()))
    assert dev[0] > 0.05
    assert min(dev[-20:]) < 0.25 * dev[0]
    layer.destroy()
