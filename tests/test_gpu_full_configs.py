"""-m gpu: the five full-size workloads in the launch configuration bench.py times.
Routing, counts, offsets and the permutation are compared for every token (bit-exact
outside the near-tie margin); outputs on a stratified sample of a few hundred tokens
(batch ends, tile edges of the shared rows, first and last row of every routed group,
every 128-row tile edge of the largest and the smallest group, plus a seeded random
draw) that the oracle evaluates one expert batch at a time."""
import functools
import numpy as np
import pytest

import bench
from paper_2502_04416_b200 import torch_io, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu



def _sample(n_tok, seed):
    if n_tok <= 64:
        return None
    return functools.partial(parity.stratified_tokens, seed=seed)


@pytest.mark.parametrize("name", ["c2_llama2_7b", "c3_llama3_8b", "c5_skew_13b"])
def test_plain_workloads_full_size(name):
    inputs = bench.prepare_inputs(name)
    w = inputs.workload
    lay = inputs.layers[0]
    if w.zipf_s:
        assert lay.select_bias_b is not None, "selection-bias fixture missing"
    layer = torch_io.layer_from_workload(inputs, w.t_max)
    for t in w.tokens:
        st = parity.check_plain_layer(layer, lay, inputs.x[:t], sample_tokens=_sample(t, t))
        assert st["differing"] <= st["near_tie"]
        assert sum(st["counts"]) == t * w.shape.top_k
        print(name, t, {k: st.get(k) for k in ("near_tie", "differing", "sampled", "max_rel", "mean_rel")},
              "counts", st["counts"])
        if w.zipf_s:                                     # the load really is skewed as designed
            share = np.array(st["counts"]) / sum(st["counts"])
            target = wl.zipf_target_shares(w.shape.n_routed, w.shape.top_k, w.zipf_s)
            assert np.abs(share - target).max() < 0.01
    layer.destroy()


@pytest.mark.parametrize("name,tokens", [("c2_llama2_7b", (100, 128)), ("c3_llama3_8b", (96,)), ("c5_skew_13b", (128,))])
def test_wide_decode_full_width(name, tokens):
    """65 to 128 rows at the full model width: the wide weights-on-M kernels (128 token columns per tile)."""
    inputs = bench.prepare_inputs(name)
    lay = inputs.layers[0]
    layer = torch_io.layer_from_workload(inputs, 128)
    for t in tokens:
        st = parity.check_plain_layer(layer, lay, inputs.x[:t])
        assert st["differing"] <= st["near_tie"]
        assert sum(st["counts"]) == t * inputs.workload.shape.top_k
    layer.destroy()


def test_hierarchical_workload_full_size():
    inputs = bench.prepare_inputs("c4_hier_8x7b")
    w = inputs.workload
    layer = torch_io.layer_from_workload(inputs, w.t_max)
    st = parity.check_hier_layer(layer, inputs, inputs.x, sample_tokens=_sample(w.t_max, 4))
    assert st["differing"] <= st["near_tie"]
    print("c4", st)
    layer.destroy()
