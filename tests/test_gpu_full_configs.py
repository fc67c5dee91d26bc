"""-m gpu: the five full-size workloads in the launch configuration bench.py times.
Routing, counts, offsets and the permutation are compared for every token (bit-exact
outside the near-tie margin); outputs on a seeded sample of tokens that the oracle
evaluates one expert batch at a time."""
import numpy as np
import pytest

import bench
from paper_2502_04416_b200 import torch_io, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

N_SAMPLE = 48


def _sample(n_tok, seed):
    if n_tok <= N_SAMPLE:
        return None
    rng = np.random.default_rng(seed)
    ids = np.sort(rng.choice(n_tok, size=N_SAMPLE, replace=False))
    ids[0], ids[-1] = 0, n_tok - 1                      # first and last row of the batch
    return ids


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
        print(name, t, {k: st[k] for k in ("near_tie", "differing", "max_rel", "mean_rel")},
              "counts", st["counts"])
        if w.zipf_s:                                     # the load really is skewed as designed
            share = np.array(st["counts"]) / sum(st["counts"])
            target = wl.zipf_target_shares(w.shape.n_routed, w.shape.top_k, w.zipf_s)
            assert np.abs(share - target).max() < 0.01
    layer.destroy()


def test_hierarchical_workload_full_size():
    inputs = bench.prepare_inputs("c4_hier_8x7b")
    w = inputs.workload
    layer = torch_io.layer_from_workload(inputs, w.t_max)
    st = parity.check_hier_layer(layer, inputs, inputs.x, sample_tokens=_sample(w.t_max, 4))
    assert st["differing"] <= st["near_tie"]
    print("c4", st)
    layer.destroy()
