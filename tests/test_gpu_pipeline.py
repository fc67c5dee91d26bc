"""-m gpu: the restructuring pipeline end to end on the GPU pieces — profile the dense FFN, pick the
shared neurons, cluster the rest (the balanced assignment itself runs on the CPU, as in the paper),
take the representatives, build the restructured layer from that partition and run its forward —
against the same chain evaluated by the CPU oracle."""
import dataclasses

import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


def test_profile_cluster_restructure_forward():
    import torch
    base = wl.shrunk(wl.WORKLOADS["c2_llama2_7b"], d_model=256, tokens=(600,), m=48)
    shape = base.shape                                    # 8 experts of 48 neurons, 2 shared, top-2
    n_r, m, k_a, q = shape.n_routed, shape.d_ff // shape.n_experts, 10, 600
    inp = wl.make_inputs(base)
    ffn = inp.layers[0]                                   # only its dense weights are used from here on
    x_cal = inp.x[:q]

    # ---- GPU: steps 1-4 on the dense FFN (every expert shared, identity order)
    dense_shape = dataclasses.replace(shape, n_shared=shape.n_experts, top_k=0)
    dense = wl.LayerInputs(dense_shape, ffn.w_gate, ffn.w_up, ffn.w_down,
                           np.arange(shape.d_ff, dtype=np.int32), np.zeros(0, dtype=np.int32))
    layer = parity.gpu_layer(dense, q)
    bits = torch.zeros((shape.d_ff, (q + 31) // 32), dtype=torch.int32, device="cuda")
    count = torch.zeros(shape.d_ff, dtype=torch.int32, device="cuda")
    layer.profile_activations(parity.to_device(x_cal, "bf16"), k_a, bits, count)
    shared_and_seeds = binding.select_shared(count, shape.n_shared * m + n_r).cpu().numpy()
    layer.destroy()
    shared, seeds = shared_and_seeds[:shape.n_shared * m], shared_and_seeds[shape.n_shared * m:]
    a_gpu = parity.unpack_activation_bits(bits.cpu().numpy().view(np.uint32), q)

    # ---- oracle: the same steps from the inputs (near-tie ATopK rows checked and carried over)
    a, _ = parity.reference_activation_matrix(a_gpu, x_cal, ffn.w_gate, ffn.w_up, k_a, "bf16")
    counts = oracle.activation_counts(a)
    np.testing.assert_array_equal(count.cpu().numpy(), counts)
    np.testing.assert_array_equal(shared, oracle.select_shared(counts, shape.n_shared * m))
    np.testing.assert_array_equal(seeds, oracle.initial_centroids(counts, shared, n_r))
    rest = np.setdiff1d(np.arange(shape.d_ff), oracle.select_shared(counts, shape.n_shared * m)).astype(np.int32)
    d0_ref = oracle.centroid_distances(a[:, rest], a[:, oracle.initial_centroids(counts, shared, n_r)])
    assign = oracle.balanced_assignment(d0_ref, m)                      # the CPU step of the paper's loop
    cent = oracle.cluster_update(a[:, rest], assign, a[:, seeds])
    d1_ref = oracle.centroid_distances(a[:, rest], cent)
    reps_ref = oracle.representatives(a[:, rest], assign, cent)

    # ---- GPU: one K-means round around that assignment
    rest_d = torch.from_numpy(rest).cuda()
    cc = torch.zeros((n_r, q), dtype=torch.int32, device="cuda")
    size = torch.zeros(n_r, dtype=torch.int32, device="cuda")
    binding.cluster_update(bits, q, torch.from_numpy(seeds.astype(np.int32)).cuda(),
                           torch.arange(n_r, dtype=torch.int32, device="cuda"), cc, size)
    s0 = binding.cluster_distances(bits, q, rest_d, cc, size).cpu().numpy()
    np.testing.assert_array_equal(s0, np.rint(d0_ref ** 2).astype(np.int64))
    assign_d = torch.from_numpy(assign.astype(np.int32)).cuda()
    binding.cluster_update(bits, q, rest_d, assign_d, cc, size)
    s1_d = binding.cluster_distances(bits, q, rest_d, cc, size)
    np.testing.assert_array_equal(s1_d.cpu().numpy(), np.rint((d1_ref * m) ** 2).astype(np.int64))
    reps = binding.cluster_representatives(s1_d, rest_d, assign_d).cpu().numpy()
    for j in range(n_r):                                               # equal distances may sit at different positions
        pos = np.nonzero(rest == reps[j])[0][0]
        assert assign[pos] == j and abs(d1_ref[pos, j] - d1_ref[reps_ref[j], j]) <= 1e-12

    # ---- the restructured layer built from that partition, forward against the oracle
    perm = np.concatenate([np.sort(shared)] + [rest[assign == j] for j in range(n_r)]).astype(np.int32)
    assert sorted(perm.tolist()) == list(range(shape.d_ff))
    lay = wl.LayerInputs(shape, ffn.w_gate, ffn.w_up, ffn.w_down, perm, reps.astype(np.int32))
    moe = parity.gpu_layer(lay, 300)
    st = parity.check_plain_layer(moe, lay, inp.x[:300])
    assert st["differing"] <= st["near_tie"]
    moe.destroy()
