"""-m gpu: the data-parallel pieces of the balanced clustering (centroid update, distance matrix,
representative neurons) through the C-ABI against the CPU oracle.  Inputs (the binary activation
matrix, the assignments) are made on the CPU; everything compared is integer and must match exactly:
the GPU's scaled squared distance against size^2 * d^2 of the oracle's real-valued definition."""
import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding

pytestmark = pytest.mark.gpu


def _activation_matrix(seed, q, d_h, k_a):
    """A [q, d_h] with K_a ones per row; a few neurons are popular, as in the paper's rate histogram."""
    rng = np.random.default_rng(seed)
    scale = np.exp(rng.normal(scale=1.0, size=d_h))
    h = rng.normal(size=(q, d_h)) * scale
    return oracle.atopk(h, k_a)


def _dev(a, dtype):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a).astype(dtype)).cuda()


def _check_distances(s_gpu, sizes, d_ref):
    want = np.rint((d_ref * sizes[None, :]) ** 2).astype(np.int64)
    np.testing.assert_array_equal(s_gpu, want)
    np.testing.assert_allclose(np.sqrt(s_gpu.astype(np.float64)) / sizes[None, :], d_ref, rtol=1e-9, atol=1e-9)


@pytest.mark.parametrize("q,n_experts,n_shared,m,k_a", [(300, 8, 2, 8, 6), (77, 4, 1, 5, 3), (2048, 8, 2, 172, 10),
                                                        (1000, 32, 4, 12, 10)])
def test_clustering_pieces(q, n_experts, n_shared, m, k_a):
    import torch
    d_h, n_r = n_experts * m, n_experts - n_shared
    a = _activation_matrix(q + m, q, d_h, k_a)
    counts = oracle.activation_counts(a)
    shared = oracle.select_shared(counts, n_shared * m)
    cent_idx = oracle.initial_centroids(counts, shared, n_r)
    rest = np.setdiff1d(np.arange(d_h), shared)                       # the N_r * m neurons to cluster
    assert len(rest) == n_r * m and np.isin(cent_idx, rest).all()
    c = a[:, rest]

    bits = _dev(oracle.pack_columns(a).view(np.int32), np.int32)
    count = torch.full((n_r, q), -7, dtype=torch.int32, device="cuda")
    size = torch.full((n_r,), -7, dtype=torch.int32, device="cuda")

    # initial centroids: cluster j = neuron cent_idx[j] alone
    binding.cluster_update(bits, q, _dev(cent_idx, np.int32), _dev(np.arange(n_r), np.int32), count, size)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(size.cpu().numpy(), 1)
    np.testing.assert_array_equal(count.cpu().numpy(), a[:, cent_idx].T)
    rest_dev = _dev(rest, np.int32)
    s0 = binding.cluster_distances(bits, q, rest_dev, count, size).cpu().numpy()
    d0 = oracle.centroid_distances(c, a[:, cent_idx])
    _check_distances(s0, np.ones(n_r), d0)
    ham = (c[:, :, None] != a[:, cent_idx][:, None, :]).sum(axis=0)   # binary centroids: Hamming distance
    np.testing.assert_array_equal(s0, ham)

    # one K-means round: balanced assignment on the CPU, update + distances + representatives on the GPU
    assign = oracle.balanced_assignment(d0, m)
    assign_dev = _dev(assign, np.int32)
    binding.cluster_update(bits, q, rest_dev, assign_dev, count, size)
    cent = oracle.cluster_update(c, assign, a[:, cent_idx])
    torch.cuda.synchronize()
    sizes = size.cpu().numpy()
    np.testing.assert_array_equal(sizes, m)
    np.testing.assert_array_equal(count.cpu().numpy().T / sizes[None, :].astype(np.float64), cent)
    s1_dev = binding.cluster_distances(bits, q, rest_dev, count, size)
    s1 = s1_dev.cpu().numpy()
    d1 = oracle.centroid_distances(c, cent)
    _check_distances(s1, sizes.astype(np.float64), d1)
    reps = binding.cluster_representatives(s1_dev, rest_dev, assign_dev).cpu().numpy()
    reps_ref = oracle.representatives(c, assign, cent)
    for j in range(n_r):
        members = np.nonzero(assign == j)[0]
        best = members[s1[members, j] == s1[members, j].min()].min()   # smallest distance, then lowest position
        assert reps[j] == rest[best]
        assert abs(d1[reps_ref[j], j] - d1[best, j]) <= 1e-12           # the oracle's pick is as close

    # a cluster without members keeps its centroid; unassigned rows are ignored
    before_c, before_s = count.clone(), size.clone()
    partial = assign.copy()
    partial[partial == 0] = -1
    partial[partial == 1] = n_r + 5
    binding.cluster_update(bits, q, rest_dev, _dev(partial, np.int32), count, size)
    want = oracle.cluster_update(c, np.where((partial >= 0) & (partial < n_r), partial, -1), cent)
    torch.cuda.synchronize()
    assert torch.equal(count[:2], before_c[:2]) and torch.equal(size[:2], before_s[:2])
    np.testing.assert_array_equal(count.cpu().numpy().T / size.cpu().numpy()[None, :].astype(np.float64), want)
    reps = binding.cluster_representatives(s1_dev, rest_dev, _dev(partial, np.int32)).cpu().numpy()
    assert reps[0] == -1 and reps[1] == -1 and (reps[2:] >= 0).all()


def test_cluster_call_contract():
    import torch
    bits = torch.zeros((8, 2), dtype=torch.int32, device="cuda")
    idx = torch.arange(8, dtype=torch.int32, device="cuda")
    count = torch.zeros((33, 40), dtype=torch.int32, device="cuda")
    size = torch.ones(33, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CmoeError) as e:
        binding.cluster_update(bits, 40, idx, idx, count, size)           # 33 clusters
    assert e.value.status == -1
    with pytest.raises(binding.CmoeError) as e:
        binding.cluster_update(bits, 100, idx, idx, count[:4], size[:4])  # 100 tokens do not fit 2 words
    assert e.value.status == -1
    s = binding.cluster_distances(bits, 40, idx[:0], count[:4], size[:4])  # no neurons: only the norms
    assert s.shape == (0, 4)
