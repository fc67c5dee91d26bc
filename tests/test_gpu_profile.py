"""-m gpu: activation profiling (H, ATopK, activation counts, shared-neuron selection) through the
C-ABI against the CPU oracle.  The top-K_a decision is taken on H as the kernel stores it (bf16 or
fp32), so the oracle's fp64 H is rounded to that type first; rows whose cut lies within one storage
ulp of the next magnitude may trade exactly those boundary neurons, everything else is bit-exact."""
import dataclasses

import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


def _dense_layer_inputs(name, d_model=None, m=None, seed=None):
    """The workload's FFN with every expert shared and neurons in original order."""
    w = wl.WORKLOADS[name]
    if d_model is not None:
        w = wl.shrunk(w, d_model=d_model, tokens=(8,), m=m)
    if seed is not None:
        w = dataclasses.replace(w, seed=seed)
    shape = dataclasses.replace(w.shape, n_shared=w.shape.n_experts, top_k=0)
    inp = wl.make_inputs(dataclasses.replace(w, shape=shape))
    lay = inp.layers[0]
    lay.neuron_perm = np.arange(shape.d_ff, dtype=np.int32)
    lay.rep_idx = np.zeros(0, dtype=np.int32)
    return shape, lay


def _check_profile(shape, lay, x, k_a, chunks, n_select):
    import torch
    q = x.shape[0]
    layer = parity.gpu_layer(lay, max(chunks))
    words = (q + 31) // 32
    bits = torch.zeros((shape.d_ff, words), dtype=torch.int32, device="cuda")
    count = torch.zeros(shape.d_ff, dtype=torch.int32, device="cuda")
    xd = parity.to_device(x, shape.dtype)
    t0 = 0
    for n in chunks:                                   # the calibration set goes through in pieces
        n = min(n, q - t0)
        if n <= 0:
            break
        layer.profile_activations(xd[t0:t0 + n], k_a, bits, count, token0=t0)
        t0 += n
    assert t0 == q
    shared = binding.select_shared(count, n_select)
    torch.cuda.synchronize()
    assert layer.status() == 0
    a_gpu = parity.unpack_activation_bits(bits.cpu().numpy().view(np.uint32), q)
    counts_gpu = count.cpu().numpy()
    shared_gpu = shared.cpu().numpy()
    layer.destroy()

    # A against the oracle (decision in the storage precision; near-tie rows checked and carried over),
    # then the integer work downstream of A: exact
    a_ref, n_patched = parity.reference_activation_matrix(a_gpu, x, lay.w_gate, lay.w_up, k_a, shape.dtype)
    np.testing.assert_array_equal(a_gpu, a_ref)
    np.testing.assert_array_equal(a_gpu.sum(axis=1), k_a)                 # K_a neurons per token
    counts_ref = oracle.activation_counts(a_ref)
    np.testing.assert_array_equal(counts_gpu, counts_ref)
    np.testing.assert_array_equal(shared_gpu, oracle.select_shared(counts_ref, n_select))
    return dict(rows=q, differing=n_patched)


SMALL = [("c2_llama2_7b", 256, 160, 300, 10, (128, 128, 64)),      # tcgen05 path, three chunks
         ("c2_llama2_7b", 256, 160, 45, 3, (40, 64)),              # decode-sized chunks
         ("c3_llama3_8b", 128, 56, 700, 10, (700,)),
         ("c2_llama2_7b", 512, 200, 130, 300, (130,))]             # K_a far from the tail: many storage ties


@pytest.mark.parametrize("name,d,m,q,k_a,chunks", SMALL, ids=[f"{s[0]}-d{s[1]}-q{s[3]}-k{s[4]}" for s in SMALL])
def test_profile_small(name, d, m, q, k_a, chunks):
    shape, lay = _dense_layer_inputs(name, d_model=d, m=m)
    rng = np.random.Generator(np.random.PCG64(77))
    x = wl.round_to_storage(rng.standard_normal((q, shape.d_model), dtype=np.float32), shape.dtype)
    _check_profile(shape, lay, x, k_a, chunks, n_select=2 * (shape.d_ff // shape.n_experts))


def test_profile_fp32_tiny():
    shape, lay = _dense_layer_inputs("c1_tiny_fp32")
    rng = np.random.Generator(np.random.PCG64(78))
    x = rng.standard_normal((64, shape.d_model), dtype=np.float32)
    st = _check_profile(shape, lay, x, 10, (64,), n_select=2 * (shape.d_ff // shape.n_experts))
    assert st["differing"] == 0


def test_profile_full_width():
    """LLaMA-2-7B-shaped FFN (d = 4096, d_h = 11008), K_a = 10 as in the paper's set-up, 512 rows."""
    shape, lay = _dense_layer_inputs("c2_llama2_7b")
    rng = np.random.Generator(np.random.PCG64(79))
    x = wl.round_to_storage(rng.standard_normal((512, shape.d_model), dtype=np.float32), shape.dtype)
    _check_profile(shape, lay, x, 10, (512,), n_select=2 * (shape.d_ff // shape.n_experts))


def test_profile_call_contract():
    import torch
    inp = wl.make_inputs(wl.shrunk(wl.WORKLOADS["c2_llama2_7b"], d_model=128, tokens=(16,), m=48))
    routed = parity.gpu_layer(inp.layers[0], 16)
    x = parity.to_device(inp.x[:16], "bf16")
    bits = torch.zeros((inp.layers[0].shape.d_ff, 1), dtype=torch.int32, device="cuda")
    count = torch.zeros(inp.layers[0].shape.d_ff, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CmoeError) as e:
        routed.profile_activations(x, 4, bits, count)             # a layer with routed experts
    assert e.value.status == -1
    routed.destroy()
    shape, lay = _dense_layer_inputs("c2_llama2_7b", d_model=128, m=48)
    layer = parity.gpu_layer(lay, 16)
    with pytest.raises(binding.CmoeError) as e:
        layer.profile_activations(x, 0, bits, count)              # k_a < 1
    assert e.value.status == -1
    with pytest.raises(binding.CmoeError) as e:
        layer.profile_activations(x, 4, bits, count, token0=20)   # bit position beyond the words given
    assert e.value.status == -4
    layer.profile_activations(x[:0], 4, bits, count)              # no rows: no-op
    torch.cuda.synchronize()
    assert int(count.sum()) == 0
    with pytest.raises(binding.CmoeError):
        binding.select_shared(count, shape.d_ff + 1)
    layer.destroy()
