"""-m gpu: the CUDA path, called through the C-ABI, against the CPU oracle on the
same seeded inputs.  Small shapes keep each expert's ragged tile tails (m = 1376,
448, 864 ...) and token counts that are not multiples of any tile."""
import ctypes as C
import dataclasses

import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

PATHS = [binding.GEMM_SIMT, binding.GEMM_AUTO]
PATH_IDS = ["simt", "auto"]


def _inputs(name, d_model=None, tokens=None, m=None, n_outer=None, seed=None):
    w = wl.WORKLOADS[name]
    if d_model is not None:
        w = wl.shrunk(w, d_model=d_model, tokens=tokens, m=m, n_outer=n_outer)
    if seed is not None:
        w = dataclasses.replace(w, seed=seed)
    return wl.make_inputs(w)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_c1_tiny_fp32(path):
    inp = _inputs("c1_tiny_fp32")
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 64)
    layer.set_gemm_path(path)
    st = parity.check_plain_layer(layer, lay, inp.x)
    assert st["differing"] == 0
    assert st["max_rel"] < 1e-4 and st["mean_rel"] < 1e-4      # fp32 end to end
    layer.destroy()


SMALL = [
    ("c2_llama2_7b", 256, None, (1, 2, 16, 77, 300)),   # 1 and 2 rows: the plain-load streamers
    ("c3_llama3_8b", 256, None, (33, 50, 64, 517)),   # 17..64 rows, more than 8 router columns: 16-row router chunks
    ("c5_skew_13b", 320, None, (129, 700)),
    ("c2_llama2_7b", 512, 200, (1000,)),       # m = 200: neither a multiple of 16 nor of 64
    ("c2_llama2_7b", 1024, 768, (1, 7, 64)),   # decode GEMMs with K split 2-4 ways per tile
]


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("name,d,m,tokens", SMALL, ids=[f"{s[0]}-d{s[1]}-m{s[2]}" for s in SMALL])
def test_small_shapes(name, d, m, tokens, path):
    inp = _inputs(name, d_model=d, tokens=tokens, m=m)
    lay = inp.layers[0]
    if wl.WORKLOADS[name].zipf_s:
        rng = np.random.default_rng(1)
        lay.select_bias_b = rng.normal(scale=0.05, size=lay.shape.n_routed).astype(np.float32)
        lay.gate_scale_u = rng.normal(scale=0.5, size=lay.shape.n_routed).astype(np.float32)
    layer = parity.gpu_layer(lay, max(tokens))
    layer.set_gemm_path(path)
    for t in tokens:
        st = parity.check_plain_layer(layer, lay, inp.x[:t])
        assert st["differing"] <= st["near_tie"]
    layer.destroy()


@pytest.mark.parametrize("tokens", [65, 100, 128, 129, 200, 256, 513, 1000])
def test_mid_size_batches(tokens):
    """65 to 1023 rows: split-K router over 64-row chunks (up to 512 rows), the wide weights-on-M kernels
    up to 128 rows, CTA-pair GEMMs from 256 rows, groups of a few dozen to a few hundred rows with ragged tiles."""
    inp = _inputs("c2_llama2_7b", d_model=512, tokens=(1000,), m=1376)
    lay = inp.layers[0]
    rng = np.random.default_rng(3)
    lay.gate_scale_u = rng.normal(scale=0.5, size=lay.shape.n_routed).astype(np.float32)
    layer = parity.gpu_layer(lay, 1000)
    st = parity.check_plain_layer(layer, lay, inp.x[:tokens])
    assert st["differing"] <= st["near_tie"]
    layer.destroy()


def test_cta_pair_gemms():
    """Expert GEMMs on tcgen05 CTA pairs (cta_group::2): groups with odd and even m-tile counts."""
    inp = _inputs("c2_llama2_7b", d_model=256, tokens=(1300, 1027), m=1376 // 4 * 4)
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 1300)
    layer.set_gemm_path(binding.GEMM_TENSOR_PAIRS)
    for t in (1300, 1027):
        st = parity.check_plain_layer(layer, lay, inp.x[:t])
        assert st["differing"] <= st["near_tie"]
    layer.destroy()


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_hierarchical_small(path):
    inp = _inputs("c4_hier_8x7b", d_model=256, tokens=(257,), m=224)
    inners = [parity.gpu_layer(lay, 8) for lay in inp.layers]
    layer = binding.Layer.create_hier(parity.to_device(inp.w_router, "bf16"), inners, 2, 300)
    layer.set_gemm_path(path)
    st = parity.check_hier_layer(layer, inp, inp.x)
    assert st["differing"] <= st["near_tie"]
    st = parity.check_hier_layer(layer, inp, inp.x[:3])          # most outer experts empty
    st = parity.check_hier_layer(layer, inp, inp.x[:100])        # 200 outer rows: router chunks straddle outer experts
    assert st["differing"] <= st["near_tie"]
    st = parity.check_hier_layer(layer, inp, inp.x[:50])         # 100 outer rows: the wide weights-on-M kernels
    assert st["differing"] <= st["near_tie"]
    layer.destroy()


def test_hierarchical_outer_near_ties():
    """Outer logits within the 1e-3 margin (Section 4.4's top-level router): two pairs of outer
    experts get router rows that differ in one coordinate by 2^-27, so whenever such a pair
    straddles the outer cut the fp32 logits cannot tell its members apart while the fp64 oracle
    can.  The CUDA choice must then be an admissible trade and everything downstream (outer
    permutation, inner routing, output) must agree once the oracle takes that choice."""
    inp = _inputs("c4_hier_8x7b", d_model=256, tokens=(600,), m=64)
    w_r = inp.w_router
    for a, b_, col in ((1, 4, 3), (2, 6, 100)):
        w_r[b_] = w_r[a]
        w_r[a, col] = np.float32(2.0 ** -20)
        w_r[b_, col] = np.float32(2.0 ** -20 * (1 + 2.0 ** -7))       # both exact in bf16
    inners = [parity.gpu_layer(lay, 8) for lay in inp.layers]
    layer = binding.Layer.create_hier(parity.to_device(w_r, "bf16"), inners, 2, 600)
    st = parity.check_hier_layer(layer, inp, inp.x)
    print("outer near-ties:", st["outer_near_tie"], "differing:", st["outer_differing"])
    assert st["outer_near_tie"] >= 50                    # the planted pairs straddle the cut often
    assert st["outer_differing"] <= st["outer_near_tie"]
    layer.destroy()


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_degenerate_structures(path):
    base = wl.shrunk(wl.WORKLOADS["c2_llama2_7b"], d_model=128, tokens=(70,), m=80)
    for n_shared, top_k in [(2, 0), (0, 2), (2, 6), (8, 0), (0, 8)]:
        shape = dataclasses.replace(base.shape, n_shared=n_shared, top_k=top_k)
        inp = wl.make_inputs(dataclasses.replace(base, shape=shape))
        lay = inp.layers[0]
        layer = parity.gpu_layer(lay, 70)
        layer.set_gemm_path(path)
        st = parity.check_plain_layer(layer, lay, inp.x)
        parity.check_plain_layer(layer, lay, inp.x[:1])       # one row: the CUDA-core path on the automatic choice
        parity.check_plain_layer(layer, lay, inp.x[5:6])
        if top_k == shape.n_routed:           # every expert on with unit gates: the dense FFN
            import torch
            got = parity.to_host(layer.forward(parity.to_device(inp.x, "bf16")))
            torch.cuda.synchronize()
            parity.check_output(got, oracle.dense_ffn(inp.x, lay.w_gate, lay.w_up, lay.w_down))
        layer.destroy()


def test_call_contract():
    import torch
    inp = _inputs("c2_llama2_7b", d_model=128, tokens=(40,), m=48)
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 32)
    x = parity.to_device(inp.x, "bf16")
    out = torch.full_like(x, 7.0)
    layer.forward(x[:0], out[:0])                                 # T = 0: no-op
    torch.cuda.synchronize()
    assert float(out.float().min()) == 7.0
    with pytest.raises(binding.CmoeError) as e:
        layer.forward(x, out)                                     # 40 > max_tokens
    assert e.value.status == -4
    with pytest.raises(binding.CmoeError) as e:
        layer.forward(x[:8], x[:8])                               # aliasing
    assert e.value.status == -1
    with pytest.raises(binding.CmoeError) as e:                   # out 16- but not 32-byte aligned: refused on the
        layer.forward(x[:8], out.view(-1)[8:8 + 8 * 128].view(8, 128))   # host, nothing is launched
    assert e.value.status == -1
    a = layer.forward(x[:32]).clone()
    b = layer.forward(x[:32]).clone()
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))  # run-to-run bit identical
    # gate parameters can be replaced after create
    u = np.linspace(-1, 1, lay.shape.n_routed).astype(np.float32)
    layer.set_gate_params(gate_scale_u=u)
    lay.gate_scale_u = u
    parity.check_plain_layer(layer, lay, inp.x[:32])
    layer.destroy()


def test_forward_host_matches_device_forward():
    """cmoe_ffn_forward_host (chunked, copies overlapped on side streams) against the device-buffer
    call: a token's result does not depend on what else is in its batch (Eq. moe_output is per x), so
    chunks processed by the same kernel family give the same bits; a ragged last chunk, a single
    chunk and pageable host memory are covered."""
    import torch
    inp = _inputs("c2_llama2_7b", d_model=256, tokens=(2900,), m=160)
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 2900)
    x = parity.to_device(inp.x, "bf16")
    ref = layer.forward(x).cpu()
    torch.cuda.synchronize()
    x_pin = x.cpu().pin_memory()
    out_pin = torch.empty_like(x_pin).pin_memory()
    for chunk in (1024, 700, 0, 2900, 5000):
        out_pin.zero_()
        layer.forward_host(x_pin, out_pin, chunk)
        torch.cuda.synchronize()
        assert layer.status() == 0
        assert torch.equal(out_pin.view(torch.int16), ref.view(torch.int16)), chunk
    for _ in range(3):                                  # back-to-back calls reuse the staging buffers
        layer.forward_host(x_pin, out_pin, 1024)
    torch.cuda.synchronize()
    assert torch.equal(out_pin.view(torch.int16), ref.view(torch.int16))
    x_page, out_page = x.cpu(), torch.zeros_like(ref)   # pageable memory: serial copies, same result
    layer.forward_host(x_page[:1500], out_page[:1500], 600)
    torch.cuda.synchronize()
    assert torch.equal(out_page[:1500].view(torch.int16), ref[:1500].view(torch.int16))
    parity.check_output(parity.to_host(out_pin), oracle.cmoe_layer_forward(inp.x, **parity.oracle_kwargs(lay))[0])
    layer.destroy()


def test_wait_timeout_is_reported_and_recovered():
    """The give-up path of the bounded device-side waits: a wait that nothing ends runs to its
    (millisecond) limit, the kernel returns normally, the layer's error word carries the code,
    cmoe_layer_status maps it to the timeout status once and clears it, and the layer then
    computes correct results again (tensor path: decode, mid-size and large batches)."""
    import torch
    inp = _inputs("c2_llama2_7b", d_model=256, tokens=(700,), m=160)
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 700)
    parity.check_plain_layer(layer, lay, inp.x[:700])
    assert layer.status() == 0
    layer.selftest_wait_timeout(2_000_000)
    torch.cuda.synchronize()
    w = C.c_int32()
    assert binding.load().cmoe_layer_status(layer._h, C.byref(w)) == -6      # CMOE_ERR_DEVICE_TIMEOUT
    assert w.value == 1                                                       # the wait's own code
    assert layer.status() == 0                                                # reported once, then cleared
    for t in (1, 64, 300, 700):
        parity.check_plain_layer(layer, lay, inp.x[:t])
    with pytest.raises(binding.CmoeError):
        layer.selftest_wait_timeout(10)                                       # limit below the documented range
    layer.destroy()


def test_launch_chaining_is_bit_identical():
    """Programmatic dependent launches change when kernels become resident, never what they compute:
    outputs and routing with chaining on and off agree bit for bit, directly and under graph replay."""
    import torch
    inp = _inputs("c2_llama2_7b", d_model=256, tokens=(1400,), m=160)
    lay = inp.layers[0]
    layer = parity.gpu_layer(lay, 1400)
    x = parity.to_device(inp.x, "bf16")
    for t in (1, 16, 64, 65, 300, 700, 1400):          # decode, mid-size and tcgen05 routers
        layer.set_launch_chaining(False)
        ref = layer.forward(x[:t]).clone()
        ref_routing = layer.routing(t, lay.shape.n_routed)
        layer.set_launch_chaining(True)
        for _ in range(3):
            got = layer.forward(x[:t]).clone()
            torch.cuda.synchronize()
            assert layer.status() == 0
            assert torch.equal(got.view(torch.int16), ref.view(torch.int16)), t
        now = layer.routing(t, lay.shape.n_routed)
        for k in ("topk_idx", "counts", "offsets", "row_token", "row_of"):
            np.testing.assert_array_equal(now[k], ref_routing[k])
        parity.check_plain_layer(layer, lay, inp.x[:t])
    out = torch.empty_like(x[:64])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        layer.forward(x[:64], out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    ref = out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        layer.forward(x[:64], out)
    for _ in range(5):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    layer.destroy()


def test_launch_chaining_hierarchical_is_bit_identical():
    """The same for a layer under a top-level router (Section 4.4): the kernels after the expert router are chained."""
    import torch
    inp = _inputs("c4_hier_8x7b", d_model=256, tokens=(300,), m=224)
    inners = [parity.gpu_layer(lay, 8) for lay in inp.layers]
    layer = binding.Layer.create_hier(parity.to_device(inp.w_router, "bf16"), inners, 2, 300)
    x = parity.to_device(inp.x, "bf16")
    for t in (3, 20, 50, 100, 300):
        layer.set_launch_chaining(False)
        ref = layer.forward(x[:t]).clone()
        layer.set_launch_chaining(True)
        for _ in range(3):
            got = layer.forward(x[:t]).clone()
            torch.cuda.synchronize()
            assert layer.status() == 0
            assert torch.equal(got.view(torch.int16), ref.view(torch.int16)), t
    layer.destroy()


@pytest.mark.parametrize("n_rows,n_k,n_groups", [(1, 2, 6), (255, 2, 6), (256, 4, 28), (257, 4, 28),
                                                 (5000, 2, 56), (16384, 4, 14), (3000, 8, 1000),
                                                 (700, 1, 3), (40, 0, 5)])
def test_token_permute_standalone(n_rows, n_k, n_groups):
    import torch
    rng = np.random.default_rng(n_rows + n_groups)
    sel = np.stack([rng.permutation(n_groups)[:n_k] for _ in range(n_rows)]).astype(np.int32)
    if n_groups > 4 and n_k:
        sel[sel == 2] = 3 if n_k == 1 else sel[sel == 2]          # an empty group when n_k == 1
    dev = torch.from_numpy(sel).cuda() if n_k else torch.zeros((n_rows, 0), dtype=torch.int32).cuda()
    cnt, off, row_token, row_of = binding.token_permute(dev, n_groups)
    torch.cuda.synchronize()
    w_cnt, w_off, w_row_token, w_row_of = oracle.token_permutation(sel, n_groups)
    np.testing.assert_array_equal(cnt.cpu().numpy(), w_cnt)
    np.testing.assert_array_equal(off.cpu().numpy(), w_off)
    np.testing.assert_array_equal(row_token.cpu().numpy(), w_row_token)
    np.testing.assert_array_equal(row_of.cpu().numpy(), w_row_of)
