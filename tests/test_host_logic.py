"""CPU-only checks: the C-ABI library builds, loads and exports every declared symbol;
argument validation that needs no device; the workload generators."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2502_04416_b200 import binding, build, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cmoe_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in cmoe.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    seen = {lib.cmoe_status_string(s).decode() for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert lib.cmoe_status_string(-99).decode() == "unknown status"


def _create(lib, cfg, perm, rep, w=1):
    out = C.c_void_p()
    st = lib.cmoe_layer_create(C.byref(cfg), w, w, w, perm.ctypes.data_as(C.c_void_p),
                               rep.ctypes.data_as(C.c_void_p), None, None, None, C.byref(out))
    return st


def test_create_validation_without_device(lib):
    d_ff, n, ns = 64, 8, 2
    perm = np.random.default_rng(0).permutation(d_ff).astype(np.int32)
    rep = perm[(ns + np.arange(n - ns)) * (d_ff // n)].astype(np.int32)
    good = dict(d_model=16, d_ff=d_ff, n_experts=n, n_shared=ns, top_k=2, max_tokens=4, dtype=0)
    cfg = lambda **kw: binding.CmoeConfig(**{**good, **kw})
    assert _create(lib, cfg(d_model=12), perm, rep) == -1          # d % 8
    assert _create(lib, cfg(n_experts=7), perm, rep) == -2         # d_ff % N
    assert _create(lib, cfg(top_k=7), perm, rep) == -1             # N_k > N_r
    assert _create(lib, cfg(dtype=5), perm, rep) == -1
    assert _create(lib, cfg(max_tokens=0), perm, rep) == -1
    assert _create(lib, cfg(), perm, rep, w=None) == -1            # null weights
    bad = perm.copy(); bad[3] = bad[4]
    assert _create(lib, cfg(), bad, rep) == -2                     # not a bijection
    bad = perm.copy(); bad[0] = d_ff
    assert _create(lib, cfg(), bad, rep) == -2
    bad_rep = rep.copy(); bad_rep[0] = perm[0]                     # a shared neuron
    assert _create(lib, cfg(), perm, bad_rep) == -3
    bad_rep = rep.copy(); bad_rep[[0, 1]] = bad_rep[[1, 0]]        # another expert's neuron
    assert _create(lib, cfg(), perm, bad_rep) == -3
    assert b"representative" in lib.cmoe_last_error()


def test_permute_argument_checks(lib):
    assert lib.cmoe_token_permute_scratch_bytes(16384, 14) == 64 * 14 * 4 // 256 * 256 + 0 \
        or lib.cmoe_token_permute_scratch_bytes(16384, 14) % 256 == 0
    assert lib.cmoe_token_permute_scratch_bytes(16384, 14) >= 64 * 14 * 4
    assert lib.cmoe_token_permute(None, 10, 2, 0, None, None, None, None, None, 0, None) == -1
    assert lib.cmoe_token_permute(None, 10, 9, 4, None, None, None, None, None, 0, None) == -1
    assert lib.cmoe_token_permute(1, 1000, 2, 4, 1, 1, 1, 1, None, 0, None) == -1   # scratch null
    assert lib.cmoe_token_permute(1, 1000, 2, 4, 1, 1, 1, 1, 256, 8, None) == -4    # too small


def test_null_layer_calls(lib):
    assert lib.cmoe_ffn_forward(None, None, 1, None, None) == -1
    assert lib.cmoe_layer_destroy(None) == 0
    w = C.c_int32()
    assert lib.cmoe_layer_status(None, C.byref(w)) == -1
    assert lib.cmoe_layer_update_bias(None, 1e-3, None, None, None) == -1
    assert lib.cmoe_layer_get_gate_params(None, None, None, None) == -1


# ------------------------------------------------------------------ workloads
def test_bf16_rounding_is_nearest_even():
    import torch
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(100000).astype(np.float32),
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38], np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(wl.f32_to_bf16_bits(a), want)
    r = wl.round_to_storage(a, "bf16")
    np.testing.assert_array_equal(wl.round_to_storage(r, "bf16"), r)       # idempotent


def test_workload_shapes_match_the_configs():
    c2, c3, c4, c5 = (wl.WORKLOADS[k].shape for k in
                      ("c2_llama2_7b", "c3_llama3_8b", "c4_hier_8x7b", "c5_skew_13b"))
    assert (c2.m, c3.m, c4.m, c5.m) == (1376, 448, 1792, 864)
    assert c2.flops_per_token() == 6 * 4096 * 1376 * 4 + 4 * 4096 * 6
    assert c2.expert_weight_bytes() == 3 * 4096 * 1376 * 2
    inp = wl.make_inputs(wl.WORKLOADS["c1_tiny_fp32"])
    lay = inp.layers[0]
    assert inp.x.shape == (64, 256) and lay.w_down.shape == (256, 1024)
    assert sorted(lay.neuron_perm) == list(range(1024))
    assert list(lay.rep_idx) == [lay.neuron_perm[(2 + j) * 128] for j in range(6)]
    again = wl.make_inputs(wl.WORKLOADS["c1_tiny_fp32"])
    np.testing.assert_array_equal(again.layers[0].w_up, lay.w_up)


def test_zipf_target_shares():
    p = wl.zipf_target_shares(14, 4, 1.2)
    assert abs(p.sum() - 1) < 1e-12 and abs(p[0] - 0.25) < 1e-12
    assert np.all(np.diff(p) <= 1e-15) and p.max() <= 0.25 + 1e-12
    raw = np.arange(1, 15) ** -1.2
    np.testing.assert_allclose(p[2:] / p[2], (raw / raw[2])[2:], rtol=1e-12)   # tail keeps its shape
