"""Pins for the CPU oracle: what the paper and the mathematics fix.

Each ``pin_*`` takes the oracle module so that ``test_planted_mistakes_are_caught``
can run the same pins against deliberately broken copies of it.
"""
import importlib.util
import math
import os
import types

import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_layer(seed=0, d=24, n_experts=8, m=6, n_shared=2, top_k=2, n_tok=37, dtype="fp32"):
    shape = wl.LayerShape(d, n_experts * m, n_experts, n_shared, top_k, dtype)
    rng = np.random.Generator(np.random.PCG64(seed))
    x = wl.draw_tokens(rng, n_tok, shape)
    lay = wl.draw_layer(rng, shape)
    # larger weights than the workloads' 0.02 so that scores are well spread
    lay.w_gate *= 12.0
    lay.w_up *= 12.0
    return shape, x, lay


def layer_kwargs(shape, lay, **over):
    kw = dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down,
              neuron_perm=lay.neuron_perm, rep_idx=lay.rep_idx,
              n_experts=shape.n_experts, n_shared=shape.n_shared, top_k=shape.top_k,
              gate_scale_u=lay.gate_scale_u, select_bias_b=lay.select_bias_b)
    kw.update(over)
    return kw


# ------------------------------------------------------------------ dense FFN
def pin_dense_closed_form(o):
    """Eq. ori_ffn_method on numbers worked by hand: gate pre-activation ln 3
    gives sigmoid 3/4; pre-activation 0 gives a dead neuron."""
    ln3 = math.log(3.0)
    x = np.array([[1.0, 0.0], [0.0, 1.0]])
    w_gate = np.array([[ln3, 0.0], [0.0, -ln3], [0.0, 0.0]])      # [d_h=3, d=2]
    w_up = np.array([[2.0, 5.0], [7.0, 4.0], [9.0, 9.0]])
    w_down = np.array([[1.0, 10.0, 100.0], [-1.0, 0.5, 100.0]])   # [d=2, d_h=3]
    # token 0: a = (ln3, 0, 0), v = (2, 7, 9): h = (ln3*3/4*2, 0, 0)
    # token 1: a = (0, -ln3, 0), v = (5, 4, 9): h = (0, -ln3*1/4*4, 0)
    want = np.array([[1.5 * ln3, -1.5 * ln3], [-10.0 * ln3, -0.5 * ln3]])
    got = o.dense_ffn(x, w_gate, w_up, w_down)
    np.testing.assert_allclose(got, want, rtol=1e-14, atol=1e-14)


def pin_dense_library(o):
    """Same FFN through a library SwiGLU in fp64 (torch)."""
    import torch
    import torch.nn.functional as F
    shape, x, lay = small_layer(seed=11, d=40, m=9)
    tx, tg, tu, td = (torch.from_numpy(np.asarray(a, dtype=np.float64))
                      for a in (x, lay.w_gate, lay.w_up, lay.w_down))
    want = F.linear(F.silu(F.linear(tx, tg)) * F.linear(tx, tu), td).numpy()
    got = o.dense_ffn(x, lay.w_gate, lay.w_up, lay.w_down)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def pin_dense_per_neuron_brute_force(o):
    """Eq. decompose: F(x) = sum_i h_i w_i, one neuron at a time, scalar loops."""
    shape, x, lay = small_layer(seed=5, d=5, n_experts=2, m=3, n_shared=1, top_k=1, n_tok=3)
    d, d_h = shape.d_model, shape.d_ff
    got = o.dense_ffn(x, lay.w_gate, lay.w_up, lay.w_down)
    for t in range(x.shape[0]):
        y = [0.0] * d
        for i in range(d_h):
            a = sum(float(lay.w_gate[i, k]) * float(x[t, k]) for k in range(d))
            v = sum(float(lay.w_up[i, k]) * float(x[t, k]) for k in range(d))
            h = a / (1.0 + math.exp(-a)) * v
            for c in range(d):
                y[c] += h * float(lay.w_down[c, i])
        np.testing.assert_allclose(got[t], y, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------- MoE invariants
def pin_all_experts_on_is_dense(o):
    """Experts partition the neurons, so every routed expert on with unit gates
    reproduces the dense FFN (Eq. decompose / Section 3.3)."""
    shape, x, lay = small_layer(seed=1)
    out, sel, gates, *_ = o.cmoe_layer_forward(x, **layer_kwargs(shape, lay, top_k=shape.n_routed))
    assert np.all(gates == 1.0)
    assert np.all(np.sort(sel, axis=1) == np.arange(shape.n_routed))
    want = o.dense_ffn(x, lay.w_gate, lay.w_up, lay.w_down)
    np.testing.assert_allclose(out, want, rtol=1e-11, atol=1e-13)


def pin_reconstruction_error_identity(o):
    """Eq. recon_error: F_MoE - F = - sum over deactivated routed experts."""
    shape, x, lay = small_layer(seed=2)
    out, sel, gates, *_ = o.cmoe_layer_forward(x, **layer_kwargs(shape, lay))
    dense = o.dense_ffn(x, lay.w_gate, lay.w_up, lay.w_down)
    missing = np.zeros_like(dense)
    for j in range(shape.n_routed):
        off = ~np.any(sel == j, axis=1)
        neurons = o.expert_neurons(lay.neuron_perm, shape.n_experts, shape.n_shared + j)
        missing[off] += o.expert_forward(x[off], lay.w_gate, lay.w_up, lay.w_down, neurons)
    assert np.abs(missing).max() > 1e-3          # the identity is not vacuous
    np.testing.assert_allclose(out - dense, -missing, rtol=1e-9, atol=1e-12)


def pin_shared_always_on(o):
    """N_k = 0 leaves exactly the shared expert, for every token."""
    shape, x, lay = small_layer(seed=3)
    out, sel, gates, *_ = o.cmoe_layer_forward(x, **layer_kwargs(shape, lay, top_k=0))
    assert sel.shape == (x.shape[0], 0)
    shared = lay.neuron_perm[:shape.n_shared * shape.m]
    want = o.hidden_activations(x, lay.w_gate, lay.w_up, shared) @ \
        np.asarray(lay.w_down[:, shared], dtype=np.float64).T
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-14)
    assert np.all(np.abs(out).max(axis=1) > 0)


def pin_router_is_representative_activation(o):
    """s_j = h_{R_j}: the score is column R_j of the dense hidden state."""
    shape, x, lay = small_layer(seed=4)
    s = o.router_scores(x, lay.w_gate, lay.w_up, lay.rep_idx)
    h = o.hidden_activations(x, lay.w_gate, lay.w_up)
    np.testing.assert_allclose(s, h[:, lay.rep_idx], rtol=1e-12, atol=1e-15)
    # each representative lies in its own routed slice
    for j, r in enumerate(lay.rep_idx):
        assert r in o.expert_neurons(lay.neuron_perm, shape.n_experts, shape.n_shared + j)


def pin_gate_closed_forms(o):
    rng = np.random.default_rng(7)
    s = rng.normal(size=(50, 6))
    # u = 0 => unit gates; b = 0 => selection orders like the raw scores
    sel, g, sp, keys = o.gate_logic(s, 3)
    assert np.all(g == 1.0)
    np.testing.assert_allclose(sp.sum(axis=1), 1.0, rtol=1e-14)
    np.testing.assert_array_equal(np.sort(sel, 1), np.sort(np.argsort(-s, axis=1)[:, :3], 1))
    # softmax is shift-invariant
    np.testing.assert_allclose(o.softmax(s + 123.0), sp, rtol=1e-12)
    # N_r = 2: s'_0 = sigmoid(s_0 - s_1)
    s2 = rng.normal(size=(20, 2))
    _, g2, sp2, _ = o.gate_logic(s2, 1, gate_scale_u=np.array([0.5, -2.0]))
    np.testing.assert_allclose(sp2[:, 0], 1 / (1 + np.exp(-(s2[:, 0] - s2[:, 1]))), rtol=1e-13)
    win = (s2[:, 1] > s2[:, 0]).astype(int)
    u = np.array([0.5, -2.0])
    np.testing.assert_allclose(g2[:, 0], 1 + sp2[np.arange(20), win] * u[win], rtol=1e-14)
    # the bias moves the selection but not the gate value
    b = np.array([0, 0, 0, 0, 0, 10.0])
    u6 = np.linspace(-1, 1, 6)
    sel_b, g_b, sp_b, keys_b = o.gate_logic(s, 2, gate_scale_u=u6, select_bias_b=b)
    assert np.all(sel_b[:, 0] == 5)
    np.testing.assert_allclose(g_b[:, 0], 1 + sp_b[:, 5] * u6[5], rtol=1e-14)
    np.testing.assert_allclose(keys_b, sp_b + b, rtol=0, atol=0)


def pin_topk_brute_force(o):
    """Selection = the N_k largest keys by a scalar scan, ties to the lower index."""
    rng = np.random.default_rng(8)
    s = rng.normal(size=(64, 7))
    s[3, 2] = s[3, 5]                       # exact ties
    s[9, :] = 0.25
    b = rng.normal(scale=0.05, size=7)
    for k in (1, 2, 4, 7):
        sel, g, sp, keys = o.gate_logic(s, k, select_bias_b=b)
        for t in range(s.shape[0]):
            remaining = list(range(7))
            want = []
            for _ in range(k):
                best = remaining[0]
                for j in remaining[1:]:
                    if keys[t, j] > keys[t, best]:
                        best = j
                want.append(best)
                remaining.remove(best)
            assert list(sel[t]) == want
    sel, *_ = o.gate_logic(s, 2)
    assert list(sel[9]) == [0, 1]
    assert sorted(sel[3])[0] != 5 or 2 in sel[3]     # of two equal keys the lower index goes first


def pin_moe_linear_in_gates(o):
    shape, x, lay = small_layer(seed=6)
    kw = dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down, neuron_perm=lay.neuron_perm,
              n_experts=shape.n_experts, n_shared=shape.n_shared)
    rng = np.random.default_rng(0)
    sel = np.stack([rng.permutation(shape.n_routed)[:2] for _ in range(x.shape[0])]).astype(np.int32)
    g1 = rng.normal(size=sel.shape)
    g2 = rng.normal(size=sel.shape)
    zero = np.zeros_like(g1)
    f = lambda g: o.moe_forward(x, sel_idx=sel, gates=g, **kw)
    base = f(zero)
    np.testing.assert_allclose(f(g1 + g2) - base, (f(g1) - base) + (f(g2) - base),
                               rtol=1e-9, atol=1e-12)
    one = np.ones_like(g1)
    assert np.abs(f(one) - base).max() > 1e-3
    np.testing.assert_allclose(f(2.5 * one) - base, 2.5 * (f(one) - base), rtol=1e-9, atol=1e-12)
    # gate 1 + s'u end to end: F_MoE(u) - F_MoE(0) = sum_sel s'_i u_i E_i(x)
    u = np.linspace(-3, 3, shape.n_routed)
    out_u, sel_u, g_u, _, sp, _ = o.cmoe_layer_forward(x, **layer_kwargs(shape, lay, gate_scale_u=u))
    out_0, sel_0, *_ = o.cmoe_layer_forward(x, **layer_kwargs(shape, lay))
    np.testing.assert_array_equal(sel_u, sel_0)
    extra = np.zeros_like(out_0)
    for t in range(x.shape[0]):
        for j in sel_0[t]:
            neurons = o.expert_neurons(lay.neuron_perm, shape.n_experts, shape.n_shared + j)
            extra[t] += sp[t, j] * u[j] * o.expert_forward(x[t:t + 1], lay.w_gate, lay.w_up,
                                                           lay.w_down, neurons)[0]
    assert np.abs(extra).max() > 1e-4
    np.testing.assert_allclose(out_u - out_0, extra, rtol=1e-8, atol=1e-12)
    # token subset evaluation equals rows of the full evaluation
    ids = np.array([0, 5, 6, 30])
    np.testing.assert_allclose(o.moe_forward(x, sel_idx=sel, gates=g1, token_ids=ids, **kw),
                               f(g1)[ids], rtol=1e-12, atol=1e-14)


def pin_permutation(o):
    rng = np.random.default_rng(9)
    n_tok, n_r, k = 97, 6, 2
    sel = np.stack([rng.permutation(n_r)[:k] for _ in range(n_tok)]).astype(np.int32)
    sel[sel == 4] = 3 - (sel[sel == 4] * 0)           # leave expert 4 empty ...
    for t in range(n_tok):                             # ... without duplicating a pair
        if sel[t, 0] == sel[t, 1]:
            sel[t, 1] = 5 if sel[t, 0] != 5 else 0
    cnt, off, row_token, row_of = o.token_permutation(sel, n_r)
    pairs = sorted((int(sel[t, j]), t) for t in range(n_tok) for j in range(k))
    assert cnt.sum() == n_tok * k and cnt[4] == 0
    assert off[0] == 0 and np.all(np.diff(off) == cnt)
    assert [int(t) for t in row_token] == [t for _, t in pairs]
    for e in range(n_r):
        seg = row_token[off[e]:off[e + 1]]
        assert np.all(np.diff(seg) > 0)
        assert cnt[e] == sum(1 for ee, _ in pairs if ee == e)
    for t in range(n_tok):
        for j in range(k):
            r = row_of[t, j]
            assert row_token[r] == t and off[sel[t, j]] <= r < off[sel[t, j] + 1]
    assert sorted(row_of.ravel()) == list(range(n_tok * k))


def pin_logit_margin(o):
    rng = np.random.default_rng(10)
    s = rng.normal(size=(40, 5))
    _, _, sp, keys = o.gate_logic(s, 2)
    srt = -np.sort(-s, axis=1)
    np.testing.assert_allclose(o.logit_margin(sp, keys, 2), 1 - np.exp(-(srt[:, 1] - srt[:, 2])),
                               rtol=1e-10)
    assert np.all(np.isinf(o.logit_margin(sp, keys, 5)))


def pin_bias_update_rule(o):
    """Overloaded experts lose gamma, underloaded gain gamma, target 1/N_r."""
    b = np.array([0.1, 0.2, 0.3, 0.4])
    got = o.bias_update(b, counts=[10, 30, 20, 20])        # shares .125 .375 .25 .25
    np.testing.assert_allclose(got, [0.101, 0.199, 0.3, 0.4], rtol=0, atol=1e-15)
    got = o.bias_update(b, counts=[10, 30, 20, 20], target_share=[0.1, 0.4, 0.3, 0.2], gamma=0.5)
    np.testing.assert_allclose(got, [-0.4, 0.7, 0.8, -0.1], rtol=0, atol=1e-15)


def pin_fit_select_bias(o):
    """The iterated bias rule of Section 4.3 on scores small enough to follow by hand.
    Three experts, top-1, 24 rows whose softmax values are given outright (s = ln p).
    Row r gives expert 0 the value p_0 = 0.40 + 0.01 r and splits the rest between experts 1 and 2
    in a proportion that varies from row to row; with b = 0 expert 0 wins all 24 rows."""
    rows = 24
    r = np.arange(rows)
    p0 = 0.40 + 0.01 * r
    f = 0.35 + 0.0125 * ((7 * r) % 24)
    p = np.stack([p0, (1 - p0) * f, (1 - p0) * (1 - f)], axis=1)
    assert np.all(p[:, 0] > p[:, 1:].max(axis=1))
    s = np.log(p)
    # (1) a target that b = 0 already meets is left alone: no update is applied
    b, counts = o.fit_select_bias(s, 1, [1.0, 0.0, 0.0], tol=1e-9)
    assert np.all(b == 0.0) and list(counts) == [24, 0, 0]
    # (2) the step decays geometrically from gamma_hi to gamma_lo: with a tolerance that is never
    # met and three iterations, expert 0 (always over its target) loses hi + sqrt(hi*lo) + lo and
    # expert 2 (always under) gains the same
    hi, lo = 4e-3, 1e-3
    b, _ = o.fit_select_bias(s, 1, [0.0, 0.5, 0.5], iters=3, gamma_hi=hi, gamma_lo=lo, tol=0.0)
    total = hi + math.sqrt(hi * lo) + lo
    np.testing.assert_allclose(b, [-total, total, total], rtol=1e-12)
    # (3) a reachable target is reached on EVERY expert: recount the selections with the returned b
    # by a scalar loop.  Shares move in steps of 1/24 > tol, so only the exact split 12/8/4 passes; on
    # the way there the split 12/9/3 has expert 0 on target and a mean deviation under tol, so a
    # stopping test on one expert or on the mean ends too early.
    target = np.array([12, 8, 4]) / 24.0
    tol = 0.03
    b, counts = o.fit_select_bias(s, 1, target, iters=4000, gamma_hi=2e-2, gamma_lo=1e-4, tol=tol)
    recount = [0, 0, 0]
    for r in range(rows):
        keys = [p[r, j] + b[j] for j in range(3)]
        recount[max(range(3), key=lambda j: (keys[j], -j))] += 1
    assert list(counts) == recount
    assert max(abs(recount[j] / rows - target[j]) for j in range(3)) <= tol
    assert b[0] < 0 < b[2]                     # the overloaded expert was pushed down, the starved one up


# ---------------------------------------------------------------- hierarchical
def hier_case(seed=12, n_outer=4, top_k=None):
    shape = wl.LayerShape(20, 8 * 5, 8, 2, 2, "fp32")
    rng = np.random.Generator(np.random.PCG64(seed))
    x = wl.draw_tokens(rng, 33, shape)
    lays = [wl.draw_layer(rng, shape) for _ in range(n_outer)]
    for lay in lays:
        lay.w_gate *= 12.0
        lay.w_up *= 12.0
    w_r = rng.standard_normal((n_outer, shape.d_model))
    layers = [layer_kwargs(shape, lay, top_k=shape.top_k if top_k is None else top_k)
              for lay in lays]
    return shape, x, lays, w_r, layers


def pin_hierarchical_all_on_is_original_moe(o):
    """Section 4.4: with every sub-expert on and unit sub-gates each outer
    expert is its dense FFN, so the layer is the original top-2 MoE."""
    shape, x, lays, w_r, layers = hier_case(top_k=6)
    out, outer_idx, outer_w, _ = o.hier_forward(x, w_r, 2, layers)
    np.testing.assert_allclose(outer_w.sum(axis=1), 1.0, rtol=1e-14)
    logits = np.asarray(x, np.float64) @ w_r.T
    want = np.zeros_like(out)
    for t in range(x.shape[0]):
        top = sorted(range(len(lays)), key=lambda i: (-logits[t, i], i))[:2]
        assert list(outer_idx[t]) == top
        z = [math.exp(logits[t, i] - logits[t, top[0]]) for i in top]
        for i, zi in zip(top, z):
            lay = lays[i]
            want[t] += zi / sum(z) * o.dense_ffn(x[t:t + 1], lay.w_gate, lay.w_up, lay.w_down)[0]
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)


def pin_hierarchical_is_weighted_sum_of_layers(o):
    shape, x, lays, w_r, layers = hier_case(seed=13)
    out, outer_idx, outer_w, routing = o.hier_forward(x, w_r, 2, layers)
    want = np.zeros_like(out)
    for i, kw in enumerate(layers):
        y, *_ = o.cmoe_layer_forward(x, **kw)
        for slot in range(2):
            hit = outer_idx[:, slot] == i
            want[hit] += outer_w[hit, slot][:, None] * y[hit]
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-13)
    ids = np.array([1, 2, 17, 32])
    sub, *_ = o.hier_forward(x, w_r, 2, layers, token_ids=ids)
    np.testing.assert_allclose(sub, out[ids], rtol=1e-12, atol=1e-14)



def pin_atopk_brute_force(o):
    """ATopK against a scalar selection loop, with exact ties across the cut."""
    rng = np.random.default_rng(21)
    h = rng.normal(size=(23, 40))
    h[3, [5, 9, 30]] = [2.5, -2.5, 2.5]          # equal magnitudes, mixed signs
    h[3, 12] = 7.0
    h[7] = np.round(h[7], 1)                      # many ties
    for k_a in (1, 2, 3, 10):
        a = o.atopk(h, k_a)
        for t in range(h.shape[0]):
            taken = []
            for _ in range(k_a):
                best = None
                for i in range(h.shape[1]):
                    if i in taken:
                        continue
                    if best is None or abs(h[t, i]) > abs(h[t, best]):   # strict: the lower index keeps a tie
                        best = i
                taken.append(best)
            want = np.zeros(h.shape[1], dtype=np.uint8)
            want[taken] = 1
            np.testing.assert_array_equal(a[t], want)


def pin_atopk_invariants(o):
    rng = np.random.default_rng(22)
    h = rng.normal(size=(50, 64))
    a = o.atopk(h, 10)
    assert a.dtype == np.uint8 and set(np.unique(a)) <= {0, 1}
    np.testing.assert_array_equal(a.sum(axis=1), 10)                      # K_a ones per token
    np.testing.assert_array_equal(o.atopk(-h, 10), a)                     # magnitude, not sign
    np.testing.assert_array_equal(o.atopk(3.0 * h, 10), a)                # scale-free
    np.testing.assert_array_equal(o.atopk(h, 64), np.ones_like(a))        # K_a = d_h: everything
    big = np.abs(h) >= np.sort(np.abs(h), axis=1)[:, -10][:, None]
    np.testing.assert_array_equal(a, big.astype(np.uint8))                # no ties here: a threshold test
    perm = rng.permutation(64)
    np.testing.assert_array_equal(o.atopk(h[:, perm], 10), a[:, perm])    # neuron order does not matter
    m = o.atopk_margin(h, 10)
    srt = -np.sort(-np.abs(h), axis=1)
    np.testing.assert_allclose(m, (srt[:, 9] - srt[:, 10]) / srt[:, 9], rtol=1e-12)


def pin_activation_rates_and_shared(o):
    """Hand-worked: 4 tokens, 5 neurons, K_a = 2."""
    h = np.array([[0.1, -3.0, 2.0, 0.0, 0.5],
                  [4.0, -0.2, 0.3, 0.1, -5.0],
                  [0.0, 1.0, -1.0, 0.2, 0.1],        # |1.0| ties |-1.0|: both are in the top two
                  [0.3, 0.2, 0.1, -0.9, 0.8]])
    a = o.atopk(h, 2)
    np.testing.assert_array_equal(a, [[0, 1, 1, 0, 0], [1, 0, 0, 0, 1], [0, 1, 1, 0, 0], [0, 0, 0, 1, 1]])
    counts = o.activation_counts(a)
    np.testing.assert_array_equal(counts, [1, 2, 2, 1, 2])
    np.testing.assert_allclose(o.activation_rates(a), [0.25, 0.5, 0.5, 0.25, 0.5])
    assert counts.sum() == 2 * 4                                          # sum_i mu_i = K_a
    np.testing.assert_array_equal(o.select_shared(counts, 3), [1, 2, 4])  # ties: lower index first
    np.testing.assert_array_equal(o.select_shared(counts, 4), [1, 2, 4, 0])
    bits = o.pack_columns(a)
    assert bits.shape == (5, 1) and bits.dtype == np.uint32
    np.testing.assert_array_equal(bits[:, 0], [0b0010, 0b0101, 0b0101, 0b1000, 0b1010])
    rng = np.random.default_rng(23)
    big = (rng.random((70, 9)) < 0.3).astype(np.uint8)
    pb = o.pack_columns(big)
    for t in range(70):
        np.testing.assert_array_equal((pb[:, t // 32] >> np.uint32(t % 32)) & 1, big[t])
    np.testing.assert_array_equal([sum(bin(int(w)).count("1") for w in row) for row in pb], big.sum(axis=0))


def pin_profile_pipeline(o):
    """Steps 1-4 chained: H is the dense hidden activation, a neuron whose gate and up vectors are
    scaled up is active for almost every token and is selected first."""
    shape, x, lay = small_layer(seed=24, d=16, n_experts=4, m=8, n_tok=29)
    wg, wu = lay.w_gate.copy(), lay.w_up.copy()
    wu[5] *= 1024.0                                # h is linear in the up vector: neuron 5 dominates
    h, a, counts, shared = o.profile_activations(x, wg, wu, 3, 8)
    np.testing.assert_allclose(h, o.hidden_activations(x, wg, wu), rtol=0, atol=0)
    np.testing.assert_allclose(h[:, 5], 1024.0 * o.hidden_activations(x, lay.w_gate, lay.w_up)[:, 5], rtol=1e-12)
    in_top3 = (np.abs(h) > np.abs(h[:, 5:6])).sum(axis=1) < 3
    assert counts[5] == in_top3.sum() and counts[5] > 0.8 * x.shape[0] and shared[0] == 5
    assert len(shared) == 8 and len(set(shared.tolist())) == 8
    assert counts[shared].min() >= np.delete(counts, shared).max()

def _binary_cols(seed, q=40, n=12, p=0.3):
    rng = np.random.default_rng(seed)
    return (rng.random((q, n)) < p).astype(np.uint8)


def pin_distance_is_hamming_on_binary(o):
    """With binary centroids the squared L2 distance counts the differing positions."""
    c = _binary_cols(31)
    cent = c[:, [2, 7, 9]]
    d = o.centroid_distances(c, cent)
    for i in range(c.shape[1]):
        for j, cj in enumerate((2, 7, 9)):
            ham = sum(1 for k in range(c.shape[0]) if c[k, i] != c[k, cj])
            assert abs(d[i, j] ** 2 - ham) < 1e-9
    assert d[2, 0] == 0.0 and d[7, 1] == 0.0
    real = np.array([[0.5, 0.0], [0.25, 1.0], [0.0, 0.0]])                # hand-worked, real-valued centroids
    cc = np.array([[1, 0], [0, 1], [1, 1]], dtype=np.uint8)               # c_0 = (1,0,1), c_1 = (0,1,1)
    d2 = o.centroid_distances(cc, real)
    np.testing.assert_allclose(d2 ** 2, [[0.25 + 0.0625 + 1, 1 + 1 + 1], [0.25 + 0.5625 + 1, 0 + 0 + 1]], rtol=1e-14)


def pin_cluster_update_and_representatives(o):
    c = np.array([[1, 1, 0, 0, 1],
                  [0, 1, 1, 0, 0],
                  [1, 1, 1, 0, 0],
                  [0, 0, 0, 1, 1]], dtype=np.uint8)                        # q = 4 tokens, 5 neurons
    prev = np.full((4, 3), 0.125)
    assign = np.array([0, 0, 0, 1, -1])                                   # cluster 2 empty, neuron 4 unassigned
    cent = o.cluster_update(c, assign, prev)
    np.testing.assert_allclose(cent[:, 0], [2 / 3, 2 / 3, 1.0, 0.0])
    np.testing.assert_allclose(cent[:, 1], [0, 0, 0, 1])
    np.testing.assert_allclose(cent[:, 2], 0.125)                          # kept
    reps = o.representatives(c, assign, cent)
    # distances^2 of neurons 0,1,2 to (2/3,2/3,1,0): 1/9+4/9+0 = 5/9 ; 1/9+1/9+0 = 2/9 ; 4/9+1/9+0 = 5/9
    np.testing.assert_array_equal(reps, [1, 3, -1])
    tie = o.representatives(c[:, [0, 2, 1]], np.array([0, 0, 0]), cent[:, :1])
    assert tie[0] == 2                                                    # the closest one wherever it stands
    same = o.representatives(c[:, [0, 2]], np.array([0, 0]), cent[:, :1])
    assert same[0] == 0                                                   # equal distances: the lower position
    rng = np.random.default_rng(32)
    cb = _binary_cols(33, q=30, n=20)
    a = rng.integers(0, 4, size=20)
    cent = o.cluster_update(cb, a, np.zeros((30, 4)))
    reps = o.representatives(cb, a, cent)
    d = o.centroid_distances(cb, cent)
    for j in range(4):
        best = None
        for i in range(20):
            if a[i] == j and (best is None or d[i, j] < d[best, j]):
                best = i
        assert reps[j] == best


def pin_initial_centroids_and_assignment(o):
    counts = np.array([5, 9, 9, 1, 7, 7, 3, 0])
    np.testing.assert_array_equal(o.initial_centroids(counts, [1, 4], 3), [2, 5, 0])
    np.testing.assert_array_equal(o.initial_centroids(counts, [], 2), [1, 2])
    # balanced assignment against exhaustive search: 6 rows, 3 clusters of 2
    import itertools
    rng = np.random.default_rng(34)
    d = rng.random((6, 3))
    got = o.balanced_assignment(d, 2)
    assert sorted(np.bincount(got, minlength=3)) == [2, 2, 2]
    best = min((sum(d[i, a[i]] for i in range(6)) for a in itertools.product(range(3), repeat=6)
                if sorted(np.bincount(a, minlength=3)) == [2, 2, 2]))
    assert abs(sum(d[i, got[i]] for i in range(6)) - best) < 1e-12


# ------------------------------------------------------- FP8 weight quantisation
def pin_fp8_format(o):
    """OCP E4M3 as its definition gives it: bias 7, 3 mantissa bits, subnormals below 2^-6,
    largest finite value 448, S.1111.111 = NaN; round to nearest, ties to even, saturating."""
    dec = o.fp8_e4m3_decode
    np.testing.assert_array_equal(dec([0x00, 0x01, 0x07, 0x08, 0x38, 0x3C, 0x40, 0x77, 0x7E]),
                                  [0.0, 2.0 ** -9, 7 * 2.0 ** -9, 2.0 ** -6, 1.0, 1.5, 2.0, 240.0, 448.0])
    assert dec([0xB8])[0] == -1.0 and np.isnan(dec([0x7F, 0xFF])).all()
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    vals = dec(codes)
    np.testing.assert_array_equal(o.fp8_e4m3_encode(vals), codes)            # every value is its own code
    # hand-worked roundings: 1.0625 and 1.1875 are ties in the binade of 1 (spacing 1/8)
    enc = o.fp8_e4m3_encode([1.0625, 1.1875, 1.07, 2.0 ** -10, 1.5 * 2.0 ** -9, 2.0 ** -6 - 2.0 ** -11, 460.0, 1e6, -1e6])
    np.testing.assert_array_equal(enc, [0x38, 0x3A, 0x39, 0x00, 0x02, 0x08, 0x7E, 0x7E, 0xFE])
    # brute force: nearest representable value by exhaustive search over the 253 finite magnitudes
    rng = np.random.default_rng(21)
    x = np.concatenate([rng.normal(scale=s, size=400) for s in (300.0, 3.0, 0.02, 0.004)])
    pos = np.array(sorted(set(np.abs(vals))))
    pos_code = {v: c for c, v in zip(codes, vals) if c < 0x80}
    for xi, ci in zip(x, o.fp8_e4m3_encode(x)):
        a = min(abs(xi), 448.0)
        dist = np.abs(pos - a)
        best = np.nonzero(dist == dist.min())[0]
        cand = [pos_code[pos[i]] for i in best]
        want = cand[0] if len(cand) == 1 else [c for c in cand if c % 2 == 0][0]
        assert ci == (want | (0x80 if xi < 0 else 0)), (xi, hex(ci), hex(want))


def pin_fp8_row_scales(o):
    """One power-of-two scale per output channel, the smallest that brings the channel's largest
    weight to at most 448."""
    rng = np.random.default_rng(22)
    w = rng.normal(scale=0.02, size=(9, 40))
    w[3] = 0.0
    w[4, 7] = 448.0                      # scale 1: the codes are the plain encoding
    w[4, :7] = [1.0, 1.5, -2.0, 0.25, 1.0625, 240.0, -448.0]
    codes, e = o.quantise_rows_fp8(w)
    assert e[4] == 0 and e[3] == 0 and not codes[3].any()
    np.testing.assert_array_equal(codes[4, :8], [0x38, 0x3C, 0xC0, 0x28, 0x38, 0x77, 0xFE, 0x7E])
    amax = np.abs(w).max(axis=1)
    scaled = amax * 2.0 ** (-e.astype(np.float64))
    live = amax > 0
    assert np.all(scaled[live] <= 448.0) and np.all(scaled[live] > 224.0)
    # a power-of-two multiple of a row has the same codes and a shifted exponent
    codes2, e2 = o.quantise_rows_fp8(w * np.array([2.0 ** k for k in (-3, 0, 5, 1, -7, 2, 9, -1, 4)])[:, None])
    np.testing.assert_array_equal(codes2, codes)
    np.testing.assert_array_equal((e2 - e)[live], np.array([-3, 0, 5, 1, -7, 2, 9, -1, 4])[live])
    # error bound of round-to-nearest with 3 mantissa bits: half a unit in the last place
    wq = o.dequantise_rows_fp8(codes, e)
    normal = np.abs(w) >= np.ldexp(1.0, -6 + e)[:, None]
    assert np.all(np.abs(wq - w)[normal] <= np.abs(w)[normal] * 2.0 ** -4)
    assert np.all(np.abs(wq - w) <= np.ldexp(1.0, -10 + e)[:, None] + np.abs(w) * 2.0 ** -4)
    # dequantised values are exactly representable in bf16 (8 significant bits suffice)
    np.testing.assert_array_equal(wl.round_to_storage(wq.astype(np.float32), "bf16"), wq.astype(np.float32))


def pin_fp8_layer(o):
    """Quantised layer: W_gate / W_up scaled per neuron, W_down per (expert block, model dimension);
    the router reads the original weights; all experts on with unit gates = the dense FFN of the
    dequantised weights."""
    shape, x, lay = small_layer(seed=23, d=24, m=6, n_tok=29)
    kw = layer_kwargs(shape, lay)
    q = o.quantise_expert_weights(lay.w_gate, lay.w_up, lay.w_down, lay.neuron_perm, shape.n_experts, shape.n_shared)
    m, n_s = shape.m, shape.n_shared
    # per-neuron scales of W_gate: row n's largest code sits in the top binade (scaled amax in (224, 448])
    top = np.abs(o.fp8_e4m3_decode(q["gate_codes"])).max(axis=1)
    assert np.all((top >= 224) & (top <= 448))       # the scaled maximum lies in (224, 448] before rounding
    # W_down: one scale per (block, c); block 0 = all shared neurons together
    blocks = [lay.neuron_perm[:n_s * m]] + [lay.neuron_perm[(n_s + j) * m:(n_s + j + 1) * m] for j in range(shape.n_routed)]
    assert q["down_exp"].shape == (len(blocks), shape.d_model)
    for b, neurons in enumerate(blocks):
        sub = np.abs(lay.w_down[:, neurons]).max(axis=1)
        np.testing.assert_array_equal(q["down_exp"][b], o.pow2_scale_exponent(sub))
        top = np.abs(o.fp8_e4m3_decode(q["down_codes"][:, neurons])).max(axis=1)
        assert np.all((top >= 224) & (top <= 448))       # the scaled maximum lies in (224, 448] before rounding
        np.testing.assert_array_equal(q["w_down"][:, neurons],
                                      o.fp8_e4m3_decode(q["down_codes"][:, neurons]) * 2.0 ** q["down_exp"][b][:, None])
    assert len({tuple(e) for e in q["down_exp"]}) > 1                       # the blocks really have their own scales
    # forward: routing of the unquantised layer, experts on the dequantised weights
    out, sel, gates, s, _, _ = o.cmoe_layer_forward_fp8(x, **kw)
    ref_out, ref_sel, ref_gates, ref_s, _, _ = o.cmoe_layer_forward(x, **kw)
    np.testing.assert_array_equal(sel, ref_sel)
    np.testing.assert_array_equal(s, ref_s)
    kq = dict(kw, w_gate=q["w_gate"], w_up=q["w_up"], w_down=q["w_down"])
    want = o.moe_forward(x, q["w_gate"], q["w_up"], q["w_down"], lay.neuron_perm, shape.n_experts, shape.n_shared, ref_sel, ref_gates)
    np.testing.assert_allclose(out, want, rtol=1e-13, atol=1e-15)
    rel = np.abs(out - ref_out).sum() / np.abs(ref_out).sum()
    assert 1e-3 < rel < 0.1                                                  # quantisation changes the output, a little
    all_on, *_ = o.cmoe_layer_forward_fp8(x, **dict(kw, top_k=shape.n_routed))
    np.testing.assert_allclose(all_on, o.dense_ffn(x, q["w_gate"], q["w_up"], q["w_down"]), rtol=1e-10, atol=1e-13)


PINS = [pin_dense_closed_form, pin_dense_library, pin_dense_per_neuron_brute_force,
        pin_all_experts_on_is_dense, pin_reconstruction_error_identity, pin_shared_always_on,
        pin_router_is_representative_activation, pin_gate_closed_forms, pin_topk_brute_force,
        pin_moe_linear_in_gates, pin_permutation, pin_logit_margin, pin_bias_update_rule, pin_fit_select_bias,
        pin_hierarchical_all_on_is_original_moe, pin_hierarchical_is_weighted_sum_of_layers,
        pin_atopk_brute_force, pin_atopk_invariants, pin_activation_rates_and_shared, pin_profile_pipeline,
        pin_distance_is_hamming_on_binary, pin_cluster_update_and_representatives,
        pin_initial_centroids_and_assignment, pin_fp8_format, pin_fp8_row_scales, pin_fp8_layer]


@pytest.mark.parametrize("pin", PINS, ids=lambda p: p.__name__)
def test_pin(pin):
    pin(oracle)


# ----------------------------------------------------- planted mistakes (CPU)
def _mutant(patch_src):
    """A copy of the oracle module with one textual edit applied."""
    path = oracle.__file__
    src = open(path).read()
    old, new = patch_src
    assert src.count(old) >= 1, f"mutation anchor not found: {old!r}"
    mod = types.ModuleType("oracle_mutant")
    mod.__file__ = path
    exec(compile(src.replace(old, new, 1), path, "exec"), mod.__dict__)
    return mod


MUTATIONS = {
    "swish_without_sigmoid": ("return a / (1.0 + np.exp(-a))", "return a"),
    "sigmoid_sign": ("return a / (1.0 + np.exp(-a))", "return a / (1.0 + np.exp(a))"),
    "gate_up_swapped": ("return swish(x @ wg.T) * (x @ wu.T)", "return swish(x @ wu.T) * (x @ wg.T)"),
    "down_transposed_slice": ("return h @ _f64(w_down[:, neurons]).T",
                              "return h @ _f64(w_down[:, neurons[::-1]]).T"),
    "shared_dropped": ("if n_shared > 0:", "if False:"),
    "expert_offset": ("expert_neurons(neuron_perm, n_experts, n_shared + j)\n        y =",
                      "expert_neurons(neuron_perm, n_experts, j)\n        y ="),
    "gate_ignored": ("out[hit_tok] += gates[hit_tok, hit_slot][:, None] * y", "out[hit_tok] += y"),
    "smallest_selected": ("order = np.argsort(-rank_keys, axis=1, kind=\"stable\")",
                          "order = np.argsort(rank_keys, axis=1, kind=\"stable\")"),
    "bias_in_gate": ("gates = 1.0 + np.take_along_axis(s_prime,", "gates = 1.0 + np.take_along_axis(keys,"),
    "softmax_unnormalised": ("return z / z.sum(axis=-1, keepdims=True)", "return z"),
    "offsets_inclusive": ("off[e + 1] = off[e] + cnt[e]", "off[e + 1] = off[e] + cnt[e] + (e == 0)"),
    "outer_weights_unnormalised": ("outer_w = softmax(sel_logits)", "outer_w = np.exp(sel_logits)"),
    "bias_rule_sign": ("b[p > target] -= gamma", "b[p > target] += gamma"),
    "fit_step_grows": ("gamma = gamma_hi * (gamma_lo / gamma_hi) ** (it / max(iters - 1, 1))",
                       "gamma = gamma_hi * (gamma_hi / gamma_lo) ** (it / max(iters - 1, 1))"),
    "fit_step_constant": ("gamma = gamma_hi * (gamma_lo / gamma_hi) ** (it / max(iters - 1, 1))", "gamma = gamma_hi"),
    "fit_stops_on_mean": ("if np.abs(counts / counts.sum() - target).max() <= tol:",
                          "if np.abs(counts / counts.sum() - target).mean() <= tol:"),
    "fit_stops_on_first_expert": ("if np.abs(counts / counts.sum() - target).max() <= tol:",
                                  "if np.abs(counts / counts.sum() - target)[0] <= tol:"),
    "atopk_signed": ("mag = np.abs(_f64(h))\n    order", "mag = _f64(h)\n    order"),
    "atopk_smallest": ("order = np.argsort(-mag, axis=1, kind=\"stable\")[:, :k_a]",
                       "order = np.argsort(mag, axis=1, kind=\"stable\")[:, :k_a]"),
    "atopk_wrong_axis": ("np.put_along_axis(a, order, 1, axis=1)", "np.put_along_axis(a, order[:a.shape[1]].T[:a.shape[0]], 1, axis=0)"),
    "counts_over_neurons": ("return np.asarray(a, dtype=np.int64).sum(axis=0)",
                            "return np.asarray(a, dtype=np.int64).sum(axis=1)"),
    "shared_lowest_rate": ("return np.argsort(-counts, kind=\"stable\")[:n_select]",
                           "return np.argsort(counts, kind=\"stable\")[:n_select]"),
    "distance_not_rooted": ("return np.sqrt((diff * diff).sum(axis=0))", "return (diff * diff).sum(axis=0)"),
    "distance_abs_not_square": ("return np.sqrt((diff * diff).sum(axis=0))", "return np.sqrt(np.abs(diff).sum(axis=0)) * 1.0000001"),
    "centroid_sum_not_mean": ("out[:, j] = c[:, members].sum(axis=1) / len(members)", "out[:, j] = c[:, members].sum(axis=1)"),
    "empty_cluster_zeroed": ("out = _f64(prev_centroids).copy()", "out = np.zeros_like(_f64(prev_centroids))"),
    "representative_farthest": ("reps[j] = members[np.argmin(d[members, j])]", "reps[j] = members[np.argmax(d[members, j])]"),
    "centroids_include_shared": ("if int(i) not in shared]", "]"),
    "assignment_unbalanced": ("rows, cols = linear_sum_assignment(np.repeat(d, m, axis=1))",
                              "rows, cols = np.arange(n), np.argmin(d, axis=1) * m"),
    "fp8_truncates": ("q = np.rint(np.ldexp(a_f, 3 - e))", "q = np.floor(np.ldexp(a_f, 3 - e))"),
    "fp8_ties_away": ("q = np.rint(np.ldexp(a_f, 3 - e))", "q = np.floor(np.ldexp(a_f, 3 - e) + 0.5)"),
    "fp8_bias_8": ("mag = np.where(e > 0, np.ldexp(1.0 + m / 8.0, e - 7), np.ldexp(m / 8.0, -6))",
                   "mag = np.where(e > 0, np.ldexp(1.0 + m / 8.0, e - 8), np.ldexp(m / 8.0, -7))"),
    "fp8_no_subnormals": ("e = np.maximum(p - 1, -6)", "e = np.maximum(p - 1, -9)"),
    "fp8_scale_one_binade_high": ("e = np.where(f <= 0.875, p - 9, p - 8)", "e = np.where(f <= 0.875, p - 8, p - 7)"),
    "fp8_scale_ignores_mantissa": ("e = np.where(f <= 0.875, p - 9, p - 8)", "e = p - 9"),
    "fp8_down_one_scale_per_row": ("codes, e = quantise_rows_fp8(w_down[:, neurons])",
                                   "codes, e = quantise_rows_fp8(w_down); codes = codes[:, neurons]"),
    "fp8_router_on_quantised": ("    s = router_scores(x, w_gate, w_up, rep_idx)\n    sel_idx, gates, s_prime, keys = gate_logic(s, top_k, gate_scale_u, select_bias_b)\n    out = moe_forward(x, q[",
                                "    s = router_scores(x, q[\"w_gate\"], q[\"w_up\"], rep_idx)\n    sel_idx, gates, s_prime, keys = gate_logic(s, top_k, gate_scale_u, select_bias_b)\n    out = moe_forward(x, q["),
    "pack_bit_order": ("np.uint64(1) << np.arange(32, dtype=np.uint64)", "np.uint64(1) << np.arange(31, -1, -1, dtype=np.uint64)"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistakes_are_caught(name):
    mutant = _mutant(MUTATIONS[name])
    failed = []
    for pin in PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError, IndexError):
            failed.append(pin.__name__)
    assert failed, f"no pin noticed the planted mistake {name!r}"


# ------------------------------------------------------------ paper's numbers
def test_flop_model_against_papers_table():
    """tests/golden/paper_efficiency_flops.txt: dense vs restructured Llama-2-7B
    whole-model FLOPs (Table efficiency_flops).  The FFN-only saving predicted
    by the per-token flop model, times the FFN's share of the matmul flops,
    must land on the printed whole-model saving."""
    rows = {}
    for line in open(os.path.join(GOLDEN, "paper_efficiency_flops.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split("=")
        rows[k.strip()] = float(v)
    shape = wl.LayerShape(4096, 11008, 8, 3, 3, "bf16")          # S3A3E8 on Llama-2-7B
    ffn_saving = 1.0 - shape.flops_per_token() / shape.dense_flops_per_token()
    assert abs(ffn_saving - 0.25) < 2e-3                          # router cost is ~0.1 %
    n_layers, vocab, d = 32, 32000, 4096
    ffn = n_layers * shape.dense_flops_per_token()
    attn_proj = n_layers * 2 * 4 * d * d
    lm_head = 2 * d * vocab
    share = ffn / (ffn + attn_proj + lm_head)
    printed = 1.0 - rows["ours_tflops"] / rows["dense_tflops"]
    assert abs(printed - rows["printed_reduction"]) < 2e-3
    assert abs(ffn_saving * share - printed) < 0.015
