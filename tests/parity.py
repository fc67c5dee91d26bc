"""GPU-vs-oracle comparison used by the -m gpu tests.

Rule: routing indices, per-expert counts, offsets and the token permutation must
match bit-exactly, except for tokens whose gap between the N_k-th and (N_k+1)-th
key is under 1e-3 in logit units; for those the CUDA path's choice must be
admissible (it only trades experts that are within that margin of the cut), the
oracle's routing is patched to that choice, and everything downstream is compared
bit-exactly / within the output tolerance again.
Outputs: max|err| <= 2e-2 * max|y| and sum|err| / sum|y| <= 5e-3.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

from oracle import cmoe_oracle as oracle
from paper_2502_04416_b200 import binding, torch_io, workloads as wl

MARGIN = 1e-3
OUT_MAX_REL = 2e-2
OUT_MEAN_REL = 5e-3


to_device, to_host, gpu_layer = torch_io.to_device, torch_io.to_host, torch_io.layer_from_inputs


def oracle_kwargs(lay: wl.LayerInputs) -> dict:
    s = lay.shape
    return dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down, neuron_perm=lay.neuron_perm,
                rep_idx=lay.rep_idx, n_experts=s.n_experts, n_shared=s.n_shared, top_k=s.top_k,
                gate_scale_u=lay.gate_scale_u, select_bias_b=lay.select_bias_b)


@dataclass
class RoutingCheck:
    sel_idx: np.ndarray       # oracle routing after patching near-tie rows to the CUDA choice
    gates: np.ndarray
    near_tie: int
    differing: int


def margin_to_cut(s_prime: np.ndarray, keys: np.ndarray, top_k: int) -> np.ndarray:
    """[rows, N_r]: distance of every expert's key from the cut (the N_k-th largest key),
    in logit units (divided by the larger of the two softmax values)."""
    n_rows, n_r = keys.shape
    order = np.argsort(-keys, axis=1, kind="stable")
    rows = np.arange(n_rows)
    cut = order[:, top_k - 1]
    kcut, scut = keys[rows, cut][:, None], s_prime[rows, cut][:, None]
    return np.abs(keys - kcut) / np.maximum(s_prime, scut)


def check_routing(gpu_idx: np.ndarray, gpu_gate: np.ndarray, gpu_keys: np.ndarray,
                  gpu_scores: np.ndarray, s: np.ndarray, top_k: int, u, b,
                  group_base: Optional[np.ndarray] = None) -> RoutingCheck:
    """Compares the CUDA routing of a set of rows with the oracle's gate logic on the
    oracle's scores ``s``.  ``group_base`` [rows] is subtracted from gpu_idx (hierarchical)."""
    sel, gates, s_prime, keys = oracle.gate_logic(s, top_k, u, b)
    n_rows, n_r = s.shape
    if top_k == 0:
        return RoutingCheck(sel, gates, 0, 0)
    local = gpu_idx - (0 if group_base is None else group_base[:, None])
    assert local.min() >= 0 and local.max() < n_r, "selected expert index out of range"
    # fp32 (tensor-core) accumulation over d <= 8192 terms against fp64: ~4e-5 absolute seen
    # on scores of magnitude ~3; 1e-4 keeps a 10x distance to the 1e-3 near-tie margin.
    np.testing.assert_allclose(gpu_scores, s, rtol=2e-4, atol=1e-4)
    np.testing.assert_allclose(gpu_keys, keys, rtol=2e-4, atol=1e-4)
    margin = oracle.logit_margin(s_prime, keys, top_k)
    near = margin < MARGIN
    same = np.sort(local, axis=1) == np.sort(sel, axis=1)
    differ = ~same.all(axis=1)
    assert not (differ & ~near).any(), \
        f"{int((differ & ~near).sum())} rows differ from the oracle with margin >= {MARGIN}"
    if differ.any():
        dist = margin_to_cut(s_prime, keys, top_k)
        uarr = np.zeros(n_r) if u is None else np.asarray(u, dtype=np.float64)
        for r in np.nonzero(differ)[0]:
            assert len(set(local[r])) == top_k
            traded = set(local[r]) ^ set(sel[r])
            assert all(dist[r, e] < MARGIN for e in traded), f"row {r}: inadmissible choice"
            sel[r] = local[r]
            gates[r] = 1.0 + s_prime[r, local[r]] * uarr[local[r]]
    # gate values, matched by expert
    o_ord, g_ord = np.argsort(sel, axis=1), np.argsort(local, axis=1)
    np.testing.assert_allclose(np.take_along_axis(gpu_gate, g_ord, 1),
                               np.take_along_axis(gates, o_ord, 1), rtol=1e-5, atol=1e-6)
    return RoutingCheck(sel, gates, int(near.sum()), int(differ.sum()))


def check_permutation(sel_global: np.ndarray, n_groups: int, gpu_idx: np.ndarray, gpu: dict):
    """Bit-exact comparison of counts / offsets / row_token / row_of; row_of is matched by
    expert because the slot order of (nearly) equal keys carries no meaning."""
    cnt, off, row_token, row_of = oracle.token_permutation(sel_global, n_groups)
    np.testing.assert_array_equal(gpu["counts"], cnt)
    np.testing.assert_array_equal(gpu["offsets"], off)
    np.testing.assert_array_equal(gpu["row_token"], row_token)
    o_ord, g_ord = np.argsort(sel_global, axis=1), np.argsort(gpu_idx, axis=1)
    np.testing.assert_array_equal(np.take_along_axis(gpu["row_of"], g_ord, 1),
                                  np.take_along_axis(row_of, o_ord, 1))
    return cnt


def check_output(got: np.ndarray, want: np.ndarray):
    err = np.abs(got.astype(np.float64) - want)
    max_rel = err.max() / np.abs(want).max()
    mean_rel = err.sum() / np.abs(want).sum()
    assert np.isfinite(got).all()
    assert max_rel <= OUT_MAX_REL, f"max|err|/max|y| = {max_rel:.3e}"
    assert mean_rel <= OUT_MEAN_REL, f"sum|err|/sum|y| = {mean_rel:.3e}"
    return max_rel, mean_rel


def check_plain_layer(layer: binding.Layer, lay: wl.LayerInputs, x: np.ndarray,
                      sample_tokens=None, expert_weights: Optional[dict] = None) -> dict:
    """One forward of a plain layer on x [T,d], compared stage by stage with the oracle.
    ``sample_tokens``: compare outputs only on these tokens (large workloads); an array, or a
    callable (n_tok, counts, offsets, row_token) -> token ids such as ``stratified_tokens``.
    ``expert_weights``: w_gate / w_up / w_down the experts multiply by when they differ from the
    layer's original weights (a quantised layer: the router still reads the originals)."""
    import torch
    s = lay.shape
    n_tok = x.shape[0]
    xd = to_device(x, s.dtype)
    out = layer.forward(xd)
    torch.cuda.synchronize()
    assert layer.status() == 0
    got = to_host(out)
    stats = dict(tokens=n_tok, launches=layer.launch_count())
    scores = oracle.router_scores(x, lay.w_gate, lay.w_up, lay.rep_idx)
    if s.n_routed > 0 and s.top_k > 0:
        r = layer.routing(n_tok, s.n_routed)
        rc = check_routing(r["topk_idx"], r["topk_gate"], r["keys"], r["scores"], scores, s.top_k,
                           lay.gate_scale_u, lay.select_bias_b)
        cnt = check_permutation(rc.sel_idx, s.n_routed, r["topk_idx"], r)
        stats.update(near_tie=rc.near_tie, differing=rc.differing, counts=cnt.tolist())
        sel, gates = rc.sel_idx, rc.gates
        if callable(sample_tokens):    # chosen from the oracle's own (patched) permutation
            _, off, row_token, _ = oracle.token_permutation(sel, s.n_routed)
            sample_tokens = sample_tokens(n_tok, cnt, off, row_token)
    else:
        sel = np.zeros((n_tok, 0), np.int32)
        gates = np.zeros((n_tok, 0))
        if callable(sample_tokens):
            sample_tokens = sample_tokens(n_tok, [], [0], [])
    ew = expert_weights or dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down)
    want = oracle.moe_forward(x, ew["w_gate"], ew["w_up"], ew["w_down"], lay.neuron_perm, s.n_experts,
                              s.n_shared, sel, gates, token_ids=sample_tokens)
    if sample_tokens is not None:
        got = got[sample_tokens]
        stats["sampled"] = len(sample_tokens)
    stats["max_rel"], stats["mean_rel"] = check_output(got, want)
    return stats


def check_outer_routing(gpu_outer_idx: np.ndarray, gpu_outer_w: np.ndarray, x: np.ndarray,
                        w_router: np.ndarray, outer_top_k: int):
    """Outer level of a hierarchical layer (Section 4.4), the same rule as the inner level: the
    selected sets must equal the oracle's except on tokens whose outer_top_k-th and next logit are
    within MARGIN; there the CUDA choice may only trade experts whose logit is within MARGIN of the
    cut, the oracle's selection is replaced by it and the weights (softmax over the selected
    logits) are recomputed for that selection.  Pure numpy: no device is touched.
    Returns (outer_idx, outer_w, near-tie tokens, differing tokens) after patching."""
    o_idx, o_w, logits = oracle.outer_router(x, w_router, outer_top_k)
    n_tok, n_outer = logits.shape
    assert gpu_outer_idx.min() >= 0 and gpu_outer_idx.max() < n_outer
    srt = -np.sort(-logits, axis=1)
    cut = srt[:, outer_top_k - 1]
    near = (cut - srt[:, outer_top_k]) < MARGIN if outer_top_k < n_outer else np.zeros(n_tok, bool)
    differ = ~(np.sort(gpu_outer_idx, 1) == np.sort(o_idx, 1)).all(axis=1)
    assert not (differ & ~near).any(), \
        f"{int((differ & ~near).sum())} tokens pick other outer experts with margin >= {MARGIN}"
    for t in np.nonzero(differ)[0]:
        assert len(set(gpu_outer_idx[t])) == outer_top_k
        traded = set(gpu_outer_idx[t]) ^ set(o_idx[t])
        assert all(abs(logits[t, e] - cut[t]) < MARGIN for e in traded), f"token {t}: inadmissible outer choice"
        order = sorted(gpu_outer_idx[t], key=lambda e: (-logits[t, e], e))     # descending logit, like the oracle
        o_idx[t] = order
        o_w[t] = oracle.softmax(logits[t, order][None, :])[0]
    go, oo = np.argsort(gpu_outer_idx, 1), np.argsort(o_idx, 1)
    np.testing.assert_allclose(np.take_along_axis(gpu_outer_w, go, 1),
                               np.take_along_axis(o_w, oo, 1), rtol=1e-4, atol=1e-6)
    return o_idx, o_w, int(near.sum()), int(differ.sum())


def stratified_tokens(n_tok: int, counts, offsets, row_token, seed: int, n_random: int = 48,
                      tile: int = 128) -> np.ndarray:
    """Tokens at which a large workload's output is compared: first and last token, the tokens
    on both sides of the first and last tile edge of the token-ordered (shared) rows, for every
    routed group the tokens of its first and last row, for the largest and the smallest non-empty
    group the tokens on both sides of every ``tile``-row edge, plus a seeded random sample.
    ``counts/offsets/row_token`` are the oracle's permutation (after near-tie patching)."""
    ids = {0, n_tok - 1}
    for e in (tile, (n_tok - 1) // tile * tile):
        ids.update(t for t in (e - 1, e) if 0 <= t < n_tok)
    counts = np.asarray(counts)
    live = np.nonzero(counts > 0)[0]
    for g in live:
        ids.add(int(row_token[offsets[g]]))
        ids.add(int(row_token[offsets[g + 1] - 1]))
    if live.size:
        big = live[np.argmax(counts[live])]
        small = live[np.argmin(counts[live])]
        for g in {int(big), int(small)}:
            for e in range(tile, int(counts[g]), tile):
                ids.add(int(row_token[offsets[g] + e - 1]))
                ids.add(int(row_token[offsets[g] + e]))
    rng = np.random.default_rng(seed)
    ids.update(int(t) for t in rng.choice(n_tok, size=min(n_random, n_tok), replace=False))
    return np.array(sorted(ids), dtype=np.int64)


def check_hier_layer(layer: binding.Layer, inputs: wl.WorkloadInputs, x: np.ndarray,
                     sample_tokens=None, expert_weights=None) -> dict:
    """Hierarchical layer: outer routing, per-outer-expert inner routing, flattened
    permutation over n_outer*N_r groups, output.  ``expert_weights``: per outer expert, the weights its
    experts multiply by when they differ from the originals (a quantised layer)."""
    import torch
    w = inputs.workload
    s = w.shape
    n_tok, ok, n_outer, nr, k = x.shape[0], w.outer_top_k, w.n_outer, s.n_routed, s.top_k
    out = layer.forward(to_device(x, s.dtype))
    torch.cuda.synchronize()
    assert layer.status() == 0
    got = to_host(out)
    r = layer.routing(n_tok, nr)
    # --- outer level
    o_idx, o_w, near_o, diff_o = check_outer_routing(r["outer_idx"], r["outer_w"], x, inputs.w_router, ok)
    _, o_off, o_row_token, _ = oracle.token_permutation(o_idx, n_outer)
    np.testing.assert_array_equal(r["outer_row_token"], o_row_token)
    # --- inner level, outer expert by outer expert (rows are grouped by outer expert)
    R = n_tok * ok
    sel_global = np.zeros((R, k), np.int32)
    gates_all = np.zeros((R, k))
    near, diff = near_o, diff_o
    for i, lay in enumerate(inputs.layers):
        rows = np.arange(o_off[i], o_off[i + 1])
        if rows.size == 0:
            continue
        toks = o_row_token[rows]
        sc = oracle.router_scores(x[toks], lay.w_gate, lay.w_up, lay.rep_idx)
        rc = check_routing(r["topk_idx"][rows], r["topk_gate"][rows], r["keys"][rows],
                           r["scores"][rows], sc, k, lay.gate_scale_u, lay.select_bias_b,
                           group_base=np.full(rows.size, i * nr))
        sel_global[rows] = rc.sel_idx + i * nr
        gates_all[rows] = rc.gates
        near += rc.near_tie
        diff += rc.differing
    cnt = check_permutation(sel_global, n_outer * nr, r["topk_idx"], r)
    # --- output on the sampled tokens
    if callable(sample_tokens):        # chosen from the permutation: routed rows hold outer rows, those hold tokens
        _, off_in, row_tok_in, _ = oracle.token_permutation(sel_global, n_outer * nr)
        sample_tokens = sample_tokens(n_tok, cnt, off_in, o_row_token[row_tok_in])
    keep = np.arange(n_tok) if sample_tokens is None else np.asarray(sample_tokens)
    want = np.zeros((len(keep), s.d_model))
    row_of_tok = {(int(o_row_token[rr]), int(i)): rr for i in range(n_outer)
                  for rr in range(o_off[i], o_off[i + 1])}
    for i, lay in enumerate(inputs.layers):
        hit = [(p, t) for p, t in enumerate(keep) if i in o_idx[t]]
        if not hit:
            continue
        pos = np.array([p for p, _ in hit])
        toks = np.array([t for _, t in hit])
        rows = np.array([row_of_tok[(int(t), i)] for t in toks])
        ew = expert_weights[i] if expert_weights is not None else dict(w_gate=lay.w_gate, w_up=lay.w_up, w_down=lay.w_down)
        y = oracle.moe_forward(x[toks], ew["w_gate"], ew["w_up"], ew["w_down"], lay.neuron_perm,
                               s.n_experts, s.n_shared, sel_global[rows] - i * nr, gates_all[rows])
        wt = np.array([o_w[t, list(o_idx[t]).index(i)] for t in toks])
        want[pos] += wt[:, None] * y
    max_rel, mean_rel = check_output(got[keep], want)
    return dict(tokens=n_tok, near_tie=near, differing=diff, outer_near_tie=near_o, outer_differing=diff_o,
                sampled=len(keep), max_rel=max_rel, mean_rel=mean_rel, launches=layer.launch_count())


# ------------------------------------------------------------ activation profiling
def unpack_activation_bits(bits: np.ndarray, q: int) -> np.ndarray:
    """[d_ff, words] uint32 bit rows -> A [q, d_ff] uint8."""
    t = np.arange(q)
    return ((bits[:, t // 32] >> (t % 32).astype(np.uint32)) & 1).T.astype(np.uint8)


def reference_activation_matrix(a_gpu: np.ndarray, x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, k_a: int,
                                dtype: str):
    """The oracle's ATopK matrix for calibration rows x, with the decision taken on H rounded to the
    storage type the kernel keeps it in.  A row whose cut lies within two storage ulps of the next
    magnitude may differ from the CUDA result by exactly such boundary neurons; that is checked here,
    and for those rows (only) the CUDA choice is carried into the returned matrix so that everything
    downstream of A can be compared exactly.  Returns (A, number of patched rows)."""
    q = x.shape[0]
    h64 = oracle.hidden_activations(x, w_gate, w_up)
    h_st = wl.round_to_storage(h64.astype(np.float32), dtype).astype(np.float64)
    a_ref = oracle.atopk(h_st, k_a)
    ulp = 2.0 ** -7 if dtype == "bf16" else 2.0 ** -20                # relative, generous by 2x
    mag = np.abs(h64)
    cut = -np.sort(-mag, axis=1)[:, k_a - 1]
    differing = np.nonzero((a_gpu != a_ref).any(axis=1))[0]
    for t in differing:
        moved = np.nonzero(a_gpu[t] != a_ref[t])[0]
        assert a_gpu[t].sum() == k_a
        assert np.all(np.abs(mag[t, moved] - cut[t]) <= 2 * ulp * cut[t]), (t, moved, mag[t, moved], cut[t])
    clear = oracle.atopk_margin(h64, k_a) > 4 * ulp
    assert not np.isin(differing, np.nonzero(clear)[0]).any()
    assert len(differing) <= max(2, 0.05 * q), f"{len(differing)} of {q} rows differ"
    patched = a_ref.copy()
    patched[differing] = a_gpu[differing]
    return patched, len(differing)
