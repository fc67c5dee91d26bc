"""CPU oracle for the forward pass of an FFN restructured into a sparse MoE.

TEST INFRASTRUCTURE ONLY.  Plain numpy in fp64, written from the paper's
equations, sharing no code with the CUDA path; only tests, the smoke check and
the benchmark's CPU-baseline leg may call it.  Inputs are whatever fp32 arrays
the caller hands in (for bf16 workloads: values already rounded to bf16);
every product and sum here is fp64.

Array conventions (the same as the C-ABI's): ``w_gate[n, :]`` and
``w_up[n, :]`` are neuron n's gate/up vectors (column n of the paper's
W_gate/W_up in R^{d x d_h}); ``w_down[:, n]`` is neuron n's output vector
(row n of the paper's W_down in R^{d_h x d}).  ``neuron_perm`` lists original
neuron indices; expert e owns ``neuron_perm[e*m:(e+1)*m]`` and experts
``0..N_s-1`` are the shared ones (Section 4.1).

Pins (tests/test_oracle_pins.py): all-experts-on = dense FFN (Eq. decompose),
the reconstruction-error identity (Eq. recon_error), router score = dense
hidden activation of the representative neuron (Eq. rep_neuron/router),
closed forms of the gate (Section 4.3), brute-force top-k, scalar per-neuron
brute force, a library fp64 SwiGLU, permutation invariants, and hierarchical
all-on = the original MoE layer (Section 4.4); for the activation profiling
stage (Appendix "Complete Activation Analysis Pipeline"): scalar brute force,
row/column invariants, sign and scale invariance of ATopK, a hand-worked case; for the
clustering pieces (Appendix "Balanced Clustering Algorithm"): squared L2 = Hamming distance
on binary vectors, a hand-worked mean, brute-force argmin, an exhaustive balanced assignment;
for the FP8 weight quantisation (Section 6): the E4M3 format's defining values, exhaustive
round trip, hand-worked ties, brute-force nearest-value search, scale-1 and power-of-two
scale cases, the rounding error bound, all-experts-on = dense FFN of the dequantised weights.
Parity unpinned (conventions the paper does not fix): the outer router's
weights for an existing MoE layer (softmax over the selected logits), the
tie-break between equal keys (lower index wins) and the NaN policy; likewise the
tie-breaks of equal magnitudes in ATopK, of equal activation counts and of equal
centroid distances (lower index or position wins); the quantisation format itself (E4M3 codes,
one power-of-two scale per output channel, router left unquantised) is a reading, the paper
names none.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


# ---------------------------------------------------------------- Section 4.1
def swish(a: np.ndarray) -> np.ndarray:
    """Swish with beta = 1 (SiLU): a * sigmoid(a)  (Eq. ori_ffn_method)."""
    a = _f64(a)
    return a / (1.0 + np.exp(-a))


def hidden_activations(x, w_gate, w_up, neurons=None) -> np.ndarray:
    """h = Swish(W_gate^T x) * (W_up^T x) for the listed neurons, all tokens
    (Eq. ori_ffn_method, first line).  x: [T,d] -> [T,len(neurons)]."""
    x = _f64(x)
    if neurons is None:
        wg, wu = _f64(w_gate), _f64(w_up)
    else:
        neurons = np.asarray(neurons, dtype=np.int64)
        wg, wu = _f64(w_gate[neurons]), _f64(w_up[neurons])
    return swish(x @ wg.T) * (x @ wu.T)


def dense_ffn(x, w_gate, w_up, w_down) -> np.ndarray:
    """F(x) = W_down^T h (Eq. ori_ffn_method)."""
    return hidden_activations(x, w_gate, w_up) @ _f64(w_down).T


def expert_forward(x, w_gate, w_up, w_down, neurons) -> np.ndarray:
    """An expert is the FFN restricted to its neurons: E(x) = sum over its
    neurons of h_i w_i (Eq. decompose with the slice of Section 4.1)."""
    neurons = np.asarray(neurons, dtype=np.int64)
    h = hidden_activations(x, w_gate, w_up, neurons)
    return h @ _f64(w_down[:, neurons]).T


def expert_neurons(neuron_perm, n_experts: int, e: int) -> np.ndarray:
    d_ff = len(neuron_perm)
    if d_ff % n_experts:
        raise ValueError("d_ff must be a multiple of the number of experts")
    m = d_ff // n_experts
    return np.asarray(neuron_perm[e * m:(e + 1) * m], dtype=np.int64)


# ---------------------------------------------------------------- Section 4.2
def router_scores(x, w_gate, w_up, rep_idx) -> np.ndarray:
    """s = G(x) = Swish(W_gate^{R T} x) * (W_up^{R T} x) (Eq. router): the
    SwiGLU activation of each routed expert's representative neuron."""
    return hidden_activations(x, w_gate, w_up, np.asarray(rep_idx, dtype=np.int64))


# ---------------------------------------------------------------- Section 4.3
def softmax(s: np.ndarray) -> np.ndarray:
    s = _f64(s)
    z = np.exp(s - s.max(axis=-1, keepdims=True))
    return z / z.sum(axis=-1, keepdims=True)


def gate_logic(s, top_k: int, gate_scale_u=None, select_bias_b=None):
    """Eq. final_gate.  s' = Softmax(s) over all N_r scores; expert i is
    selected iff s'_i + b_i is among the N_k largest keys; a selected expert's
    gate is 1 + s'_i u_i (the bias takes no part in the gate value).
    Equal keys: the lower index wins.  NaN keys rank below everything.

    Returns (sel_idx [T,N_k] int32 in descending-key order, gates [T,N_k],
    s_prime [T,N_r], keys [T,N_r])."""
    s = _f64(s)
    n_tok, n_r = s.shape
    if not 0 <= top_k <= n_r:
        raise ValueError("top_k must lie in [0, N_r]")
    u = np.zeros(n_r) if gate_scale_u is None else _f64(gate_scale_u)
    b = np.zeros(n_r) if select_bias_b is None else _f64(select_bias_b)
    s_prime = softmax(s)
    keys = s_prime + b
    rank_keys = np.where(np.isnan(keys), -np.inf, keys)
    order = np.argsort(-rank_keys, axis=1, kind="stable")   # full sort of all N_r keys
    sel_idx = order[:, :top_k].astype(np.int32)
    gates = 1.0 + np.take_along_axis(s_prime, sel_idx.astype(np.int64), axis=1) * u[sel_idx]
    return sel_idx, gates, s_prime, keys


def logit_margin(s_prime, keys, top_k: int) -> np.ndarray:
    """Per token: gap between the N_k-th and (N_k+1)-th key, expressed in logit
    (pre-softmax) units: (key_p - key_q) / max(s'_p, s'_q).  With b = 0 this is
    1 - exp(-(s_p - s_q)) ~ s_p - s_q.  +inf when no (N_k+1)-th key exists."""
    keys = _f64(keys)
    n_tok, n_r = keys.shape
    if top_k == 0 or top_k >= n_r:
        return np.full(n_tok, np.inf)
    order = np.argsort(-keys, axis=1, kind="stable")
    p, q = order[:, top_k - 1], order[:, top_k]
    rows = np.arange(n_tok)
    gap = keys[rows, p] - keys[rows, q]
    return gap / np.maximum(s_prime[rows, p], s_prime[rows, q])


# ------------------------------------------------------- Eq. moe_output
def moe_forward(x, w_gate, w_up, w_down, neuron_perm, n_experts: int, n_shared: int,
                sel_idx, gates, token_ids=None) -> np.ndarray:
    """F_MoE(x) = E^s(x) + sum_i g_i E_i^r(x) (Eq. moe_output) with the gate
    values given; terms with g_i = 0 (unselected experts) are skipped.  The
    N_s shared experts form one always-on expert.  Routed experts are added in
    ascending expert index.  ``token_ids`` restricts the evaluation to a
    subset of tokens (used to sample outputs of large workloads)."""
    x = _f64(x)
    sel_idx = np.asarray(sel_idx)
    gates = _f64(gates)
    if token_ids is not None:
        token_ids = np.asarray(token_ids, dtype=np.int64)
        x, sel_idx, gates = x[token_ids], sel_idx[token_ids], gates[token_ids]
    n_r = n_experts - n_shared
    m = len(neuron_perm) // n_experts
    out = np.zeros_like(x)
    if n_shared > 0:
        shared = np.asarray(neuron_perm[:n_shared * m], dtype=np.int64)
        out += expert_forward(x, w_gate, w_up, w_down, shared)
    for j in range(n_r):
        hit_tok, hit_slot = np.nonzero(sel_idx == j)
        if hit_tok.size == 0:
            continue
        neurons = expert_neurons(neuron_perm, n_experts, n_shared + j)
        y = expert_forward(x[hit_tok], w_gate, w_up, w_down, neurons)
        out[hit_tok] += gates[hit_tok, hit_slot][:, None] * y
    return out


def cmoe_layer_forward(x, w_gate, w_up, w_down, neuron_perm, rep_idx, n_experts: int,
                       n_shared: int, top_k: int, gate_scale_u=None, select_bias_b=None):
    """Router (Eq. router) -> gates (Eq. final_gate) -> experts and combine
    (Eq. moe_output).  Returns (out, sel_idx, gates, s, s_prime, keys)."""
    s = router_scores(x, w_gate, w_up, rep_idx)
    sel_idx, gates, s_prime, keys = gate_logic(s, top_k, gate_scale_u, select_bias_b)
    out = moe_forward(x, w_gate, w_up, w_down, neuron_perm, n_experts, n_shared,
                      sel_idx, gates)
    return out, sel_idx, gates, s, s_prime, keys


# ------------------------------------------- token histogram and permutation
def token_permutation(sel_idx, n_groups: int):
    """Expert-contiguous order of the selected (token, expert) pairs.  The
    paper only says that the top-N_k experts are activated; this is the one
    canonical way to list the pairs: sorted by (expert, token).

    cnt[e]      = number of tokens that selected e
    off         = exclusive prefix sum of cnt (length n_groups + 1)
    row_token[r]= token at row r;  rows off[e]..off[e+1]-1 belong to expert e,
                  tokens ascending
    row_of[t,j] = row holding the pair (t, sel_idx[t, j])
    """
    sel_idx = np.asarray(sel_idx)
    n_tok, n_k = sel_idx.shape
    cnt = np.zeros(n_groups, dtype=np.int32)
    for t in range(n_tok):
        for j in range(n_k):
            cnt[sel_idx[t, j]] += 1
    off = np.zeros(n_groups + 1, dtype=np.int32)
    for e in range(n_groups):
        off[e + 1] = off[e] + cnt[e]
    fill = off[:-1].copy()
    row_token = np.full(n_tok * n_k, -1, dtype=np.int32)
    row_of = np.full((n_tok, n_k), -1, dtype=np.int32)
    for t in range(n_tok):                      # ascending token => stable
        for j in range(n_k):
            e = sel_idx[t, j]
            r = fill[e]
            fill[e] += 1
            row_token[r] = t
            row_of[t, j] = r
    return cnt, off, row_token, row_of


# ---------------------------------------------------------------- Section 4.4
def outer_router(x, w_router, outer_top_k: int):
    """Top-level router of an existing MoE layer: logits l = W_r x, the
    outer_top_k largest logits are selected (ties: lower index), weights =
    softmax over the selected logits.  (The paper only says that the top-level
    router selects primary experts; this is the Mixtral-style convention.)"""
    logits = _f64(x) @ _f64(w_router).T
    order = np.argsort(-np.where(np.isnan(logits), -np.inf, logits), axis=1, kind="stable")
    outer_idx = order[:, :outer_top_k].astype(np.int32)
    sel_logits = np.take_along_axis(logits, outer_idx.astype(np.int64), axis=1)
    outer_w = softmax(sel_logits)
    return outer_idx, outer_w, logits


def hier_forward(x, w_router, outer_top_k: int, layers: Sequence[dict], token_ids=None):
    """Section 4.4: every expert E_i of an existing MoE layer is replaced by
    E_i^s + sum_j g'_{i,j} E^r_{i,j}; the output is sum over the selected
    outer experts of w_i times that.  ``layers[i]`` holds the keyword
    arguments of cmoe_layer_forward for outer expert i.
    Returns (out, outer_idx, outer_w, per-expert routing list)."""
    x = _f64(x)
    outer_idx, outer_w, _ = outer_router(x, w_router, outer_top_k)
    keep = np.arange(x.shape[0]) if token_ids is None else np.asarray(token_ids, dtype=np.int64)
    out = np.zeros((len(keep), x.shape[1]))
    routing = []
    for i, layer in enumerate(layers):
        tok, slot = np.nonzero(outer_idx == i)          # tok ascending
        routing.append(None)
        if tok.size == 0:
            continue
        s = router_scores(x[tok], layer["w_gate"], layer["w_up"], layer["rep_idx"])
        sel_idx, gates, s_prime, keys = gate_logic(
            s, layer["top_k"], layer.get("gate_scale_u"), layer.get("select_bias_b"))
        routing[i] = dict(tokens=tok, sel_idx=sel_idx, gates=gates, s=s,
                          s_prime=s_prime, keys=keys)
        in_keep = np.isin(tok, keep)
        if not in_keep.any():
            continue
        sub = np.nonzero(in_keep)[0]
        y = moe_forward(x[tok], layer["w_gate"], layer["w_up"], layer["w_down"],
                        layer["neuron_perm"], layer["n_experts"], layer["n_shared"],
                        sel_idx, gates, token_ids=sub)
        dst = np.searchsorted(keep, tok[sub])
        out[dst] += outer_w[tok[sub], slot[sub]][:, None] * y
    return out, outer_idx, outer_w, routing


# ---------------------------------------------------------------- Section 4.3
def bias_update(select_bias_b, counts, target_share=None, gamma: float = 1e-3):
    """One step of the load-balancing rule: with p_i the fraction of routed
    assignments that went to expert i and p* the target (uniform 1/N_r in the
    paper), b_i decreases by gamma if p_i > p*, increases by gamma if p_i < p*."""
    b = _f64(select_bias_b).copy()
    counts = _f64(counts)
    p = counts / counts.sum()
    target = np.full_like(p, 1.0 / len(p)) if target_share is None else _f64(target_share)
    b[p > target] -= gamma
    b[p < target] += gamma
    return b


def fit_select_bias(s, top_k: int, target_share, iters: int = 4000,
                    gamma_hi: float = 2e-2, gamma_lo: float = 1e-4, tol: float = 3e-3):
    """Iterate bias_update on fixed router scores with a geometrically decaying
    step until every expert's share is within ``tol`` of its target.  Produces
    the selection bias of the skewed-load workload (an input to both sides)."""
    s_prime = softmax(s)
    n_tok, n_r = s_prime.shape
    b = np.zeros(n_r)
    target = _f64(target_share)
    for it in range(iters):
        order = np.argsort(-(s_prime + b), axis=1, kind="stable")[:, :top_k]
        counts = np.bincount(order.ravel(), minlength=n_r)
        if np.abs(counts / counts.sum() - target).max() <= tol:
            break
        gamma = gamma_hi * (gamma_lo / gamma_hi) ** (it / max(iters - 1, 1))
        b = bias_update(b, counts, target, gamma)
    return b, counts


# ------------------------------------------- Section 4.1 / Appendix: profiling
def atopk(h, k_a: int) -> np.ndarray:
    """Binary activation matrix A (Eq. atopk_appendix): A[t, i] = 1 when |h[t, i]|
    is among the K_a largest magnitudes of row t.  Equal magnitudes at the cut
    go to the lower neuron index (a convention; the paper does not fix it).
    h: [q, d_h] -> uint8 [q, d_h]."""
    mag = np.abs(_f64(h))
    order = np.argsort(-mag, axis=1, kind="stable")[:, :k_a]
    a = np.zeros(mag.shape, dtype=np.uint8)
    np.put_along_axis(a, order, 1, axis=1)
    return a


def atopk_margin(h, k_a: int) -> np.ndarray:
    """Relative gap between the K_a-th and (K_a+1)-th largest |h| of each row,
    (m_K - m_{K+1}) / m_K: how far a row is from a different ATopK set."""
    mag = -np.sort(-np.abs(_f64(h)), axis=1)
    if k_a >= mag.shape[1]:
        return np.full(mag.shape[0], np.inf)
    top, nxt = mag[:, k_a - 1], mag[:, k_a]
    return (top - nxt) / np.maximum(top, np.finfo(F64).tiny)


def activation_counts(a) -> np.ndarray:
    """Number of tokens for which each neuron is active; mu_i = counts_i / q
    (Eq. mu_appendix).  a: [q, d_h] -> int64 [d_h]."""
    return np.asarray(a, dtype=np.int64).sum(axis=0)


def activation_rates(a) -> np.ndarray:
    a = np.asarray(a)
    return activation_counts(a) / F64(a.shape[0])


def select_shared(counts, n_select: int) -> np.ndarray:
    """The n_select = N_s*m neurons with the highest activation rate
    (Eq. S_Ns_appendix), listed from the highest rate down; equal rates go to
    the lower neuron index."""
    counts = np.asarray(counts, dtype=np.int64)
    return np.argsort(-counts, kind="stable")[:n_select].astype(np.int64)


def pack_columns(a) -> np.ndarray:
    """Bit-packed columns of A: word [i, t // 32] holds A[t, i] in bit t % 32
    (the storage both sides use for the activation feature vectors c_i)."""
    a = np.asarray(a, dtype=np.uint8)
    q, d_h = a.shape
    words = (q + 31) // 32
    padded = np.zeros((words * 32, d_h), dtype=np.uint8)
    padded[:q] = a
    bits = padded.reshape(words, 32, d_h).astype(np.uint64)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))[None, :, None]
    return (bits * weights).sum(axis=1).astype(np.uint32).T.copy()


def profile_activations(x, w_gate, w_up, k_a: int, n_select: int):
    """Steps 1-4 of the profiling pipeline on calibration rows x [q, d]:
    H (Eq. h_matrix_appendix), A (ATopK), counts (q * mu), shared-neuron list."""
    h = hidden_activations(x, w_gate, w_up)
    a = atopk(h, k_a)
    counts = activation_counts(a)
    return h, a, counts, select_shared(counts, n_select)


# ------------------------------- Appendix: balanced clustering of routed neurons
def initial_centroids(counts, shared_idx, n_routed: int) -> np.ndarray:
    """Neuron indices of the N_r initial centroids: the remaining (non-shared)
    neurons with the highest activation rates, highest first, ties to the lower index."""
    counts = np.asarray(counts, dtype=np.int64)
    shared = set(int(i) for i in np.asarray(shared_idx).ravel())
    order = [int(i) for i in np.argsort(-counts, kind="stable") if int(i) not in shared]
    return np.asarray(order[:n_routed], dtype=np.int64)


def centroid_distances(c, centroids) -> np.ndarray:
    """d[i, j] = || c_i - chat_j ||_2 over the q calibration tokens.
    c: [q, n] activation feature vectors (columns of A); centroids: [q, N_r]."""
    c, centroids = _f64(c), _f64(centroids)
    diff = c[:, :, None] - centroids[:, None, :]
    return np.sqrt((diff * diff).sum(axis=0))


def cluster_update(c, assign, prev_centroids) -> np.ndarray:
    """chat_j <- mean of the c_i assigned to cluster j; a cluster without members
    keeps its previous centroid.  assign: [n] cluster of each neuron (-1: none)."""
    c = _f64(c)
    assign = np.asarray(assign, dtype=np.int64)
    out = _f64(prev_centroids).copy()
    for j in range(out.shape[1]):
        members = np.nonzero(assign == j)[0]
        if len(members) > 0:
            out[:, j] = c[:, members].sum(axis=1) / len(members)
    return out


def representatives(c, assign, centroids) -> np.ndarray:
    """R_j = argmin over the neurons of cluster j of || c_i - chat_j ||_2
    (Eq. rep_neuron); equal distances go to the lower position.  Returns the
    position in c's columns for each cluster (-1 for an empty cluster)."""
    d = centroid_distances(c, centroids)
    assign = np.asarray(assign, dtype=np.int64)
    reps = np.full(d.shape[1], -1, dtype=np.int64)
    for j in range(d.shape[1]):
        members = np.nonzero(assign == j)[0]
        if len(members) > 0:
            reps[j] = members[np.argmin(d[members, j])]      # argmin returns the first minimum
    return reps


def balanced_assignment(d, m: int) -> np.ndarray:
    """Assignment T with every row in exactly one cluster and every cluster holding m
    rows that minimises sum_ij T_ij d_ij (Eq. con_1_appendix), solved as the paper does:
    each column repeated m times, then a linear assignment (library routine)."""
    from scipy.optimize import linear_sum_assignment
    d = _f64(d)
    n, n_r = d.shape
    assert n == n_r * m
    rows, cols = linear_sum_assignment(np.repeat(d, m, axis=1))
    assign = np.empty(n, dtype=np.int64)
    assign[rows] = cols // m
    return assign


# ------------------- Section 6 "Compatibility with Other Efficiency Techniques"
# Post-training weight quantisation of the restructured experts.  The paper only states that
# the restructured FFN composes with post-training quantisation and fixes no format; the
# reading taken here: weight-only FP8 in the OCP E4M3 encoding (1 sign, 4 exponent bits with
# bias 7, 3 mantissa bits, subnormals, largest finite value 448, no infinities; S.1111.111 is
# NaN) with ONE POWER-OF-TWO scale per output channel, as in the OCP microscaling formats'
# E8M0 scales.  Output channel = a neuron's row of W_gate / W_up, and a row of an expert's
# block of W_down^T (one scale per (expert, model dimension); the N_s shared experts form one
# block).  Activations, the router's representative rows and all arithmetic stay as they are.
# Because the scale is a power of two, w / scale is exact in any binary format, so the code
# chosen by round-to-nearest-even does not depend on the precision it is computed in, and the
# dequantised weight code * scale is again exact (also in bf16).

E4M3_MAX = 448.0


def fp8_e4m3_decode(codes) -> np.ndarray:
    """Value of each E4M3 code byte: (-1)^s * 2^(E-7) * (1 + M/8) for E > 0,
    (-1)^s * 2^-6 * (M/8) for E = 0; codes 0x7F / 0xFF are NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    s, e, m = c >> 7, (c >> 3) & 0xF, c & 0x7
    mag = np.where(e > 0, np.ldexp(1.0 + m / 8.0, e - 7), np.ldexp(m / 8.0, -6))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return np.where(s == 1, -mag, mag)


def fp8_e4m3_encode(v) -> np.ndarray:
    """Nearest E4M3 code of each value, ties to the even mantissa, magnitudes beyond 448
    saturate to +-448 (no infinities in this format); NaN -> 0x7F."""
    v = _f64(v)
    a = np.abs(v)
    out = np.zeros(v.shape, dtype=np.uint8)
    fin = ~np.isnan(v)
    a_f = np.where(fin, np.minimum(a, E4M3_MAX), 0.0)
    # spacing of representable values around a: 2^(e-3) in the binade 2^e, 2^-9 below 2^-6
    _, p = np.frexp(a_f)                       # a = f * 2^p, f in [0.5, 1)  =>  binade exponent p - 1
    e = np.maximum(p - 1, -6)
    q = np.rint(np.ldexp(a_f, 3 - e))          # a / 2^(e-3), rounded half to even; in [0, 16]
    # q = 16 means the value rounded up into the next binade
    bump = q >= 16
    e = np.where(bump, e + 1, e)
    q = np.where(bump, 8.0, q)
    normal = q >= 8                            # q in [8, 15]: 1.M with M = q - 8; below: subnormal, M = q
    field_e = np.where(normal, e + 7, 0).astype(np.int64)
    field_m = np.where(normal, q - 8, q).astype(np.int64)
    code = (field_e << 3) | field_m
    code = np.where(code > 0x7E, 0x7E, code)   # cannot exceed 448 after the clamp; kept as a guard
    sign = (np.signbit(v) & fin).astype(np.int64) << 7
    out = np.where(fin, code | sign, 0x7F).astype(np.uint8)
    return out


def pow2_scale_exponent(amax) -> np.ndarray:
    """Smallest integer e with amax * 2^-e <= 448 (so that the channel's largest weight uses the
    top of the E4M3 range); 0 for an all-zero channel."""
    amax = _f64(amax)
    f, p = np.frexp(amax)                      # amax = f * 2^p, f in [0.5, 1);  448 = 0.875 * 2^9
    e = np.where(f <= 0.875, p - 9, p - 8)
    return np.where(amax > 0, e, 0).astype(np.int64)


def quantise_rows_fp8(w):
    """Per-row (output-channel) power-of-two scale and E4M3 codes of a weight matrix [rows, k].
    Returns (codes uint8 [rows, k], scale_exponent int64 [rows]); weight ~ decode(code) * 2^e."""
    w = _f64(w)
    e = pow2_scale_exponent(np.abs(w).max(axis=1)) if w.shape[1] else np.zeros(w.shape[0], np.int64)
    codes = fp8_e4m3_encode(np.ldexp(w, -e[:, None]))
    return codes, e


def dequantise_rows_fp8(codes, scale_exponent) -> np.ndarray:
    return np.ldexp(fp8_e4m3_decode(codes), np.asarray(scale_exponent, dtype=np.int64)[:, None])


def quantise_expert_weights(w_gate, w_up, w_down, neuron_perm, n_experts: int, n_shared: int):
    """FP8 weight-only quantisation of a restructured layer.  W_gate and W_up: one scale per
    neuron (row).  W_down: one scale per (expert block, model dimension), the block being the
    expert's slice of neurons (all shared experts together form block 0).  Returns a dict with
    the dequantised matrices in the original layout (``w_gate``, ``w_up``, ``w_down``: what a
    forward pass of the quantised layer multiplies by) and the codes / scale exponents:
    ``gate_codes, gate_exp, up_codes, up_exp`` by original neuron, ``down_codes`` [d, d_ff] by
    original neuron column, ``down_exp`` [1 + N_r, d] by block."""
    w_down = _f64(w_down)
    d_ff = len(neuron_perm)
    m = d_ff // n_experts
    n_r = n_experts - n_shared
    g_codes, g_exp = quantise_rows_fp8(w_gate)
    u_codes, u_exp = quantise_rows_fp8(w_up)
    blocks = []
    if n_shared > 0:
        blocks.append(np.asarray(neuron_perm[:n_shared * m], dtype=np.int64))
    for j in range(n_r):
        blocks.append(expert_neurons(neuron_perm, n_experts, n_shared + j))
    d_codes = np.zeros(w_down.shape, dtype=np.uint8)
    d_exp = np.zeros((len(blocks), w_down.shape[0]), dtype=np.int64)
    w_down_q = np.zeros_like(w_down)
    for b, neurons in enumerate(blocks):
        codes, e = quantise_rows_fp8(w_down[:, neurons])
        d_codes[:, neurons] = codes
        d_exp[b] = e
        w_down_q[:, neurons] = dequantise_rows_fp8(codes, e)
    return dict(w_gate=dequantise_rows_fp8(g_codes, g_exp), w_up=dequantise_rows_fp8(u_codes, u_exp),
                w_down=w_down_q, gate_codes=g_codes, gate_exp=g_exp, up_codes=u_codes, up_exp=u_exp,
                down_codes=d_codes, down_exp=d_exp, has_shared_block=n_shared > 0)


def cmoe_layer_forward_fp8(x, w_gate, w_up, w_down, neuron_perm, rep_idx, n_experts: int,
                           n_shared: int, top_k: int, gate_scale_u=None, select_bias_b=None):
    """Forward of the layer with FP8-quantised expert weights: the router (Eq. router) reads the
    ORIGINAL representative rows, so the routing is that of the unquantised layer; the experts
    (Eq. moe_output) multiply by the dequantised weights.  Returns what cmoe_layer_forward does."""
    q = quantise_expert_weights(w_gate, w_up, w_down, neuron_perm, n_experts, n_shared)
    s = router_scores(x, w_gate, w_up, rep_idx)
    sel_idx, gates, s_prime, keys = gate_logic(s, top_k, gate_scale_u, select_bias_b)
    out = moe_forward(x, q["w_gate"], q["w_up"], q["w_down"], neuron_perm, n_experts, n_shared,
                      sel_idx, gates)
    return out, sel_idx, gates, s, s_prime, keys
