"""CPU tests of the comparison rules the -m gpu tests apply (tests/parity.py): the outer near-tie
rule of hierarchical layers and the stratified token sample.  The "CUDA result" here is made up
on the host from the oracle's own, so no device is needed."""
import numpy as np
import pytest

from oracle import cmoe_oracle as oracle
from tests import parity


def _outer_case():
    """5 tokens, 4 outer experts, top-2, d = 4 with unit-vector tokens so that the logits are
    the router's columns: token t sees logits w_router[:, t % 4] scaled by its own length."""
    w_router = np.array([[0.90, 0.10, 0.50, 0.30],
                         [0.50, 0.70, 0.500004, 0.10],     # token 2: experts 0/1/2 within 4e-6
                         [0.499995, 0.20, 0.500002, 0.20],  # token 0: experts 1/2 within 5e-6 of each other
                         [0.10, 0.60, 0.10, 0.2995]])       # token 3: experts 0/3 5e-4 apart
    x = np.eye(4)[[0, 1, 2, 3, 0]]
    return x, w_router


def test_outer_rule_accepts_equal_and_admissible_choices():
    x, w_r = _outer_case()
    o_idx, o_w, logits = oracle.outer_router(x, w_r, 2)
    assert o_idx.tolist() == [[0, 1], [1, 3], [1, 2], [0, 3], [0, 1]]
    # identical choice: nothing is patched
    idx, w, near, diff = parity.check_outer_routing(o_idx.copy(), o_w.copy(), x, w_r, 2)
    assert diff == 0 and near == 3 and np.array_equal(idx, o_idx)      # tokens 0, 2, 4 are near-ties
    # token 0 trades expert 1 for expert 2 (5e-6 below the cut): admissible, patched, weights recomputed
    g_idx, g_w = o_idx.copy(), o_w.copy()
    g_idx[0] = [0, 2]
    z = np.exp(np.array([0.90, 0.499995]) - 0.90)
    g_w[0] = z / z.sum()
    idx, w, near, diff = parity.check_outer_routing(g_idx, g_w, x, w_r, 2)
    assert diff == 1 and idx[0].tolist() == [0, 2] and idx[4].tolist() == [0, 1]
    np.testing.assert_allclose(w[0], g_w[0], rtol=1e-12)
    np.testing.assert_allclose(w[1:], o_w[1:], rtol=0, atol=0)
    # the order in which the CUDA path lists the pair carries no meaning
    g_idx[0], g_w[0] = [2, 0], g_w[0][::-1].copy()
    parity.check_outer_routing(g_idx, g_w, x, w_r, 2)


def test_outer_rule_rejects_inadmissible_choices():
    x, w_r = _outer_case()
    o_idx, o_w, _ = oracle.outer_router(x, w_r, 2)
    # token 1: clear margins (0.7, 0.6 | 0.2): any other set is an error
    g = o_idx.copy(); g[1] = [1, 2]
    with pytest.raises(AssertionError):
        parity.check_outer_routing(g, o_w.copy(), x, w_r, 2)
    # token 0 is a near-tie between experts 1 and 2, but dropping expert 0 (0.4 above the cut) is not admissible
    g = o_idx.copy(); g[0] = [1, 2]
    with pytest.raises(AssertionError):
        parity.check_outer_routing(g, o_w.copy(), x, w_r, 2)
    # token 3: the runner-up is 5e-4 below the cut, a near-tie by the 1e-3 rule; the weights must
    # then be those of the traded selection, not the oracle's original ones
    g = o_idx.copy(); g[3] = [0, 1]
    with pytest.raises(AssertionError):
        parity.check_outer_routing(g, o_w.copy(), x, w_r, 2)      # expert 1 (0.10) is far from the cut
    # wrong weights on an untouched token
    bad_w = o_w.copy(); bad_w[1] = bad_w[1][::-1]
    with pytest.raises(AssertionError):
        parity.check_outer_routing(o_idx.copy(), bad_w, x, w_r, 2)


def test_stratified_sample_covers_the_edges():
    rng = np.random.default_rng(0)
    n_tok, n_groups, n_k = 3000, 6, 2
    keys = rng.random((n_tok, n_groups)) * np.array([4.0, 1, 1, 1, 1, 0.75])      # group 0 large, group 5 small
    sel = np.argsort(-keys, axis=1)[:, :n_k].astype(np.int32)
    cnt, off, row_token, _ = oracle.token_permutation(sel, n_groups)
    ids = parity.stratified_tokens(n_tok, cnt, off, row_token, seed=1)
    assert np.all(np.diff(ids) > 0) and ids[0] == 0 and ids[-1] == n_tok - 1
    assert {127, 128, 2943, 2944} <= set(ids.tolist())
    for g in range(n_groups):
        assert row_token[off[g]] in ids and row_token[off[g + 1] - 1] in ids
    big, small = int(np.argmax(cnt)), int(np.argmin(cnt))
    assert cnt[big] > 256 and cnt[small] > 128
    for g in (big, small):
        for e in range(128, cnt[g], 128):
            assert row_token[off[g] + e - 1] in ids and row_token[off[g] + e] in ids
    assert len(ids) < 400
    # a layer without routed experts still gets the batch ends, the shared tile edges and the random draw
    ids0 = parity.stratified_tokens(n_tok, [], [0], [], seed=1)
    assert {0, 127, 128, n_tok - 1} <= set(ids0.tolist())
