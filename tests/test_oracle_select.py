"""Pins of the oracle's cost-aware draft selection (Algorithm 1, Eqs. 7-10) against an
independent set-based evaluation, the worked example of Fig. 3, and the prefix-consistency
property stated in Sec. 4.2.  CPU only."""
import numpy as np
import pytest

import oracle
import synth


def _bits(pairs, L, E):
    W = (L * E + 31) // 32
    out = np.zeros(W, dtype=np.uint32)
    for (l, e) in pairs:
        b = l * E + e
        out[b >> 5] |= np.uint32(1 << (b & 31))
    return out


def _set_based(parent, P, sets, gamma, eps, B0=frozenset(), global_cost=False):
    """Algorithm 1 with Python sets of (layer, expert) pairs; scores in float32."""
    n = len(parent)
    traj = []
    for i in range(n):
        traj.append(set(sets[i]) | (traj[parent[i]] if parent[i] >= 0 else set()))
    B, S, costs = set(B0), [], []
    while len(S) < min(gamma, n):
        best, bs, bc = None, None, None
        for i in range(n):
            if i in S:
                continue
            cost = len(traj[i]) if global_cost else len(traj[i] - B)
            score = np.float32(P[i]) / (np.float32(cost) + np.float32(eps))
            if best is None or score > bs:
                best, bs, bc = i, score, cost
        S.append(best)
        costs.append(bc)
        if not global_cost:
            B |= traj[best]
    return S, costs, B


def _unpack(pred, L, E):
    sets = []
    for row in pred:
        s = set()
        for w, word in enumerate(row):
            for b in range(32):
                if (int(word) >> b) & 1:
                    bit = w * 32 + b
                    s.add((bit // E, bit % E))
        sets.append(s)
    return sets


@pytest.mark.parametrize("L,E,K,depth,gamma,glob", [(4, 32, 4, 3, 4, False), (6, 64, 8, 3, 8, False),
                                                    (3, 16, 2, 4, 6, False), (4, 32, 4, 3, 5, True)])
def test_selection_matches_set_based_algorithm(L, E, K, depth, gamma, glob):
    parent, P, pred = synth.make_draft_tree(L, E, K, depth=depth)
    sel, costs, buf = oracle.select_drafts(parent, P, pred, gamma, eps=1e-6, global_cost=glob)
    S, C, B = _set_based(list(parent), list(P), _unpack(pred, L, E), gamma, 1e-6, global_cost=glob)
    assert list(sel) == S and list(costs) == C
    if not glob:
        np.testing.assert_array_equal(buf, _bits(B, L, E))
        assert sel[0] == 0  # the root has P = 1 and the smallest path footprint


def test_fig3_worked_example():
    """Fig. 3: gamma = 2.  Step 1 picks the root t0 and puts its 4 predicted experts in B.
    Step 2: t1 has the higher cumulative probability (0.53) but 3 new experts, score 0.17;
    t2 introduces 2 new experts and scores 0.20, so S = {t0, t2}.  The figure does not print
    P(t2); every value consistent with a printed 0.20 at cost 2 (and below 0.53) must give t2."""
    L, E = 1, 16
    root = {(0, 1), (0, 2), (0, 3), (0, 4)}
    t1 = {(0, 5), (0, 6), (0, 7), (0, 1)}            # 3 new experts
    t2 = {(0, 2), (0, 3), (0, 8), (0, 9)}            # reuses two covered experts, 2 new
    pred = np.stack([_bits(s, L, E) for s in (root, t1, t2)])
    assert float(np.float32(0.53) / np.float32(3)) // 0.01 * 0.01 == pytest.approx(0.17)
    for p2 in (0.40, 0.41, 0.419):
        sel, costs, _ = oracle.select_drafts([-1, 0, 0], [1.0, 0.53, p2], pred, 2, eps=1e-6)
        assert list(sel) == [0, 2] and list(costs) == [4, 2]
        assert 0.20 <= p2 / 2 < 0.21
    # acceptance-only ranking (no cost) would have taken t1: zero predicted sets -> cost 0 for all
    sel, _, _ = oracle.select_drafts([-1, 0, 0], [1.0, 0.53, 0.41], np.zeros_like(pred), 2, eps=1e-6)
    assert list(sel) == [0, 1]


def test_prefix_consistency_and_buffer_effect():
    parent, P, pred = synth.make_draft_tree(5, 48, 6, depth=4)
    n = len(parent)
    sel, costs, buf = oracle.select_drafts(parent, P, pred, n, eps=1e-6)
    pos = {int(node): i for i, node in enumerate(sel)}
    assert sorted(pos) == list(range(n))
    for c in range(1, n):              # a child never precedes its parent (Sec. 4.2)
        assert pos[int(parent[c])] < pos[c]
    # dynamic buffer: a preloaded buffer can only lower costs, and a full buffer makes every
    # cost zero, reducing the rule to ranking by cumulative probability (ties to lower index)
    full = np.full(pred.shape[1], 0xFFFFFFFF, dtype=np.uint32)
    sel_f, costs_f, _ = oracle.select_drafts(parent, P, pred, n, eps=1e-6, buffer0=full)
    assert set(costs_f) == {0}
    order = sorted(range(n), key=lambda i: (-float(P[i]), i))
    assert list(sel_f) == order


def test_global_cost_variant_does_not_update_buffer():
    parent, P, pred = synth.make_draft_tree(4, 32, 4, depth=3)
    b0 = np.zeros(pred.shape[1], dtype=np.uint32)
    b0[0] = 0xF0F0
    sel, costs, buf = oracle.select_drafts(parent, P, pred, 5, eps=1e-6, buffer0=b0, global_cost=True)
    np.testing.assert_array_equal(buf, b0)
    # costs are path footprints |E_traj|, independent of the buffer (Eq. 10)
    sets = _unpack(pred, 4, 32)
    for node, c in zip(sel, costs):
        traj, i = set(), int(node)
        while i >= 0:
            traj |= sets[i]
            i = int(parent[i])
        assert c == len(traj)
