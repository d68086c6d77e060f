"""Pins for the oracle's group-limited routing (published DeepSeek-V3 rule): reduction to the plain
sigmoid top-k, an independent sort-based evaluation, structural properties, bias and scale.  CPU only."""
import numpy as np
import pytest

import oracle


def _cfg(E, k, ng, kg, scale=1.0):
    return oracle.Config(H=8, I=8, E=E, top_k=k, score=oracle.SCORE_SIGMOID, routed_scale=scale, n_group=ng,
                         topk_group=kg)


def _sort_based(logits, bias, k, ng, kg, scale):
    """Independent evaluation with numpy sorts (lexicographic keys give the tie rules)."""
    T, E = logits.shape
    gs = E // ng
    s = 1.0 / (1.0 + np.exp(-logits))
    c = s + (0.0 if bias is None else bias.astype(np.float64))
    ids = np.empty((T, k), dtype=np.int32)
    w = np.empty((T, k))
    for t in range(T):
        grp = c[t].reshape(ng, gs)
        top2 = -np.sort(-grp, axis=1)[:, :2].sum(1) if gs >= 2 else grp[:, 0]
        order = np.lexsort((np.arange(ng), -top2))          # score descending, index ascending
        kept = np.zeros(ng, dtype=bool)
        kept[order[:kg]] = True
        cand = [e for e in range(E) if kept[e // gs]]
        cand.sort(key=lambda e: (-c[t, e], e))
        ids[t] = cand[:k]
        w[t] = scale * s[t, ids[t]] / (s[t, ids[t]].sum() + 1e-20)
    return ids, w


def test_one_group_without_bias_is_the_plain_sigmoid_topk():
    rs = np.random.RandomState(0)
    logits = rs.normal(0, 1, (50, 64))
    ids_g, w_g, _ = oracle.topk_grouped(_cfg(64, 6, 1, 1, 2.5), logits)
    ids_p, w_p, _ = oracle.topk(oracle.Config(H=8, I=8, E=64, top_k=6, score=oracle.SCORE_SIGMOID, routed_scale=2.5), logits)
    np.testing.assert_array_equal(ids_g, ids_p)
    np.testing.assert_allclose(w_g, w_p, rtol=1e-13)


@pytest.mark.parametrize("E,k,ng,kg", [(256, 8, 8, 4), (64, 6, 4, 2), (32, 4, 8, 3), (16, 2, 16, 5)])
def test_matches_sort_based_evaluation(E, k, ng, kg):
    rs = np.random.RandomState(E + k)
    logits = rs.normal(0, 1.5, (40, E))
    logits[3] = np.round(logits[3])            # many exact ties in one token
    logits[4] = 0.0                            # everything tied
    bias = rs.normal(0, 0.2, E).astype(np.float32)
    bias[5] = bias[6]                          # tied biases too
    for b in (None, bias):
        ids, w, gap = oracle.topk_grouped(_cfg(E, k, ng, kg, 2.5), logits, b)
        ids_r, w_r = _sort_based(logits, b, k, ng, kg, 2.5)
        np.testing.assert_array_equal(ids, ids_r)
        np.testing.assert_allclose(w, w_r, rtol=1e-13)
        assert (gap >= 0).all()


def test_structure_bias_and_scale():
    E, k, ng, kg = 64, 8, 8, 2
    gs = E // ng
    rs = np.random.RandomState(9)
    logits = rs.normal(0, 1, (30, E))
    ids, w, _ = oracle.topk_grouped(_cfg(E, k, ng, kg, 2.5), logits)
    for t in range(30):
        assert len(set(ids[t] // gs)) <= kg                      # at most topk_group groups are used
        assert len(set(ids[t])) == k
    np.testing.assert_allclose(w.sum(1), 2.5, rtol=1e-12)        # weights sum to the routed scale
    # a large bias forces an expert in (and its group), but weights keep using the unbiased score
    bias = np.zeros(E, dtype=np.float32)
    bias[37] = 10.0
    ids_b, w_b, _ = oracle.topk_grouped(_cfg(E, k, ng, kg, 1.0), logits, bias)
    assert (ids_b[:, 0] == 37).all()
    s = 1.0 / (1.0 + np.exp(-logits))
    sel = np.take_along_axis(s, ids_b.astype(np.int64), 1)
    np.testing.assert_allclose(w_b, sel / sel.sum(1, keepdims=True), rtol=1e-12)
    # a bias that is constant inside every group and ordered across groups selects the groups by itself
    gb = np.repeat(np.arange(ng, dtype=np.float32) * 3.0, gs)
    ids_c, _, _ = oracle.topk_grouped(_cfg(E, k, ng, kg, 1.0), logits, gb)
    assert set(np.unique(ids_c // gs)) <= {ng - 1, ng - 2} and (np.sort(ids_c, axis=1) == np.arange(E - gs, E)).all()
    ids_d, _, _ = oracle.topk_grouped(_cfg(E, 12, ng, kg, 1.0), logits, gb)       # k > group size: both kept groups are used
    assert set(np.unique(ids_d // gs)) == {ng - 1, ng - 2}
