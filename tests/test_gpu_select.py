"""GPU parity of the cost-aware draft selection kernel (Algorithm 1) against the oracle:
selected nodes, their costs and the final expert buffer must be bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth

pytestmark = pytest.mark.gpu


def _run(parent, P, pred, gamma, eps=1e-6, buffer0=None, global_cost=False):
    dev = "cuda"
    tp = torch.from_numpy(parent).to(dev)
    tP = torch.from_numpy(P).to(dev)
    tpred = torch.from_numpy(pred.view(np.int32)).to(dev)
    tb = None if buffer0 is None else torch.from_numpy(buffer0.view(np.int32)).to(dev)
    sel, costs, buf, nsel, _ = moev.select_drafts(tp, tP, tpred, gamma, eps, tb, global_cost)
    torch.cuda.synchronize()
    k = int(nsel.item())
    return sel.cpu().numpy()[:k], costs.cpu().numpy()[:k], buf.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("L,E,K,depth,branch,gamma", [
    (58, 256, 8, 3, 2, 4),      # DeepSeek-V3.1-sized footprint, the paper's tree (3 steps x top-2) and budget
    (94, 128, 8, 3, 2, 4),      # Qwen3-235B-sized
    (36, 128, 4, 3, 2, 4),      # GPT-OSS-sized
    (58, 256, 8, 5, 2, 16),     # deeper tree, larger budget
    (4, 32, 4, 6, 3, 64),       # 1093 nodes: more nodes than threads' warps, many rounds
    (1, 16, 2, 2, 2, 100)])     # budget larger than the tree
def test_selection_matches_oracle(L, E, K, depth, branch, gamma):
    parent, P, pred = synth.make_draft_tree(L, E, K, depth=depth, branch=branch)
    for glob in (False, True):
        s_ref, c_ref, b_ref = oracle.select_drafts(parent, P, pred, gamma, eps=1e-6, global_cost=glob)
        s, c, b = _run(parent, P, pred, gamma, global_cost=glob)
        np.testing.assert_array_equal(s, s_ref)
        np.testing.assert_array_equal(c, c_ref)
        np.testing.assert_array_equal(b, b_ref)


@pytest.mark.parametrize("L,E,K,depth,gamma,ties", [
    (58, 256, 8, 7, 64, False),    # 255 nodes x 464 words: footprints over 8 CTAs' shared memory
    (58, 256, 8, 9, 128, False),   # 1023 nodes: 32 CTAs
    (94, 128, 8, 6, 40, True),     # 127 nodes x 376 words, coarse probabilities (many exact score ties), initial buffer
    (61, 96, 6, 7, 300, False)])   # 183 words (not a multiple of four), budget larger than the tree
def test_selection_long_bitmaps_several_ctas(L, E, K, depth, gamma, ties):
    """Bitmaps too long for one CTA's shared memory take the cooperative multi-CTA kernel: same
    selections, costs and final buffer, bit for bit."""
    parent, P, pred = synth.make_draft_tree(L, E, K, depth=depth)
    b0 = None
    if ties:
        P = (np.round(P * 8) / 8).astype(np.float32)
        P[0] = 1.0
        b0 = np.random.RandomState(5).randint(0, 2 ** 32, size=pred.shape[1], dtype=np.uint64).astype(np.uint32)
        b0 &= np.random.RandomState(6).randint(0, 2 ** 32, size=pred.shape[1], dtype=np.uint64).astype(np.uint32)
    eps = 0.5 if ties else 1e-6
    s_ref, c_ref, b_ref = oracle.select_drafts(parent, P, pred, gamma, eps=eps, buffer0=b0)
    for rep in range(2):                                     # twice: the control words are reset per call
        s, c, b = _run(parent, P, pred, gamma, eps=eps, buffer0=b0)
        np.testing.assert_array_equal(s, s_ref)
        np.testing.assert_array_equal(c, c_ref)
        np.testing.assert_array_equal(b, b_ref)


def test_selection_with_initial_buffer_and_ties():
    parent, P, pred = synth.make_draft_tree(8, 64, 4, depth=4)
    b0 = np.random.RandomState(3).randint(0, 2 ** 32, size=pred.shape[1], dtype=np.uint64).astype(np.uint32)
    P = np.round(P * 8) / 8                      # coarse probabilities: many exact score ties
    P[0] = 1.0
    P = P.astype(np.float32)
    s_ref, c_ref, b_ref = oracle.select_drafts(parent, P, pred, 12, eps=0.5, buffer0=b0)
    s, c, b = _run(parent, P, pred, 12, eps=0.5, buffer0=b0)
    np.testing.assert_array_equal(s, s_ref)
    np.testing.assert_array_equal(c, c_ref)
    np.testing.assert_array_equal(b, b_ref)


def test_selection_rejects_bad_arguments():
    parent, P, pred = synth.make_draft_tree(2, 16, 2, depth=2)
    tp = torch.from_numpy(parent).cuda()
    tP = torch.from_numpy(P).cuda()
    tpred = torch.from_numpy(pred.view(np.int32)).cuda()
    with pytest.raises(moev.MoevError):
        moev.select_drafts(tp, tP, tpred, 0)
    with pytest.raises(moev.MoevError):
        moev.select_drafts(tp, tP, tpred, 2, eps=0.0)


def test_selection_then_verify_union_matches_buffer():
    """End to end with the verification layer: when the predicted sets are the nodes' true routing
    (single layer), the expert buffer the selection ends with is exactly the union the router
    kernels report for the selected tokens."""
    shape = synth.SHAPES["tiny"]
    parent, P, pred = synth.make_draft_tree(1, shape.E, shape.top_k, depth=4, branch=2, seed_tag="e2e-tree")
    wr, x_all = synth.make_tree_verify_inputs(shape, parent, pred, device="cuda")
    gamma = 8
    tp, tP = torch.from_numpy(parent).cuda(), torch.from_numpy(P).cuda()
    tpred = torch.from_numpy(pred.view(np.int32)).cuda()
    sel, costs, buf, nsel, _ = moev.select_drafts(tp, tP, tpred, gamma, 1e-6)
    torch.cuda.synchronize()
    w = synth.make_expert_weights(shape, layer=0, device="cuda")
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt, shape.afmt,
                          shape.score, moev.IMPL_AUTO, shape.routed_scale)
    v = moev.MoeVerifier(cfg)
    d = {"router_w": wr}
    d.update({k: t for k, t in w.items() if t is not None})
    L = moev.binding.make_layer(d)
    out = v.alloc_out(gamma, diagnostics=True)
    v.verify(L, x_all[sel.long()].contiguous(), gamma, out)
    v.status_sync()
    U = int(out["n_active"].item())
    bits = buf.cpu().numpy().view(np.uint32)
    assert U == int(sum(bin(int(b)).count("1") for b in bits))
    union = out["union_ids"].cpu().numpy()[:U]
    expect = [e for e in range(shape.E) if (int(bits[e >> 5]) >> (e & 31)) & 1]
    np.testing.assert_array_equal(union, np.array(expect, dtype=np.int32))
    assert int(costs.sum().item()) == U          # marginal costs add up to the final footprint
    v.close()
