"""Pins of the CPU oracle against things that are NOT the oracle: library casts, float64
library matmul/topk/softmax, brute force on tiny inputs, closed forms, invariants, and the
figures the paper prints (tests/golden/paper_byte_model.txt).  CPU only."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import dense_weights, rel_err, small_shape, torch_dense_layer, torch_ffn

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_byte_model.txt")


def _gold():
    d = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split()
            d[k] = float(v)
    return d


def _ocfg(s: synth.Shape) -> oracle.Config:
    return oracle.Config(s.H, s.I, s.E, s.top_k, s.n_shared, s.wfmt, s.afmt, s.score, s.routed_scale)


def _mk(shape, gamma, routing="iid", layer=0, **kw):
    w = synth.make_expert_weights(shape, layer=layer)
    fn = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing,
          "clustered": synth.make_clustered_routing}[routing]
    wr, x = fn(shape, gamma, layer=layer, **kw)
    return w, wr, x, synth.layer_to_numpy(wr, w), synth.to_numpy(x)


# ------------------------------------------------------------------ decoders

def test_bf16_decoder_exhaustive_vs_torch():
    codes = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16)
    ref = codes.view(torch.bfloat16).to(torch.float64).numpy()
    for c in range(0, 65536, 7):  # stride keeps it fast; every exponent and sign is hit
        got = oracle.decode_bf16(c)
        assert (np.isnan(got) and np.isnan(ref[c])) or got == ref[c]


def test_e4m3_decoder_exhaustive_vs_torch():
    ref = torch.arange(256, dtype=torch.int32).to(torch.uint8).view(torch.float8_e4m3fn).to(torch.float64)
    for c in range(256):
        got = oracle.decode_e4m3(c)
        assert (np.isnan(got) and np.isnan(ref[c].item())) or got == ref[c].item()
    assert oracle.decode_e4m3(0x7E) == 448.0 and oracle.decode_e4m3(0x01) == 2.0 ** -9


def test_e8m0_decoder_exhaustive_vs_torch():
    ref = torch.arange(256, dtype=torch.int32).to(torch.uint8).view(torch.float8_e8m0fnu).to(torch.float64)
    for c in range(256):
        got = oracle.decode_e8m0(c)
        assert (np.isnan(got) and np.isnan(ref[c].item())) or got == ref[c].item()
    assert oracle.decode_e8m0(127) == 1.0


def test_e2m1_decoder_value_table():
    # OCP microscaling e2m1 value set
    table = [0, .5, 1, 1.5, 2, 3, 4, 6]
    for c in range(16):
        v = oracle.decode_e2m1(c)
        assert abs(v) == table[c & 7]
        assert (np.signbit(v)) == bool(c & 8)


@pytest.mark.parametrize("base,dims", [("deepseek", dict(H=384, I=256, E=3)),
                                       ("gptoss", dict(H=160, I=96, E=3)),
                                       ("qwen", dict(H=128, I=64, E=3)),
                                       ("tiny", dict(H=64, I=32, E=3))])
def test_row_decoder_vs_torch_casts(base, dims):
    shape = small_shape(base, **dims)
    w = synth.make_expert_weights(shape)
    dw = dense_weights(shape, w)
    for name, N, K in (("gate", shape.I, shape.H), ("down", shape.H, shape.I)):
        wn, sn = synth.to_numpy(w["w_" + name]), synth.to_numpy(w["s_" + name])
        for e, n in itertools.product(range(shape.E), (0, N // 2, N - 1)):
            got = oracle.decode_weight_row(shape.wfmt, wn, sn, e, N, K, n)
            np.testing.assert_array_equal(got, dw[name][e, n].numpy())


def test_fp8_block_scale_uses_both_block_indices():
    # a row in the second 128-row block and columns in the third 128-col block must pick s[1,2]
    shape = small_shape("deepseek", H=384, I=256, E=1, n_shared=0)
    codes = np.full((1, 256, 384), 0x38, dtype=np.uint8)  # e4m3 0x38 = 1.0
    s = np.arange(1, 7, dtype=np.float32).reshape(1, 2, 3)
    row = oracle.decode_weight_row(shape.wfmt, codes, s, 0, 256, 384, 130)
    assert row[0] == 4.0 and row[127] == 4.0 and row[128] == 5.0 and row[383] == 6.0


def test_mxfp4_nibble_order_and_scale():
    packed = np.array([[[0x21, 0xF7] + [0] * 14]], dtype=np.uint8)  # K=32
    sc = np.array([[[128]]], dtype=np.uint8)  # 2^1
    row = oracle.decode_weight_row(synth.W_MXFP4, packed, sc, 0, 1, 32, 0)
    # byte 0x21: low nibble 1 (0.5) is element 0, high nibble 2 (1.0) is element 1
    assert list(row[:4]) == [1.0, 2.0, 12.0, -12.0]


# -------------------------------------------------------------------- router

@pytest.mark.parametrize("base", ["tiny", "qwen"])
def test_logits_equal_float64_matmul(base):
    shape = small_shape(base, H=192, E=24)
    wr, x = synth.make_iid_routing(shape, 9)
    got = oracle.router_logits(_ocfg(shape), synth.to_numpy(x), synth.to_numpy(wr), 9)
    ref = (x.to(torch.float64) @ wr.to(torch.float64).T).numpy()
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_logit_carrier_is_exact():
    shape = small_shape("deepseek", H=512, I=128, E=64, n_shared=0)
    wr, x = synth.make_scattered_routing(shape, 11)
    got = oracle.router_logits(_ocfg(shape), synth.to_numpy(x), synth.to_numpy(wr), 11)
    np.testing.assert_array_equal(got, x[:, :64].to(torch.float64).numpy())


def _rank_topk(l, k):
    """O(E^2) rank count: rank(e) = #{e' : l[e'] > l[e] or (l[e'] == l[e] and e' < e)}."""
    E = len(l)
    rank = [sum(1 for f in range(E) if l[f] > l[e] or (l[f] == l[e] and f < e)) for e in range(E)]
    out = [0] * k
    for e in range(E):
        if rank[e] < k:
            out[rank[e]] = e
    return out


@pytest.mark.parametrize("score", [synth.SCORE_SOFTMAX, synth.SCORE_SIGMOID])
def test_topk_vs_rank_count_and_torch(score):
    rs = np.random.RandomState(5)
    cfg = oracle.Config(H=8, I=8, E=24, top_k=5, score=score, routed_scale=1.0)
    logits = rs.randn(13, 24)
    logits[3, :] = np.round(logits[3, :] * 2) / 2  # many exact ties in this row
    ids, w, gap = oracle.topk(cfg, logits)
    for t in range(13):
        assert list(ids[t]) == _rank_topk(list(logits[t]), 5)
    t_ids = torch.topk(torch.from_numpy(logits), 5, dim=1).indices.numpy()
    for t in range(13):
        if t != 3:
            assert list(ids[t]) == list(t_ids[t])
    srt = -np.sort(-logits, axis=1)
    np.testing.assert_allclose(gap, srt[:, 4] - srt[:, 5], atol=0)


def test_topk_tie_goes_to_lower_id():
    cfg = oracle.Config(H=8, I=8, E=4, top_k=2)
    ids, w, gap = oracle.topk(cfg, np.array([[1.0, 1.0, 1.0, 0.0]]))
    assert list(ids[0]) == [0, 1] and gap[0] == 0.0
    np.testing.assert_allclose(w[0], [0.5, 0.5])


def test_router_weights_softmax_and_sigmoid_vs_torch():
    rs = np.random.RandomState(6)
    logits = rs.randn(7, 32) * 2
    tl = torch.from_numpy(logits)
    cfg = oracle.Config(H=8, I=8, E=32, top_k=4, score=synth.SCORE_SOFTMAX)
    ids, w, _ = oracle.topk(cfg, logits)
    full = torch.softmax(tl, dim=1).gather(1, torch.from_numpy(ids).long())
    np.testing.assert_allclose(w, (full / full.sum(1, keepdim=True)).numpy(), rtol=1e-13)
    np.testing.assert_allclose(w.sum(1), 1.0, rtol=1e-14)
    cfg2 = oracle.Config(H=8, I=8, E=32, top_k=4, score=synth.SCORE_SIGMOID, routed_scale=2.5)
    ids2, w2, _ = oracle.topk(cfg2, logits)
    np.testing.assert_array_equal(ids, ids2)  # selection is on the raw logits in both modes
    sg = torch.sigmoid(tl).gather(1, torch.from_numpy(ids2).long())
    np.testing.assert_allclose(w2, (2.5 * sg / sg.sum(1, keepdim=True)).numpy(), rtol=1e-13)
    np.testing.assert_allclose(w2.sum(1), 2.5, rtol=1e-14)


# ---------------------------------------------------------------- union/perm

def test_union_perm_vs_numpy_routines():
    rs = np.random.RandomState(7)
    E, k, gamma = 40, 4, 17
    ids = np.stack([rs.choice(E, k, replace=False) for _ in range(gamma)]).astype(np.int32)
    U, uni, off, perm, inv = oracle.union_perm(E, k, ids)
    flat = ids.reshape(-1)
    ref_uni, ref_cnt = np.unique(flat, return_counts=True)
    assert U == len(ref_uni)
    np.testing.assert_array_equal(uni, ref_uni)
    np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(ref_cnt)]))
    np.testing.assert_array_equal(perm, np.argsort(flat, kind="stable"))
    np.testing.assert_array_equal(inv[perm], np.arange(gamma * k))
    assert off[-1] == gamma * k


def test_union_invariants_and_paper_ar_rows():
    g = _gold()
    # gamma = 1 => the union is exactly the token's top-k (the paper's autoregressive rows)
    for name, key in (("deepseek", "ar_active_experts_deepseek"), ("qwen", "ar_active_experts_qwen"),
                      ("gptoss", "ar_active_experts_gptoss")):
        s = synth.SHAPES[name]
        rs = np.random.RandomState(1)
        cfg = oracle.Config(H=8, I=8, E=s.E, top_k=s.top_k)
        ids, _, _ = oracle.topk(cfg, rs.randn(1, s.E))
        U = oracle.union_perm(s.E, s.top_k, ids)[0]
        assert U == s.top_k == g[key]
    # identical tokens => U = k ; bounds k <= U <= min(E, gamma k)
    cfg = oracle.Config(H=8, I=8, E=64, top_k=8)
    rs = np.random.RandomState(2)
    row = rs.randn(1, 64)
    ids, _, _ = oracle.topk(cfg, np.repeat(row, 9, axis=0))
    assert oracle.union_perm(64, 8, ids)[0] == 8
    for gamma in (1, 2, 5, 32):
        ids, _, _ = oracle.topk(cfg, rs.randn(gamma, 64))
        U = oracle.union_perm(64, 8, ids)[0]
        assert 8 <= U <= min(64, 8 * gamma) and U == len(set(ids.reshape(-1).tolist()))


def test_union_mean_matches_closed_form_for_iid_routing():
    E, k, gamma = 128, 8, 16
    cfg = oracle.Config(H=8, I=8, E=E, top_k=k)
    rs = np.random.RandomState(3)
    us = []
    for _ in range(200):
        ids, _, _ = oracle.topk(cfg, rs.randn(gamma, E))
        us.append(oracle.union_perm(E, k, ids)[0])
    closed = E * (1 - (1 - k / E) ** gamma)  # = 82.4 for this (Qwen-shaped) case
    assert abs(np.mean(us) - closed) < 1.0


@pytest.mark.parametrize("gamma,U", [(1, 8), (8, 8), (8, 64), (32, 100), (32, 256), (128, 16)])
def test_exact_union_generator(gamma, U):
    shape = small_shape("deepseek", H=512, I=128, n_shared=0)
    wr, x = synth.make_exact_union_routing(shape, gamma, U)
    res = oracle.moe_verify(_ocfg(shape), {"router_w": synth.to_numpy(wr)}, synth.to_numpy(x), gamma,
                            skip_ffn=True)
    assert res.n_active == U
    assert res.gap.min() >= 0.25


# ----------------------------------------------------------------------- FFN

@pytest.mark.parametrize("base,dims", [("tiny", dict(H=64, I=48, E=3)),
                                       ("qwen", dict(H=128, I=64, E=3)),
                                       ("deepseek", dict(H=256, I=384, E=2)),
                                       ("gptoss", dict(H=160, I=96, E=3))])
def test_expert_ffn_vs_torch_float64(base, dims):
    shape = small_shape(base, **dims)
    w = synth.make_expert_weights(shape)
    dw = dense_weights(shape, w)
    xs = torch.randn(5, shape.H, dtype=torch.float64, generator=torch.Generator().manual_seed(1))
    layer = synth.layer_to_numpy(torch.zeros(shape.E, shape.H), w)
    for e in range(shape.E):
        got = oracle.expert_ffn(_ocfg(shape), layer, e, xs.numpy())
        np.testing.assert_allclose(got, torch_ffn(dw, e, xs).numpy(), rtol=1e-10, atol=1e-18)
    if shape.n_shared:
        got = oracle.expert_ffn(_ocfg(shape), layer, 0, xs.numpy(), shared=True)
        np.testing.assert_allclose(got, torch_ffn(dw, 0, xs, "sh_").numpy(), rtol=1e-10, atol=1e-18)


def test_ffn_is_not_symmetric_in_gate_and_up():
    # swapping gate and up must change the result (catches a transposed operand)
    shape = small_shape("tiny", H=32, I=16, E=1)
    w = synth.make_expert_weights(shape)
    layer = synth.layer_to_numpy(torch.zeros(1, 32), w)
    sw = dict(layer, w_gate=layer["w_up"], w_up=layer["w_gate"])
    xs = np.random.RandomState(0).randn(2, 32)
    a = oracle.expert_ffn(_ocfg(shape), layer, 0, xs)
    b = oracle.expert_ffn(_ocfg(shape), sw, 0, xs)
    assert np.abs(a - b).max() > 1e-3 * np.abs(a).max()


# --------------------------------------------------------------- whole layer

@pytest.mark.parametrize("base,dims,gamma", [
    ("tiny", {}, 8),
    ("qwen", dict(H=128, I=64, E=16, top_k=4), 6),
    ("deepseek", dict(H=256, I=128, E=32, top_k=4), 6),
    ("gptoss", dict(H=160, I=96, E=16), 5)])
def test_layer_vs_bruteforce_dense_and_torch(base, dims, gamma):
    shape = small_shape(base, **dims)
    w, wr, x, layer, xn = _mk(shape, gamma)
    res = oracle.moe_verify(_ocfg(shape), layer, xn, gamma)
    assert res.gap.min() > 1e-9
    dense = oracle.moe_dense(_ocfg(shape), layer, xn, gamma)
    np.testing.assert_allclose(res.y, dense, rtol=1e-11, atol=1e-16)
    ref = torch_dense_layer(shape, wr, w, x).numpy()
    assert rel_err(res.y, ref) < 1e-11
    assert res.n_active == len(set(res.topk_ids.reshape(-1).tolist()))


def test_single_token_is_explicit_sum_over_its_topk():
    shape = small_shape("deepseek", H=256, I=128, E=32, top_k=4)
    w, wr, x, layer, xn = _mk(shape, 4)
    res = oracle.moe_verify(_ocfg(shape), layer, xn, 4)
    xd = x.to(torch.float64).numpy()
    for t in range(4):
        acc = np.zeros(shape.H)
        for j in range(shape.top_k):
            acc += res.topk_w[t, j] * oracle.expert_ffn(_ocfg(shape), layer, int(res.topk_ids[t, j]),
                                                        xd[t:t + 1])[0]
        acc += oracle.expert_ffn(_ocfg(shape), layer, 0, xd[t:t + 1], shared=True)[0]
        np.testing.assert_allclose(res.y[t], acc, rtol=1e-11, atol=1e-16)
        # and the one-token call gives the same row: the layer is per-token
        one = oracle.moe_verify(_ocfg(shape), layer, np.ascontiguousarray(xn[t:t + 1]), 1)
        np.testing.assert_allclose(one.y[0], res.y[t], rtol=1e-12, atol=1e-18)
        assert one.n_active == shape.top_k


def test_linearity_in_combine_weights():
    shape = small_shape("qwen", H=128, I=64, E=16, top_k=4)
    w, wr, x, layer, xn = _mk(shape, 5)
    cfg = _ocfg(shape)
    rs = np.random.RandomState(4)
    w1, w2 = rs.randn(5, 4), rs.randn(5, 4)
    y1 = oracle.moe_verify(cfg, layer, xn, 5, override_w=w1).y
    y2 = oracle.moe_verify(cfg, layer, xn, 5, override_w=w2).y
    y12 = oracle.moe_verify(cfg, layer, xn, 5, override_w=2.0 * w1 - 3.0 * w2).y
    np.testing.assert_allclose(y12, 2.0 * y1 - 3.0 * y2, rtol=1e-10, atol=1e-15)
    y0 = oracle.moe_verify(cfg, layer, xn, 5, override_w=np.zeros((5, 4))).y
    assert np.all(y0 == 0)


def test_shared_expert_only_when_routed_weights_are_zero():
    shape = small_shape("deepseek", H=256, I=128, E=16, top_k=4)
    w, wr, x, layer, xn = _mk(shape, 3)
    y = oracle.moe_verify(_ocfg(shape), layer, xn, 3, override_w=np.zeros((3, 4))).y
    ref = torch_ffn(dense_weights(shape, w), 0, x.to(torch.float64), "sh_").numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-10, atol=1e-18)


def test_identical_experts_reduce_to_one_dense_ffn_and_zero_up_gives_zero():
    shape = small_shape("tiny", H=64, I=32, E=8, top_k=3)
    w, wr, x, layer, xn = _mk(shape, 6)
    for n in ("w_gate", "w_up", "w_down"):
        w[n][:] = w[n][0]
    layer = synth.layer_to_numpy(wr, w)
    y = oracle.moe_verify(_ocfg(shape), layer, xn, 6).y
    ref = torch_ffn(dense_weights(shape, w), 0, x.to(torch.float64)).numpy()  # weights sum to 1
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-18)
    w["w_up"].zero_()
    y = oracle.moe_verify(_ocfg(shape), synth.layer_to_numpy(wr, w), xn, 6).y
    assert np.all(y == 0)


def test_token_permutation_equivariance():
    shape = small_shape("gptoss", H=160, I=96, E=16)
    w, wr, x, layer, xn = _mk(shape, 7)
    p = np.random.RandomState(8).permutation(7)
    a = oracle.moe_verify(_ocfg(shape), layer, xn, 7)
    b = oracle.moe_verify(_ocfg(shape), layer, np.ascontiguousarray(xn[p]), 7)
    np.testing.assert_allclose(b.y, a.y[p], rtol=1e-12, atol=1e-18)
    np.testing.assert_array_equal(b.topk_ids, a.topk_ids[p])
    assert a.n_active == b.n_active


def test_clustered_routing_shrinks_the_union():
    shape = small_shape("deepseek", H=512, I=128, n_shared=0)
    cfg = _ocfg(shape)
    us, uc = [], []
    for layer in range(4):
        wr, x = synth.make_scattered_routing(shape, 64, layer=layer)
        us.append(oracle.moe_verify(cfg, {"router_w": synth.to_numpy(wr)}, synth.to_numpy(x), 64,
                                    skip_ffn=True).n_active)
        wr, x = synth.make_clustered_routing(shape, 64, layer=layer)
        uc.append(oracle.moe_verify(cfg, {"router_w": synth.to_numpy(wr)}, synth.to_numpy(x), 64,
                                    skip_ffn=True).n_active)
    closed = 256 * (1 - (1 - 8 / 256) ** 64)  # 222.4
    assert abs(np.mean(us) - closed) < 8
    assert np.mean(uc) < 0.75 * np.mean(us)


# ---------------------------------------------------------------- byte model

def test_byte_model_matches_paper_figures():
    g = _gold()
    ds = _ocfg(synth.SHAPES["deepseek"])
    assert oracle.expert_code_bytes(ds) == 3 * 7168 * 2048 == 44040192
    assert round(oracle.expert_code_bytes(ds) / 1e6, 2) == g["deepseek_fp8_expert_MB"]
    assert oracle.expert_scale_bytes(ds) == 3 * 56 * 16 * 4 == 10752
    traffic_gb = g["deepseek_delta_experts"] * g["deepseek_moe_layers"] * oracle.expert_code_bytes(ds) / 1e9
    assert round(traffic_gb, 1) == g["deepseek_delta_traffic_GB"]
    qw = _ocfg(synth.SHAPES["qwen"])
    marg = (g["qwen_hbm_GB_baseline"] - g["qwen_hbm_GB_ecospec"]) * 1e9 / (
        (g["qwen_experts_baseline"] - g["qwen_experts_ecospec"]) * g["qwen_moe_layers"])
    assert abs(marg / oracle.expert_code_bytes(qw) - 1) < 0.03  # Table 2 / Table 3 marginal bytes
    oss = _ocfg(synth.SHAPES["gptoss"])
    assert oracle.expert_code_bytes(oss) + oracle.expert_scale_bytes(oss) == 13219200
    for name in synth.SHAPES:
        s = synth.SHAPES[name]
        assert s.code_bytes_per_expert() == oracle.expert_code_bytes(_ocfg(s))
        assert s.scale_bytes_per_expert() == oracle.expert_scale_bytes(_ocfg(s))


def test_zipf_routing_is_skewed_and_has_a_margin():
    """The skewed generator concentrates assignments on few experts; logits are exact through
    the carrier, so the oracle's ids are the top-k of the constructed logits."""
    shape = small_shape("deepseek", H=256, I=128, E=64)
    wr, x = synth.make_zipf_routing(shape, 128, alpha=1.5)
    res = oracle.moe_verify(_ocfg(shape), {"router_w": synth.to_numpy(wr)}, synth.to_numpy(x), 128, skip_ffn=True)
    counts = np.bincount(res.topk_ids.reshape(-1), minlength=shape.E)
    assert counts.max() >= 64 and (counts == 0).sum() >= 1
    logits = x[:, :shape.E].float().numpy().astype(np.float64)
    np.testing.assert_array_equal(np.sort(res.topk_ids, axis=1),
                                  np.sort(np.argsort(-logits, axis=1, kind="stable")[:, :shape.top_k], axis=1))
