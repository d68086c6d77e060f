"""Pins for the oracle's GPT-OSS expert form (ffn_kind 1: clamped gate/up, sigmoid(1.702 g),
(u + 1) factor, biases) -- special cases that reduce to library routines or closed forms.  CPU only."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import dense_weights, small_shape


def _cfg(s, kind=1):
    return oracle.Config(s.H, s.I, s.E, s.top_k, s.n_shared, s.wfmt, s.afmt, s.score, s.routed_scale, kind)


def _layer(shape, seed=0, with_bias=True):
    w = synth.make_expert_weights(shape, layer=seed, device="cpu")
    d = {k: synth.to_numpy(v) for k, v in w.items() if v is not None}
    rs = np.random.RandomState(seed + 7)
    if with_bias:
        d["b_gate"] = rs.normal(0, 0.5, (shape.E, shape.I)).astype(np.float32)
        d["b_up"] = rs.normal(0, 0.5, (shape.E, shape.I)).astype(np.float32)
        d["b_down"] = rs.normal(0, 0.5, (shape.E, shape.H)).astype(np.float32)
    return w, d


def test_zero_up_projection_reduces_to_gated_unit_of_library_sigmoid():
    """W_up = 0, b_up = 0: u + 1 = 1, so h = g sigmoid(1.702 g); with alpha folded into a
    rescaled silu, h = silu(1.702 g) / 1.702 (torch's silu), out = W_d h + b_d."""
    shape = small_shape("tiny", H=64, I=32, E=4)
    w, d = _layer(shape)
    d["w_up"] = np.zeros_like(d["w_up"])
    d["b_up"] = np.zeros_like(d["b_up"])
    xs = np.random.RandomState(1).normal(0, 1, (5, shape.H))
    dw = dense_weights(shape, w)
    Wg, Wd = dw["gate"], dw["down"]
    for e in range(shape.E):
        out = oracle.expert_ffn(_cfg(shape), d, e, xs)
        g = torch.from_numpy(xs) @ Wg[e].double().T + torch.from_numpy(d["b_gate"][e]).double()
        assert float(g.max()) < 7.0            # no clamping in this case
        h = torch.nn.functional.silu(1.702 * g) / 1.702
        ref = h @ Wd[e].double().T + torch.from_numpy(d["b_down"][e]).double()
        np.testing.assert_allclose(out, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_clamps_saturate():
    """Huge inputs: g clamps to 7 (or stays very negative, where g sigmoid(1.702 g) -> 0) and u to +-7,
    so h takes one of three values per element: 7 s 8, 7 s (-6) or ~0, with s = sigmoid(11.914)."""
    shape = small_shape("tiny", H=64, I=32, E=2)
    w, d = _layer(shape, with_bias=False)
    d["w_down"] = np.zeros_like(d["w_down"])
    d["w_down"][:, :, :] = 0.0
    # identity-like down projection to read h: H >= I, W_d[e, i, i] = 1
    for i in range(shape.I):
        d["w_down"][:, i, i] = 1.0
    xs = np.random.RandomState(2).normal(0, 1, (3, shape.H)) * 1e5
    out = oracle.expert_ffn(_cfg(shape), d, 0, xs)[:, :shape.I]
    s = 1.0 / (1.0 + np.exp(-1.702 * 7.0))
    allowed = np.array([7 * s * 8, 7 * s * -6, 0.0])
    dist = np.abs(out[..., None] - allowed).min(-1)
    assert dist.max() < 1e-9
    assert (np.abs(out - 7 * s * 8) < 1e-9).any() and (np.abs(out - 7 * s * -6) < 1e-9).any()


def test_zero_weights_leave_the_bias_closed_form():
    """All weight matrices zero: out = b_d + 0 (W_d = 0) for every token, and with W_g = W_u = 0 only,
    out = W_d ((b_u + 1) b_g sigmoid(1.702 b_g)) + b_d, independent of x."""
    shape = small_shape("tiny", H=64, I=32, E=3)
    w, d = _layer(shape)
    Wd = dense_weights(shape, w)["down"]
    d0 = dict(d, w_gate=np.zeros_like(d["w_gate"]), w_up=np.zeros_like(d["w_up"]))
    xs = np.random.RandomState(3).normal(0, 1, (4, shape.H))
    for e in range(shape.E):
        bg, bu, bd = (d[k][e].astype(np.float64) for k in ("b_gate", "b_up", "b_down"))
        g, u = np.minimum(bg, 7.0), np.clip(bu, -7.0, 7.0)
        h = g / (1.0 + np.exp(-1.702 * g)) * (u + 1.0)
        ref = Wd[e].double().numpy() @ h + bd
        out = oracle.expert_ffn(_cfg(shape), d0, e, xs)
        np.testing.assert_allclose(out, np.broadcast_to(ref, out.shape), rtol=1e-12, atol=1e-12)
        d00 = dict(d0, w_down=np.zeros_like(d["w_down"]))
        np.testing.assert_allclose(oracle.expert_ffn(_cfg(shape), d00, e, xs), np.broadcast_to(bd, out.shape))


def test_layer_combines_biased_experts_with_router_weights():
    """Whole layer, all weights zero: y_t = sum_j w[t, j] * b_down[ids[t, j]] (the down bias is inside
    the expert, hence weighted); and ffn_kind 0 ignores the bias pointers."""
    shape = small_shape("tiny", H=64, I=32, E=8, top_k=2)
    w, d = _layer(shape)
    wr, x = synth.make_iid_routing(shape, 6)
    d["router_w"] = synth.to_numpy(wr)
    z = dict(d, w_gate=np.zeros_like(d["w_gate"]), w_up=np.zeros_like(d["w_up"]), w_down=np.zeros_like(d["w_down"]))
    res = oracle.moe_verify(_cfg(shape), z, synth.to_numpy(x), 6)
    ref = np.einsum("tj,tjh->th", res.topk_w, d["b_down"][res.topk_ids].astype(np.float64))
    np.testing.assert_allclose(res.y, ref, rtol=1e-12, atol=1e-14)
    a = oracle.moe_verify(_cfg(shape, 0), d, synth.to_numpy(x), 6).y
    nb = {k: v for k, v in d.items() if not k.startswith("b_")}
    b = oracle.moe_verify(_cfg(shape, 0), nb, synth.to_numpy(x), 6).y
    np.testing.assert_array_equal(a, b)
    # and the biased form differs from the bias-free one
    assert np.abs(oracle.moe_verify(_cfg(shape), d, synth.to_numpy(x), 6).y - a).max() > 1e-3
