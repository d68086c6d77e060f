"""Pins for the FP8-activation variant of the oracle (1x128 scales in front of both expert
GEMMs, as deployed DeepSeek-V3 inference does; not in the paper).  Each pin checks the
oracle against something other than its own arithmetic: torch's e4m3 cast (a library
routine), closed forms, and an independent numpy evaluation of the quantised FFN."""
import numpy as np
import pytest
import torch

import oracle
import synth
from helpers import dense_weights, small_shape


def _torch_e4m3_codes(v: np.ndarray) -> np.ndarray:
    return torch.from_numpy(v.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def test_encode_e4m3_matches_torch_cast():
    rng = np.random.default_rng(3)
    vals = np.concatenate([
        rng.normal(0, 1, 4000), rng.normal(0, 100, 4000), rng.uniform(-448, 448, 4000),
        rng.uniform(-0.02, 0.02, 4000),                         # subnormal range (step 2^-9)
        np.array([0.0, -0.0, 448.0, -448.0, 447.9, 2 ** -9, 2 ** -10, 3 * 2 ** -10, 0.9 * 2 ** -10]),
    ]).astype(np.float32)
    got = np.array([oracle.encode_e4m3(float(v)) for v in vals], dtype=np.uint8)
    np.testing.assert_array_equal(got, _torch_e4m3_codes(vals))


def test_encode_e4m3_midpoints_go_to_even_codes_and_large_values_saturate():
    for c in range(0, 0x7E):
        lo, hi = oracle.decode_e4m3(c), oracle.decode_e4m3(c + 1)
        mid = np.float32((lo + hi) / 2)          # exactly representable in binary32
        assert float(mid) == (lo + hi) / 2
        want = c if c % 2 == 0 else c + 1
        assert oracle.encode_e4m3(float(mid)) == want
        assert oracle.encode_e4m3(-float(mid)) == want | 0x80
    for v in (448.0, 460.0, 1e6, 3e38):
        assert oracle.encode_e4m3(v) == 0x7E and oracle.encode_e4m3(-v) == 0xFE
    for c in range(0x7F):                          # every code is a fixed point
        assert oracle.encode_e4m3(oracle.decode_e4m3(c)) == c


@pytest.mark.parametrize("mode", [1, 2])
def test_act_quant_blocks_against_torch_and_closed_forms(mode):
    rng = np.random.default_rng(11)
    x = (rng.normal(0, 1, (5, 448)) * np.array([1e-3, 1, 30, 1e3, 1])[:, None]).astype(np.float32)
    x[4, 128:256] = 0.0                            # an all-zero block
    codes, scales = oracle.act_quant(x, mode)
    assert codes.shape == x.shape and scales.shape == (5, 4)   # 448 = 3.5 blocks: the last one is short
    for r in range(5):
        for b in range(4):
            blk = x[r, 128 * b:128 * (b + 1)]
            amax = np.abs(blk).max()
            if amax == 0:
                s = np.float32(1.0)
            elif mode == 1:
                s = np.float32(amax) / np.float32(448.0)
            else:                                   # smallest power of two >= amax / 448
                v = float(np.float32(amax) / np.float32(448.0))
                s = np.float32(2.0 ** np.ceil(np.log2(v)))
                assert s >= v > s / 2
            assert scales[r, b] == s
            np.testing.assert_array_equal(codes[r, 128 * b:128 * (b + 1)], _torch_e4m3_codes(blk / s))
    # the block maximum maps to the top of the range (mode 1: exactly 448), so nothing saturates
    deq = np.vectorize(oracle.decode_e4m3)(codes) * np.repeat(scales, 128, axis=1)[:, :448]
    if mode == 1:
        assert np.abs(np.vectorize(oracle.decode_e4m3)(codes[0, :128])).max() == 448.0
    # e4m3 keeps 4 significant bits: relative error <= 2^-4 for values above the subnormal range of the block
    big = np.abs(x) >= np.repeat(scales, 128, axis=1)[:, :448] * 2.0 ** -6
    assert (np.abs(deq - x)[big] <= np.abs(x)[big] * 2.0 ** -4 * (1 + 1e-6)).all()


def test_act_quant_is_the_identity_on_representable_rows():
    # a row of e4m3-representable values whose maximum is 448 quantises to itself (mode 1: s = 1)
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 0x7F, 256).astype(np.uint8)
    codes[17] = 0x7E
    codes[128 + 5] = 0x7E
    x = np.vectorize(oracle.decode_e4m3)(codes).astype(np.float32) * np.where(rng.random(256) < 0.5, -1, 1).astype(np.float32)
    q, s = oracle.act_quant(x, 1)
    assert (s == 1.0).all()
    np.testing.assert_array_equal(np.vectorize(oracle.decode_e4m3)(q).astype(np.float32), x)


def _numpy_quantised_ffn(shape, w, layer_np, e, xs, mode):
    """Independent evaluation: dequantise the expert's weights with numpy, quantise with torch's cast."""
    def qdq(v):
        out = np.zeros_like(v, dtype=np.float64)
        for b0 in range(0, v.shape[0], 128):
            blk = v[b0:b0 + 128].astype(np.float32)
            amax = np.abs(blk).max()
            if amax == 0:
                continue
            s = np.float32(amax) / np.float32(448.0)
            if mode == 2:
                s = np.float32(2.0 ** np.ceil(np.log2(float(s))))
            q = torch.from_numpy(blk / s).to(torch.float8_e4m3fn).to(torch.float32).numpy()
            out[b0:b0 + 128] = q.astype(np.float64) * float(s)
        return out
    dw = dense_weights(shape, w)                    # torch's own casts
    Wg, Wu, Wd = (dw[k][e].numpy() for k in ("gate", "up", "down"))
    ys = []
    for x in xs:
        xq = qdq(x)
        g, u = Wg @ xq, Wu @ xq
        h = g / (1 + np.exp(-g)) * u
        ys.append(Wd @ qdq(h.astype(np.float32)))
    return np.stack(ys)


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("base", ["deepseek", "qwen"])
def test_quantised_expert_ffn_against_numpy(base, mode):
    shape = small_shape(base, H=384, I=256, E=4)
    w = synth.make_expert_weights(shape, layer=0, device="cpu")
    layer_np = synth.layer_to_numpy(None, w)
    rng = np.random.default_rng(7)
    xs = rng.normal(0, 1, (3, shape.H)).astype(np.float32).astype(np.float64)
    cfg = oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt, shape.afmt, shape.score,
                        act_quant=mode)
    got = oracle.expert_ffn(cfg, layer_np, 2, xs)
    want = _numpy_quantised_ffn(shape, w, layer_np, 2, xs, mode)
    # h values that differ in the last binary32 bit between the two evaluations may land on
    # different codes; everything else agrees to rounding
    err = np.abs(got - want).max() / np.abs(want).max()
    assert err < 2e-3, err
    plain = oracle.expert_ffn(oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt,
                                            shape.afmt, shape.score), layer_np, 2, xs)
    rel = np.abs(got - plain).max() / np.abs(plain).max()
    assert 1e-4 < rel < 0.2, rel                    # the quantisation is visible, and small


def test_layer_with_quantised_activations_keeps_routing_and_linearity():
    shape = small_shape("deepseek", H=256, I=128, E=8)
    w = synth.make_expert_weights(shape, layer=1, device="cpu")
    wr, x = synth.make_iid_routing(shape, 6, layer=1, device="cpu")
    layer_np = synth.layer_to_numpy(wr, w)
    xn = synth.to_numpy(x)
    base = oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt, shape.afmt, shape.score)
    qcfg = oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt, shape.afmt, shape.score,
                         act_quant=1)
    a, b = oracle.moe_verify(base, layer_np, xn, 6), oracle.moe_verify(qcfg, layer_np, xn, 6)
    np.testing.assert_array_equal(a.topk_ids, b.topk_ids)          # the router sees the unquantised x
    np.testing.assert_array_equal(a.topk_w, b.topk_w)
    # y = sum_j w_j FFN_q(x) + shared: explicit sum over the selected experts with the single-expert routine
    xd = x.to(torch.float64).numpy()
    for t in range(6):
        y = np.zeros(shape.H)
        for j in range(shape.top_k):
            y += b.topk_w[t, j] * oracle.expert_ffn(qcfg, layer_np, int(b.topk_ids[t, j]), xd[t:t + 1])[0]
        for s in range(shape.n_shared):
            y += oracle.expert_ffn(qcfg, layer_np, s, xd[t:t + 1], shared=True)[0]
        np.testing.assert_allclose(b.y[t], y, rtol=1e-12, atol=1e-14)
