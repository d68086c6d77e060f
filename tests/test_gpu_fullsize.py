"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Routing tables (ids, union, offsets, permutation, n_active) are compared bit-exactly for all
gamma tokens (the oracle's routing is cheap).  Outputs are compared on sampled tokens: the layer
is per-token, so the oracle evaluates just those rows of x (same ids by construction, checked)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import Y_TOL, gcfg, ocfg, run_gpu
from helpers import rel_err

pytestmark = pytest.mark.gpu

ROUTING = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing,
           "clustered": synth.make_clustered_routing, "exact": synth.make_exact_union_routing}


@pytest.fixture(scope="module")
def layers():
    cache = {}

    def get(name):
        if name not in cache:
            cache.clear()  # one full-size layer on the device / host at a time
            shape = synth.SHAPES[name]
            w = synth.make_expert_weights(shape, device="cuda")
            cache[name] = (shape, w, {k: synth.to_numpy(v) for k, v in w.items()})
        return cache[name]

    yield get
    cache.clear()
    torch.cuda.empty_cache()


def _check(layers, name, gamma, routing, sample, **kw):
    shape, w, w_host = layers(name)
    wr, x = ROUTING[routing](shape, gamma, device="cuda", **kw)
    res = run_gpu(shape, wr, w, x, gamma)
    host = dict(w_host, router_w=synth.to_numpy(wr))
    xn = synth.to_numpy(x)
    ref = oracle.moe_verify(ocfg(shape), host, xn, gamma, skip_ffn=True)
    U = ref.n_active
    assert int(res["n_active"][0]) == U
    np.testing.assert_array_equal(res["topk_ids"], ref.topk_ids)
    np.testing.assert_array_equal(res["union_ids"][:U], ref.union_ids)
    np.testing.assert_array_equal(res["offsets"][:U + 1], ref.offsets)
    np.testing.assert_array_equal(res["perm"], ref.perm)
    np.testing.assert_allclose(res["topk_w"], ref.topk_w, rtol=1e-5, atol=1e-7)
    assert np.isfinite(res["y"]).all()
    rows = sorted(set(sample))
    sub = oracle.moe_verify(ocfg(shape), host, np.ascontiguousarray(xn[rows]), len(rows))
    np.testing.assert_array_equal(sub.topk_ids, ref.topk_ids[rows])
    err = rel_err(res["y"][rows], sub.y)
    assert err <= Y_TOL[shape.wfmt], f"{name}: output rel err {err:.3e}"
    return U, err


def test_deepseek_fp8_gamma64_scattered_full(layers):
    U, err = _check(layers, "deepseek", 64, "scattered", [0, 31, 63])
    assert 200 <= U <= 245          # E (1 - (1 - k/E)^gamma) = 222.4


def test_deepseek_fp8_gamma64_clustered_full(layers):
    U, err = _check(layers, "deepseek", 64, "clustered", [0, 5, 40])
    assert 60 <= U <= 180


@pytest.mark.parametrize("gamma,U", [(1, 8), (8, 64), (128, 8), (128, 256)])
def test_deepseek_fp8_exact_union_full(layers, gamma, U):
    """Corners of the unique-expert sweep: one token; every token alone on its experts; 128
    tokens on 8 experts (token runs split into several units); every expert active."""
    got, err = _check(layers, "deepseek", gamma, "exact", [0, gamma - 1], U=U)
    assert got == U


def test_qwen_bf16_gamma64_full(layers):
    U, err = _check(layers, "qwen", 64, "iid", [0, 17, 63])
    assert 110 <= U <= 128          # 125.9 expected


def test_gptoss_mxfp4_gamma64_full(layers):
    U, err = _check(layers, "gptoss", 64, "iid", [0, 33, 63])
    assert 95 <= U <= 125           # 111.2 expected
