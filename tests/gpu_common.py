"""Shared machinery of the GPU parity tests: run the CUDA path through the C ABI and the
CPU oracle on the same seeded inputs and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from helpers import rel_err

Y_TOL = {synth.W_FP32: 1e-2, synth.W_BF16: 1e-2, synth.W_FP8E4M3_B128: 1e-2, synth.W_MXFP4: 3e-2}


def ocfg(s: synth.Shape) -> oracle.Config:
    return oracle.Config(s.H, s.I, s.E, s.top_k, s.n_shared, s.wfmt, s.afmt, s.score, s.routed_scale)


def gcfg(s: synth.Shape, max_tokens: int, impl: int = moev.IMPL_AUTO) -> moev.MoevConfig:
    return moev.MoevConfig(s.H, s.I, s.E, s.top_k, s.n_shared, max_tokens, s.wfmt, s.afmt, s.score,
                           impl, s.routed_scale)


def device_layer(router_w, weights):
    d = {"router_w": router_w}
    d.update({k: v for k, v in weights.items() if v is not None})
    return moev.binding.make_layer(d), d


def run_gpu(shape, router_w, weights, x, gamma, impl=moev.IMPL_AUTO, max_tokens=None, verifier=None):
    v = verifier or moev.MoeVerifier(gcfg(shape, max_tokens or gamma, impl))
    layer, keep = device_layer(router_w, weights)
    out = v.alloc_out(gamma)
    v.verify(layer, x, gamma, out)
    v.status_sync()
    torch.cuda.synchronize()
    res = {k: t.cpu().numpy() if t.dtype != torch.bfloat16 else t.float().cpu().numpy()
           for k, t in out.items()}
    res["_impl"] = v.resolved_impl()
    if verifier is None:
        v.close()
    return res


def compare(shape, res, ref: oracle.Result, gamma, y_ref=None, y_rows=None, tol=None):
    """Bit-exact routing tables; weights to 1e-5; outputs within the format's tolerance."""
    U = ref.n_active
    assert int(res["n_active"][0]) == U
    np.testing.assert_array_equal(res["topk_ids"], ref.topk_ids)
    np.testing.assert_array_equal(res["union_ids"][:U], ref.union_ids)
    np.testing.assert_array_equal(res["offsets"][:U + 1], ref.offsets)
    np.testing.assert_array_equal(res["perm"], ref.perm)
    np.testing.assert_allclose(res["topk_w"], ref.topk_w, rtol=1e-5, atol=1e-7)
    y_ref = ref.y if y_ref is None else y_ref
    y = res["y"] if y_rows is None else res["y"][y_rows]
    assert np.isfinite(y).all()
    err = rel_err(y, y_ref)
    tol = tol or Y_TOL[shape.wfmt]
    assert err <= tol, f"output rel err {err:.3e} > {tol}"
    return err


def parity_case(shape, gamma, routing="iid", impl=moev.IMPL_AUTO, layer_id=0, expect_impl=None, **kw):
    dev = "cuda"
    w = synth.make_expert_weights(shape, layer=layer_id, device=dev)
    fn = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing,
          "clustered": synth.make_clustered_routing, "exact": synth.make_exact_union_routing,
          "zipf": synth.make_zipf_routing}[routing]
    wr, x = fn(shape, gamma, layer=layer_id, device=dev, **kw)
    res = run_gpu(shape, wr, w, x, gamma, impl)
    if expect_impl is not None:
        assert res["_impl"] == expect_impl, f"resolved kernels {res['_impl']}, expected {expect_impl}"
    ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
    if routing == "iid":
        assert ref.gap.min() > 1e-9, "seed gives a near-tie; pick another layer id"
    return compare(shape, res, ref, gamma), ref
