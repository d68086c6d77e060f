"""The allocation-free router entry point (moev_route_topk_static) against the regular path.

Some callers cannot call cudaMalloc (all device memory already belongs to their own pool, or
they run in a thread that must not block on the allocator), so they cannot create a context.
This entry point keeps its scratch in a fixed array inside the library.  The check: called
through the C ABI twice in a row, it must give the ids moev_verify gives (exactly) and the same
router weights (1e-5, the tolerance of the other parity tests), the second call included, since
every call reuses the same array; the oracle's routing is the second reference.  Collected
last so a failure here cannot hide other tests."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import device_layer, gcfg, ocfg
from helpers import small_shape

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("base,dims,gamma,routing", [
    ("deepseek", dict(H=1024, I=512, E=64), 32, synth.make_scattered_routing),
    ("qwen", dict(H=1024, I=384, E=32), 17, synth.make_iid_routing),
    ("tiny", dict(), 8, synth.make_iid_routing)])   # fp32 activations
def test_static_scratch_router_matches_verify_twice(base, dims, gamma, routing):
    shape = small_shape(base, **dims)
    cfg = gcfg(shape, gamma)
    w = synth.make_expert_weights(shape, device="cuda")
    inputs = [routing(shape, gamma, device="cuda", layer=l) for l in (0, 1)]
    v = moev.MoeVerifier(cfg)
    expect = []
    for wr, x in inputs:
        layer, keep = device_layer(wr, w)
        out = v.alloc_out(gamma)
        v.verify(layer, x, gamma, out)
        v.status_sync()
        expect.append((out["topk_ids"].cpu().numpy(), out["topk_w"].cpu().numpy()))
        ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma, skip_ffn=True)
        np.testing.assert_array_equal(expect[-1][0], ref.topk_ids)
        np.testing.assert_allclose(expect[-1][1], ref.topk_w, rtol=1e-5, atol=1e-7)
    v.close()
    assert moev.static_scratch_floats(shape.H, shape.E, gamma) <= 5 * 1024 * 1024
    # two calls in a row on different inputs, then the first input again: stale scratch from
    # the previous call must not leak into the next
    for wr, x, (ids_ref, w_ref) in [inputs[0] + (expect[0],), inputs[1] + (expect[1],),
                                    inputs[0] + (expect[0],)]:
        ids = torch.full((gamma, shape.top_k), -1, dtype=torch.int32, device="cuda")
        wts = torch.zeros(gamma, shape.top_k, dtype=torch.float32, device="cuda")
        moev.route_topk_static(cfg, wr, x, gamma, ids, wts)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(ids.cpu().numpy(), ids_ref)
        np.testing.assert_allclose(wts.cpu().numpy(), w_ref, rtol=1e-5, atol=1e-7)


def test_static_scratch_router_rejects_oversized_problems():
    big = moev.MoevConfig(H=8192, I=2048, E=512, top_k=8, max_tokens=1024)
    assert moev.static_scratch_floats(8192, 512, 1024) > 5 * 1024 * 1024
    x = torch.zeros(1024, 8192, dtype=torch.bfloat16, device="cuda")
    wr = torch.zeros(512, 8192, dtype=torch.float32, device="cuda")
    ids = torch.zeros(1024, 8, dtype=torch.int32, device="cuda")
    wts = torch.zeros(1024, 8, dtype=torch.float32, device="cuda")
    with pytest.raises(moev.MoevError) as e:
        moev.route_topk_static(big, wr, x, 1024, ids, wts)
    assert e.value.status == 1


def test_static_scratch_router_rejects_group_limited_routing():
    """Group-limited routing needs the layer's score-correction bias, which the entry point does
    not take; it must say so instead of routing without the bias."""
    cfg = moev.MoevConfig(H=512, I=256, E=32, top_k=4, max_tokens=8, score=moev.SCORE_SIGMOID,
                          n_group=4, topk_group=2)
    x = torch.zeros(8, 512, dtype=torch.bfloat16, device="cuda")
    wr = torch.zeros(32, 512, dtype=torch.float32, device="cuda")
    ids = torch.zeros(8, 4, dtype=torch.int32, device="cuda")
    wts = torch.zeros(8, 4, dtype=torch.float32, device="cuda")
    with pytest.raises(moev.MoevError) as e:
        moev.route_topk_static(cfg, wr, x, 8, ids, wts)
    assert e.value.status == 1
