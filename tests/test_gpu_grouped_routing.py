"""GPU parity of the group-limited routing (sigmoid scores + score-correction bias, top groups by the
sum of their two best experts, routed scale) against the oracle: ids, union and permutation
bit-exact, weights to 1e-5, outputs within the format's tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import compare
from helpers import small_shape

pytestmark = pytest.mark.gpu


def _run(shape, gamma, n_group, topk_group, scale, routing, impl=moev.IMPL_AUTO, bias_sd=0.1, seed=0):
    dev = "cuda"
    w = synth.make_expert_weights(shape, layer=seed, device=dev)
    fn = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing,
          "clustered": synth.make_clustered_routing}[routing]
    wr, x = fn(shape, gamma, layer=seed, device=dev)
    g = torch.Generator(device="cpu").manual_seed(77 + seed)
    bias = (torch.randn(shape.E, generator=g) * bias_sd).float()
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt, shape.afmt,
                          synth.SCORE_SIGMOID, impl, scale, 0, n_group, topk_group)
    v = moev.MoeVerifier(cfg)
    d = {"router_w": wr, "router_bias": bias.to(dev)}
    d.update({k: t for k, t in w.items() if t is not None})
    L = moev.binding.make_layer(d)
    out = v.alloc_out(gamma)
    v.verify(L, x, gamma, out)
    v.status_sync()
    torch.cuda.synchronize()
    res = {k: (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in out.items()}
    v.close()
    host = synth.layer_to_numpy(wr, w)
    host["router_bias"] = bias.numpy()
    ocfg = oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt, shape.afmt,
                         synth.SCORE_SIGMOID, scale, 0, n_group, topk_group)
    ref = oracle.moe_verify(ocfg, host, synth.to_numpy(x), gamma)
    gs = shape.E // n_group
    assert all(len(set(ref.topk_ids[t] // gs)) <= topk_group for t in range(gamma))
    return compare(shape, res, ref, gamma), ref


@pytest.mark.parametrize("routing", ["iid", "scattered", "clustered"])
def test_deepseek_rule_reduced_shape(routing):
    """8 groups, 4 kept, top-8, routed scale 2.5: the published DeepSeek-V3 settings on a reduced layer."""
    shape = small_shape("deepseek", H=1024, I=512, E=64)
    err, ref = _run(shape, 32, 8, 4, 2.5, routing)
    np.testing.assert_allclose(ref.topk_w.sum(1), 2.5, rtol=1e-9)


@pytest.mark.parametrize("n_group,topk_group,k", [(1, 1, 8), (4, 1, 8), (16, 5, 6), (64, 8, 8), (2, 2, 8)])
def test_group_shapes(n_group, topk_group, k):
    shape = small_shape("deepseek", H=512, I=256, E=64, top_k=k)
    _run(shape, 19, n_group, topk_group, 1.0, "iid", seed=n_group)


def test_large_biases_and_cuda_core_kernels():
    shape = small_shape("deepseek", H=512, I=256, E=64)
    _run(shape, 12, 8, 4, 2.5, "scattered", impl=moev.IMPL_SIMT, bias_sd=1.0, seed=3)


def test_full_router_shape():
    """The DeepSeek-V3.1 router shape (256 experts, H = 7168, 8 groups of 32, 4 kept) with thin experts."""
    shape = small_shape("deepseek", H=7168, I=128, E=256)
    _run(shape, 64, 8, 4, 2.5, "scattered")


@pytest.mark.parametrize("E,H,n_group,topk_group,k,gamma,routing,bias_sd", [
    (256, 7168, 8, 4, 8, 4, "iid", 0.1),          # the published DeepSeek-V3 settings at the paper's gamma
    (256, 7168, 8, 4, 8, 8, "scattered", 0.1),    # exact logits with exact ties
    (256, 2048, 8, 4, 8, 1, "clustered", 1.0),    # one row; biases as large as the scores
    (256, 1024, 1, 1, 8, 7, "iid", 0.1),          # one group of 256: eight slots per group
    (256, 1024, 2, 1, 6, 5, "iid", 0.3),
    (512, 1024, 8, 3, 8, 6, "iid", 0.1),          # sixteen experts per lane, two slots per group
    (128, 1024, 4, 2, 4, 13, "iid", 0.1),         # one router row per CTA: 16 rows per CTA
    (128, 1024, 4, 4, 8, 16, "scattered", 0.1),
    (256, 2048, 8, 4, 8, 12, "iid", 0.1),         # 9 to 16 rows with two router rows per CTA: two token groups of 8
    (256, 2048, 8, 4, 8, 16, "clustered", 0.1),
])
def test_group_limited_routing_on_fp64_logits(E, H, n_group, topk_group, k, gamma, routing, bias_sd):
    """Small calls whose groups are whole 32-expert slots take the routing path with fp64 logits from the
    start; the group rule is applied to those logits by one warp per token."""
    shape = small_shape("deepseek", H=H, I=256, E=E, top_k=k)
    _run(shape, gamma, n_group, topk_group, 2.5, routing, bias_sd=bias_sd, seed=gamma)


def test_bad_group_configs_are_rejected():
    for ng, kg, score in [(3, 1, synth.SCORE_SIGMOID), (8, 9, synth.SCORE_SIGMOID), (8, 4, synth.SCORE_SOFTMAX),
                          (64, 4, synth.SCORE_SIGMOID)]:
        with pytest.raises(moev.MoevError):
            moev.MoeVerifier(moev.MoevConfig(256, 128, 64, 8, 0, 8, synth.W_BF16, synth.ACT_BF16, score,
                                             moev.IMPL_AUTO, 1.0, 0, ng, kg))
