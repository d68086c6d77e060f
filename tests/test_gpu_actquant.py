"""GPU parity for the FP8-activation variant (1x128 scales in front of both expert GEMMs):
the CUDA path through the C ABI against the CPU fp64 oracle with the same quantisation rule.
The codes of x are decided by the same binary32 operations on both sides; the codes of h depend
on g and u, which the two sides accumulate differently, so a few of them differ by one step:
outputs are compared within the format's tolerance, routing tables bit for bit."""
import dataclasses

import numpy as np
import pytest

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import compare, gcfg, ocfg, run_gpu
from helpers import small_shape

pytestmark = pytest.mark.gpu


def _case(shape, gamma, mode, impl, routing=synth.make_iid_routing, expect_impl=None, layer_id=0, **kw):
    dev = "cuda"
    w = synth.make_expert_weights(shape, layer=layer_id, device=dev)
    wr, x = routing(shape, gamma, layer=layer_id, device=dev, **kw)
    v = moev.MoeVerifier(dataclasses.replace(gcfg(shape, gamma, impl), act_quant=mode))
    res = run_gpu(shape, wr, w, x, gamma, impl, verifier=v)
    v.close()
    if expect_impl is not None:
        assert res["_impl"] == expect_impl
    ref = oracle.moe_verify(dataclasses.replace(ocfg(shape), act_quant=mode), synth.layer_to_numpy(wr, w),
                            synth.to_numpy(x), gamma)
    plain = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
    err = compare(shape, res, ref, gamma)
    # the variant is what was computed: the unquantised layer is further away than the tolerance allows to confuse
    gap = np.abs(ref.y - plain.y).max() / np.abs(plain.y).max()
    assert err < gap, (err, gap)
    return err, ref


@pytest.mark.parametrize("impl", [moev.IMPL_SIMT, moev.IMPL_AUTO])
@pytest.mark.parametrize("mode", [moev.ACTQ_FP8_B128, moev.ACTQ_FP8_B128_POW2])
@pytest.mark.parametrize("gamma", [1, 19])
def test_deepseek_shaped_fp8_activations(impl, mode, gamma):
    shape = small_shape("deepseek", H=1024, I=512, E=64)
    _case(shape, gamma, mode, impl, routing=synth.make_scattered_routing,
          expect_impl=moev.IMPL_TCGEN05 if impl == moev.IMPL_AUTO else moev.IMPL_SIMT)


@pytest.mark.parametrize("gamma,U,n_shared", [(40, 8, 1), (33, 8, 2), (100, 8, 0)])
def test_fp8_activations_many_tokens_per_expert(gamma, U, n_shared):
    """Units of more than eight tokens (the wide column path of the epilogue), several units per
    expert, shared experts; calls this dense would take the two-phase schedule without the variant."""
    shape = small_shape("deepseek", H=640, I=384, E=32, n_shared=n_shared)
    err, ref = _case(shape, gamma, moev.ACTQ_FP8_B128, moev.IMPL_AUTO, routing=synth.make_exact_union_routing,
                     expect_impl=moev.IMPL_TCGEN05, U=U)
    assert ref.n_active == U


@pytest.mark.parametrize("base,kw", [("qwen", dict(H=512, I=256, E=32)), ("gptoss", dict(H=704, I=320, E=32)),
                                     ("tiny", dict())])
def test_fp8_activations_other_weight_formats_run_on_cuda_cores(base, kw):
    shape = small_shape(base, **kw) if kw else synth.SHAPES["tiny"]
    _case(shape, 9, moev.ACTQ_FP8_B128, moev.IMPL_AUTO, expect_impl=moev.IMPL_SIMT)
