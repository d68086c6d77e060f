"""GPU parity of the GPT-OSS expert form (ffn_kind 1: biases, clamps, sigmoid(1.702 g), u + 1)
against the oracle: MXFP4 on the tensor-core kernel and on CUDA cores, bf16 / fp32 on CUDA cores."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import Y_TOL, compare
from helpers import small_shape

pytestmark = pytest.mark.gpu


def _run(shape, gamma, impl, x_gain=1.0, bias_sd=0.5, seed=0):
    dev = "cuda"
    w = synth.make_expert_weights(shape, layer=seed, device=dev)
    wr, x = synth.make_iid_routing(shape, gamma, layer=seed, device=dev)
    if x_gain != 1.0:
        x = (x.float() * x_gain).to(x.dtype)
    g = torch.Generator(device="cpu").manual_seed(1234 + seed)
    biases = {"b_gate": torch.randn(shape.E, shape.I, generator=g) * bias_sd,
              "b_up": torch.randn(shape.E, shape.I, generator=g) * bias_sd,
              "b_down": torch.randn(shape.E, shape.H, generator=g) * bias_sd}
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, 0, gamma, shape.wfmt, shape.afmt, shape.score,
                          impl, shape.routed_scale, moev.binding.FFN_GPTOSS)
    v = moev.MoeVerifier(cfg)
    d = {"router_w": wr}
    d.update({k: t for k, t in w.items() if t is not None})
    d.update({k: t.to(dev).contiguous() for k, t in biases.items()})
    L = moev.binding.make_layer(d)
    out = v.alloc_out(gamma)
    v.verify(L, x, gamma, out)
    v.status_sync()
    torch.cuda.synchronize()
    res = {k: (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in out.items()}
    resolved = v.resolved_impl()
    v.close()
    host = synth.layer_to_numpy(wr, w)
    host.update({k: t.numpy() for k, t in biases.items()})
    ocfg = oracle.Config(shape.H, shape.I, shape.E, shape.top_k, 0, shape.wfmt, shape.afmt, shape.score,
                         shape.routed_scale, oracle.FFN_GPTOSS)
    ref = oracle.moe_verify(ocfg, host, synth.to_numpy(x), gamma)
    assert ref.gap.min() > 1e-9
    return compare(shape, res, ref, gamma), resolved


@pytest.mark.parametrize("impl", [moev.IMPL_SIMT, moev.IMPL_AUTO])
@pytest.mark.parametrize("gamma", [1, 8, 19, 40])
def test_gptoss_form_mxfp4_ragged(impl, gamma):
    shape = small_shape("gptoss", H=704, I=320, E=32)
    err, resolved = _run(shape, gamma, impl)
    if impl == moev.IMPL_AUTO:
        assert resolved == moev.IMPL_TCGEN05     # the MXFP4 tensor-core kernel serves the biased form


@pytest.mark.parametrize("impl", [moev.IMPL_SIMT, moev.IMPL_AUTO])
def test_gptoss_form_clamps_active(impl):
    """Activations scaled up so that a good share of the gate / up pre-activations hit the clamps."""
    shape = small_shape("gptoss", H=704, I=320, E=32)
    _run(shape, 12, impl, x_gain=24.0, bias_sd=2.0, seed=1)


@pytest.mark.parametrize("base,kw", [("tiny", dict(H=256, I=128, E=16)), ("qwen", dict(H=512, I=256, E=32))])
def test_gptoss_form_other_formats_run_on_cuda_cores(base, kw):
    shape = small_shape(base, **kw)
    err, resolved = _run(shape, 9, moev.IMPL_AUTO)
    assert resolved == moev.IMPL_SIMT


def test_gptoss_form_rejects_shared_experts():
    with pytest.raises(moev.MoevError):
        moev.MoeVerifier(moev.MoevConfig(256, 128, 16, 2, 1, 8, synth.W_BF16, synth.ACT_BF16, synth.SCORE_SOFTMAX,
                                         moev.IMPL_AUTO, 1.0, moev.binding.FFN_GPTOSS))
