"""GPU parity: the CUDA path (through the C ABI) against the CPU fp64 oracle, element by
element on the same seeded inputs.  Integer results bit-exact; router weights 1e-5;
outputs max_t(max_i|y-ref| / max_i|ref|) <= 1e-2 (fp32/bf16/fp8) or 3e-2 (mxfp4)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_12696_b200 as moev
import synth
from gpu_common import compare, device_layer, gcfg, ocfg, parity_case, run_gpu
from helpers import small_shape

pytestmark = pytest.mark.gpu

IMPLS = [moev.IMPL_SIMT, moev.IMPL_AUTO]


@pytest.mark.parametrize("impl", IMPLS)
def test_tiny_config(impl):
    parity_case(synth.SHAPES["tiny"], 8, impl=impl)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("gamma", [1, 16, 33])
def test_qwen_shaped_reduced(impl, gamma):
    shape = small_shape("qwen", H=1024, I=384, E=32)
    parity_case(shape, gamma, impl=impl)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("routing", ["scattered", "clustered"])
def test_deepseek_shaped_reduced(impl, routing):
    shape = small_shape("deepseek", H=1024, I=512, E=64)
    err, ref = parity_case(shape, 32, routing=routing, impl=impl)
    assert 8 <= ref.n_active <= 64


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("gamma", [1, 8, 19])
def test_gptoss_shaped_reduced_ragged(impl, gamma):
    # 704 = 5.5 * 128 and 320 = 2.5 * 128: several tiles and a ragged tail (half a chunk) in both dims;
    # the tensor-core kernel needs multiples of 64
    shape = small_shape("gptoss", H=704, I=320, E=32)
    parity_case(shape, gamma, impl=impl, expect_impl=moev.IMPL_TCGEN05 if impl == moev.IMPL_AUTO else moev.IMPL_SIMT)


@pytest.mark.parametrize("gamma", [3, 19])
def test_gptoss_shaped_not_multiple_of_64_runs_on_cuda_cores(gamma):
    # 736 = 5.75 * 128 and 352 = 2.75 * 128: served by the CUDA-core kernels
    shape = small_shape("gptoss", H=736, I=352, E=32)
    parity_case(shape, gamma, expect_impl=moev.IMPL_SIMT)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("gamma,U,n_shared", [(40, 4, 0), (33, 8, 0), (21, 12, 1), (64, 4, 2)])
def test_gptoss_shaped_many_tokens_per_expert(impl, gamma, U, n_shared):
    """MXFP4 with more tokens per expert than one work unit holds (runs of 16), with and
    without shared experts, on ragged dimensions."""
    shape = small_shape("gptoss", H=704, I=320, E=32, n_shared=n_shared)
    err, ref = parity_case(shape, gamma, routing="exact", impl=impl, U=U,
                           expect_impl=moev.IMPL_TCGEN05 if impl == moev.IMPL_AUTO else moev.IMPL_SIMT)
    assert ref.n_active == U


@pytest.mark.parametrize("H,I,gamma", [(320, 704, 9), (512, 512, 17), (256, 256, 5), (640, 1088, 12), (2880, 2880, 6)])
def test_gptoss_shapes_two_phase_kernel(H, I, gamma):
    """Shapes of the MXFP4 tensor-core kernel's two task kinds: I > H (more gate/up slices than
    W_down tile pairs, ragged last chunk in both phases), scale rows whose length is a multiple of
    four bytes, the smallest shape it serves (a single K chunk and a single task of each kind per
    unit), an odd number of 128-row tiles of H, and the full GPT-OSS dimensions with few experts."""
    shape = small_shape("gptoss", H=H, I=I, E=8 if H == 2880 else 16)
    err, ref = parity_case(shape, gamma, expect_impl=moev.IMPL_TCGEN05)


def test_gptoss_repeated_calls_reuse_scratch():
    """Two different calls on one context: the h scratch rows and progress counters of the
    MXFP4 kernel carry nothing over from the previous call."""
    shape = small_shape("gptoss", H=704, I=320, E=32)
    dev = "cuda"
    w = synth.make_expert_weights(shape, layer=0, device=dev)
    v = moev.MoeVerifier(gcfg(shape, 48))
    for layer_id, gamma, routing in [(1, 48, synth.make_iid_routing), (2, 7, synth.make_scattered_routing),
                                     (3, 31, synth.make_iid_routing)]:
        wr, x = routing(shape, gamma, layer=layer_id, device=dev)
        res = run_gpu(shape, wr, w, x, gamma, moev.IMPL_AUTO, verifier=v)
        ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
        compare(shape, res, ref, gamma)
    v.close()


@pytest.mark.parametrize("base,kw,gamma,routing", [
    ("qwen", dict(H=1024, I=384, E=176, top_k=6), 7, "iid"),        # more experts than SMs: two router rows per CTA; E no multiple of 32
    ("qwen", dict(H=1024, I=384, E=176, top_k=6), 8, "scattered"),  # exact logits with exact ties
    ("deepseek", dict(H=512, I=256, E=512), 8, "iid"),              # sixteen experts per lane in the selection
    ("deepseek", dict(H=512, I=256, E=512), 3, "clustered"),
    ("deepseek", dict(H=8192, I=256, E=32), 5, "iid"),              # rows of 8192 columns: one full pass of the logit kernel
    ("gptoss", dict(H=704, I=320, E=32), 2, "iid"),
    ("tiny", dict(), 8, "iid"), ("tiny", dict(E=24, top_k=24), 4, "iid"),   # fp32 activations; top-k = E
    ("gptoss", dict(H=704, I=320, E=32), 13, "iid"),                # 9 to 16 rows, one router row per CTA: 16 rows of x per CTA
    ("qwen", dict(H=1024, I=384, E=96), 16, "scattered"),
])
def test_smallest_calls_fp64_logit_routing(base, kw, gamma, routing):
    """Calls of at most eight rows (sixteen where a CTA holds one router row and the rows fit its
    shared memory) take the routing path that evaluates all logits in fp64 (no candidate stage): ids, weights, union, offsets and permutation bit for bit against the oracle,
    outputs within the format's tolerance, twice on one context (the second call meets the first
    call's workspace)."""
    shape = small_shape(base, **kw)
    w = synth.make_expert_weights(shape, device="cuda")
    fn = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing, "clustered": synth.make_clustered_routing}[routing]
    v = moev.MoeVerifier(gcfg(shape, 16))
    for layer in (0, 1):
        wr, x = fn(shape, gamma, layer=layer, device="cuda")
        res = run_gpu(shape, wr, w, x, gamma, verifier=v)
        ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
        if routing == "iid" and ref.gap.min() <= 1e-9:
            continue  # a near-tie in the fp64 logits leaves the ids undefined
        compare(shape, res, ref, gamma)
    v.close()


@pytest.mark.parametrize("gamma,routing", [(10, "iid"), (14, "scattered"), (29, "clustered")])
def test_cluster_routing_path_with_two_router_rows_per_cta_shape(gamma, routing):
    """9 to 32 rows on a shape the fp64-logit path does not take beyond 8 rows (more experts than SMs):
    split-K partials + refinement by a thread-block cluster per token, with clusters of eight (10 rows),
    of four because eight would not fit two thirds of the machine (14 rows), and of two (29 rows)."""
    shape = small_shape("deepseek", H=2048, I=256, E=256)
    parity_case(shape, gamma, routing=routing)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("gamma,U", [(1, 8), (8, 8), (8, 64), (32, 40), (128, 8), (128, 64)])
def test_exact_union_cases(impl, gamma, U):
    """Degenerate groupings: all tokens on the same k experts (m_e = gamma), every expert
    used, one token only."""
    shape = small_shape("deepseek", H=512, I=256, E=64)
    err, ref = parity_case(shape, gamma, routing="exact", impl=impl, U=U)
    assert ref.n_active == U


@pytest.mark.parametrize("base,kw,gamma", [("deepseek", dict(H=512, I=256, E=64), 512),
                                           ("gptoss", dict(H=704, I=320, E=32), 200),
                                           ("qwen", dict(H=512, I=256, E=32), 260)])
def test_batched_verification_skewed_routing(base, kw, gamma):
    """Many rows per call (several requests' trees at once) with Zipf-skewed routing: hot
    experts receive hundreds of tokens (many work units each), cold ones none."""
    shape = small_shape(base, **kw)
    err, ref = parity_case(shape, gamma, routing="zipf", alpha=1.5)
    counts = np.bincount(ref.topk_ids.reshape(-1), minlength=shape.E)
    assert counts.max() >= gamma // 2 and ref.n_active <= shape.E


@pytest.mark.parametrize("gamma,U,n_shared", [(100, 8, 1), (77, 16, 0), (128, 8, 2), (33, 8, 1)])
def test_many_tokens_per_expert_two_phase_schedule(gamma, U, n_shared):
    """FP8 calls with many tokens per streamed expert take the two-phase schedule (gate/up tasks
    write h tiles to scratch, down tasks own a pair of H tiles): odd number of H tiles (the last
    down task has one tile), three I slices, token runs that do not fill a unit, shared experts."""
    shape = small_shape("deepseek", H=640, I=384, E=32, n_shared=n_shared)
    err, ref = parity_case(shape, gamma, routing="exact", U=U)
    assert ref.n_active == U


@pytest.mark.parametrize("gamma,n_shared", [(5, 0), (40, 1)])
def test_fp8_wide_intermediate_runs_fold_scale_schedule(gamma, n_shared):
    """Block-scaled FP8 with I > 4096 (33 slices of 128): the tensor-core kernel has no per-token
    quantised activations for such shapes and runs the schedule whose producer warps fold the
    weight block scale into the activations of every K chunk; units of up to 32 tokens."""
    shape = small_shape("deepseek", H=512, I=4224, E=4, top_k=2, n_shared=n_shared)
    parity_case(shape, gamma, routing="scattered", expect_impl=moev.IMPL_TCGEN05)


@pytest.mark.parametrize("impl", IMPLS)
def test_topk_equals_E_and_two_shared(impl):
    shape = small_shape("deepseek", H=256, I=128, E=8, top_k=8, n_shared=2)
    err, ref = parity_case(shape, 5, routing="scattered", impl=impl)
    assert ref.n_active == 8


@pytest.mark.parametrize("impl", IMPLS)
def test_exact_logit_ties_break_to_lower_id(impl):
    shape = small_shape("qwen", H=256, I=128, E=32, top_k=4)
    w = synth.make_expert_weights(shape, device="cuda")
    wr, x = synth.make_scattered_routing(shape, 6, device="cuda")
    x = x.clone()
    x[:, :32] = 0.0          # all 32 logits tie at 0 -> ids must be 0,1,2,3
    x[3, 7] = 1.0            # one clear winner, then ties
    res = run_gpu(shape, wr, w, x, 6, impl)
    ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), 6)
    assert list(ref.topk_ids[0]) == [0, 1, 2, 3] and list(ref.topk_ids[3]) == [7, 0, 1, 2]
    compare(shape, res, ref, 6)


@pytest.mark.parametrize("base,kw,gamma", [("deepseek", dict(H=1024, I=512, E=64), 24), ("gptoss", dict(H=704, I=320, E=32), 24),
                                           ("qwen", dict(H=1024, I=384, E=32), 24),
                                           ("deepseek", dict(H=1024, I=512, E=64), 6), ("gptoss", dict(H=704, I=320, E=32), 5)])
def test_pipelined_layers_match_oracle(base, kw, gamma):
    """moev_verify_pipeline: three independent layers in one call (the router of layer l + 1
    overlaps the tail of layer l) give each layer's oracle result; run twice back to back.  Both the
    routing of larger calls and that of the smallest ones (logits in fp64 from the start), whose
    first kernel also writes workspace the previous layer still reads and must wait for it."""
    shape = small_shape(base, **kw)
    n = 3
    v = moev.MoeVerifier(gcfg(shape, gamma))
    layers, keep, xs, refs = [], [], [], []
    for l in range(n):
        w = synth.make_expert_weights(shape, layer=l, device="cuda")
        wr, x = synth.make_scattered_routing(shape, gamma, layer=l, device="cuda") if shape.E <= shape.H and base != "qwen" \
            else synth.make_iid_routing(shape, gamma, layer=l, device="cuda")
        L, d = device_layer(wr, w)
        layers.append(L); keep.append(d); xs.append(x)
        refs.append(oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma))
    for rep in range(2):
        outs = [v.alloc_out(gamma) for _ in range(n)]
        v.verify_pipeline(layers, xs, gamma, outs)
        v.status_sync()
        torch.cuda.synchronize()
        for l in range(n):
            res = {k: (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in outs[l].items()}
            compare(shape, res, refs[l], gamma)
    v.close()


@pytest.mark.parametrize("base,kw,gamma,prefetch", [("deepseek", dict(H=1024, I=512, E=64), 24, False),
                                                    ("deepseek", dict(H=1024, I=512, E=64), 8, True),
                                                    ("gptoss", dict(H=704, I=320, E=32), 24, False),
                                                    ("qwen", dict(H=1024, I=384, E=32), 40, True)])
def test_chained_dependent_layers_match_oracle(base, kw, gamma, prefetch):
    """moev_verify_chain: four dependent layers in one call, layer l + 1 verifying the output of
    layer l.  Every layer is checked against the oracle evaluated on the input that layer actually
    saw (x0, then the previous layer's bf16 output as the device produced it): the routing tables
    bit for bit, the output within the format's tolerance.  A layer that read its input before the
    previous one had finished would fail both.  The inputs are rescaled between the layers by the
    test's own router (logits come from the hidden state itself), so ties and near-ties occur as
    they fall.  Run twice; with the weight prefetch on, a (partly wrong) expert prediction must not
    change any result."""
    shape = small_shape(base, **kw)
    n = 4
    v = moev.MoeVerifier(gcfg(shape, gamma))
    v.prefetch_enable(prefetch)
    layers, keep, hosts = [], [], []
    for l in range(n):
        w = synth.make_expert_weights(shape, layer=l, device="cuda")
        wr, x = synth.make_iid_routing(shape, gamma, layer=l, device="cuda")
        wr = wr * 50.0  # the layer outputs are small: keep the logits of later layers well separated
        d = {"router_w": wr}
        d.update({k: t for k, t in w.items() if t is not None})
        if prefetch:
            d["predicted_ids"] = torch.arange(l, l + 6, dtype=torch.int32, device="cuda") % shape.E
        layers.append(moev.binding.make_layer(d)); keep.append(d)
        hosts.append(synth.layer_to_numpy(wr, w))
        if l == 0:
            x0 = x
    for rep in range(2):
        outs = [v.alloc_out(gamma) for _ in range(n)]
        v.verify_chain(layers, x0, gamma, outs)
        v.status_sync()
        torch.cuda.synchronize()
        x_in, compared = x0, 0
        for l in range(n):
            ref = oracle.moe_verify(ocfg(shape), hosts[l], synth.to_numpy(x_in), gamma)
            res = {k: (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in outs[l].items()}
            if ref.gap.min() > 1e-9:   # (a near-tie in the fp64 logits leaves the ids undefined)
                compare(shape, res, ref, gamma)
                compared += 1
            x_in = outs[l]["y"]
        assert compared >= n - 1
    v.close()


def test_expert_kernel_span_stamps():
    """moev_ffn_span_*: with the stamps on, the expert kernel's working time of the last call is positive and
    shorter than the call; the results do not change; off again, the stamps stay as they were."""
    shape = small_shape("deepseek", H=1024, I=512, E=64)
    gamma = 8
    v = moev.MoeVerifier(gcfg(shape, gamma))
    assert v.ffn_span_read() == 0.0
    w = synth.make_expert_weights(shape, device="cuda")
    wr, x = synth.make_iid_routing(shape, gamma, device="cuda")
    ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
    v.ffn_span_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    res = run_gpu(shape, wr, w, x, gamma, verifier=v)   # warm-up
    e0.record()
    res = run_gpu(shape, wr, w, x, gamma, verifier=v)
    e1.record()
    torch.cuda.synchronize()
    span = v.ffn_span_read()
    assert 0.0 < span < e0.elapsed_time(e1) * 1e3
    compare(shape, res, ref, gamma)
    v.ffn_span_enable(False)
    run_gpu(shape, wr, w, x, gamma, verifier=v)
    assert v.ffn_span_read() == span
    v.close()


def test_context_reuse_and_smaller_gamma():
    """One context, several calls with different gamma: workspace state must not leak."""
    shape = small_shape("qwen", H=512, I=256, E=16, top_k=4)
    v = moev.MoeVerifier(gcfg(shape, 64))
    w = synth.make_expert_weights(shape, device="cuda")
    for gamma in (64, 3, 17, 64):
        wr, x = synth.make_iid_routing(shape, gamma, device="cuda", layer=gamma)
        res = run_gpu(shape, wr, w, x, gamma, verifier=v)
        ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
        compare(shape, res, ref, gamma)
    v.close()


def test_verify_host_matches_verify():
    shape = small_shape("deepseek", H=512, I=256, E=32)
    v = moev.MoeVerifier(gcfg(shape, 16))
    w = synth.make_expert_weights(shape, device="cuda")
    wr, x = synth.make_scattered_routing(shape, 16, device="cuda")
    layer, keep = device_layer(wr, w)
    out = v.alloc_out(16)
    v.verify(layer, x, 16, out)
    torch.cuda.synchronize()
    xh = x.cpu().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    nh = torch.zeros(1, dtype=torch.int32).pin_memory()
    v.verify_host(layer, xh, 16, yh, nh)
    assert int(nh[0]) == int(out["n_active"][0])
    ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), 16)
    from helpers import rel_err
    assert rel_err(yh.float().numpy(), ref.y) <= 1e-2
    v.close()


def test_invalid_arguments_are_rejected_before_launch():
    shape = small_shape("qwen", H=256, I=128, E=16, top_k=4)
    with pytest.raises(moev.MoevError) as e:
        moev.MoeVerifier(moev.MoevConfig(H=250, I=128, E=16, top_k=4))
    assert e.value.status == 1
    with pytest.raises(moev.MoevError):
        moev.MoeVerifier(moev.MoevConfig(H=256, I=128, E=16, top_k=17))
    v = moev.MoeVerifier(gcfg(shape, 8))
    w = synth.make_expert_weights(shape, device="cuda")
    wr, x = synth.make_iid_routing(shape, 8, device="cuda")
    layer, keep = device_layer(wr, w)
    out = v.alloc_out(8)
    for gamma in (0, 9):
        with pytest.raises(moev.MoevError) as e:
            v.verify(layer, x, gamma, out)
        assert e.value.status == 1
    with pytest.raises(moev.MoevError):  # misaligned x
        v.verify(layer, x.view(-1)[1:257], 1, out)
    if v.resolved_impl() == moev.IMPL_TCGEN05:  # expert weights at a 16-byte offset: the TMA descriptors need 32
        off = dict(keep)
        flat = torch.empty(keep["w_up"].numel() + 8, dtype=keep["w_up"].dtype, device="cuda")
        off["w_up"] = flat[8:].view_as(keep["w_up"])
        assert off["w_up"].data_ptr() % 32 == 16
        with pytest.raises(moev.MoevError) as e:
            v.verify(moev.binding.make_layer(off), x, 8, out)
        assert e.value.status == 1
    bad = dict(keep)
    bad.pop("w_up")
    with pytest.raises(moev.MoevError):
        v.verify(moev.binding.make_layer(bad), x, 8, out)
    with pytest.raises(moev.MoevError):
        v.verify(layer, x, 8, {"y": out["y"]})  # n_active missing
    v.verify(layer, x, 8, out)  # still usable afterwards
    v.status_sync()
    v.close()
