"""Child process of test_gpu_timeout.py: loads the test-hook build of the library (millisecond wait
budgets, a switch that withholds the schedulers' final message / inflates the selection kernel's
barrier target) and drives every expert-kernel body and the cooperative selection kernel through
its time-out path.  Prints one JSON object."""
import ctypes as C
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np  # noqa: E402
import torch  # noqa: E402

import paper_2607_12696_b200.binding as binding  # noqa: E402
from paper_2607_12696_b200.build import TEST_LIB  # noqa: E402

binding._LIB_PATH = TEST_LIB  # before the first lib() call
import oracle  # noqa: E402
import paper_2607_12696_b200 as moev  # noqa: E402
import synth  # noqa: E402
from gpu_common import compare, device_layer, gcfg, ocfg  # noqa: E402
from helpers import small_shape  # noqa: E402


def withhold(on: bool):
    L = moev.lib()
    L.moev_test_withhold.restype = C.c_int32
    assert L.moev_test_withhold(C.c_int32(int(on))) == 0


def layer_case(name, shape, gamma, routing, **kw):
    """normal call -> parity; withheld call -> MOEV_ETIMEOUT, status word cleared; normal call -> parity."""
    w = synth.make_expert_weights(shape, device="cuda")
    wr, x = routing(shape, gamma, device="cuda", **kw)
    layer, keep = device_layer(wr, w)
    ref = oracle.moe_verify(ocfg(shape), synth.layer_to_numpy(wr, w), synth.to_numpy(x), gamma)
    v = moev.MoeVerifier(gcfg(shape, gamma))
    rec = {"impl": v.resolved_impl()}

    def run_and_compare():
        out = v.alloc_out(gamma)
        v.verify(layer, x, gamma, out)
        v.status_sync()
        res = {k: (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy() for k, t in out.items()}
        return compare(shape, res, ref, gamma)

    rec["err_before"] = run_and_compare()
    withhold(True)
    out = v.alloc_out(gamma)
    t0 = time.perf_counter()
    v.verify(layer, x, gamma, out)
    try:
        v.status_sync()
        rec["timeout_status"] = 0
    except moev.MoevError as e:
        rec["timeout_status"] = e.status
    rec["timeout_wall_s"] = time.perf_counter() - t0
    withhold(False)
    try:
        v.status_sync()          # the status word was cleared by the read that reported the time-out
        rec["status_after"] = 0
    except moev.MoevError as e:
        rec["status_after"] = e.status
    rec["err_after"] = run_and_compare()
    rec["err_after2"] = run_and_compare()
    v.close()
    return name, rec


def select_case():
    """cooperative selection kernel: barrier target one arrival too high -> n_selected = -1; then normal."""
    n_layers, E, K, gamma = 58, 256, 8, 16
    parent, P, pred = synth.make_draft_tree(n_layers, E, K, depth=7, branch=2, seed_tag="timeout-tree")
    tp, tP = torch.from_numpy(parent).cuda(), torch.from_numpy(P).cuda()
    tpred = torch.from_numpy(pred.view(np.int32)).cuda()
    ref = oracle.select_drafts(parent, P, pred, gamma, 1e-6)
    rec = {}
    withhold(True)
    t0 = time.perf_counter()
    out = moev.select_drafts(tp, tP, tpred, gamma, 1e-6)
    torch.cuda.synchronize()
    rec["timeout_wall_s"] = time.perf_counter() - t0
    rec["n_selected_withheld"] = int(out[3].item())
    withhold(False)
    out = moev.select_drafts(tp, tP, tpred, gamma, 1e-6)
    torch.cuda.synchronize()
    rec["n_selected_after"] = int(out[3].item())
    rec["selected_match"] = bool(np.array_equal(out[0].cpu().numpy()[:len(ref[0])], np.asarray(ref[0])))
    return "select_grid", rec


def main():
    torch.cuda.set_device(0)
    res = {}
    cases = [
        ("fp8_single_phase", small_shape("deepseek", H=1024, I=512, E=64), 16, synth.make_scattered_routing, {}),
        ("fp8_two_phase", small_shape("deepseek", H=640, I=384, E=32), 100, synth.make_exact_union_routing, {"U": 8}),
        ("fp8_fold_scale", small_shape("deepseek", H=512, I=4224, E=4, top_k=2), 5, synth.make_scattered_routing, {}),
        ("bf16", small_shape("qwen", H=1024, I=384, E=32), 16, synth.make_iid_routing, {}),
        ("mxfp4", small_shape("gptoss", H=704, I=320, E=32), 19, synth.make_iid_routing, {}),
    ]
    for name, shape, gamma, routing, kw in cases:
        k, rec = layer_case(name, shape, gamma, routing, **kw)
        res[k] = rec
    k, rec = select_case()
    res[k] = rec
    print("RESULT " + json.dumps(res))


if __name__ == "__main__":
    main()
