"""CPU-side checks of the C-ABI library: it loads, and exports every symbol the header
declares.  No compute call is made (no GPU needed)."""
import os
import re

import paper_2607_12696_b200 as moev

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moev.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moev_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert "moev_verify" in names and "moev_create" in names and len(names) >= 10
    L = moev.lib()
    for n in names:
        assert hasattr(L, n), f"libmoev.so does not export {n}"
    assert set(moev.binding.EXPORTS) == set(names)


def test_byte_model_through_the_abi():
    ds = moev.MoevConfig(7168, 2048, 256, 8, 1, wfmt=moev.W_FP8E4M3_B128, score=moev.SCORE_SIGMOID)
    assert moev.expert_code_bytes(ds) == 44040192       # Fig. 1(c): 44.04 MB
    assert moev.expert_bytes(ds) == 44050944
    oss = moev.MoevConfig(2880, 2880, 128, 4, wfmt=moev.W_MXFP4)
    assert moev.expert_bytes(oss) == 13219200
    qw = moev.MoevConfig(4096, 1536, 128, 8, wfmt=moev.W_BF16)
    assert moev.expert_bytes(qw) == 37748736


def test_create_fails_loudly_without_a_device():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    with pytest.raises(moev.MoevError):
        moev.MoeVerifier(moev.MoevConfig(256, 128, 16, 2))


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_12696_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"


def test_select_drafts_rejects_misaligned_workspace_before_any_cuda_call():
    """Argument validation comes first, so this needs no device: the control words behind the
    footprints are read as 8- and 16-byte quantities, hence the 16-byte rule of the header."""
    import ctypes as C
    L = moev.lib()
    buf = (C.c_uint32 * 4096)()
    base = C.addressof(buf)
    base += (-base) % 16
    ok_args = dict(n=4, W=1, gamma=2)
    for off, expect in ((4, 1), (8, 1)):
        st = L.moev_select_drafts(ok_args["n"], ok_args["W"], base + 1024, base + 2048, base + 3072, None,
                                  ok_args["gamma"], 1e-6, 0, base + 4096 + off, base + 8192, None, None, None, None)
        assert st == expect


def test_static_router_rejects_group_limited_routing_before_any_cuda_call():
    import ctypes as C
    cfg = moev.MoevConfig(256, 128, 16, 2, score=moev.SCORE_SIGMOID, n_group=4, topk_group=2, max_tokens=8).c()
    buf = (C.c_uint8 * 65536)()
    base = C.addressof(buf)
    base += (-base) % 16
    st = moev.lib().moev_route_topk_static(C.byref(cfg), base, base + 16384, 4, base + 32768, base + 49152, None)
    assert st == 1
