"""The C-ABI library loads and exports every symbol the header declares; host-side
argument checks work without a GPU (no compute calls here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def aiq():
    from paper_2512_14090_b200 import build
    build.build()
    from paper_2512_14090_b200 import binding
    return binding


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "aiq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aiq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(aiq):
    declared = _declared_symbols()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(aiq.lib, name), name
    assert sorted(aiq.EXPORTS) == declared


def test_binding_constants_equal_the_header(aiq):
    text = open(os.path.join(ROOT, "include", "aiq.h")).read()
    m = re.search(r"#define\s+AIQ_STATIC_WORKSPACE_BYTES\s+\((\d+)u \* (\d+)u \* (\d+)u\)", text)
    assert m and int(m.group(1)) * int(m.group(2)) * int(m.group(3)) == aiq.STATIC_WORKSPACE_BYTES
    for name in ("OK", "ERR_INVALID_ARG", "ERR_UNSUPPORTED_BITS", "ERR_SHAPE", "ERR_WORKSPACE_TOO_SMALL",
                 "ERR_CUDA", "ERR_NOT_SM100", "ERR_NONFINITE", "ERR_TIMEOUT"):
        m = re.search(r"\bAIQ_%s = (\d+)" % name, text)
        assert m and int(m.group(1)) == getattr(aiq, name), name


def test_status_strings(aiq):
    seen = {aiq.status_string(i) for i in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert aiq.status_string(12345) == "unknown status"


def test_packed_row_bytes(aiq):
    assert aiq.aiq_packed_row_bytes(27, 4) == 16
    assert aiq.aiq_packed_row_bytes(9, 8) == 32
    assert aiq.aiq_packed_row_bytes(576, 16) == 1152
    assert aiq.aiq_packed_row_bytes(33, 32) == 256
    assert aiq.aiq_packed_row_bytes(10, 5) == 0
    assert aiq.aiq_packed_row_bytes(0, 8) == 0


def test_host_side_argument_checks(aiq):
    one = C.c_void_p(256)
    assert aiq.lib.aiq_quantize_layer(one, 4, 4, 3, one, one, None, None) == aiq.ERR_UNSUPPORTED_BITS
    assert "bits=3" in aiq.last_error()
    assert aiq.lib.aiq_quantize_layer(None, 4, 4, 8, one, one, None, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_quantize_layer(one, 0, 4, 8, one, one, None, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_qlinear(one, one, None, 4, 4, 7, one, 1, one, None, 0, None) == aiq.ERR_UNSUPPORTED_BITS
    assert aiq.lib.aiq_qlinear(one, one, None, 4, 4, 8, one, 0, one, None, 0, None) == aiq.ERR_INVALID_ARG
    assert aiq.aiq_qlinear_workspace_bytes(4096, 4096, 4, 1) > 0
    assert aiq.aiq_qlinear_workspace_bytes(4096, 4096, 16, 1) == 0      # plain kernel only
    assert aiq.aiq_qlinear_workspace_bytes(4096, 4000, 4, 1) == 0
    assert aiq.aiq_qlinear_workspace_bytes(64, 512, 8, 1) == 0
    assert aiq.lib.aiq_fold_bn(None, one, one, one, one, 1, 1, 1e-5, one, one, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_forward(None, one, one, 1, one, one, 0, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_eval_schemes(None, one, 1, one, one, 1, one, None, None, one, 0, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_scheme_ai(None, one, 1, None, None, None) == aiq.ERR_INVALID_ARG
    assert aiq.lib.aiq_model_num_layers(None) == -1
    assert aiq.lib.aiq_workspace_bytes(None, 1, 1) == 0


def test_model_bytes_and_wiring_checks(aiq):
    from aiq_workloads import resnet20, mobilenet_v2, tiny_net
    for arch in (resnet20(), mobilenet_v2("cifar"), mobilenet_v2("imagenet"), tiny_net()):
        desc, keep = aiq.arch_desc(arch)
        nbytes = aiq.lib.aiq_model_bytes(C.byref(desc))
        n_w = sum(l["cout"] * (1 if l["kind"] == "dw" else l["cin"]) * l["k"] ** 2 for l in arch["layers"])
        # folded fp32 + bank at 4/8/16/32 bits = 4 + 7.5 bytes per weight, plus padding
        assert nbytes >= n_w * 11.5
    bad = resnet20()
    bad["layers"][3]["cin"] = 17
    desc, keep = aiq.arch_desc(bad)
    assert aiq.lib.aiq_model_bytes(C.byref(desc)) == 0
    assert "channels" in aiq.last_error()
    cyc = tiny_net()
    cyc["layers"][1]["input"] = 2       # 1 <- 2 <- 1
    desc, keep = aiq.arch_desc(cyc)
    assert aiq.lib.aiq_model_bytes(C.byref(desc)) == 0
    assert "cycle" in aiq.last_error()
    nofc = tiny_net()
    nofc["layers"] = nofc["layers"][:-1]
    desc, keep = aiq.arch_desc(nofc)
    assert aiq.lib.aiq_model_bytes(C.byref(desc)) == 0
    res = tiny_net()
    res["layers"][6]["residual"] = 0    # 8 channels at 8x8 vs 16 at 4x4
    desc, keep = aiq.arch_desc(res)
    assert aiq.lib.aiq_model_bytes(C.byref(desc)) == 0
    assert "residual" in aiq.last_error()
