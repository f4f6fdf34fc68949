"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2410_21271_b200 as eora
from paper_2410_21271_b200 import build as eora_build


@pytest.fixture(scope="module")
def lib():
    eora_build.build()
    return eora.lib()


def declared_functions():
    inc = os.path.dirname(eora.HEADER_PATH)
    names = set()
    for h in sorted(os.listdir(inc)):                       # every header of include/
        if not h.endswith(".h"):
            continue
        text = open(os.path.join(inc, h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(eora_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"eora_linear_create", "eora_linear_forward", "eora_linear_destroy", "eora_solve", "eora_solve_loss",
            "eora_solve_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert lib.eora_version() >= 100


def test_struct_layout_matches_header():
    assert ctypes.sizeof(eora.eora_linear_config) == 12 * 4
    assert ctypes.sizeof(eora.eora_linear_weights) == 10 * ctypes.sizeof(ctypes.c_void_p)
    # field order as declared in the header
    hdr = open(os.path.join(os.path.dirname(__file__), "..", "include", "eora_linear.h")).read()
    body = hdr[hdr.index("typedef struct {", hdr.index("} eora_linear_config;")):hdr.index("} eora_linear_weights;")]
    names = re.findall(r"const void\* (\w+);", body)
    assert names == [f[0] for f in eora.eora_linear_weights._fields_]


def test_solve_config_layout_and_argument_checks(lib):
    assert ctypes.sizeof(eora.eora_solve_config) == 6 * 4
    hdr = open(os.path.join(os.path.dirname(eora.HEADER_PATH), "eora_solve.h")).read()
    body = hdr[hdr.index("typedef struct {"):hdr.index("} eora_solve_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for decl in re.findall(r"int32_t ([^;]+);", body) for f in decl.split(",")]
    assert fields == [f[0] for f in eora.eora_solve_config._fields_]
    good = eora.eora_solve_config(256, 128, 64, 16, 0, 0)
    assert eora.eora_solve_workspace_bytes(good) > 4 * (256 * 128 + 128 * 128 + 256 * 256)
    for bad in (eora.eora_solve_config(0, 128, 64, 16, 0, 0), eora.eora_solve_config(256, 128, 64, 0, 0, 0),
                eora.eora_solve_config(256, 128, 64, 500, 100, 0), eora.eora_solve_config(8, 128, 64, 16, 0, 0)):
        assert eora.eora_solve_workspace_bytes(bad) == 0
    assert lib.eora_solve_workspace_bytes(None) == 0
    assert lib.eora_solve(None, None, None, None, None, None, None, None, 0, None) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_solve_loss(None, None, None, None, None, None, None, None, 0, None) == eora.EORA_ERR_NULL_ARG


def test_status_strings(lib):
    seen = set()
    for s in range(0, -8, -1):
        txt = eora.eora_status_string(s)
        assert txt and txt != "unknown status"
        seen.add(txt)
    assert len(seen) == 8
    assert eora.eora_status_string(-99) == "unknown status"


def good_cfg(**kw):
    c = eora.eora_linear_config()
    c.d_in, c.d_out, c.rank = 256, 64, 64
    c.w_format, c.w_bits, c.w_group = eora.EORA_W_QUANT, 4, 128
    c.ab_format, c.ab_group = eora.EORA_AB_F16, 128
    c.x_dtype, c.y_dtype, c.max_m, c.kernel_policy = 0, 0, 8, 0
    for k, v in kw.items():
        setattr(c, k, v)
    return c


def test_create_rejects_bad_arguments_without_a_device(lib):
    w = eora.eora_linear_weights()
    assert eora.eora_linear_create_status(None, w) == eora.EORA_ERR_NULL_ARG
    assert eora.eora_linear_create_status(good_cfg(), None) == eora.EORA_ERR_NULL_ARG
    bad = [dict(d_in=100), dict(d_out=40), dict(rank=12), dict(rank=-8), dict(max_m=0), dict(w_group=96),
           dict(w_group=192), dict(d_in=0)]
    for kw in bad:
        assert eora.eora_linear_create_status(good_cfg(**kw), w) == eora.EORA_ERR_BAD_SHAPE, kw
    unsupported = [dict(w_bits=2), dict(w_bits=8), dict(w_format=7), dict(ab_format=5), dict(x_dtype=3),
                   dict(y_dtype=9), dict(kernel_policy=4)]
    for kw in unsupported:
        assert eora.eora_linear_create_status(good_cfg(**kw), w) == eora.EORA_ERR_UNSUPPORTED, kw
    assert eora.eora_linear_create_status(good_cfg(ab_format=eora.EORA_AB_Q4, rank=32), w) == eora.EORA_ERR_BAD_SHAPE
    # valid config, but the weight pointers are NULL / misaligned
    assert eora.eora_linear_create_status(good_cfg(), w) == eora.EORA_ERR_NULL_ARG
    w.w_codes = w.w_scales = w.w_zeros = 4096
    assert eora.eora_linear_create_status(good_cfg(), w) == eora.EORA_ERR_NULL_ARG      # A, B missing
    w.a = w.b = 4096
    w.w_codes = 4100
    assert eora.eora_linear_create_status(good_cfg(), w) == eora.EORA_ERR_MISALIGNED
    # 2:4 + 4-bit backbone: 4 bits only, a group like the quantised backbone, and the position words
    w.w_codes = 4096
    sq = dict(w_format=eora.EORA_W_SPARSE24_Q4)
    assert eora.eora_linear_create_status(good_cfg(w_bits=3, **sq), w) == eora.EORA_ERR_UNSUPPORTED
    assert eora.eora_linear_create_status(good_cfg(w_group=96, **sq), w) == eora.EORA_ERR_BAD_SHAPE
    assert eora.eora_linear_create_status(good_cfg(**sq), w) == eora.EORA_ERR_NULL_ARG  # w_meta missing
    w.w_meta = 4104
    assert eora.eora_linear_create_status(good_cfg(**sq), w) == eora.EORA_ERR_MISALIGNED


def test_calls_on_null_handle(lib):
    assert lib.eora_linear_destroy(None) == eora.EORA_OK
    assert lib.eora_linear_forward(None, None, 1, None, None) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_forward_host(None, None, 1, None, None) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_path(None, 1) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_launches(None, 1) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_dump(None, 0, None, None) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_last_device_status(None) == eora.EORA_ERR_NULL_ARG
    assert lib.eora_linear_weight_bytes(None) == 0 and lib.eora_linear_scratch_bytes(None) == 0
