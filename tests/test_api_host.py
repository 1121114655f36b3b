"""Host-side behaviour of the C ABI (no GPU needed): the library loads, exports every
symbol the header declares, and rejects bad requests before any device work."""
import ctypes
import os
import re

import pytest

from paper_2412_19867_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2412_19867_b200 import build
    build.build()
    return b.load()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "wfq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(wfq_[a-z0-9_]+)\s*\(", header))
    assert declared == set(b.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.wfq_version() >= 100


def _create(lib, *args):
    plan = ctypes.c_void_p()
    st = lib.wfq_plan_create(ctypes.byref(plan), *args)
    return st, plan


def test_plan_create_validation(lib):
    ok = (1, 64, 64, 32, 32, 4, 3, 32, 8)
    st, plan = _create(lib, *ok)
    assert st == b.WFQ_OK and plan.value
    assert lib.wfq_plan_destroy(plan) == b.WFQ_OK
    assert lib.wfq_plan_create(None, *ok) == b.WFQ_ERR_INVALID_ARG
    bad = {
        (0, 64, 64, 32, 32, 4, 3, 32, 8): b.WFQ_ERR_INVALID_ARG,    # N < 1
        (1, 64, 64, -1, 32, 4, 3, 32, 8): b.WFQ_ERR_INVALID_ARG,    # H < 1
        (1, 64, 64, 32, 32, 4, 5, 32, 8): b.WFQ_ERR_UNSUPPORTED,    # r != 3
        (1, 64, 64, 32, 32, 3, 3, 32, 8): b.WFQ_ERR_UNSUPPORTED,    # m not in {2,4,6}
        (1, 64, 64, 32, 32, 8, 3, 32, 8): b.WFQ_ERR_UNSUPPORTED,
        (1, 64, 64, 32, 32, 4, 3, 32, 4): b.WFQ_ERR_UNSUPPORTED,    # bits != 8
        (1, 64, 64, 32, 32, 4, 3, 48, 8): b.WFQ_ERR_UNSUPPORTED,    # group not multiple of 32
        (1, 96, 64, 32, 32, 4, 3, 64, 8): b.WFQ_ERR_UNSUPPORTED,    # C % group != 0
        (1, 512, 64, 32, 32, 4, 3, 512, 8): b.WFQ_ERR_UNSUPPORTED,  # group > 256
        (4096, 1280, 64, 512, 512, 4, 3, 64, 8): b.WFQ_ERR_UNSUPPORTED,  # index overflow
    }
    for args, want in bad.items():
        st, plan = _create(lib, *args)
        assert st == want, args
        assert not plan.value


def test_workspace_size_and_order_of_calls(lib):
    N, C, K, H, W, m, gs = 2, 64, 96, 13, 9, 6, 32
    st, plan = _create(lib, N, C, K, H, W, m, 3, gs, 8)
    assert st == b.WFQ_OK
    n, P = m + 2, (m + 2) ** 2
    T = N * (-(-H // m)) * (-(-W // m))
    Tp = (T + 31) // 32 * 32            # row pitch of Y
    Ts = (T + 127) // 128 * 128         # row pitch of sX
    up = lambda v: (v + 1023) // 1024 * 1024
    want = up(P * T * C) + up(P * (C // gs) * Ts * 4) + up(P * K * Tp * 4)
    assert lib.wfq_plan_workspace_bytes(plan) == want
    assert lib.wfq_plan_workspace_bytes(None) == 0
    # nothing may run before workspace + filters exist
    fake = ctypes.c_void_p(4096)
    assert lib.wfq_conv_forward(plan, fake, fake, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_input_transform_quantize(plan, fake, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_gemm_dequantize(plan, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_output_transform(plan, fake, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_conv_forward_host(plan, fake, fake, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_debug_gemm_acc32(plan, fake, None) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_check_device_status(plan, None, None) == b.WFQ_ERR_NOT_PREPARED
    ptr, nb = ctypes.c_void_p(), ctypes.c_size_t()
    assert lib.wfq_debug_get(plan, b.WFQ_BUF_XQ, ctypes.byref(ptr), ctypes.byref(nb)) == b.WFQ_ERR_NOT_PREPARED
    assert lib.wfq_debug_get(plan, 99, ctypes.byref(ptr), ctypes.byref(nb)) == b.WFQ_ERR_INVALID_ARG
    # workspace checks happen before any driver call
    assert lib.wfq_plan_set_workspace(plan, None, want) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_workspace(plan, ctypes.c_void_p(1024), want - 1) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_workspace(plan, ctypes.c_void_p(1024 + 16), want) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_input_dtype(plan, 7) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_input_dtype(plan, b.WFQ_BF16) == b.WFQ_ERR_INVALID_ARG     # bf16: output only
    assert lib.wfq_plan_set_output_dtype(plan, 3) == b.WFQ_ERR_INVALID_ARG
    for dt in (b.WFQ_BF16, b.WFQ_F16, b.WFQ_F32):
        assert lib.wfq_plan_set_output_dtype(plan, dt) == b.WFQ_OK
    assert lib.wfq_plan_set_input_dtype(plan, b.WFQ_F16) == b.WFQ_OK
    assert lib.wfq_prepare_filters(plan, None, None, None, None, None) == b.WFQ_ERR_INVALID_ARG
    # a zero or non-finite scale is rejected before any device work
    zero = (ctypes.c_float * 8)(*([1.0] * 7 + [0.0]))
    assert lib.wfq_prepare_filters(plan, fake, ctypes.cast(zero, ctypes.c_void_p), None, None,
                                   None) == b.WFQ_ERR_INVALID_ARG
    inf = (ctypes.c_float * 8)(*([1.0] * 7 + [float("inf")]))
    assert lib.wfq_prepare_filters(plan, fake, None, ctypes.cast(inf, ctypes.c_void_p), None,
                                   None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_destroy(plan) == b.WFQ_OK
    assert lib.wfq_plan_destroy(None) == b.WFQ_OK


def test_null_plan_is_rejected_everywhere(lib):
    fake = ctypes.c_void_p(4096)
    assert lib.wfq_conv_forward(None, fake, fake, None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_input_dtype(None, 0) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_workspace(None, fake, 0) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_prepare_filters(None, fake, None, None, None, None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_check_device_status(None, None, None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_conv_forward_host_async(None, fake, fake, None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_epilogue(None, None, 0) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_output_dtype(None, 0) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_full_quant(None, 0, 0) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_plan_set_weight_bits(None, 8) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_filters_bytes(None) == 0
    assert lib.wfq_filters_export(None, fake, 0, None) == b.WFQ_ERR_INVALID_ARG
    assert lib.wfq_filters_import(None, fake, 0, None) == b.WFQ_ERR_INVALID_ARG


def test_weight_bits_and_blob_size(lib):
    st, plan = _create(lib, 1, 64, 96, 8, 8, 4, 3, 32, 8)
    assert st == b.WFQ_OK
    full = lib.wfq_filters_bytes(plan)
    codes, scales = 36 * 96 * 64, 36 * 2 * 128 * 4
    assert full == 256 + codes + scales
    for bits in (0, 2, 5, 16):
        assert lib.wfq_plan_set_weight_bits(plan, bits) == b.WFQ_ERR_UNSUPPORTED
    assert lib.wfq_plan_set_weight_bits(plan, 4) == b.WFQ_OK
    assert lib.wfq_filters_bytes(plan) == 256 + codes // 2 + scales
    assert lib.wfq_plan_set_weight_bits(plan, 8) == b.WFQ_OK
    assert lib.wfq_filters_bytes(plan) == full
    assert lib.wfq_plan_destroy(plan) == b.WFQ_OK


def test_status_strings(lib):
    seen = {b.status_string(i) for i in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert b.status_string(123) == "unknown status"


def test_binding_raises_instead_of_falling_back():
    with pytest.raises(b.WfqError) as e:
        b.wfq_plan_create(1, 64, 64, 8, 8, 5, 3, 32, 8)
    assert e.value.status == b.WFQ_ERR_UNSUPPORTED
