"""The allocation-free filter quantization entry point against wfq_prepare_filters.

Hosts that cannot call cudaMalloc when filters arrive (a framework whose pool owns the
device, a latency-critical loop, a fixed memory budget) use
wfq_quantize_filters_static, which keeps its intermediate in an array built into the
library.  Both entry points must give the same codes and scales; the built-in array is
shared by all calls, so two calls in a row (the second on a smaller layer, which leaves
the first call's values behind in the array) are both checked.  This file is collected
last on purpose: a failure here must not hide the results of the other tests.
"""
import numpy as np
import pytest

from paper_2412_19867_b200 import binding as b
from paper_2412_19867_b200 import workloads as wl
from paper_2412_19867_b200.workloads import Layer

pytestmark = pytest.mark.gpu


def _both_ways(layer):
    import torch
    from tests.gpu_util import make_conv, codes_close, scales_close
    conv, (x, w, sB, sG) = make_conv(layer)                    # wfq_prepare_filters
    want_q = conv.buffer(b.WFQ_BUF_WQ).cpu().numpy()
    want_s = conv.buffer(b.WFQ_BUF_SW).cpu().numpy()[:, :, :layer.K]     # rows are padded to 128
    wd = torch.from_numpy(w).cuda()
    # outputs pre-filled so that unwritten elements would show
    got_q = torch.full(want_q.shape, 99, dtype=torch.int8, device="cuda")
    got_s = torch.full(want_s.shape, float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    b.wfq_quantize_filters_static(wd.data_ptr(), layer.K, layer.C, layer.m, layer.gs, list(sG),
                                  got_q.data_ptr(), got_s.data_ptr(), stream)
    torch.cuda.synchronize()
    codes_close(got_q.cpu().numpy(), want_q)
    scales_close(got_s.cpu().numpy(), want_s, rtol=1e-6)
    assert np.array_equal(got_q.cpu().numpy(), want_q)         # same kernels: identical
    # and directly against the CPU oracle's offline filter path
    from oracle import oracle as orc
    ref = orc.prepare_filters(w, layer.m, layer.gs, orc.matrices(layer.m, sB, sG))
    codes_close(got_q.cpu().numpy(), ref.Wq)
    scales_close(got_s.cpu().numpy(), ref.sW.transpose(0, 2, 1), rtol=1e-6)
    conv.close()


def test_static_scratch_matches_prepare_filters_twice_in_a_row():
    _both_ways(Layer(1, 256, 192, 8, 8, 6, 64, "f16", "silu_outlier", "kaiming_chan", 8, 0, 0))
    _both_ways(Layer(1, 64, 40, 8, 8, 4, 32, "f32", "gauss_outlier", "gauss_chan", 8, 1, 0))


def test_static_scratch_rejects_oversized_and_bad_requests():
    import torch
    dummy = torch.zeros(16, dtype=torch.float32, device="cuda")
    ptr = dummy.data_ptr()
    K = C = 1280                                               # 36*1280*1280 floats > 4 Mi
    assert 36 * K * C > b.WFQ_STATIC_SCRATCH_FLOATS
    with pytest.raises(b.WfqError) as e:
        b.wfq_quantize_filters_static(ptr, K, C, 4, 64, None, ptr, ptr, 0)
    assert e.value.status == b.WFQ_ERR_SCRATCH_TOO_SMALL
    with pytest.raises(b.WfqError) as e:
        b.wfq_quantize_filters_static(0, 32, 32, 4, 32, None, ptr, ptr, 0)
    assert e.value.status == b.WFQ_ERR_INVALID_ARG
    with pytest.raises(b.WfqError) as e:
        b.wfq_quantize_filters_static(ptr, 32, 48, 4, 32, None, ptr, ptr, 0)
    assert e.value.status == b.WFQ_ERR_UNSUPPORTED
