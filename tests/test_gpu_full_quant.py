"""GPU parity of the fully quantized transforms (Section 4.1, Eqs. quant-B and quant-y) against
the CPU oracle (`oracle/full_quant.py`), through the C ABI.

Both sides decide every quantizer in fp64 from exact inputs and multiply integer codes exactly, so
the bars are: integer-transform codes and scales of stage 1 bit exact; the integer output
transform fed with the same fp32 Y equal up to the fp32 rounding of the result; end to end, the
GPU's y equals the oracle's output transform continued from the GPU's own Y (fp32 rounding), and
differs from the all-oracle result only through the fp32 accumulation order of Y (a code of Y
that flips moves one tile by a quantization step), which is bounded in relative L2 norm."""
import numpy as np
import pytest

from paper_2412_19867_b200 import workloads as wl
from paper_2412_19867_b200.workloads import Layer

pytestmark = pytest.mark.gpu

LAYERS = [
    Layer(2, 64, 32, 12, 12, 4, 32, "f16", "silu_outlier", "kaiming_chan", 8, 0, 0),
    Layer(1, 64, 48, 13, 11, 6, 64, "f16", "silu_outlier", "kaiming_chan", 8, 1, 0),     # ragged edges
    Layer(1, 128, 32, 8, 8, 4, 128, "f32", "gauss_outlier", "gauss_chan", 8, 2, 0),
    Layer(1, 256, 16, 12, 6, 6, 256, "f16", "silu_outlier", "kaiming", 8, 3, 0),
    Layer(2, 64, 24, 7, 10, 2, 32, "f16", "silu_outlier", "kaiming_chan", 8, 4, 0),       # F(2,3)
]
MODES = [("tile", 1), ("row", 2)]


def _setup(layer, scales="given"):
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    x, w, sB, sG = wl.make_tensors(layer)
    if scales == "standard":
        sB = sG = None
    conv, tensors = gu.make_conv(layer, (x, w, sB, sG))
    return torch, orc, b, gu, conv, tensors


@pytest.mark.parametrize("layer", LAYERS, ids=lambda L: L.name)
def test_integer_input_transform_is_bit_exact(layer):
    from oracle import full_quant as fq
    torch, orc, b, gu, conv, (x, w, sB, sG) = _setup(layer)
    ref = fq.wfq_full(x, w, layer.m, layer.gs, sB, sG, quant_input=True, quant_output=False)
    b.wfq_plan_set_full_quant(conv.plan, 1, b.WFQ_Y_FP32)
    xd = torch.from_numpy(x).to("cuda:0")
    b.wfq_input_transform_quantize(conv.plan, xd.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    Xq = conv.buffer(b.WFQ_BUF_XQ).cpu().numpy()
    sX = conv.buffer(b.WFQ_BUF_SX).cpu().numpy()[:, :, :conv.T]
    assert np.array_equal(Xq, ref.Xq), f"{np.mean(Xq != ref.Xq):.2e} of the codes differ"
    assert np.array_equal(sX, ref.sX.transpose(0, 2, 1)), "group scales differ"
    # and the floating-point transform of the same plan still runs after switching back
    b.wfq_plan_set_full_quant(conv.plan, 0, b.WFQ_Y_FP32)
    b.wfq_input_transform_quantize(conv.plan, xd.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    gu.codes_close(conv.buffer(b.WFQ_BUF_XQ).cpu().numpy(), orc.wfq(x, w, layer.m, layer.gs, sB, sG).Xq)
    conv.close()


@pytest.mark.parametrize("mode,mode_id", MODES)
@pytest.mark.parametrize("layer", LAYERS, ids=lambda L: L.name)
def test_integer_output_transform_on_the_same_y(layer, mode, mode_id):
    from oracle import full_quant as fq
    torch, orc, b, gu, conv, (x, w, sB, sG) = _setup(layer)
    ref = orc.wfq(x, w, layer.m, layer.gs, sB, sG)
    Y32 = ref.Y.astype(np.float32)                                    # [P][T][K], what the GPU buffer holds
    Yp = np.zeros((conv.P, layer.K, conv.Tp), dtype=np.float32)
    Yp[:, :, :conv.T] = Y32.transpose(0, 2, 1)
    conv.write_buffer(b.WFQ_BUF_Y, torch.from_numpy(Yp))
    AT = ref.mats.VA * ref.mats.sA[None, :]
    ytile, parts = fq.output_transform_int(Y32.astype(np.float64), AT, mode)
    want = orc.scatter_tiles(ytile, layer.N, layer.H, layer.W, layer.m)
    b.wfq_plan_set_full_quant(conv.plan, 0, mode_id)
    y = torch.full((layer.N, layer.K, layer.H, layer.W), float("nan"), dtype=torch.float32, device="cuda:0")
    b.wfq_output_transform(conv.plan, y.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    assert np.isfinite(got).all()
    err = np.max(np.abs(got - want)) / np.max(np.abs(want))
    assert err <= 2e-7, err                                           # one fp32 rounding of the result
    conv.close()


@pytest.mark.parametrize("mode,mode_id", MODES)
@pytest.mark.parametrize("layer", LAYERS[:2], ids=lambda L: L.name)
def test_fully_quantized_forward(layer, mode, mode_id):
    from oracle import full_quant as fq
    torch, orc, b, gu, conv, (x, w, sB, sG) = _setup(layer)
    ref = fq.wfq_full(x, w, layer.m, layer.gs, sB, sG, quant_input=True, quant_output=True, y_scale=mode)
    b.wfq_plan_set_full_quant(conv.plan, 1, mode_id)
    xd = torch.from_numpy(x).to("cuda:0")
    got = conv.forward(xd).cpu().numpy()
    conv.check_status()
    assert np.isfinite(got).all()
    # continued from the GPU's own Y: the integer output transform is reproduced exactly
    Y_gpu = conv.buffer(b.WFQ_BUF_Y).cpu().numpy()[:, :, :conv.T].transpose(0, 2, 1).astype(np.float64)
    ytile, _ = fq.output_transform_int(np.ascontiguousarray(Y_gpu), ref.AT, mode)
    cont = orc.scatter_tiles(ytile, layer.N, layer.H, layer.W, layer.m)
    assert np.max(np.abs(got - cont)) <= 2e-7 * np.max(np.abs(cont))
    # against the all-oracle pipeline: Y agrees to fp32 accumulation, a few codes of Y may flip
    assert gu.max_rel(Y_gpu, ref.Y) <= 1e-5
    rel_l2 = np.linalg.norm(got - ref.y) / np.linalg.norm(ref.y)
    assert rel_l2 <= 1e-2, rel_l2
    # host-buffer entry point takes the same path
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty(got.shape, dtype=torch.float32).pin_memory()
    conv.forward_host(xh, yh)
    assert np.array_equal(yh.numpy(), got)
    conv.close()


def test_learned_scales_help_the_integer_output_transform():
    """Section 3.2 / 4.1: with Y quantized per tile, the standard F(6,3) scales lose the signal
    and the paper's learned scales recover most of it; the GPU shows what the oracle shows."""
    from oracle import full_quant as fq
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = Layer(1, 64, 64, 24, 24, 6, 32, "f32", "gauss", "kaiming", 8, 5, 0)
    x, w, _, _ = wl.make_tensors(L)
    direct = orc.direct(x, w)
    learned = wl.LEARNED_F63
    out = {}
    for name, sB, sG in (("standard", None, None),
                         ("learned", np.array(learned["SB"], np.float32), np.array(learned["SG"], np.float32))):
        conv, _ = gu.make_conv(L, (x, w, sB, sG))
        b.wfq_plan_set_full_quant(conv.plan, 1, b.WFQ_Y_TILE)
        got = conv.forward(torch.from_numpy(x).to("cuda:0")).cpu().numpy()
        conv.check_status()
        ref = fq.wfq_full(x, w, L.m, L.gs, sB, sG, quant_input=True, quant_output=True, y_scale="tile")
        out[name] = (orc.sqnr_db(direct, got), orc.sqnr_db(direct, ref.y))
        conv.close()
    print(out)
    for name in out:
        assert abs(out[name][0] - out[name][1]) <= 0.5, out
    assert out["learned"][0] >= out["standard"][0] + 10.0, out


def test_full_quant_arguments_are_checked():
    from paper_2412_19867_b200 import binding as b
    plan = b.wfq_plan_create(1, 64, 64, 8, 8, 4, 3, 32, 8)
    with pytest.raises(b.WfqError):
        b.wfq_plan_set_full_quant(plan, 2, b.WFQ_Y_FP32)
    with pytest.raises(b.WfqError):
        b.wfq_plan_set_full_quant(plan, 0, 3)
    b.wfq_plan_set_full_quant(plan, 1, b.WFQ_Y_ROW)
    b.wfq_plan_destroy(plan)
