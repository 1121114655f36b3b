"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded tensors.

Bars:
  * int32 group accumulators: bit exact given identical int8 operands;
  * int8 Winograd-domain tensors: bit exact except at most 1e-4 of the elements, off
    by one LSB (fp32 transform on the GPU vs fp64-then-round in the oracle);
  * final fp32 output: max |y - y_ref| <= 2e-3 * max |y_ref|.
Stage-wise bars for the fp32 stages fed with the oracle's operands are derived from
fp32 rounding and written next to the checks in gpu_util.py.
"""
import numpy as np
import pytest

from paper_2412_19867_b200 import workloads as wl
from paper_2412_19867_b200.workloads import Layer

pytestmark = pytest.mark.gpu


def _check(layer, tensors=None, **kw):
    from tests.gpu_util import check_layer_all_levels
    rep = check_layer_all_levels(layer, tensors, **kw)
    print(layer.name, {k: (f"{v:.3e}" if isinstance(v, float) else v) for k, v in rep.items()})
    return rep


def test_config1_full():
    _check(wl.config_layers(1)[0])


# Reduced copies of the other configurations: same tile size, group size, dtype and
# distributions, sizes the oracle finishes in seconds, several 128-tile blocks with a
# ragged tail, ragged image edges, C != K, K not a multiple of the channel block.
SMALL = [
    Layer(3, 64, 64, 28, 28, 6, 64, "f16", "relu_heavy", "kaiming", 2, 0, 1),       # T=75
    Layer(6, 128, 96, 14, 14, 6, 64, "f16", "relu_heavy", "kaiming", 2, 1, 1),      # ragged 14/6
    Layer(9, 128, 128, 7, 7, 6, 64, "f16", "relu_heavy", "kaiming", 2, 3, 1),       # 7x7 images
    Layer(3, 128, 128, 28, 28, 4, 32, "f16", "relu_heavy", "kaiming", 3, 0, 1),     # T=147
    Layer(3, 128, 64, 28, 28, 4, 128, "f16", "relu_heavy", "kaiming", 3, 2, 1),
    Layer(4, 256, 64, 14, 14, 6, 32, "f16", "relu_heavy", "kaiming", 3, 9, 1),
    Layer(4, 256, 64, 14, 14, 6, 128, "f16", "relu_heavy", "kaiming", 3, 11, 1),    # two-pass K1
    Layer(1, 320, 320, 32, 32, 4, 64, "f16", "silu_outlier", "kaiming_chan", 4, 0, 1),  # C=2.5 stages
    Layer(1, 320, 160, 48, 40, 6, 64, "f16", "silu_outlier", "kaiming_chan", 5, 6, 1),  # H != W
    Layer(1, 256, 64, 20, 20, 4, 256, "f32", "gauss_outlier", "gauss_chan", 1, 0, 2),   # gs=256, fp32
    Layer(2, 32, 40, 9, 11, 4, 32, "f32", "gauss_outlier", "gauss_chan", 1, 0, 3),      # odd W, K=40
    Layer(1, 96, 32, 13, 13, 6, 96, "f16", "silu_outlier", "kaiming_chan", 4, 0, 4),    # gs=96
    # few tiles, many output channels, groups of 32: output channels on the accumulator rows,
    # four groups per chunk; with whole 128-channel stages and with a 32-channel last stage
    Layer(1, 128, 128, 8, 8, 4, 32, "f16", "silu_outlier", "kaiming_chan", 4, 0, 5),
    Layer(2, 160, 192, 8, 8, 4, 32, "f16", "silu_outlier", "kaiming_chan", 4, 0, 6),
    # groups that straddle the 128-channel stages of the contraction, several groups per unit,
    # a partial last stage; both orientations
    Layer(1, 192, 40, 13, 13, 6, 96, "f16", "silu_outlier", "kaiming_chan", 4, 0, 7),
    Layer(1, 320, 64, 8, 8, 4, 160, "f16", "silu_outlier", "kaiming_chan", 4, 0, 8),    # swapped
    Layer(2, 512, 64, 12, 12, 4, 256, "f16", "silu_outlier", "kaiming_chan", 4, 0, 9),
    # swapped contraction with the 48-column block: one and two column blocks, groups of 64 and 32
    Layer(1, 128, 256, 24, 24, 4, 64, "f16", "silu_outlier", "kaiming_chan", 5, 8, 3),  # T = 36
    Layer(1, 128, 256, 24, 24, 4, 32, "f16", "silu_outlier", "kaiming_chan", 5, 8, 4),
    Layer(1, 64, 128, 36, 40, 4, 64, "f16", "silu_outlier", "kaiming_chan", 5, 8, 5),   # T = 90
    # tensor-core input transform: column chunks with a ragged last chunk (3-D boxes), whole
    # tile rows in several boxes, an odd number of operand tiles per CTA, groups of 32
    Layer(1, 64, 32, 24, 136, 4, 64, "f16", "silu_outlier", "kaiming_chan", 5, 0, 1),   # W = 136: chunks
    Layer(1, 128, 32, 20, 64, 6, 32, "f16", "silu_outlier", "kaiming_chan", 5, 5, 1),   # 11 tiles per row
    Layer(5, 64, 32, 10, 16, 6, 64, "f16", "relu_heavy", "kaiming", 2, 0, 2),           # 3 tiles per row
    # 16-byte staging of the input transform (fp16, W a multiple of 8) with the other group paths:
    # groups of 256 (four lanes per group) and of 96 (group read twice from shared memory)
    Layer(1, 512, 32, 16, 16, 6, 256, "f16", "silu_outlier", "kaiming_chan", 5, 9, 1),
    Layer(2, 192, 32, 12, 24, 4, 96, "f16", "silu_outlier", "kaiming_chan", 5, 9, 2),
    # F(2,3) (the textbook tile, 16 positions): even and odd widths, fp16 and fp32, 16-byte staging,
    # both orientations of the contraction
    Layer(2, 64, 96, 18, 24, 2, 64, "f16", "silu_outlier", "kaiming_chan", 5, 9, 3),
    Layer(1, 128, 40, 9, 11, 2, 32, "f32", "gauss_outlier", "gauss_chan", 5, 9, 4),
    Layer(1, 128, 256, 8, 6, 2, 128, "f16", "relu_heavy", "kaiming", 5, 9, 5),
]


@pytest.mark.parametrize("layer", SMALL, ids=lambda L: L.name)
def test_reduced_configs(layer):
    _check(layer)


@pytest.mark.parametrize("layer", [L for L in SMALL if L.dtype == "f16" and L.gs in (32, 64) and L.C % 64 == 0],
                         ids=lambda L: L.name)
def test_reduced_configs_tensor_core_input_transform(layer):
    """The same layers with the tensor-core input transform selected."""
    _check(layer, k1_kernel=2)


def test_tiny_brute_force_shape():
    """C = K = group = 32, one tile per image."""
    for m in (4, 6):
        _check(Layer(1, 32, 32, m, m, m, 32, "f32", "gauss_outlier", "gauss_chan", 1, 0, 10 + m))


def test_all_zero_input_and_zero_groups():
    L = Layer(1, 64, 32, 8, 8, 4, 32, "f16", "zeros", "kaiming", 9, 0, 0)
    x, w, sB, sG = wl.make_tensors(L)
    rep = _check(L, (x, w, sB, sG))
    # one all-zero channel group, one group with a single outlier
    L2 = Layer(1, 64, 32, 8, 8, 4, 32, "f16", "silu_outlier", "kaiming", 9, 1, 0)
    x, w, sB, sG = wl.make_tensors(L2)
    x[:, :32] = 0
    x[0, 40, 3, 3] = 3000.0
    _check(L2, (x, w, sB, sG))


def test_negative_and_standard_scales():
    L = Layer(2, 64, 64, 12, 12, 6, 32, "f16", "silu_outlier", "kaiming_chan", 9, 2, 0)
    x, w, sB, sG = wl.make_tensors(L)
    _check(L, (x, w, None, None))                       # NULL scales = the standard ones
    sB2 = sB.copy(); sB2[[0, 3]] *= -1
    sG2 = sG.copy(); sG2[[1, 3]] *= -1
    _check(L, (x, w, sB2, sG2))
    learned = wl.LEARNED_F63                              # the paper's learned F(6,3) scales
    _check(L, (x, w, np.array(learned["SB"], np.float32), np.array(learned["SG"], np.float32)))


@pytest.mark.parametrize("m,H,W", [(4, 16, 16), (4, 9, 14), (4, 7, 7), (6, 12, 12), (6, 13, 11), (2, 8, 10), (2, 7, 9)],
                         ids=["f43_w16", "f43_w14", "f43_w7", "f63_w12", "f63_w11", "f23_w10", "f23_w9"])
def test_bias_and_activation_epilogue(m, H, W):
    """y = act(conv + bias) fused into the output transform, every store variant; the
    setting can be changed and cleared between calls on one plan."""
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = Layer(2, 64, 40, H, W, m, 32, "f16", "silu_outlier", "kaiming_chan", 9, 2, 50 + W)
    conv, (x, w, sB, sG) = gu.make_conv(L)
    xd = torch.from_numpy(x).to("cuda:0")
    ref = orc.wfq(x, w, L.m, L.gs, sB, sG).y
    scale = float(np.max(np.abs(ref)))
    rng = np.random.default_rng(7)
    bias = (rng.standard_normal(L.K) * 0.5 * scale).astype(np.float32)
    bd = torch.from_numpy(bias).to("cuda:0")
    for act_id, act in ((b.WFQ_ACT_RELU, "relu"), (b.WFQ_ACT_SILU, "silu"), (b.WFQ_ACT_NONE, "none")):
        for use_bias in (True, False):
            if act == "none" and not use_bias:
                continue
            conv.set_epilogue(bd if use_bias else None, act_id)
            y = conv.forward(xd).cpu().numpy()
            conv.check_status()
            want = orc.epilogue(ref, bias if use_bias else None, act)
            err = float(np.max(np.abs(y - want))) / scale
            assert err <= gu.FINAL_TOL, (act, use_bias, err)
    conv.set_epilogue(None, b.WFQ_ACT_NONE)
    y = conv.forward(xd).cpu().numpy()
    assert float(np.max(np.abs(y - ref))) / scale <= gu.FINAL_TOL
    with pytest.raises(b.WfqError):
        b.wfq_plan_set_epilogue(conv.plan, None, 7)
    conv.close()


@pytest.mark.parametrize("m,H,W", [(4, 16, 16), (4, 9, 14), (4, 7, 7), (6, 12, 12), (6, 13, 11), (2, 8, 10), (2, 7, 9)],
                         ids=["f43_w16", "f43_w14", "f43_w7", "f63_w12", "f63_w11", "f23_w10", "f23_w9"])
def test_fp16_output(m, H, W):
    """y written as fp16 or bf16 by every store variant equals the fp32 result rounded once, with
    and without an epilogue, through the device and the host-buffer entry points, and in the
    fully quantized mode."""
    import torch
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = Layer(2, 64, 40, H, W, m, 32, "f16", "silu_outlier", "kaiming_chan", 9, 4, 60 + W)
    conv, (x, w, sB, sG) = gu.make_conv(L)
    xd = torch.from_numpy(x).to("cuda:0")
    bias = torch.linspace(-1.0, 1.0, L.K, dtype=torch.float32, device="cuda:0")
    for epi in (False, True):
        for fq_mode in ((0, b.WFQ_Y_FP32), (1, b.WFQ_Y_TILE)):
            conv.set_epilogue(bias if epi else None, b.WFQ_ACT_SILU if epi else b.WFQ_ACT_NONE)
            b.wfq_plan_set_full_quant(conv.plan, *fq_mode)
            conv.set_output_dtype("f32")
            y32 = conv.forward(xd)
            for name, dt in (("f16", torch.float16), ("bf16", torch.bfloat16)):
                conv.set_output_dtype(name)
                y16 = conv.forward(xd)
                conv.check_status()
                assert y16.dtype == dt
                assert torch.equal(y16, y32.to(dt)), (epi, fq_mode, name)
                xh = torch.from_numpy(x).pin_memory()
                yh = torch.empty(y16.shape, dtype=dt).pin_memory()
                conv.forward_host(xh, yh)
                assert torch.equal(yh, y16.cpu())
    conv.close()


@pytest.mark.parametrize("layer", [
    Layer(2, 128, 96, 24, 24, 4, 64, "f16", "silu_outlier", "kaiming_chan", 9, 5, 1),
    Layer(1, 192, 200, 12, 12, 6, 32, "f16", "silu_outlier", "kaiming_chan", 9, 5, 2),
], ids=lambda L: L.name)
def test_contraction_shapes_agree(layer):
    """Every orientation / column block the debug option can force gives the library's own
    result: bit for bit within an orientation (same arithmetic per element), to fp32 rounding
    across orientations (the two scales are multiplied in the other order)."""
    import torch
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    _check(layer)
    conv, (x, w, sB, sG) = gu.make_conv(layer)
    xd = torch.from_numpy(x).to("cuda:0")
    ys = {}
    for shape in (0, 116, 164, 216, 232, 248, 264):
        b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_GEMM_SHAPE, shape)
        ys[shape] = conv.forward(xd).cpu().numpy()
        conv.check_status()
    scale = float(np.max(np.abs(ys[0])))
    assert np.array_equal(ys[116], ys[164])
    for shape in (232, 248, 264):
        assert np.array_equal(ys[216], ys[shape]), shape
    assert float(np.max(np.abs(ys[116] - ys[216]))) <= 1e-5 * scale
    assert np.array_equal(ys[0], ys[116]) or np.array_equal(ys[0], ys[216])
    with pytest.raises(b.WfqError):
        b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_GEMM_SHAPE, 132)
    conv.close()


@pytest.mark.parametrize("layer", [
    Layer(1, 64, 32, 13, 11, 6, 64, "f16", "silu_outlier", "kaiming_chan", 9, 8, 1),      # ragged edges
    Layer(3, 192, 32, 20, 24, 4, 32, "f32", "gauss_outlier", "gauss_chan", 9, 8, 2),      # fp32, two groups per item
    Layer(2, 256, 32, 28, 28, 6, 128, "f16", "relu_heavy", "kaiming", 9, 8, 3),           # two lanes per group
    Layer(1, 192, 32, 12, 24, 4, 96, "f16", "silu_outlier", "kaiming_chan", 9, 8, 4),     # generic group size
    Layer(2, 128, 48, 56, 56, 6, 64, "f16", "relu_heavy", "kaiming", 9, 8, 5),            # several items per CTA
    Layer(1, 512, 32, 16, 16, 4, 256, "f16", "silu_outlier", "kaiming_chan", 9, 8, 6),    # four lanes per group
    Layer(2, 64, 32, 10, 14, 2, 64, "f16", "silu_outlier", "kaiming_chan", 9, 8, 7),      # F(2,3)
    Layer(2, 128, 32, 21, 26, 4, 32, "f16", "silu_outlier", "kaiming_chan", 9, 8, 8),     # tensor cores, F(4,3), groups of 32
    Layer(1, 320, 32, 64, 64, 4, 64, "f16", "silu_outlier", "kaiming_chan", 9, 8, 9),     # tensor cores, several items per CTA
    # tensor cores: images narrower than the 8-column box, tile rows shorter than a work item
    # (whole tiles of the item outside the image), an odd number of tile columns, groups of 32 with F(6,3)
    Layer(9, 128, 32, 7, 7, 6, 64, "f16", "relu_heavy", "kaiming", 9, 8, 10),
    Layer(2, 64, 32, 5, 5, 4, 32, "f16", "silu_outlier", "kaiming_chan", 9, 8, 11),
    Layer(3, 128, 40, 30, 18, 6, 32, "f16", "silu_outlier", "kaiming_chan", 9, 8, 12),
    # tensor cores, groups of 128 and 256 (two and four boxes of channels per tile), the other tile size each
    Layer(2, 256, 32, 22, 20, 4, 128, "f16", "silu_outlier", "kaiming_chan", 9, 8, 13),
    Layer(1, 512, 32, 20, 26, 6, 256, "f16", "silu_outlier", "kaiming_chan", 9, 8, 14),
], ids=lambda L: L.name)
def test_nhwc_input_matches_nchw(layer):
    """x given as [N][H][W][C].  With the plain NHWC kernel (TMA-staged strips, debug option 1) the
    codes and scales of stage 1 and the final output equal the NCHW path's bit for bit; with the
    library's choice (the tensor-core NHWC kernel where it applies) the codes agree with the
    oracle's within the usual bars; also through the host-buffer entry point, and back to NCHW."""
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = layer
    conv, (x, w, sB, sG) = gu.make_conv(L)
    xd = torch.from_numpy(x).to("cuda:0")
    xn = xd.permute(0, 2, 3, 1).contiguous()
    y0 = conv.forward(xd)
    xq0 = conv.buffer(b.WFQ_BUF_XQ).clone()
    sx0 = conv.buffer(b.WFQ_BUF_SX)[:, :, :conv.T].clone()
    ref = orc.wfq(x, w, L.m, L.gs, sB=sB, sG=sG)
    conv.set_input_layout("nhwc")
    b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, 1)
    conv.buffer(b.WFQ_BUF_XQ).fill_(99)
    y1 = conv.forward(xn)
    conv.check_status()
    assert torch.equal(conv.buffer(b.WFQ_BUF_XQ), xq0)
    assert torch.equal(conv.buffer(b.WFQ_BUF_SX)[:, :, :conv.T], sx0)
    assert torch.equal(y0, y1)
    b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, 0)
    conv.buffer(b.WFQ_BUF_XQ).fill_(99)
    y2 = conv.forward(xn)
    conv.check_status()
    xq2 = conv.buffer(b.WFQ_BUF_XQ).cpu().numpy()
    gu.codes_close(xq2, ref.Xq)
    assert np.mean(xq2 != xq0.cpu().numpy()) <= 1e-4
    gu.scales_close(conv.buffer(b.WFQ_BUF_SX).cpu().numpy()[:, :, :conv.T], ref.sX.transpose(0, 2, 1))
    assert gu.max_rel(y2.cpu().numpy(), ref.y) <= gu.FINAL_TOL or np.any(xq2 != ref.Xq)
    yh = torch.empty(y0.shape, dtype=torch.float32).pin_memory()
    conv.forward_host(xn.cpu().pin_memory(), yh)
    assert torch.equal(yh, y2.cpu())
    with pytest.raises(b.WfqError):
        b.wfq_plan_set_full_quant(conv.plan, 1, b.WFQ_Y_FP32)
    conv.set_input_layout("nchw")
    assert torch.equal(conv.forward(xd), y0)
    conv.close()


def test_filters_export_and_import():
    """A plan made ready from an exported blob computes what the plan that prepared the filters
    computes (also for another batch and image size, and in the fully quantized mode); a blob
    for other parameters or a damaged one is refused and leaves the plan unprepared."""
    import torch
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = Layer(2, 128, 72, 20, 24, 6, 64, "f16", "silu_outlier", "kaiming_chan", 9, 7, 1)
    conv, (x, w, sB, sG) = gu.make_conv(L)
    blob = b.wfq_filters_export(conv.plan, conv._stream())
    assert len(blob) == b.wfq_filters_bytes(conv.plan)
    xd = torch.from_numpy(x).to("cuda:0")
    for N, H, W in ((L.N, L.H, L.W), (1, 9, 14)):
        a = b.Conv(N, L.C, L.K, H, W, L.m, L.gs, L.dtype)
        a.prepare(torch.from_numpy(w).to("cuda:0"), list(sB), list(sG))
        c = b.Conv(N, L.C, L.K, H, W, L.m, L.gs, L.dtype)
        b.wfq_filters_import(c.plan, blob, c._stream())
        xs = xd[:N, :, :H, :W].contiguous()
        for mode in ((0, b.WFQ_Y_FP32), (1, b.WFQ_Y_ROW)):
            b.wfq_plan_set_full_quant(a.plan, *mode)
            b.wfq_plan_set_full_quant(c.plan, *mode)
            assert torch.equal(a.forward(xs), c.forward(xs))
        c.check_status()
        a.close(); c.close()
    other = b.Conv(1, L.C, L.K + 8, 8, 8, L.m, L.gs, L.dtype)
    with pytest.raises(b.WfqError):
        b.wfq_filters_import(other.plan, blob)
    bad = bytearray(bytes(blob)); bad[0] ^= 0xff
    same = b.Conv(1, L.C, L.K, 8, 8, L.m, L.gs, L.dtype)
    with pytest.raises(b.WfqError):
        b.wfq_filters_import(same.plan, bytes(bad))
    with pytest.raises(b.WfqError):
        b.wfq_filters_import(same.plan, bytes(blob)[:1000])
    with pytest.raises(b.WfqError):                      # still not prepared
        same.forward(torch.zeros((1, L.C, 8, 8), dtype=torch.float16, device="cuda:0"))
    with pytest.raises(b.WfqError):
        b.wfq_filters_export(same.plan)
    other.close(); same.close(); conv.close()


W4_LAYERS = [
    Layer(2, 64, 96, 18, 24, 2, 64, "f16", "silu_outlier", "kaiming_chan", 5, 9, 3),       # F(2,3)
    Layer(3, 128, 128, 28, 28, 4, 32, "f16", "relu_heavy", "kaiming", 3, 0, 1),            # T=147
    Layer(6, 128, 96, 14, 14, 6, 64, "f16", "relu_heavy", "kaiming", 2, 1, 1),             # ragged 14/6
    Layer(1, 320, 64, 8, 8, 4, 160, "f16", "silu_outlier", "kaiming_chan", 4, 0, 8),       # swapped contraction
    Layer(1, 256, 64, 20, 20, 4, 256, "f32", "gauss_outlier", "gauss_chan", 1, 0, 2),      # gs=256, fp32
]


@pytest.mark.parametrize("layer", W4_LAYERS, ids=lambda L: L.name)
def test_four_bit_weights(layer):
    """W4A8 (Section 5's naming: filter codes in [-7, 7], activations at 8 bits): every level of the
    check against the oracle with its filters quantized to 4 bits, and the loss against W8A8 is
    what the oracle shows."""
    rep = _check(layer, w_bits=4)
    x, w, sB, sG = wl.make_tensors(layer)
    from oracle import oracle as orc
    from tests import gpu_util as gu
    direct = orc.direct(x, w)
    want4 = orc.sqnr_db(direct, gu.oracle_wfq(x, w, layer, sB, sG, 4).y)
    want8 = orc.sqnr_db(direct, gu.oracle_wfq(x, w, layer, sB, sG, 8).y)
    assert abs(rep["sqnr_vs_direct_db"] - want4) <= 0.1, (rep, want4)
    assert want4 < want8 - 10.0, (want4, want8)          # 4 bits fewer: about 24 dB in theory


def test_four_bit_weights_blob_and_switching():
    """The exported blob of a 4-bit plan stores two codes per byte (half the code section, the
    documented nibble order), imports into a plan created for 8 bits, and switching the width
    un-prepares the plan."""
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests import gpu_util as gu
    L = Layer(2, 128, 72, 20, 24, 6, 64, "f16", "silu_outlier", "kaiming_chan", 9, 7, 1)
    conv8, (x, w, sB, sG) = gu.make_conv(L)
    conv4, _ = gu.make_conv(L, (x, w, sB, sG), w_bits=4)
    codes = conv4.P * L.K * L.C
    assert b.wfq_filters_bytes(conv8.plan) - b.wfq_filters_bytes(conv4.plan) == codes // 2
    blob = bytes(b.wfq_filters_export(conv4.plan, conv4._stream()))
    assert len(blob) == b.wfq_filters_bytes(conv4.plan)
    ref = orc.prepare_filters(w, L.m, L.gs, orc.matrices(L.m, sB, sG, None), bits=4)
    q = ref.Wq.reshape(-1).astype(np.int16)                               # [P][K][C], codes in [-7, 7]
    packed = ((q[0::2] & 0xF) | ((q[1::2] & 0xF) << 4)).astype(np.uint8)
    got = np.frombuffer(blob, dtype=np.uint8, count=codes // 2, offset=256)
    assert np.mean(got != packed) <= gu.CODE_MISMATCH_RATE
    xd = torch.from_numpy(x).to("cuda:0")
    y4 = conv4.forward(xd).clone()
    y8 = conv8.forward(xd).clone()
    assert not torch.equal(y4, y8)
    # a plan created for 8 bits takes the blob's width
    c = b.Conv(L.N, L.C, L.K, L.H, L.W, L.m, L.gs, L.dtype)
    b.wfq_filters_import(c.plan, blob, c._stream())
    assert torch.equal(c.forward(xd), y4)
    assert b.wfq_filters_bytes(c.plan) == len(blob)
    c.check_status()
    # a truncated 4-bit blob is refused
    d = b.Conv(1, L.C, L.K, 8, 8, L.m, L.gs, L.dtype)
    with pytest.raises(b.WfqError):
        b.wfq_filters_import(d.plan, blob[:len(blob) - 16])
    # switching the width: not prepared until the filters are quantized again; then 8-bit results
    conv4.set_weight_bits(8)
    with pytest.raises(b.WfqError):
        conv4.forward(xd)
    conv4.prepare(torch.from_numpy(w).to("cuda:0"), list(sB), list(sG))
    assert torch.equal(conv4.forward(xd), y8)
    with pytest.raises(b.WfqError):
        conv4.set_weight_bits(5)
    for o in (conv8, conv4, c, d):
        o.close()


def test_asynchronous_host_buffer_entry_point():
    """Two layers through wfq_conv_forward_host_async on two streams, repeatedly, against the
    synchronous entry point (one of them large enough for the chunked path)."""
    import torch
    from tests import gpu_util as gu
    layers = [Layer(4, 64, 192, 64, 64, 4, 32, "f16", "silu_outlier", "kaiming_chan", 9, 6, 1),
              Layer(1, 64, 32, 13, 11, 6, 64, "f16", "silu_outlier", "kaiming_chan", 9, 6, 2)]
    convs, xs, want, got = [], [], [], []
    for L in layers:
        conv, (x, w, sB, sG) = gu.make_conv(L)
        xh = torch.from_numpy(x).pin_memory()
        yh = torch.empty((L.N, L.K, L.H, L.W), dtype=torch.float32).pin_memory()
        conv.forward_host(xh, yh)
        convs.append(conv); xs.append(xh); want.append(yh.clone())
        got.append(torch.full(yh.shape, float("nan"), dtype=torch.float32).pin_memory())
    streams = [torch.cuda.Stream("cuda:0") for _ in layers]
    for rep in range(3):
        for conv, xh, yh, st in zip(convs, xs, got, streams):
            conv.forward_host_async(xh, yh, st)
        for st in streams:
            st.synchronize()
        for a, b_ in zip(want, got):
            assert torch.equal(a, b_)
        for yh in got:
            yh.fill_(float("nan"))
    for conv in convs:
        conv.check_status()
        conv.close()


def test_host_buffer_entry_point_matches_device_one():
    import torch
    from tests.gpu_util import make_conv
    L = wl.config_layers(1)[0]
    conv, (x, w, sB, sG) = make_conv(L)
    xd = torch.from_numpy(x).cuda()
    y_dev = conv.forward(xd)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty(y_dev.shape, dtype=torch.float32).pin_memory()
    conv.forward_host(xh, yh)
    assert torch.equal(yh, y_dev.cpu())
    conv.close()


def test_host_buffer_entry_point_in_chunks_matches_device_one():
    """A batch large enough for the pipelined host path (chunks of whole images on two
    internal streams): same bits as the device entry point, twice in a row."""
    import torch
    from tests.gpu_util import make_conv
    L = Layer(8, 64, 128, 56, 56, 6, 64, "f16", "relu_heavy", "kaiming", 2, 0, 7)
    conv, (x, w, sB, sG) = make_conv(L)
    xd = torch.from_numpy(x).cuda()
    y_dev = conv.forward(xd).cpu()
    xh = torch.from_numpy(x).pin_memory()
    for _ in range(2):
        yh = torch.zeros(y_dev.shape, dtype=torch.float32).pin_memory()
        conv.forward_host(xh, yh)
        assert torch.equal(yh, y_dev)
    conv.check_status()
    # the same batch handed over as NHWC (tensor-core input transform in the chunks' plans) with bf16 output
    conv.set_input_layout("nhwc")
    conv.set_output_dtype("bf16")
    xn = xd.permute(0, 2, 3, 1).contiguous()
    y_dev = conv.forward(xn).cpu()
    xnh = xn.cpu().pin_memory()
    for _ in range(2):
        yh = torch.zeros(y_dev.shape, dtype=torch.bfloat16).pin_memory()
        conv.forward_host(xnh, yh)
        assert torch.equal(yh, y_dev)
    conv.check_status()
    conv.close()


@pytest.mark.parametrize("layer", [
    Layer(2, 128, 32, 24, 24, 6, 64, "f16", "silu_outlier", "kaiming_chan", 5, 6, 2),
    Layer(2, 64, 32, 20, 40, 4, 32, "f16", "silu_outlier", "kaiming_chan", 5, 6, 3),
    Layer(1, 256, 32, 18, 16, 6, 128, "f16", "silu_outlier", "kaiming_chan", 5, 6, 4),
], ids=lambda L: L.name)
def test_input_transform_kernels_agree(layer):
    """The tensor-core input transform, the cp.async one with 16-byte copies (what an aligned
    fp16 x with W a multiple of 8 gets) and the one with 4-byte copies (debug option, or a
    misaligned x, which neither a TMA descriptor nor a 16-byte copy can take) against the
    oracle and against each other on the same layer."""
    import torch
    from oracle import oracle as orc
    from paper_2412_19867_b200 import binding as b
    from tests.gpu_util import make_conv, codes_close, scales_close
    L = layer
    conv, (x, w, sB, sG) = make_conv(L)
    ref = orc.wfq(x, w[:1], L.m, L.gs, sB=sB, sG=sG)
    xbuf = torch.zeros(x.size + 8, dtype=torch.float16, device="cuda")
    got = []
    for force, offset in ((2, 0), (1, 0), (2, 2), (3, 0), (0, 0)):          # offset in elements: 4-byte aligned only
        xd = xbuf[offset:offset + x.size].view(x.shape)
        xd.copy_(torch.from_numpy(x))
        b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, force)
        conv.buffer(b.WFQ_BUF_XQ).fill_(99)
        b.wfq_input_transform_quantize(conv.plan, xd.data_ptr(), conv._stream())
        torch.cuda.synchronize()
        conv.check_status()
        xq = conv.buffer(b.WFQ_BUF_XQ).cpu().numpy()
        codes_close(xq, ref.Xq)
        scales_close(conv.buffer(b.WFQ_BUF_SX).cpu().numpy()[:, :, :conv.T], ref.sX.transpose(0, 2, 1))
        got.append(xq)
    assert np.mean(got[0] != got[1]) <= 1e-4
    for other in got[2:]:
        assert np.array_equal(got[1], other)                # all from the cp.async kernel, either copy width
    conv.close()


def test_bounded_waits_run_out_and_report():
    """A load that never arrives: the waits for it end by themselves after the (shortened)
    limit, the kernel records WFQ_ERR_TIMEOUT with the id of the wait in the status word,
    drains, frees its tensor memory and returns; a fresh plan then computes correctly."""
    import torch
    from paper_2412_19867_b200 import binding as b
    from tests.gpu_util import make_conv, max_rel
    from oracle import oracle as orc
    L = Layer(1, 64, 64, 16, 16, 4, 64, "f16", "silu_outlier", "kaiming_chan", 9, 5, 0)
    # (option, value, stage call, expected wait ids)
    # (the roles up- and downstream of the starved one run out at about the same time: any of the
    # kernel's waits may be the first to record itself)
    cases = [(b.WFQ_DEBUG_SKIP_INPUT_ITEM, 1, "k1", set(range(8, 14))),   # tensor-core input transform
             (b.WFQ_DEBUG_SKIP_INPUT_ITEM, 1, "k1n", set(range(8, 14))),  # the same for NHWC input
             (b.WFQ_DEBUG_SKIP_GEMM_STAGE, 0, "k2", set(range(1, 8)))]    # contraction
    for option, value, stage, want in cases:
        conv, (x, w, sB, sG) = make_conv(L)
        xd = torch.from_numpy(x).cuda()
        y = conv.forward(xd)                                  # a clean call first
        torch.cuda.synchronize()
        conv.check_status()
        b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_WAIT_CYCLES, 2_000_000)   # about 1 ms
        b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, 0 if stage == "k1n" else 2)
        b.wfq_plan_set_debug_option(conv.plan, option, value)
        if stage == "k1":
            b.wfq_input_transform_quantize(conv.plan, xd.data_ptr(), conv._stream())
        elif stage == "k1n":
            conv.set_input_layout("nhwc")
            xn = xd.permute(0, 2, 3, 1).contiguous()
            b.wfq_input_transform_quantize(conv.plan, xn.data_ptr(), conv._stream())
        else:
            b.wfq_gemm_dequantize(conv.plan, conv._stream())
        torch.cuda.synchronize()                              # the kernel ended by itself
        st, where = b.wfq_check_device_status(conv.plan, conv._stream())
        assert st == b.WFQ_ERR_TIMEOUT, (stage, st)
        assert where in want, (stage, where)
        conv.close()
        # the context is intact: a fresh plan gives the right answer
        conv, _ = make_conv(L, (x, w, sB, sG))
        y2 = conv.forward(xd)
        torch.cuda.synchronize()
        conv.check_status()
        assert torch.equal(y, y2)
        ref = orc.wfq(x, w, L.m, L.gs, sB=sB, sG=sG)
        assert max_rel(y2.cpu().numpy(), ref.y) <= 2e-3
        conv.close()


def test_misaligned_or_null_device_pointers_are_rejected():
    import torch
    from paper_2412_19867_b200 import binding as b
    from tests.gpu_util import make_conv
    L = wl.config_layers(1)[0]
    conv, _ = make_conv(L)
    y = torch.empty(L.N * L.K * L.H * L.W + 4, dtype=torch.float32, device="cuda")
    x = torch.zeros(L.N * L.C * L.H * L.W, dtype=torch.float32, device="cuda")
    with pytest.raises(b.WfqError):
        b.wfq_conv_forward(conv.plan, x.data_ptr(), y.data_ptr() + 4, 0)
    with pytest.raises(b.WfqError):
        b.wfq_conv_forward(conv.plan, 0, y.data_ptr(), 0)
    conv.close()
