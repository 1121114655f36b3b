"""Helpers for the GPU parity tests: run a layer through the C ABI and compare every
level with the CPU oracle on the same seeded tensors."""
import numpy as np

from oracle import oracle as orc
from paper_2412_19867_b200 import binding as b
from paper_2412_19867_b200 import workloads as wl

# Parity bars (see the test module's docstring)
CODE_MISMATCH_RATE = 1e-4      # fraction of int8 codes allowed to differ, by 1 LSB only
SCALE_RTOL = 1e-5              # fp32 group scales: fp32 transform vs fp64-then-round
FINAL_TOL = 2e-3               # max |y - y_ref| / max |y_ref|


def make_conv(layer, tensors=None, device="cuda:0", w_bits=8):
    import torch
    x, w, sB, sG = wl.make_tensors(layer) if tensors is None else tensors
    conv = b.Conv(layer.N, layer.C, layer.K, layer.H, layer.W, layer.m, layer.gs, layer.dtype, device)
    if w_bits != 8:
        conv.set_weight_bits(w_bits)
    conv.prepare(torch.from_numpy(w).to(device), None if sB is None else list(sB),
                 None if sG is None else list(sG))
    return conv, (x, w, sB, sG)


def padded(a, pitch):
    """Zero-pad the last axis of a float array to `pitch` (the row pitch of sX / sW)."""
    out = np.zeros(a.shape[:-1] + (pitch,), dtype=np.float32)
    out[..., :a.shape[-1]] = a
    return out


def codes_close(got, want):
    """int8 tensors: identical except at most CODE_MISMATCH_RATE of elements off by one."""
    got = np.asarray(got).astype(np.int16)
    want = np.asarray(want).astype(np.int16)
    assert got.shape == want.shape
    diff = np.abs(got - want)
    rate = float(np.mean(diff != 0))
    assert diff.max() <= 1, f"code differs by {diff.max()} LSB"
    assert rate <= CODE_MISMATCH_RATE, f"code mismatch rate {rate:.3e}"
    return rate


def scales_close(got, want, rtol=SCALE_RTOL):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    assert np.all((want == 0) == (got == 0)), "zero-group pattern differs"
    nz = want != 0
    if nz.any():
        rel = np.abs(got[nz] - want[nz]) / np.abs(want[nz])
        assert rel.max() <= rtol, f"scale relative error {rel.max():.3e}"


def max_rel(got, want):
    want = np.asarray(want, dtype=np.float64)
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - want)) / max(np.max(np.abs(want)), 1e-300))


def oracle_wfq(x, w, layer, sB, sG, w_bits=8, **kw):
    """The oracle's pipeline with the filters quantized to w_bits (activations: 8 bits)."""
    filters = None
    if w_bits != 8:
        filters = orc.prepare_filters(w, layer.m, layer.gs, orc.matrices(layer.m, sB, sG, None), bits=w_bits)
    return orc.wfq(x, w, layer.m, layer.gs, sB=sB, sG=sG, filters=filters, **kw)


def check_layer_all_levels(layer, tensors=None, final_tol=FINAL_TOL, k1_kernel=0, w_bits=8):
    """Filters, stage 1, raw int32 group sums, stage 2, stage 3 and end to end.
    k1_kernel: input-transform kernel (0 = the library's choice, 2 = tensor cores where they apply);
    w_bits: bit width of the filter codes."""
    import torch
    conv, (x, w, sB, sG) = make_conv(layer, tensors, w_bits=w_bits)
    b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, k1_kernel)
    dev = conv.device
    ref = oracle_wfq(x, w, layer, sB, sG, w_bits)
    if w_bits != 8:
        assert np.abs(ref.Wq).max() == 2 ** (w_bits - 1) - 1
    report = {}

    # offline filter path
    report["wq_rate"] = codes_close(conv.buffer(b.WFQ_BUF_WQ).cpu().numpy(), ref.Wq)
    sw_all = conv.buffer(b.WFQ_BUF_SW).cpu().numpy()
    scales_close(sw_all[:, :, :layer.K], ref.sW.transpose(0, 2, 1), rtol=1e-6)
    assert not sw_all[:, :, layer.K:].any(), "sW padding columns must be zero"

    # stage 1: fused input transform + quantize
    xd = torch.from_numpy(x).to(dev)
    b.wfq_input_transform_quantize(conv.plan, xd.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    report["xq_rate"] = codes_close(conv.buffer(b.WFQ_BUF_XQ).cpu().numpy(), ref.Xq)
    scales_close(conv.buffer(b.WFQ_BUF_SX).cpu().numpy()[:, :, :conv.T], ref.sX.transpose(0, 2, 1))

    # identical int8 operands from here on: the oracle's codes and scales
    conv.write_buffer(b.WFQ_BUF_XQ, torch.from_numpy(ref.Xq))
    conv.write_buffer(b.WFQ_BUF_SX, torch.from_numpy(padded(ref.sX.transpose(0, 2, 1), conv.Ts)))
    conv.write_buffer(b.WFQ_BUF_WQ, torch.from_numpy(ref.Wq))
    conv.write_buffer(b.WFQ_BUF_SW, torch.from_numpy(padded(ref.sW.transpose(0, 2, 1), conv.Kp)))

    # level 1: int32 group accumulators, bit exact
    acc = torch.empty(ref.acc.shape, dtype=torch.int32, device=dev)
    b.wfq_debug_gemm_acc32(conv.plan, acc.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    conv.check_status()
    assert np.array_equal(acc.cpu().numpy(), ref.acc), "int32 group accumulators differ"

    # stage 2: dequantized Y
    b.wfq_gemm_dequantize(conv.plan, conv._stream())
    torch.cuda.synchronize()
    conv.check_status()
    Y = conv.buffer(b.WFQ_BUF_Y).cpu().numpy()[:, :, :conv.T]           # [P][K][T]
    report["Y_rel"] = max_rel(Y.transpose(0, 2, 1), ref.Y)
    assert report["Y_rel"] <= 1e-5, report

    # stage 3: output transform fed with the oracle's Y
    Yp = np.zeros((conv.P, layer.K, conv.Tp), dtype=np.float32)
    Yp[:, :, :conv.T] = ref.Y.transpose(0, 2, 1)
    conv.write_buffer(b.WFQ_BUF_Y, torch.from_numpy(Yp))
    y = torch.empty((layer.N, layer.K, layer.H, layer.W), dtype=torch.float32, device=dev)
    b.wfq_output_transform(conv.plan, y.data_ptr(), conv._stream())
    torch.cuda.synchronize()
    report["y3_rel"] = max_rel(y.cpu().numpy(), ref.y)
    # fp32 output transform: eps * (max row L1 norm of A^T)^2 = 6e-8 * 67^2 = 2.7e-4 worst case
    assert report["y3_rel"] <= 2e-4, report

    # end to end through wfq_conv_forward (filters re-prepared by the library)
    conv.prepare(torch.from_numpy(w).to(dev), None if sB is None else list(sB),
                 None if sG is None else list(sG))
    y.fill_(float("nan"))
    conv.forward(xd, y)
    torch.cuda.synchronize()
    conv.check_status()
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all(), "output has unwritten or non-finite elements"
    report["y_rel"] = max_rel(yh, ref.y)
    if report["y_rel"] > final_tol:
        # A code that is off by one LSB (allowed at level 2) moves its tile's outputs by a
        # quantization step times the gain of the output transform: compare with the
        # oracle continued from the GPU's codes and scales (see sampled_tiles_final_check).
        Xq_gpu = conv.buffer(b.WFQ_BUF_XQ).cpu().numpy()
        assert np.any(Xq_gpu != ref.Xq), report
        codes_close(Xq_gpu, ref.Xq)
        sX_gpu = np.ascontiguousarray(conv.buffer(b.WFQ_BUF_SX).cpu().numpy()[:, :, :conv.T].transpose(0, 2, 1))
        Y2 = orc.dequantize(orc.contract(Xq_gpu, ref.Wq, layer.gs), sX_gpu, ref.sW)
        y2 = orc.scatter_tiles(orc.output_transform(Y2, layer.m, ref.mats), layer.N, layer.H, layer.W, layer.m)
        report["y_rel_from_gpu_codes"] = max_rel(yh, y2)
        assert report["y_rel_from_gpu_codes"] <= final_tol, report
    else:
        assert report["y_rel"] <= final_tol, report
    report["sqnr_vs_direct_db"] = orc.sqnr_db(orc.direct(x, w), yh)
    conv.close()
    return report


def sampled_tiles_final_check(layer, conv, yh, ref, tiles, ks, tol=FINAL_TOL):
    """Level 3 on sampled tiles: max |y - y_ref| / max |y| per tile against the oracle.

    Levels 2 and 3 interact: one int8 code that is off by one LSB (level 2 allows that for
    1e-4 of the elements) moves the outputs of its tile by one quantization step of its
    group times the filter codes times the gain of the output transform (up to 32 for
    F(6,3)), which can exceed 2e-3 of max |y| when the group holds an outlier.  A tile that
    contains such a code is therefore compared with the oracle's pipeline continued from
    the GPU's codes and scales for that tile (contraction, dequantization and output
    transform by the oracle); all other tiles with the oracle's own codes.  Returns
    (worst error, number of tiles that needed the continuation)."""
    import torch
    m = layer.m
    geo = orc.geometry(layer.N, layer.H, layer.W, m)
    scale = float(np.max(np.abs(yh)))
    tt = torch.from_numpy(tiles).to(conv.device)
    Xq = conv.buffer(b.WFQ_BUF_XQ)[:, tt].cpu().numpy()
    sX = conv.buffer(b.WFQ_BUF_SX)[:, :, tt].cpu().numpy().transpose(0, 2, 1)      # [P][t][G]
    differs = np.any(Xq != ref.Xq, axis=(0, 2))                                       # per sampled tile
    ytile = ref.ytile
    if differs.any():
        idx = np.nonzero(differs)[0]
        acc = orc.contract(Xq[:, idx], ref.Wq, layer.gs)
        Y = orc.dequantize(acc, np.ascontiguousarray(sX[:, idx]), ref.sW)
        ytile = ref.ytile.copy()
        ytile[idx] = orc.output_transform(Y, m, ref.mats)
    worst = 0.0
    for i, t in enumerate(tiles):
        tw, th, img = t % geo.TW, (t // geo.TW) % geo.TH, t // (geo.TW * geo.TH)
        hh, ww = min(m, layer.H - th * m), min(m, layer.W - tw * m)
        got = yh[img][ks][:, th * m:th * m + hh, tw * m:tw * m + ww]
        worst = max(worst, float(np.max(np.abs(got - ytile[i][:, :hh, :ww]))) / scale)
    assert worst <= tol, worst
    return worst, int(differs.sum())
