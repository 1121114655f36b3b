"""Full-size parity on sampled outputs: every layer of the benchmark configurations is
run at its real size, in the launch configuration the benchmark times, and compared
with the oracle on sampled tiles (the oracle evaluates the pipeline for a list of tiles;
group scales are per tile and per output channel, so a tile's result does not depend
on the other tiles).  Properties that hold at any size are checked on the whole output."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2412_19867_b200 import binding as b
from paper_2412_19867_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# every configured layer: 1 + 4 + 12 + 3 + 10 (configuration 1 is also run in full by
# test_gpu_parity.py)
FULL = [L for cfg in (2, 3, 4, 5) for L in wl.config_layers(cfg)]


# the tensor-core input transform at full size: one layer per staging mode and tile size
TC_FULL = [wl.config_layers(2)[i] for i in (0, 1, 2, 3)] + wl.config_layers(4) + [wl.config_layers(5)[i] for i in (5, 6)]


@pytest.mark.parametrize("layer", TC_FULL, ids=lambda L: L.name)
def test_full_size_sampled_tiles_tensor_core_input_transform(layer):
    test_full_size_sampled_tiles(layer, k1_kernel=2)


# NHWC input at full size (the tensor-core kernel that takes the TMA boxes as operands; groups of 128
# go to the plain NHWC kernel): both tile sizes, groups of 32 / 64 / 128, one and many items per CTA
NHWC_FULL = ([wl.config_layers(5)[i] for i in (0, 4, 5, 9)] + [wl.config_layers(2)[i] for i in (0, 3)] +
             [wl.config_layers(3)[i] for i in (0, 8, 9)])


@pytest.mark.parametrize("layer", NHWC_FULL, ids=lambda L: L.name)
def test_full_size_sampled_tiles_nhwc_input(layer):
    test_full_size_sampled_tiles(layer, nhwc=True)


@pytest.mark.parametrize("layer", FULL, ids=lambda L: L.name)
def test_full_size_sampled_tiles(layer, k1_kernel=0, nhwc=False):
    import torch
    from tests.gpu_util import make_conv, codes_close, scales_close, max_rel, FINAL_TOL
    conv, (x, w, sB, sG) = make_conv(layer)
    b.wfq_plan_set_debug_option(conv.plan, b.WFQ_DEBUG_INPUT_TRANSFORM_KERNEL, k1_kernel)
    xd = torch.from_numpy(x).cuda()
    if nhwc:
        conv.set_input_layout("nhwc")
        xd = xd.permute(0, 2, 3, 1).contiguous()
    y = conv.forward(xd)
    torch.cuda.synchronize()
    conv.check_status()
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()

    rng = np.random.default_rng(layer.seed)
    T = conv.T
    nt = min(T, 24)
    tiles = np.unique(np.concatenate([[0, T - 1], rng.integers(0, T, nt)]))
    ks = np.unique(np.concatenate([[0, layer.K - 1], rng.integers(0, layer.K, 46)]))
    ref = orc.wfq(x, w[ks], layer.m, layer.gs, sB=sB, sG=sG, tiles=tiles)

    Xq = conv.buffer(b.WFQ_BUF_XQ)[:, torch.from_numpy(tiles).cuda()].cpu().numpy()
    codes_close(Xq, ref.Xq)
    sX = conv.buffer(b.WFQ_BUF_SX)[:, :, torch.from_numpy(tiles).cuda()].cpu().numpy()
    scales_close(sX, ref.sX.transpose(0, 2, 1))
    Wq = conv.buffer(b.WFQ_BUF_WQ)[:, torch.from_numpy(ks).cuda()].cpu().numpy()
    codes_close(Wq, ref.Wq)

    from tests.gpu_util import sampled_tiles_final_check
    worst, continued = sampled_tiles_final_check(layer, conv, yh, ref, tiles, ks)
    print(layer.name, f"worst {worst:.2e}", "tiles compared from the GPU's codes:", continued)
    conv.close()
