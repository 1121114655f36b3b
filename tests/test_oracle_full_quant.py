"""Pins of the fully quantized pipeline (Section 4.1, Eqs. quant-B, quant-Y, quant-y) in
``oracle/full_quant.py``: its integer matrix products against independent numpy loops,
its limits against the pinned first part of the oracle and against direct convolution,
hand-made quantizer cases, and the paper's qualitative claims about where quantization
hurts (the output transform, because of the dynamic range of Y across the Winograd
positions) on seeded synthetic layers."""
import numpy as np
import pytest

from oracle import full_quant as fq
from oracle import oracle as orc
from paper_2412_19867_b200 import workloads as wl
from paper_2412_19867_b200.workloads import Layer


def _layer(m=6, gs=32, C=64, K=32, H=12, W=12, N=1, seed_variant=0, act="gauss_outlier"):
    L = Layer(N, C, K, H, W, m, gs, "f16", act, "kaiming", 7, 0, seed_variant)
    return L, wl.make_tensors(L)


def test_quantize_sym_hand_cases():
    v = np.array([[1.0, -2.0, 0.5, 0.0], [0.0, 0.0, 0.0, 0.0]])
    q, s = fq.quantize_sym(v, axes=(1,), bits=8)
    assert s.shape == (2, 1) and s[0, 0] == 2.0 / 127 and s[1, 0] == 0.0
    # 1/(2/127) = 63.5 -> 64 (half to even); -2 -> -127; 0.5 -> 31.75 -> 32
    assert q.tolist() == [[64, -127, 32, 0], [0, 0, 0, 0]]
    q4, s4 = fq.quantize_sym(np.array([7.0, -3.5, 1.0]), axes=(0,), bits=4)
    assert s4[0] == 1.0 and q4.tolist() == [7, -4, 1]          # -3.5 -> -4 (even)
    assert np.all(np.abs(q) <= 127)


def test_gather_patches_matches_oracle_input_transform_with_identity():
    # the patches, transformed by the first part's fp64 routine, equal B^T d B computed here
    L, (x, w, sB, sG) = _layer(m=4, H=7, W=9)
    mats = orc.matrices(L.m, sB, sG)
    d = fq.gather_patches(x, L.m)
    BT = mats.sB[:, None] * mats.VB
    mine = np.einsum("ia,tcab,jb->tcij", BT, d, BT).reshape(d.shape[0], L.C, -1).transpose(2, 0, 1)
    ref = orc.input_transform(x, L.m, mats)
    assert np.max(np.abs(mine - ref)) <= 1e-12 * np.max(np.abs(ref))


@pytest.mark.parametrize("m", [4, 6])
def test_integer_products_are_exact(m):
    L, (x, w, sB, sG) = _layer(m=m, C=32, K=8, H=2 * m, W=m)
    r = fq.wfq_full(x, w, m, L.gs, sB=sB, sG=sG)
    # Eq. quant-B, brute force over one tile and a few channels
    BTq, xq = r.inp.BTq, r.inp.xq
    n = m + 2
    for c in (0, 5, 31):
        want = np.zeros((n, n), dtype=np.int64)
        for i in range(n):
            for j in range(n):
                for a in range(n):
                    for b in range(n):
                        want[i, j] += BTq[i, a] * xq[1, c, a, b] * BTq[j, b]
        assert np.array_equal(r.inp.prod[1, c], want)
    # the real-valued X~ is that product times the three scales
    g = 5 // L.gs
    assert np.allclose(r.Xt[:, 1, 5].reshape(n, n), r.inp.prod[1, 5] * r.inp.sqB ** 2 * r.inp.sqx[1, g], rtol=1e-15)
    # Eq. quant-y, brute force
    ATq, Yq = r.out.ATq, r.out.Yq
    want = np.zeros((m, m), dtype=np.int64)
    for u in range(m):
        for v in range(m):
            for i in range(n):
                for j in range(n):
                    want[u, v] += ATq[u, i] * Yq[0, 3, i, j] * ATq[v, j]
    assert np.array_equal(r.out.prod[0, 3], want)
    assert np.all(np.abs(Yq) <= 127) and np.all(np.abs(xq) <= 127)


def test_switching_both_integer_transforms_off_is_the_pinned_pipeline():
    L, (x, w, sB, sG) = _layer(m=6, H=13, W=8)
    a = fq.wfq_full(x, w, L.m, L.gs, sB=sB, sG=sG, quant_input=False, quant_output=False)
    b = orc.wfq(x, w, L.m, L.gs, sB=sB, sG=sG)
    assert np.array_equal(a.Xq, b.Xq) and np.array_equal(a.acc, b.acc)
    assert np.array_equal(a.y, b.y)


def test_many_bits_recover_the_partly_quantized_pipeline():
    # with 16-bit matrices, inputs and Y the integer transforms are accurate to ~1e-4 (8 bits:
    # ~1e-2), so they approach the floating-point transforms of oracle.wfq
    L, (x, w, sB, sG) = _layer(m=4, H=8, W=8, act="relu_heavy")
    ref = orc.wfq(x, w, L.m, L.gs, sB=sB, sG=sG)
    mats = orc.matrices(L.m, sB, sG)
    BT = mats.sB[:, None] * mats.VB
    d = fq.gather_patches(x, L.m)
    X8, _ = fq.input_transform_int(d, BT, L.gs, bits=8, mat_bits=8)
    X16, _ = fq.input_transform_int(d, BT, L.gs, bits=16, mat_bits=16)
    e8 = np.max(np.abs(X8 - ref.Xt)) / np.max(np.abs(ref.Xt))
    e16 = np.max(np.abs(X16 - ref.Xt)) / np.max(np.abs(ref.Xt))
    assert e16 <= 2e-4 and 1e-3 < e8 < 5e-2
    AT = mats.VA * mats.sA[None, :]
    # the output side needs many more bits for the same accuracy (the dynamic range of Y
    # across the positions): the error falls by about 2^-4 per four bits
    errs = []
    for bits in (8, 12, 16, 20):
        yb, _ = fq.output_transform_int(ref.Y, AT, "tile", bits=bits, mat_bits=16)
        errs.append(np.max(np.abs(yb - ref.ytile)) / np.max(np.abs(ref.ytile)))
    assert errs[0] > errs[1] > errs[2] > errs[3] and errs[3] <= 5e-3 and errs[0] > 0.1
    with pytest.raises(ValueError):
        fq.input_transform_int(d, BT, L.gs, bits=24, mat_bits=24)      # would overflow int64


def test_scale_cancellation_survives_only_without_output_quantization():
    # S_A S_B S_G = I.  Rescaling S_G by f (hence S_A by 1/f) multiplies position (i, j) of W
    # and of Y by f_i f_j: the group-wise int8 codes do not change (each group lies in one
    # position) and the floating-point output transform undoes the factor, so without the
    # integer output transform the result is the same; with it, Y is quantized with one
    # scale per tile and the result depends on how the factors spread Y's positions: this
    # is the stage where the choice of scales matters (Section 4.1)
    L, (x, w, sB, sG) = _layer(m=6, H=12, W=12)
    n = L.m + 2
    rng = np.random.default_rng(5)
    f = np.exp(rng.uniform(-1.5, 1.5, n))
    base = fq.wfq_full(x, w, L.m, L.gs, sB=sB, sG=sG, quant_input=False, quant_output=False)
    resc = fq.wfq_full(x, w, L.m, L.gs, sB=sB, sG=sG * f, quant_input=False, quant_output=False)
    assert np.array_equal(base.Xq, resc.Xq)
    # (the filters are rounded to fp32 after the scaling, so a code at a tie may flip, and
    # one flipped code moves an output by a quantization step times the transform's gain)
    assert np.mean(base.Wq != resc.Wq) <= 1e-4
    assert np.max(np.abs(base.y - resc.y)) <= 2e-2 * np.max(np.abs(base.y))
    assert np.median(np.abs(base.y - resc.y)) <= 1e-6 * np.max(np.abs(base.y))
    on_a = fq.wfq_full(x, w, L.m, L.gs, sB=sB, sG=sG, quant_input=False, quant_output=True)
    on_b = fq.wfq_full(x, w, L.m, L.gs, sB=sB, sG=sG * f, quant_input=False, quant_output=True)
    assert np.median(np.abs(on_a.y - on_b.y)) > 1e-3 * np.max(np.abs(on_a.y))


def test_output_transform_is_where_quantization_hurts_and_pixel_scales_would_not():
    # Section 3.2: input transform and Hadamard stage quantize well, the output transform
    # does not (tile or row scales), pixel-wise scales would (but are not integer kernels)
    L, (x, w, _, _) = _layer(m=6, C=64, K=32, H=24, W=24, act="gauss_outlier")
    sB, sG = np.array(wl.STD_SB[6]), np.array(wl.STD_SG[6])
    direct = orc.direct(x, w)
    sq = {}
    for name, kw in {"hadamard only": dict(quant_input=False, quant_output=False),
                     "+ input": dict(quant_input=True, quant_output=False),
                     "+ output, tile": dict(quant_input=False, quant_output=True, y_scale="tile"),
                     "+ output, row": dict(quant_input=False, quant_output=True, y_scale="row"),
                     "+ output, pixel": dict(quant_input=False, quant_output=True, y_scale="pixel")}.items():
        sq[name] = orc.sqnr_db(direct, fq.wfq_full(x, w, 6, L.gs, sB=sB, sG=sG, **kw).y)
    print({k: round(v, 1) for k, v in sq.items()})
    assert sq["+ output, tile"] < sq["hadamard only"] - 6.0        # at least a factor two in amplitude
    assert sq["+ output, row"] > sq["+ output, tile"]
    assert sq["+ output, pixel"] > sq["+ output, row"]
    # the spread of Y across the positions is what the tile scale cannot cover
    spread = fq.position_spread(fq.wfq_full(x, w, 6, L.gs, sB=sB, sG=sG, quant_input=False, quant_output=False).Y)
    assert spread.min() < 0.05 and spread.max() == 1.0
