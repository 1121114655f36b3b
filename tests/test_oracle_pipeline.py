"""Pins for the CPU oracle's pipeline (CPU only).

Each stage is tied to something other than itself: a library routine
(scipy correlate, numpy integer einsum), the Winograd identity against the direct
convolution, invariants (scale cancellation, sign symmetry of the codes), closed
forms on hand-made inputs, and special cases where the quantized result must equal
the direct convolution.
"""
import numpy as np
import pytest
from scipy.signal import correlate2d

from oracle import oracle as orc
from paper_2412_19867_b200 import workloads as wl


def _rand_layer(rng, N, C, K, H, W):
    x = rng.standard_normal((N, C, H, W))
    w = rng.standard_normal((K, C, 3, 3))
    return x, w


def _custom_scales(rng, m):
    n = m + 2
    sB = (np.array(wl.STD_SB[m]) * np.exp(0.3 * rng.standard_normal(n))).astype(np.float32)
    sG = (np.array(wl.STD_SG[m]) * np.exp(0.3 * rng.standard_normal(n))).astype(np.float32)
    sB[1] = -sB[1]  # signs are allowed
    return sB, sG


def test_direct_matches_library_correlation():
    rng = np.random.default_rng(1)
    x, w = _rand_layer(rng, 2, 3, 4, 5, 7)
    y = orc.direct(x, w)
    for n in range(2):
        for k in range(4):
            ref = sum(correlate2d(x[n, c], w[k, c], mode="same", boundary="fill") for c in range(3))
            np.testing.assert_allclose(y[n, k], ref, rtol=0, atol=1e-12)


def test_direct_single_tap_shifts():
    """A filter with one nonzero tap shifts the image (catches swapped/negated offsets)."""
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 1, 6, 5))
    for a in range(3):
        for b in range(3):
            w = np.zeros((1, 1, 3, 3))
            w[0, 0, a, b] = 1.0
            y = orc.direct(x, w)[0, 0]
            xp = np.pad(x[0, 0], 1)
            np.testing.assert_array_equal(y, xp[a:a + 6, b:b + 5])


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("shape", [(1, 2, 3, 7, 7), (2, 3, 2, 14, 9), (1, 1, 1, 4, 6), (1, 2, 2, 13, 56)])
def test_unquantized_winograd_equals_direct(m, shape):
    rng = np.random.default_rng(3)
    x, w = _rand_layer(rng, *shape)
    ref = orc.direct(x, w)
    y = orc.unquantized(x, w, m)
    assert np.max(np.abs(y - ref)) <= 1e-10 * np.max(np.abs(ref))


@pytest.mark.parametrize("m", [2, 4, 6])
def test_scaling_invariance_unquantized(m):
    """Any nonzero S_B, S_G with S_A = (S_B S_G)^-1 give the same result."""
    rng = np.random.default_rng(4)
    x, w = _rand_layer(rng, 1, 3, 2, 11, 8)
    ref = orc.direct(x, w)
    sB, sG = _custom_scales(rng, m)
    y = orc.unquantized(x, w, m, sB=sB, sG=sG)
    assert np.max(np.abs(y - ref)) <= 1e-10 * np.max(np.abs(ref))
    # a wrong S_A must be visible (the check is not vacuous)
    bad = orc.unquantized(x, w, m, sB=sB, sG=sG, sA=np.ones(m + 2))
    assert np.max(np.abs(bad - ref)) > 1e-3 * np.max(np.abs(ref))


def test_quantizer_brute_force_and_properties():
    rng = np.random.default_rng(5)
    v = rng.standard_normal((7, 64)).astype(np.float32) * np.float32(3.7)
    v[2, :32] = 0.0                      # an all-zero group
    v[3, 5] = 1000.0                     # an outlier
    q, s = orc.quantize_groups(v, 32)
    assert q.dtype == np.int8 and s.shape == (7, 2)
    for r in range(7):
        for g in range(2):
            grp = v[r, 32 * g:32 * g + 32]
            amax = np.max(np.abs(grp))
            if amax == 0:
                assert s[r, g] == 0 and not q[r, 32 * g:32 * g + 32].any()
                continue
            # brute force, python floats rounded to fp32 at each step
            scale = np.float32(amax) / np.float32(127.0)
            inv = np.float32(127.0) / np.float32(amax)
            assert s[r, g] == scale
            for e in range(32):
                prod = np.float32(grp[e]) * inv
                want = int(np.clip(np.rint(prod), -127, 127))   # np.rint: half to even
                assert q[r, 32 * g + e] == want
            qq = q[r, 32 * g:32 * g + 32].astype(np.float64)
            assert np.max(np.abs(qq)) == 127                       # abs-max element hits the end
            assert np.all(np.abs(grp - scale * qq) <= 0.5 * scale * (1 + 1e-5))
    assert np.abs(q).max() <= 127


def test_quantizer_ties_round_half_to_even_and_idempotent():
    # amax = 127 -> inv = 1 exactly, so values k + 0.5 are exact ties
    v = np.zeros((1, 32), dtype=np.float32)
    v[0, :8] = [127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5]
    q, s = orc.quantize_groups(v, 32)
    assert s[0, 0] == 1.0
    assert list(q[0, :8]) == [127, 0, 2, 2, 0, -2, -2, 126]
    # on-grid values are reproduced exactly (idempotence)
    grid = (np.arange(-16, 16) * 7 % 255 - 127).astype(np.float32)[None, :]
    grid[0, 0] = 127.0
    q2, s2 = orc.quantize_groups(grid * np.float32(0.25), 32)
    np.testing.assert_array_equal(q2[0].astype(np.float32), grid[0])


@pytest.mark.parametrize("bits", [4, 6])
def test_quantizer_other_bit_widths_brute_force(bits):
    """The same quantizer with 2^(bits-1) - 1 in place of 127 (4 bits: the weight side of the
    W4A8 setting, Section 5): scale, every code by brute force, error at most half a step."""
    qmax = 2 ** (bits - 1) - 1
    v = np.linspace(-1, 1, 32, dtype=np.float32)[None, :]
    q, s = orc.quantize_groups(v, 32, bits=bits)
    assert q.max() == qmax and q.min() == -qmax and s[0, 0] == np.float32(1.0) / np.float32(qmax)
    rng = np.random.default_rng(50 + bits)
    v = rng.standard_normal((5, 64)).astype(np.float32) * np.float32(0.37)
    v[1, 32:] = 0.0
    v[2, 7] = 55.0
    q, s = orc.quantize_groups(v, 32, bits=bits)
    for r in range(5):
        for g in range(2):
            grp = v[r, 32 * g:32 * g + 32]
            amax = np.max(np.abs(grp))
            if amax == 0:
                assert s[r, g] == 0 and not q[r, 32 * g:32 * g + 32].any()
                continue
            scale = np.float32(amax) / np.float32(qmax)
            inv = np.float32(qmax) / np.float32(amax)
            assert s[r, g] == scale
            want = [int(np.clip(np.rint(np.float32(e) * inv), -qmax, qmax)) for e in grp]
            assert list(q[r, 32 * g:32 * g + 32]) == want
            assert np.max(np.abs(want)) == qmax
            assert np.all(np.abs(grp - np.float64(scale) * np.array(want)) <= 0.5 * scale * (1 + 1e-5))
    # ties at inv = 1: half to even, as at 8 bits
    t = np.zeros((1, 32), dtype=np.float32)
    t[0, :6] = [qmax, 0.5, 1.5, 2.5, -0.5, -1.5]
    q, s = orc.quantize_groups(t, 32, bits=bits)
    assert s[0, 0] == 1.0 and list(q[0, :6]) == [qmax, 0, 2, 2, 0, -2]


def test_four_bit_filters_cost_about_four_bits_of_sqnr():
    """Filters at 4 bits with activations at 8 (through `filters=`): the error of the result is
    dominated by the filter codes' step, 127/7 = 18 times coarser, so the SQNR against the direct
    convolution falls by about 20 log10(18) = 25 dB (within a few dB on random data)."""
    from paper_2412_19867_b200 import workloads as wl
    L = wl.Layer(1, 64, 32, 12, 12, 4, 32, "f32", "gauss", "kaiming", 8, 11, 0)
    x, w, sB, sG = wl.make_tensors(L)
    direct = orc.direct(x, w)
    f4 = orc.prepare_filters(w, L.m, L.gs, orc.matrices(L.m, sB, sG, None), bits=4)
    assert np.abs(f4.Wq).max() == 7
    r8 = orc.wfq(x, w, L.m, L.gs, sB, sG)
    r4 = orc.wfq(x, w, L.m, L.gs, sB, sG, filters=f4)
    assert np.array_equal(r4.Xq, r8.Xq)                       # the activation side is untouched
    drop = orc.sqnr_db(direct, r8.y) - orc.sqnr_db(direct, r4.y)
    assert 18.0 <= drop <= 30.0, drop


def test_contract_matches_integer_einsum_and_bound():
    rng = np.random.default_rng(6)
    P, T, K, C, gs = 3, 5, 4, 64, 32
    Xq = rng.integers(-127, 128, (P, T, C), dtype=np.int8)
    Wq = rng.integers(-127, 128, (P, K, C), dtype=np.int8)
    Xq[0, 0, :] = 127
    Wq[0, 0, :] = -127                                       # the extreme case
    acc = orc.contract(Xq, Wq, gs)
    ref = np.einsum("ptgc,pkgc->ptkg", Xq.reshape(P, T, 2, gs).astype(np.int64),
                    Wq.reshape(P, K, 2, gs).astype(np.int64))
    np.testing.assert_array_equal(acc, ref)
    assert acc[0, 0, 0, 0] == -gs * 127 * 127
    assert np.abs(acc).max() <= gs * 127 * 127


def test_dequantize_closed_form():
    P, T, K, G = 2, 3, 2, 2
    acc = np.arange(P * T * K * G, dtype=np.int32).reshape(P, T, K, G) - 7
    sX = (1.0 + np.arange(P * T * G, dtype=np.float32).reshape(P, T, G)) / 8
    sW = (2.0 + np.arange(P * K * G, dtype=np.float32).reshape(P, K, G)) / 4
    Y = orc.dequantize(acc, sX, sW)
    for p in range(P):
        for t in range(T):
            for k in range(K):
                want = sum(float(acc[p, t, k, g]) * float(sX[p, t, g]) * float(sW[p, k, g]) for g in range(G))
                assert Y[p, t, k] == pytest.approx(want, rel=1e-15)


@pytest.mark.parametrize("m", [2, 4, 6])
def test_one_channel_per_group_equals_direct(m):
    """With a single nonzero channel per group every nonzero maps to +-127 and
    dequantizes to 127*fl32(amax/127): the quantized pipeline must reproduce the direct
    convolution up to fp32 rounding of the transformed values and scales."""
    rng = np.random.default_rng(7)
    gs, C, K = 32, 64, 3
    x = np.zeros((2, C, 9, 10))
    w = np.zeros((K, C, 3, 3))
    x[:, ::gs] = rng.standard_normal((2, C // gs, 9, 10))
    w[:, ::gs] = rng.standard_normal((K, C // gs, 3, 3))
    sB, sG = _custom_scales(rng, m)
    res = orc.wfq(x, w, m, gs, sB=sB, sG=sG)
    ref = orc.direct(x, w)
    nz = res.Xq[res.Xq != 0]
    assert np.all(np.abs(nz) == 127)
    assert np.max(np.abs(res.y - ref)) <= 2e-5 * np.max(np.abs(ref))


@pytest.mark.parametrize("m,gs", [(4, 32), (6, 64)])
def test_quantized_error_within_a_priori_bound(m, gs):
    """|Y - Y_exact| <= sum_c (|X| sW/2 + |W| sX/2 + sX sW/4), pushed through |A^T| (x) |A^T|."""
    rng = np.random.default_rng(8)
    C, K = 2 * gs, 5
    x = rng.standard_normal((1, C, 2 * m + 1, m + 2))
    w = 0.1 * rng.standard_normal((K, C, 3, 3))
    res = orc.wfq(x, w, m, gs)
    mats = res.mats
    P, T, _ = res.Xq.shape
    G = C // gs
    Yexact = orc.hadamard_f64(res.Xt, res.Wt)
    sXf = np.repeat(res.sX.astype(np.float64), gs, axis=2)          # [P][T][C]
    sWf = np.repeat(res.sW.astype(np.float64), gs, axis=2)          # [P][K][C]
    bound = (np.einsum("ptc,pkc->ptk", np.abs(res.Xt), sWf) / 2
             + np.einsum("ptc,pkc->ptk", sXf, np.abs(res.Wt)) / 2
             + np.einsum("ptc,pkc->ptk", sXf, sWf) / 4) * (1 + 1e-5) + 1e-12
    assert np.all(np.abs(res.Y - Yexact) <= bound)
    # output-space bound
    n = m + 2
    AT = np.abs(mats.VA * mats.sA[None, :])                          # |A^T| (m x n)
    Bt = bound.reshape(n, n, T, K)
    ybound = np.einsum("ui,ijtk,vj->tkuv", AT, Bt, AT)
    ref = orc.direct(x, w)
    yb = orc.scatter_tiles(ybound, 1, x.shape[2], x.shape[3], m)
    assert np.all(np.abs(res.y - ref) <= yb + 1e-9 * np.abs(ref).max())
    assert orc.sqnr_db(ref, res.y) > 15.0


@pytest.mark.parametrize("m", [2, 4, 6])
def test_codes_invariant_to_scales_up_to_sign(m):
    """Groups run along channels at a fixed position, so multiplying a position by
    sB_i sB_j scales the whole group: codes change only by the sign of that product."""
    rng = np.random.default_rng(9)
    x, w = _rand_layer(rng, 1, 64, 4, 2 * m, 2 * m)
    base = orc.wfq(x, w, m, 32)
    sB, sG = _custom_scales(rng, m)
    alt = orc.wfq(x, w, m, 32, sB=sB, sG=sG)
    n = m + 2
    ratio = sB.astype(np.float64) / np.array(wl.STD_SB[m])
    sign = np.sign(np.outer(ratio, ratio)).reshape(n * n)[:, None, None].astype(np.int16)
    diff = np.abs(alt.Xq.astype(np.int16) - sign * base.Xq.astype(np.int16))
    assert diff.max() <= 1 and np.mean(diff != 0) < 1e-3
    assert np.max(np.abs(alt.y - base.y)) <= 2e-2 * np.max(np.abs(base.y))


def test_tile_subset_equals_full_run():
    rng = np.random.default_rng(10)
    x, w = _rand_layer(rng, 2, 32, 3, 10, 7)
    full = orc.wfq(x, w, 4, 32)
    tiles = np.array([0, 5, 7, 11])
    part = orc.wfq(x, w, 4, 32, tiles=tiles)
    np.testing.assert_array_equal(part.Xq, full.Xq[:, tiles])
    np.testing.assert_array_equal(part.ytile, full.ytile[tiles])
    geo = orc.geometry(2, 10, 7, 4)
    assert geo.T == 2 * 3 * 2 and full.ytile.shape == (geo.T, 3, 4, 4)


def test_ragged_edges_do_not_raise_group_maxima():
    """Zero fill beyond the image only adds zeros to a patch: an image embedded in a
    larger zero canvas gives the same outputs inside."""
    rng = np.random.default_rng(11)
    x, w = _rand_layer(rng, 1, 32, 2, 7, 7)
    a = orc.wfq(x, w, 6, 32).y
    assert a.shape == (1, 2, 7, 7)
    ref = orc.direct(x, w)
    assert orc.sqnr_db(ref, a) > 15.0


def test_all_zero_input_gives_zero_output_without_nan():
    x = np.zeros((1, 32, 6, 6))
    w = np.random.default_rng(12).standard_normal((2, 32, 3, 3))
    res = orc.wfq(x, w, 4, 32)
    assert not res.Xq.any() and not res.sX.any()
    assert np.all(res.y == 0.0)


@pytest.mark.parametrize("cfg", [1])
def test_config1_quality_sanity(cfg):
    layer = wl.config_layers(cfg)[0]
    x, w, sB, sG = wl.make_tensors(layer)
    res = orc.wfq(x, w, layer.m, layer.gs, sB=sB, sG=sG)
    ref = orc.direct(x, w)
    assert orc.sqnr_db(ref, res.y) > 15.0
    assert np.abs(res.acc).max() <= layer.gs * 127 * 127


def test_workload_generators_are_seeded_and_shaped():
    for cfg, count in [(1, 1), (2, 4), (3, 12), (4, 3), (5, 10)]:
        layers = wl.config_layers(cfg)
        assert len(layers) == count
        for L in layers:
            assert L.C % L.gs == 0
    L = wl.config_layers(4)[2]
    a = wl.make_tensors(L)
    b = wl.make_tensors(L)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(u, v)
    assert a[0].dtype == np.float16 and a[0].shape == (2, 1280, 16, 16)
    assert a[1].shape == (1280, 1280, 3, 3) and a[2].shape == (6,)


def test_epilogue_hand_values():
    """Bias per output channel, then ReLU / SiLU: hand-computed values (silu(1) = 1 / (1 + 1/e),
    silu(0) = 0, silu(-t) = silu(t) - t)."""
    y = np.array([[[[1.0, -2.0]], [[0.5, 0.0]]]])          # [1][2][1][2]
    bias = np.array([0.0, -0.5])
    np.testing.assert_allclose(orc.epilogue(y, bias, "none"), [[[[1.0, -2.0]], [[0.0, -0.5]]]])
    np.testing.assert_allclose(orc.epilogue(y, bias, "relu"), [[[[1.0, 0.0]], [[0.0, 0.0]]]])
    s = orc.epilogue(y, None, "silu")
    e = 2.718281828459045
    np.testing.assert_allclose(s[0, 0, 0, 0], 1.0 / (1.0 + 1.0 / e), rtol=1e-15)
    assert s[0, 1, 0, 1] == 0.0
    np.testing.assert_allclose(s[0, 0, 0, 1], 2.0 / (1.0 + e * e) * e * e - 2.0, rtol=1e-13)
    t = np.linspace(-5, 5, 11).reshape(1, 1, 1, 11)
    np.testing.assert_allclose(orc.epilogue(-t, None, "silu"), orc.epilogue(t, None, "silu") - t, atol=1e-15)
    with pytest.raises(ValueError):
        orc.epilogue(y, None, "gelu")
