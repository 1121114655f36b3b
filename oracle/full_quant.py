"""CPU oracle, second part (test infrastructure): the paper's *fully* quantized pipeline.

``oracle.wfq`` quantizes only the Winograd-domain input and filters (Eq. quant-Y) and runs
both transforms in floating point.  Section 4.1 goes further: the input transform and the
output transform are integer matrix products as well,

    X~ = s_qB^2 s_qx  Q(S_B V_B / s_qB)  Q(x / s_qx)   Q(V_B^T S_B / s_qB)     (Eq. quant-B)
    Y~ = s_qW s_qX    Q(W / s_qW) Q(X~ / s_qX)                                 (Eq. quant-Y)
    y~ = s_qA^2 s_qY  Q(V_A S_A / s_qA)  Q(Y~ / s_qY)  Q(S_A V_A^T / s_qA)     (Eq. quant-y)

and Section 3.2 / 4.1 say that Y needs one scale per output tile or per row / column for
the integer arithmetic to work, which is where the dynamic range of Y across the
Winograd positions hurts and where the learned scales S_B, S_G help.

Plain numpy, fp64 and int64, small layers only; the steps follow the three equations in
order.  It reuses the first part of the oracle for the pieces the two have in common
(matrices, filter path, group quantizer, integer contraction, dequantization) and shares
nothing with the CUDA path.

Readings where the paper is silent (listed in the design notes as well):
  * Q is the quantizer of Section 2: symmetric, codes in [-(2^(b-1)-1), 2^(b-1)-1],
    round half to even, scale = abs-max / (2^(b-1)-1), dynamic.
  * s_qB and s_qA are scalars in the equations (they appear squared): one scale per
    transform matrix.
  * s_qx: one scale per (tile, group of `group_size` consecutive input channels), shared
    by the n x n patches of those channels (a scalar per matrix product factors out).
  * s_qY: ``y_scale = "tile"`` one scale per (tile, output channel), i.e. per n x n matrix
    Y~; ``"row"`` one scale per row of that matrix for the product with the right-hand
    matrix, whose result is quantized again per column for the left-hand product (each
    1-D pass is then an integer matrix product with scales that factor out);
    ``"pixel"`` one scale per element (the paper's remark that this would be accurate but
    rules out integer kernels: the products are then not integer products; kept as the
    reference point).
"""
from types import SimpleNamespace

import numpy as np

from . import oracle as orc


def qmax_of(bits):
    return 2 ** (bits - 1) - 1


def quantize_sym(v, axes, bits=8):
    """Symmetric abs-max quantizer (Section 2) with one scale per slice over `axes`.

    Returns (integer codes as int64, scales broadcastable against v).  A slice whose
    abs-max is zero gets scale 0 and codes 0."""
    v = np.asarray(v, dtype=np.float64)
    q = qmax_of(bits)
    amax = np.max(np.abs(v), axis=axes, keepdims=True)
    s = amax / q
    safe = np.where(s > 0, s, 1.0)
    codes = np.clip(np.rint(v / safe), -q, q).astype(np.int64)
    codes = np.where(s > 0, codes, 0)
    return codes, s


def gather_patches(x, m, tiles=None):
    """d[t][c][a][b]: the n x n input patch of tile t and channel c (zeros outside the image)."""
    x = np.asarray(x, dtype=np.float64)
    N, C, H, W = x.shape
    geo = orc.geometry(N, H, W, m)
    n = geo.n
    xp = np.zeros((N, C, geo.TH * m + 2, geo.TW * m + 2))
    xp[:, :, 1:H + 1, 1:W + 1] = x
    ids = np.arange(geo.T) if tiles is None else np.asarray(tiles)
    d = np.empty((len(ids), C, n, n))
    for i, t in enumerate(ids):
        tw, th, img = t % geo.TW, (t // geo.TW) % geo.TH, t // (geo.TW * geo.TH)
        d[i] = xp[img, :, th * m:th * m + n, tw * m:tw * m + n]
    return d


def input_transform_int(d, BT, gs, bits=8, mat_bits=8):
    """Eq. quant-B on patches d[t][c][n][n]: returns X~[P][t][c] (fp64) and the integer parts."""
    T, C, n, _ = d.shape
    if bits + 2 * mat_bits + 6 > 62:
        raise ValueError("the integer products would not fit int64")
    BTq, sqB = quantize_sym(BT, axes=(0, 1), bits=mat_bits)                   # one scale per matrix
    dg = d.reshape(T, C // gs, gs, n, n)
    xq, sqx = quantize_sym(dg, axes=(2, 3, 4), bits=bits)                     # per (tile, group)
    xq = xq.reshape(T, C, n, n)
    prod = np.einsum("ia,tcab,jb->tcij", BTq, xq, BTq)                        # exact in int64
    scale = (sqB.reshape(()) ** 2) * np.repeat(sqx.reshape(T, C // gs), gs, axis=1)
    Xt = prod.astype(np.float64) * scale[:, :, None, None]
    return (np.ascontiguousarray(Xt.reshape(T, C, n * n).transpose(2, 0, 1)),
            SimpleNamespace(BTq=BTq, sqB=float(sqB.reshape(())), xq=xq, sqx=sqx.reshape(T, C // gs), prod=prod))


def output_transform_int(Y, AT, y_scale="tile", bits=8, mat_bits=8):
    """Eq. quant-y on Y[P][t][k] (fp64): returns y tiles [t][k][m][m] and the integer parts."""
    P, T, K = Y.shape
    m, n = AT.shape
    if bits + 2 * mat_bits + 6 > 62:
        raise ValueError("the integer products would not fit int64")
    Yt = np.ascontiguousarray(Y.transpose(1, 2, 0)).reshape(T, K, n, n)
    ATq, sqA = quantize_sym(AT, axes=(0, 1), bits=mat_bits)
    sA = float(sqA.reshape(()))
    if y_scale == "tile":
        Yq, sqY = quantize_sym(Yt, axes=(2, 3), bits=bits)
        prod = np.einsum("ui,tkij,vj->tkuv", ATq, Yq, ATq)                    # exact in int64
        y = prod.astype(np.float64) * (sA * sA) * sqY
        return y, SimpleNamespace(ATq=ATq, sqA=sA, Yq=Yq, sqY=sqY, prod=prod)
    if y_scale == "row":
        Yq, sr = quantize_sym(Yt, axes=(3,), bits=bits)                       # one scale per row i
        Z = np.einsum("tkij,vj->tkiv", Yq, ATq).astype(np.float64) * sA * sr  # rows keep their scale
        Zq, sc = quantize_sym(Z, axes=(2,), bits=bits)                        # one scale per column v
        prod = np.einsum("ui,tkiv->tkuv", ATq, Zq)
        y = prod.astype(np.float64) * sA * sc
        return y, SimpleNamespace(ATq=ATq, sqA=sA, Yq=Yq, sqY=sr, prod=prod)
    if y_scale == "pixel":
        # every element its own scale: exact up to the matrix codes (not an integer product)
        y = np.einsum("ui,tkij,vj->tkuv", ATq * sA, Yt, ATq * sA)
        return y, SimpleNamespace(ATq=ATq, sqA=sA, Yq=None, sqY=None, prod=None)
    raise ValueError(y_scale)


def wfq_full(x, w, m, gs, sB=None, sG=None, sA=None, bits=8, mat_bits=8, tiles=None,
             quant_input=True, quant_output=True, y_scale="tile"):
    """The fully quantized pipeline of Section 4.1 with every intermediate kept.

    quant_input / quant_output switch the integer input / output transform on (Eqs.
    quant-B / quant-y); with both off this is ``oracle.wfq`` step for step.  Returns a
    namespace with Xt (X~, fp64), Xq, sX, Wq, sW, acc, Y, ytile, y and the per-stage
    integer parts ``inp`` / ``out``."""
    N, C, H, W = x.shape
    mats = orc.matrices(m, sB, sG, sA)
    f = orc.prepare_filters(w, m, gs, mats, bits)
    BT = mats.sB[:, None] * mats.VB                      # S_B V_B
    AT = mats.VA * mats.sA[None, :]                      # V_A S_A (m x n)
    inp = out = None
    if quant_input:
        Xt, inp = input_transform_int(gather_patches(x, m, tiles), BT, gs, bits, mat_bits)
    else:
        Xt = orc.input_transform(x, m, mats, tiles)
    X32 = Xt.astype(np.float32)
    Xq, sX = orc.quantize_groups(X32, gs, bits)
    acc = orc.contract(Xq, f.Wq, gs)
    Y = orc.dequantize(acc, sX, f.sW)
    if quant_output:
        ytile, out = output_transform_int(Y, AT, y_scale, bits, mat_bits)
    else:
        ytile = orc.output_transform(Y, m, mats)
    y = orc.scatter_tiles(ytile, N, H, W, m) if tiles is None else None
    return SimpleNamespace(mats=mats, BT=BT, AT=AT, Xt=Xt, X32=X32, Xq=Xq, sX=sX, Wq=f.Wq, sW=f.sW, acc=acc,
                           Y=Y, ytile=ytile, y=y, inp=inp, out=out)


def position_spread(Y):
    """Dynamic range of Y across the Winograd positions (caption of the dynamic-range
    figure, Section 3.2): the standard deviation of Y at each of the n x n positions over
    tiles and output channels, relative to the largest one.  Input Y[P][t][k]."""
    P = Y.shape[0]
    n = int(round(P ** 0.5))
    sd = np.std(np.asarray(Y, dtype=np.float64).reshape(P, -1), axis=1)
    return (sd / max(sd.max(), 1e-300)).reshape(n, n)
