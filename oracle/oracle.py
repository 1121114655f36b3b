"""CPU oracle for the group-wise int8-quantized Winograd convolution (test infrastructure).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares nothing with the CUDA path.  The heavy loops are plain C
(``wfq_oracle.c``, compiled here with gcc); this file sequences the steps in the
paper's order and keeps every intermediate so each level of the CUDA path can be
compared with it:

    (a) ``direct``        fp64 direct 3x3 convolution (the definition, Section 3.1)
    (b) ``wfq``           the quantized pipeline of Section 4.1: scaled input/filter
                          transforms -> group-wise int8 quantization in the Winograd
                          domain -> per-position integer contraction per channel group
                          -> dequantization (Eq. quant-Y) -> scaled output transform
    (c) ``unquantized``   the same transforms with an fp64 Hadamard stage, used to pin
                          the transforms to (a)

Readings where the paper is silent (symmetric abs-max, -127..127, half-to-even,
reciprocal multiply in fp32, zero group -> scale 0) are stated in the C source next
to the quantizer.
"""
import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

from . import winograd_matrices as wm

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wfq_oracle.c")
_LIB = os.path.join(_HERE, "_wfq_oracle.so")
_lib = None


def build(force=False):
    """Compile the C oracle with gcc (OpenMP over outer loops, no BLAS, no intrinsics)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", _LIB + ".tmp", _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.wfq_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads():
    return int(lib().wfq_oracle_num_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def geometry(N, H, W, m):
    n = m + 2
    TH, TW = -(-H // m), -(-W // m)
    return SimpleNamespace(n=n, P=n * n, TH=TH, TW=TW, T=N * TH * TW)


def matrices(m, sB=None, sG=None, sA=None):
    """fp64 V_A (m x n), V_B (n x n), V_G (n x 3) and the scale vectors.

    ``sB``/``sG`` default to the standard scales.  If ``sA`` is not given it is
    derived from the scaling condition S_A S_B S_G = I in fp64 and then rounded to
    fp32 (the value a library taking fp32 scale vectors would hold).
    """
    VA, VB, VG = wm.vandermonde_parts_f64(m)
    sA_std, sB_std, sG_std = wm.standard_scales_f64(m)
    sB = sB_std if sB is None else _f64(sB)
    sG = sG_std if sG is None else _f64(sG)
    if sA is None:
        sA = (1.0 / (sB * sG)).astype(np.float32).astype(np.float64)
    else:
        sA = _f64(sA)
    return SimpleNamespace(VA=VA, VB=VB, VG=VG, sA=sA, sB=sB, sG=sG)


def direct(x, w):
    """fp64 direct convolution, stride 1, padding 1, cross-correlation, no bias."""
    x, w = _f64(x), _f64(w)
    N, C, H, W = x.shape
    K = w.shape[0]
    assert w.shape == (K, C, 3, 3)
    y = np.empty((N, K, H, W), dtype=np.float64)
    d = ctypes.c_double
    lib().wfq_oracle_direct(_p(x, d), _p(w, d), _p(y, d), N, C, K, H, W)
    return y


def filter_transform(w, mats):
    w = _f64(w)
    K, C = w.shape[:2]
    n = mats.VG.shape[0]
    Wt = np.empty((n * n, K, C), dtype=np.float64)
    d = ctypes.c_double
    lib().wfq_oracle_filter_transform(_p(w, d), _p(_f64(mats.VG), d), _p(_f64(mats.sG), d),
                                      K, C, n, _p(Wt, d))
    return Wt


def input_transform(x, m, mats, tiles=None):
    x = _f64(x)
    N, C, H, W = x.shape
    geo = geometry(N, H, W, m)
    if tiles is None:
        tptr, nt = None, geo.T
    else:
        tiles = np.ascontiguousarray(tiles, dtype=np.int64)
        tptr, nt = _p(tiles, ctypes.c_int64), len(tiles)
    Xt = np.empty((geo.P, nt, C), dtype=np.float64)
    d = ctypes.c_double
    lib().wfq_oracle_input_transform(_p(x, d), _p(_f64(mats.VB), d), _p(_f64(mats.sB), d),
                                     N, C, H, W, m, tptr, ctypes.c_int64(nt), _p(Xt, d))
    return Xt


def quantize_groups(v32, gs, bits=8):
    """v32[..., C] fp32 -> (int8 codes [..., C], fp32 scales [..., C/gs])."""
    v32 = np.ascontiguousarray(v32, dtype=np.float32)
    C = v32.shape[-1]
    assert C % gs == 0
    rows = v32.size // C
    q = np.empty(v32.shape, dtype=np.int8)
    s = np.empty(v32.shape[:-1] + (C // gs,), dtype=np.float32)
    qmax = 2 ** (bits - 1) - 1
    lib().wfq_oracle_quantize_groups(_p(v32, ctypes.c_float), ctypes.c_int64(rows), C, gs, qmax,
                                     _p(q, ctypes.c_int8), _p(s, ctypes.c_float))
    return q, s


def contract(Xq, Wq, gs):
    Xq = np.ascontiguousarray(Xq, dtype=np.int8)
    Wq = np.ascontiguousarray(Wq, dtype=np.int8)
    P, T, C = Xq.shape
    K = Wq.shape[1]
    assert Wq.shape == (P, K, C)
    acc = np.empty((P, T, K, C // gs), dtype=np.int32)
    lib().wfq_oracle_contract(_p(Xq, ctypes.c_int8), _p(Wq, ctypes.c_int8), P, ctypes.c_int64(T),
                              K, C, gs, _p(acc, ctypes.c_int32))
    return acc


def dequantize(acc, sX, sW):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    sX = np.ascontiguousarray(sX, dtype=np.float32)
    sW = np.ascontiguousarray(sW, dtype=np.float32)
    P, T, K, G = acc.shape
    assert sX.shape == (P, T, G) and sW.shape == (P, K, G)
    Y = np.empty((P, T, K), dtype=np.float64)
    lib().wfq_oracle_dequantize(_p(acc, ctypes.c_int32), _p(sX, ctypes.c_float),
                                _p(sW, ctypes.c_float), P, ctypes.c_int64(T), K, G,
                                _p(Y, ctypes.c_double))
    return Y


def hadamard_f64(Xt, Wt):
    Xt, Wt = _f64(Xt), _f64(Wt)
    P, T, C = Xt.shape
    K = Wt.shape[1]
    Y = np.empty((P, T, K), dtype=np.float64)
    d = ctypes.c_double
    lib().wfq_oracle_hadamard_f64(_p(Xt, d), _p(Wt, d), P, ctypes.c_int64(T), K, C, _p(Y, d))
    return Y


def output_transform(Y, m, mats):
    Y = _f64(Y)
    P, T, K = Y.shape
    yt = np.empty((T, K, m, m), dtype=np.float64)
    d = ctypes.c_double
    lib().wfq_oracle_output_transform(_p(Y, d), _p(_f64(mats.VA), d), _p(_f64(mats.sA), d),
                                      ctypes.c_int64(T), K, m, _p(yt, d))
    return yt


def scatter_tiles(ytile, N, H, W, m, tiles=None):
    ytile = _f64(ytile)
    nt, K = ytile.shape[:2]
    y = np.zeros((N, K, H, W), dtype=np.float64)
    if tiles is None:
        tptr = None
    else:
        tiles = np.ascontiguousarray(tiles, dtype=np.int64)
        tptr = _p(tiles, ctypes.c_int64)
    d = ctypes.c_double
    lib().wfq_oracle_scatter_tiles(_p(ytile, d), tptr, ctypes.c_int64(nt), N, K, H, W, m, _p(y, d))
    return y


def prepare_filters(w, m, gs, mats, bits=8):
    """Offline filter path: transform (fp64), one rounding to fp32, group quantization."""
    Wt = filter_transform(w, mats)
    W32 = Wt.astype(np.float32)
    Wq, sW = quantize_groups(W32, gs, bits)
    return SimpleNamespace(Wt=Wt, W32=W32, Wq=Wq, sW=sW)


def wfq(x, w, m, gs, sB=None, sG=None, sA=None, bits=8, tiles=None, filters=None):
    """The quantized Winograd pipeline with every intermediate kept.

    x[N][C][H][W] (any float dtype; converted exactly to fp64), w[K][C][3][3].
    ``tiles``: optional list of tile ids to evaluate (sampled parity at full size);
    then ``y`` is None and ``ytile`` holds the m x m outputs of those tiles.
    Returns a namespace with Xt, X32, Xq, sX[P][T][G], Wq, sW[P][K][G],
    acc[P][T][K][G], Y[P][T][K], ytile[T][K][m][m], y[N][K][H][W] (fp64).
    """
    N, C, H, W = x.shape
    mats = matrices(m, sB, sG, sA)
    f = prepare_filters(w, m, gs, mats, bits) if filters is None else filters
    Xt = input_transform(x, m, mats, tiles)
    X32 = Xt.astype(np.float32)            # the single rounding before quantization
    Xq, sX = quantize_groups(X32, gs, bits)
    acc = contract(Xq, f.Wq, gs)
    Y = dequantize(acc, sX, f.sW)
    ytile = output_transform(Y, m, mats)
    y = scatter_tiles(ytile, N, H, W, m) if tiles is None else None
    return SimpleNamespace(mats=mats, Xt=Xt, X32=X32, Xq=Xq, sX=sX, Wt=f.Wt, W32=f.W32,
                           Wq=f.Wq, sW=f.sW, acc=acc, Y=Y, ytile=ytile, y=y)


def unquantized(x, w, m, sB=None, sG=None, sA=None, derive_sA_exact=True):
    """Winograd pipeline without quantization (fp64 throughout)."""
    N, C, H, W = x.shape
    mats = matrices(m, sB, sG, sA)
    if sA is None and derive_sA_exact:
        mats.sA = 1.0 / (mats.sB * mats.sG)
    Y = hadamard_f64(input_transform(x, m, mats), filter_transform(w, mats))
    return scatter_tiles(output_transform(Y, m, mats), N, H, W, m)


def epilogue(y, bias=None, act="none"):
    """Bias per output channel and activation on y[N][K][H][W] (fp64): none, relu, silu."""
    y = np.asarray(y, dtype=np.float64)
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :, None, None]
    if act == "relu":
        return np.maximum(y, 0.0)
    if act == "silu":
        return y / (1.0 + np.exp(-y))
    if act != "none":
        raise ValueError(act)
    return y


def sqnr_db(ref, test):
    ref = np.asarray(ref, dtype=np.float64)
    err = np.asarray(test, dtype=np.float64) - ref
    return 10.0 * np.log10(np.sum(ref * ref) / max(np.sum(err * err), 1e-300))
