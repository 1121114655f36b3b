"""Seeded synthetic layers and tensors (shared by the tests, the benchmark and the oracle runs).

This module draws random inputs only; it holds none of the method's arithmetic
(no transform, no quantizer).  The layer shapes are those of the benchmark
configurations (ResNet-18/34-style stages and SD-like UNet conv blocks); the value
distributions imitate the activations and filters of such networks:

* ``gauss_outlier``  N(0,1), each element x20 with probability 0.01   (fp32)
* ``relu_heavy``     relu(t), t ~ Student-t(4): half-normal body, heavy tail (fp16)
* ``silu_outlier``   silu(z), z ~ N(0,1), each element x50 with probability 0.005 (fp16)
* filters ``gauss_chan``  N(0, 0.05^2) x per-output-channel factor exp(U[ln .3, ln 3])
* filters ``kaiming``     N(0, 2/(9C))
* filters ``kaiming_chan`` Kaiming x per-output-channel factor exp(U[ln .1, ln 10])
* transform scales: the standard scale vectors printed in the paper's supplementary
  (plain data, listed below) times exp(0.1 z) per entry (log-normal(0, 0.1)),
  with S_A left to the library (derived from S_A S_B S_G = I).

Seeds: 241219867 + 1000*config + 10*layer + variant.
"""
from dataclasses import dataclass, replace

import numpy as np

BASE_SEED = 241219867

# Standard F(m,3) scale vectors as printed in the paper's supplementary section
# "Standard Winograd transforms" (input data for both sides, like the learned table).
STD_SB = {2: [1.0, 2.0, 2.0, -1.0],
          4: [4.0, -6.0, -6.0, 24.0, 24.0, 1.0],
          6: [1.0, -4.5, -4.5, 90.0, 90.0, 45.0 / 32.0, 45.0 / 32.0, 1.0]}
STD_SG = {2: [1.0, 0.5, 0.5, 1.0],
          4: [1.0 / 4, -1.0 / 6, -1.0 / 6, 1.0 / 24, 1.0 / 24, 1.0],
          6: [1.0, -2.0 / 9, -2.0 / 9, 1.0 / 90, 1.0 / 90, 32.0 / 45, 32.0 / 45, 1.0]}

# Learned F(6,3) scales, table "Comparison between standard Winograd scales and our
# learned Winograd scales" (values rounded to 3-4 digits as printed).
LEARNED_F63 = dict(
    SA=[0.525, 0.354, 0.351, 0.0601, 0.0609, 0.491, 0.490, 0.519],
    SB=[-1.378, -4.908, -4.912, 90.366, 90.362, 1.820, 1.823, 1.386],
    SG=[-1.382, -0.576, -0.579, 0.184, 0.182, 1.119, 1.120, 1.391])


@dataclass(frozen=True)
class Layer:
    """One 3x3 stride-1 pad-1 convolution layer evaluated as F(m,3)."""
    N: int
    C: int
    K: int
    H: int
    W: int
    m: int
    gs: int
    dtype: str = "f16"            # input dtype: "f16" or "f32"
    act: str = "silu_outlier"
    filt: str = "kaiming_chan"
    cfg: int = 0
    idx: int = 0
    variant: int = 0

    @property
    def seed(self):
        return BASE_SEED + 1000 * self.cfg + 10 * self.idx + self.variant

    @property
    def name(self):
        return (f"cfg{self.cfg}.{self.idx}:N{self.N}_C{self.C}_K{self.K}_"
                f"{self.H}x{self.W}_F{self.m}_g{self.gs}_{self.dtype}")

    @property
    def direct_ops(self):
        """Direct-convolution-equivalent operations, 2*N*K*C*H*W*9."""
        return 2 * self.N * self.K * self.C * self.H * self.W * 9

    def scaled(self, **kw):
        return replace(self, **kw)


def config_layers(cfg):
    """The benchmark configurations, 1-based like the configuration list."""
    if cfg == 1:
        return [Layer(1, 64, 64, 32, 32, 4, 32, "f32", "gauss_outlier", "gauss_chan", 1, 0)]
    if cfg == 2:
        return [Layer(32, c, c, h, h, 6, 64, "f16", "relu_heavy", "kaiming", 2, i)
                for i, (c, h) in enumerate([(64, 56), (128, 28), (256, 14), (512, 7)])]
    if cfg == 3:
        out, i = [], 0
        for m in (4, 6):
            for (c, h) in ((128, 28), (256, 14)):
                for gs in (32, 64, 128):
                    out.append(Layer(64, c, c, h, h, m, gs, "f16", "relu_heavy", "kaiming", 3, i))
                    i += 1
        return out
    if cfg == 4:
        return [Layer(2, c, c, h, h, 4, 64, "f16", "silu_outlier", "kaiming_chan", 4, i)
                for i, (c, h) in enumerate([(320, 64), (640, 32), (1280, 16)])]
    if cfg == 5:
        out, i = [], 0
        for m in (4, 6):
            for (c, k, h) in ((320, 320, 128), (320, 640, 64), (640, 640, 64),
                              (640, 1280, 32), (1280, 1280, 32)):
                out.append(Layer(1, c, k, h, h, m, 64, "f16", "silu_outlier", "kaiming_chan", 5, i))
                i += 1
        return out
    raise ValueError(f"unknown config {cfg}")


def _activations(rng, layer):
    shape = (layer.N, layer.C, layer.H, layer.W)
    if layer.act == "gauss_outlier":
        x = rng.standard_normal(shape)
        x = np.where(rng.random(shape) < 0.01, 20.0 * x, x)
    elif layer.act == "relu_heavy":
        x = np.maximum(rng.standard_t(4, shape), 0.0)
    elif layer.act == "silu_outlier":
        z = rng.standard_normal(shape)
        x = z / (1.0 + np.exp(-z))
        x = np.where(rng.random(shape) < 0.005, 50.0 * x, x)
    elif layer.act == "gauss":
        x = rng.standard_normal(shape)          # the random-noise inputs of the data-free setting
    elif layer.act == "zeros":
        x = np.zeros(shape)
    else:
        raise ValueError(layer.act)
    return x.astype(np.float16 if layer.dtype == "f16" else np.float32)


def _filters(rng, layer):
    shape = (layer.K, layer.C, 3, 3)
    if layer.filt == "gauss_chan":
        w = 0.05 * rng.standard_normal(shape)
        w *= np.exp(rng.uniform(np.log(0.3), np.log(3.0), (layer.K, 1, 1, 1)))
    elif layer.filt == "kaiming":
        w = np.sqrt(2.0 / (9 * layer.C)) * rng.standard_normal(shape)
    elif layer.filt == "kaiming_chan":
        w = np.sqrt(2.0 / (9 * layer.C)) * rng.standard_normal(shape)
        w *= np.exp(rng.uniform(np.log(0.1), np.log(10.0), (layer.K, 1, 1, 1)))
    else:
        raise ValueError(layer.filt)
    return w.astype(np.float32)


def _scales(rng, layer):
    n = layer.m + 2
    sB = np.array(STD_SB[layer.m]) * np.exp(0.1 * rng.standard_normal(n))
    sG = np.array(STD_SG[layer.m]) * np.exp(0.1 * rng.standard_normal(n))
    return sB.astype(np.float32), sG.astype(np.float32)


def make_tensors(layer):
    """(x, w, sB, sG) for a layer: x fp16/fp32 NCHW, w fp32 [K][C][3][3], fp32 scale vectors."""
    rng = np.random.default_rng(layer.seed)
    x = _activations(rng, layer)
    w = _filters(rng, layer)
    sB, sG = _scales(rng, layer)
    return x, w, sB, sG
