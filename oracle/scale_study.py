"""Dynamic range of the Winograd-domain output and a data-free scale fit (test
infrastructure, CPU oracle only).

Section 3.2 observes that the positions of Y have very different dynamic ranges (its
dynamic-range figure: relative standard deviation per position), which is what breaks
the integer output transform of Eq. quant-y, and Section 4.2 / Algorithm 1 learn the
diagonal scales S_B, S_G on random-noise inputs so that the fully quantized result tracks
the direct convolution.  This module measures both on seeded synthetic layers with the
oracle of ``full_quant.py``:

    python -m oracle.scale_study            # prints the tables (about a minute)

  * ``position_table``  relative standard deviation of Y at the n x n positions;
  * ``stage_sqnr``      SQNR against direct convolution with the stages quantized one
                        after the other (Hadamard stage, + integer input transform,
                        + integer output transform with a tile or a row scale);
  * ``fit_scales``      a derivative-free stand-in for Algorithm 1: Gaussian-noise
                        inputs, the SQNR of the fully quantized layer as the objective,
                        one shared scale set for all layers, coordinate search on the
                        logarithms of S_G with S_B fixed (only the products S_B S_G
                        = 1 / S_A reach the output transform) instead of SGD through the
                        quantizers.  It needs no data, weights of the layers only.
"""
import numpy as np

from . import full_quant as fq
from . import oracle as orc
from . import winograd_matrices as wm


def noise_layers(m, shapes=((32, 16, 12), (64, 16, 2 * 6)), seed=0):
    """[(x, w)]: Gaussian-noise inputs (fp16 values) and Kaiming-normal 3x3 filters."""
    rng = np.random.default_rng(241219867 + seed)
    out = []
    for C, K, H in shapes:
        x = rng.standard_normal((1, C, H, H)).astype(np.float16).astype(np.float64)
        w = (np.sqrt(2.0 / (9 * C)) * rng.standard_normal((K, C, 3, 3))).astype(np.float32)
        out.append((x, w))
    return out


def mean_sqnr(layers, m, gs, sB, sG, **kw):
    vals = []
    for x, w in layers:
        y = fq.wfq_full(x, w, m, gs, sB=sB, sG=sG, **kw).y
        vals.append(orc.sqnr_db(orc.direct(x, w), y))
    return float(np.mean(vals))


def stage_sqnr(layers, m, gs, sB, sG):
    return {"hadamard": mean_sqnr(layers, m, gs, sB, sG, quant_input=False, quant_output=False),
            "+input": mean_sqnr(layers, m, gs, sB, sG, quant_input=True, quant_output=False),
            "+output(tile)": mean_sqnr(layers, m, gs, sB, sG, quant_input=True, quant_output=True, y_scale="tile"),
            "+output(row)": mean_sqnr(layers, m, gs, sB, sG, quant_input=True, quant_output=True, y_scale="row")}


def position_table(layers, m, gs, sB, sG):
    x, w = layers[0]
    Y = fq.wfq_full(x, w, m, gs, sB=sB, sG=sG, quant_input=False, quant_output=False).Y
    return fq.position_spread(Y)


def fit_scales(layers, m, gs, y_scale="tile", sweeps=4, step=4.0, verbose=False):
    """Coordinate search for S_G (S_B standard): maximise the mean SQNR of the fully
    quantized layers.  Returns (sB, sG, history of the objective)."""
    sA_std, sB, sG0 = wm.standard_scales_f64(m)
    n = m + 2
    logf = np.zeros(n)

    def objective(lf):
        return mean_sqnr(layers, m, gs, sB, sG0 * np.exp(lf), quant_input=True, quant_output=True,
                         y_scale=y_scale)

    best = objective(logf)
    hist = [best]
    for _ in range(sweeps):
        for i in range(n):
            for sign in (+1.0, -1.0):
                trial = logf.copy()
                trial[i] += sign * np.log(step)
                val = objective(trial)
                if val > best:
                    best, logf = val, trial
        hist.append(best)
        if verbose:
            print(f"  step x{step:.2f}: {best:.2f} dB")
        step = np.sqrt(step)
    return sB, sG0 * np.exp(logf), hist


def main():
    np.set_printoptions(precision=3, suppress=True, linewidth=140)
    m, gs = 6, 32
    layers = noise_layers(m)
    sA_std, sB_std, sG_std = wm.standard_scales_f64(m)
    learned = dict(SB=[-1.378, -4.908, -4.912, 90.366, 90.362, 1.820, 1.823, 1.386],
                   SG=[-1.382, -0.576, -0.579, 0.184, 0.182, 1.119, 1.120, 1.391])   # the paper's table
    print("F(6,3), groups of", gs, "- Gaussian-noise inputs, Kaiming filters")
    sets = {"standard scales": (sB_std, sG_std),
            "the paper's learned scales": (np.array(learned["SB"]), np.array(learned["SG"]))}
    print("fitting S_G by coordinate search (tile scale for Y) ...")
    sBf, sGf, hist = fit_scales(layers, m, gs, "tile", verbose=True)
    sets["fitted here"] = (sBf, sGf)
    for name, (sB, sG) in sets.items():
        print(f"\n{name}: S_A = {1.0 / (np.asarray(sB) * np.asarray(sG))}")
        print("  SQNR vs direct convolution [dB]:", {k: round(v, 1) for k, v in stage_sqnr(layers, m, gs, sB, sG).items()})
        print("  relative standard deviation of Y per position:")
        print(position_table(layers, m, gs, sB, sG))


if __name__ == "__main__":
    main()
