"""The dynamic-range diagnostic and the data-free scale fit of ``oracle/scale_study.py``
against the paper's qualitative claims (Sections 3.2, 4.2; the table of learned scales)."""
import numpy as np

from oracle import scale_study as st
from oracle import winograd_matrices as wm
from paper_2412_19867_b200 import workloads as wl


def test_standard_scales_have_the_cross_and_the_learned_table_flattens_it():
    layers = st.noise_layers(6, shapes=((32, 16, 12),))
    _, sB, sG = wm.standard_scales_f64(6)
    std = st.position_table(layers, 6, 32, sB, sG)
    lrn = st.position_table(layers, 6, 32, np.array(wl.LEARNED_F63["SB"]), np.array(wl.LEARNED_F63["SG"]))
    # rows / columns 3 and 4 (the points +-2) are the small ones: the 'cross'
    assert std[3, 3] < 0.01 and std[0, 0] > 0.5 and std[3, 0] < 0.1
    assert lrn.min() > 10 * std.min()
    s_std = st.stage_sqnr(layers, 6, 32, sB, sG)
    s_lrn = st.stage_sqnr(layers, 6, 32, np.array(wl.LEARNED_F63["SB"]), np.array(wl.LEARNED_F63["SG"]))
    # input transform and Hadamard stage: small effect either way; output transform: the
    # standard scales collapse, the learned ones recover most of it
    assert abs(s_std["hadamard"] - s_std["+input"]) < 1.5 and abs(s_lrn["hadamard"] - s_lrn["+input"]) < 1.5
    assert s_std["+output(tile)"] < 0.0 and s_lrn["+output(tile)"] > s_std["+output(tile)"] + 15.0
    assert s_lrn["+output(row)"] > s_lrn["+output(tile)"]


def test_data_free_fit_improves_on_the_standard_scales():
    layers = st.noise_layers(6, shapes=((32, 8, 12),))
    _, sB0, sG0 = wm.standard_scales_f64(6)
    before = st.mean_sqnr(layers, 6, 32, sB0, sG0, quant_input=True, quant_output=True, y_scale="tile")
    sB, sG, hist = st.fit_scales(layers, 6, 32, "tile", sweeps=2)
    assert hist[-1] >= hist[0] and hist[-1] > before + 10.0
    # S_A = 1/(S_B S_G) moved the way the paper's table does: the +-2 points' entries shrink
    sA = 1.0 / (sB * sG)
    assert abs(sA[3]) < 0.5 and abs(sA[4]) < 0.5
    # and it generalises to a layer it was not fitted on
    other = st.noise_layers(6, shapes=((64, 8, 12),), seed=3)
    assert st.mean_sqnr(other, 6, 32, sB, sG, quant_input=True, quant_output=True, y_scale="tile") > \
        st.mean_sqnr(other, 6, 32, sB0, sG0, quant_input=True, quant_output=True, y_scale="tile") + 10.0
