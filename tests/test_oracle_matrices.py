"""Pins for the oracle's transformation matrices (CPU only).

The matrices are rebuilt in exact rationals from the interpolation points and
checked against (1) the values the paper prints, entry by entry, (2) the defining
property of a minimal filtering algorithm F(m,3) on all basis vectors (exact), and
(3) the scaling condition S_A S_B S_G = I.
"""
from fractions import Fraction as Fr

import pytest

from oracle import winograd_matrices as wm
from tests.golden_io import read_printed, read_table


def _check(name, rebuilt, printed, errata, tag):
    fixes = {(r, c): (p, f) for (mn, r, c, p, f) in errata if mn == tag}
    assert len(rebuilt) == len(printed) and len(rebuilt[0]) == len(printed[0]), name
    for r, (ra, rb) in enumerate(zip(rebuilt, printed)):
        for c, (a, b) in enumerate(zip(ra, rb)):
            if (r, c) in fixes:
                p, f = fixes[(r, c)]
                assert b == p, f"{name}[{r}][{c}]: fixture does not hold the printed typo"
                assert a == f, f"{name}[{r}][{c}]: rebuilt {a} != corrected {f}"
            else:
                assert a == b, f"{name}[{r}][{c}]: rebuilt {a} != printed {b}"


@pytest.mark.parametrize("m,fixture", [(4, "winograd_f43_printed.txt"),
                                       (6, "winograd_f63_printed.txt")])
def test_rebuilt_matrices_equal_printed(m, fixture):
    mats, errata = read_printed(fixture)
    n = m + 2
    std = wm.STANDARD_SCALES[m]
    assert std["SA"] == mats["SA"][0] and std["SB"] == mats["SB"][0] and std["SG"] == mats["SG"][0]
    pts = wm.POINTS[m]
    _check("V_nxm", wm.vandermonde(pts, m), mats["V_nxm"], errata, "V_nxm")
    _check("V_nx3", wm.vandermonde(pts, 3), mats["V_nx3"], errata, "V_nx3")
    VA, VB, VG = wm.vandermonde_parts(m)
    _check("V_nxn_invT", VB, mats["V_nxn_invT"], errata, "V_nxn_invT")
    AT, BT, G = wm.scaled_matrices(m)
    div = mats["BT_div"][0][0] if "BT_div" in mats else Fr(1)
    _check("AT", AT, mats["AT"], errata, "AT")
    _check("BT", BT, [[v / div for v in row] for row in mats["BT"]], errata, "BT")
    _check("G", G, mats["G"], errata, "G")
    assert len(errata) == (0 if m == 4 else 4)
    assert len(VB) == n and len(VA) == m and len(VG) == n


def test_f23_matrices_equal_the_textbook_ones():
    """F(2,3) is not printed in the paper: the rebuilt matrices are pinned to the textbook ones."""
    mats, errata = read_printed("winograd_f23_textbook.txt")
    assert not errata
    std = wm.STANDARD_SCALES[2]
    assert std["SA"] == mats["SA"][0] and std["SB"] == mats["SB"][0] and std["SG"] == mats["SG"][0]
    AT, BT, G = wm.scaled_matrices(2)
    assert AT == mats["AT"] and BT == mats["BT"] and G == mats["G"]


@pytest.mark.parametrize("m", [2, 4, 6])
def test_scaling_condition_standard(m):
    std = wm.STANDARD_SCALES[m]
    assert all(a * b * g == 1 for a, b, g in zip(std["SA"], std["SB"], std["SG"]))


def _conv1d_via_winograd(AT, BT, G, d, g):
    Gg = [sum(G[i][k] * g[k] for k in range(3)) for i in range(len(G))]
    Bd = [sum(BT[i][k] * d[k] for k in range(len(d))) for i in range(len(BT))]
    had = [a * b for a, b in zip(Gg, Bd)]
    return [sum(AT[u][i] * had[i] for i in range(len(had))) for u in range(len(AT))]


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("scales", ["standard", "custom"])
def test_minimal_filtering_identity_exact(m, scales):
    """A^T[(G g) .* (B^T d)] == sum_k d[u+k] g[k] for every pair of basis vectors."""
    n = m + 2
    if scales == "standard":
        AT, BT, G = wm.scaled_matrices(m)
    else:
        SB = [Fr(3, 7) * (-1) ** i * (i + 1) for i in range(n)]
        SG = [Fr(5, 2 + i) for i in range(n)]
        SA = [1 / (b * g) for b, g in zip(SB, SG)]
        AT, BT, G = wm.scaled_matrices(m, SA, SB, SG)
    for a in range(n):
        d = [Fr(int(i == a)) for i in range(n)]
        for b in range(3):
            g = [Fr(int(i == b)) for i in range(3)]
            want = [sum(d[u + k] * g[k] for k in range(3)) for u in range(m)]
            assert _conv1d_via_winograd(AT, BT, G, d, g) == want


def test_inverse_is_exact():
    for m in (2, 4, 6):
        V = wm.vandermonde(wm.POINTS[m], m + 2)
        I = wm.matmul(V, wm.inverse(V))
        assert all(I[i][j] == int(i == j) for i in range(m + 2) for j in range(m + 2))


def test_learned_scales_table_multiplies_to_one():
    rows = read_table("learned_scales_f63.txt")
    assert len(rows) == 8
    for sa, sb, sg in rows:
        assert abs(sa * sb * sg - 1.0) < 2e-3
    # the workloads module carries the same printed values as input data
    from paper_2412_19867_b200.workloads import LEARNED_F63
    assert [r[0] for r in rows] == LEARNED_F63["SA"]
    assert [r[1] for r in rows] == LEARNED_F63["SB"]
    assert [r[2] for r in rows] == LEARNED_F63["SG"]
