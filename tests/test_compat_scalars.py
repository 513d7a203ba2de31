"""Compatibility scalars and the risk certificate: oracle pins (paper-printed value, closed forms, invariants) and the
library's host functions against the oracle.  No GPU needed."""
import math
import os

import numpy as np
import pytest

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import build as cbuild
from paper_2609_32420_b200 import carnator as cn

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "risk_certificate_paper.txt")


@pytest.fixture(scope="module", autouse=True)
def _built():
    cbuild.build_library()


def _golden():
    row = [ln for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")][0].split()
    return int(row[0]), int(row[1]), float(row[2]), int(row[3]), float(row[4]), float(row[5]), float(row[6])


def test_oracle_reproduces_the_printed_certificate():
    n, u, alpha, total, coverage, bound, delta = _golden()
    ub = orc.clopper_pearson_upper(u, n, alpha)
    assert round(100 * ub, 2) == bound                    # 4.50 %
    assert round(100 * n / total, 2) == coverage          # 71.43 %
    assert 100 * ub <= delta                              # satisfies the 5 % risk constraint
    assert abs(ub - (1 - alpha ** (1 / n))) < 1e-12       # closed form for u = 0


def test_library_bound_matches_oracle_and_printed_value():
    n, u, alpha, _, _, bound, _ = _golden()
    assert round(100 * cn.clopper_pearson_upper(u, n, alpha), 2) == bound
    for (uu, nn, aa) in [(0, 50, 0.1), (1, 50, 0.1), (3, 70, 0.05), (10, 30, 0.1), (29, 30, 0.2), (0, 1, 0.5)]:
        assert abs(cn.clopper_pearson_upper(uu, nn, aa) - orc.clopper_pearson_upper(uu, nn, aa)) < 1e-9
    assert cn.clopper_pearson_upper(5, 5, 0.1) == 1.0
    assert math.isnan(cn.clopper_pearson_upper(6, 5, 0.1))


def test_bound_is_the_binomial_tail_solution():
    """Definition: at p = U the probability of seeing <= u unsafe cases among n is alpha."""
    from scipy.stats import binom
    for (u, n, a) in [(0, 50, 0.1), (2, 40, 0.05), (7, 25, 0.1)]:
        assert abs(binom.cdf(u, n, orc.clopper_pearson_upper(u, n, a)) - a) < 1e-9


def test_delta_e00_closed_forms_and_invariants():
    rng = np.random.default_rng(0)
    for _ in range(20):
        x = [rng.uniform(0, 100), rng.uniform(-80, 80), rng.uniform(-80, 80)]
        y = [rng.uniform(0, 100), rng.uniform(-80, 80), rng.uniform(-80, 80)]
        assert orc.delta_e00(x, x) == 0.0
        assert abs(orc.delta_e00(x, y) - orc.delta_e00(y, x)) < 1e-12
        assert abs(cn.delta_e00(x, y) - orc.delta_e00(x, y)) < 1e-9
    # achromatic pair: only the lightness term remains, dE = |dL| / S_L
    L1, L2 = 35.0, 61.0
    Lb = 0.5 * (L1 + L2)
    SL = 1 + 0.015 * (Lb - 50) ** 2 / math.sqrt(20 + (Lb - 50) ** 2)
    assert abs(orc.delta_e00([L1, 0, 0], [L2, 0, 0]) - (L2 - L1) / SL) < 1e-12
    # near the neutral axis a* is stretched by 1.5 (G -> 1/2): (50, e, 0) vs (50, -e, 0) -> 3 e
    e = 1e-4
    assert abs(orc.delta_e00([50, e, 0], [50, -e, 0]) / (3 * e) - 1) < 1e-3


PAIRS = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "ciede2000_published_pairs.txt")


def _pairs():
    rows = [[float(x) for x in ln.split()] for ln in open(PAIRS) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 34
    return rows


def test_delta_e00_reproduces_the_published_check_pairs():
    """Pins the hue half of the formula: T, the hue-difference and mean-hue wrap branches, and the rotation term
    (sign and position), none of which the closed forms above reach."""
    for i, r in enumerate(_pairs()):
        assert abs(orc.delta_e00(r[0:3], r[3:6]) - r[6]) <= 1e-4, f"pair {i + 1}"
        assert abs(orc.delta_e00(r[3:6], r[0:3]) - r[6]) <= 1e-4, f"pair {i + 1} swapped"
        assert abs(cn.delta_e00(r[0:3], r[3:6]) - r[6]) <= 1e-4, f"pair {i + 1} (library)"


def test_context_discrepancy_is_the_largest_difference_over_shared_nouns():
    rows = _pairs()
    assert orc.context_discrepancy([], []) == 0.0 == cn.context_discrepancy([], [])      # no shared noun
    for sel in ([0], [3, 16, 24], [33, 18, 6, 20], list(range(34))):
        q, j = [rows[i][0:3] for i in sel], [rows[i][3:6] for i in sel]
        want = max(rows[i][6] for i in sel)                                              # published values
        assert abs(orc.context_discrepancy(q, j) - want) <= 1e-4
        assert abs(cn.context_discrepancy(q, j) - orc.context_discrepancy(q, j)) < 1e-9
    assert math.isnan(cn.lib().carnator_context_discrepancy(None, None, 2))


def test_shape_size_and_gate():
    yy, xx = np.mgrid[0:40, 0:60]
    disk = ((yy - 20) ** 2 + (xx - 30) ** 2 <= 15 ** 2).astype(np.uint8)
    big = ((np.mgrid[0:90, 0:90][0] - 45) ** 2 + (np.mgrid[0:90, 0:90][1] - 45) ** 2 <= 40 ** 2).astype(np.uint8)
    square = np.zeros((30, 30), dtype=np.uint8); square[5:25, 8:20] = 1
    # scale and translation drop out after bounding-box normalisation
    assert orc.shape_discrepancy(disk, big, 32) < 0.03
    assert orc.shape_discrepancy(square, square, 32) == 0.0
    d_sq = orc.shape_discrepancy(disk, square, 32)
    assert abs(d_sq - (1 - 2 * (math.pi / 4) / (math.pi / 4 + 1))) < 0.03      # disk vs its full box: Dice = 2a/(a+1), a = pi/4
    for (a, b) in [(disk, big), (disk, square), (square, big)]:
        assert abs(cn.shape_discrepancy(a, b, 32) - orc.shape_discrepancy(a, b, 32)) < 1e-12
    assert orc.size_discrepancy(0.2, 0.1) == pytest.approx(math.log(2))
    assert cn.size_discrepancy(0.1, 0.2) == pytest.approx(math.log(2))
    tau = [1.62, 2.17, 1.00, 7.58]                       # the thresholds the paper reports
    assert cn.compatibility_gate([1.0, 2.0, 0.5, 7.58], tau) == 1 == orc.compatibility_gate([1.0, 2.0, 0.5, 7.58], tau)
    assert cn.compatibility_gate([1.0, 2.2, 0.5, 7.0], tau) == 0 == orc.compatibility_gate([1.0, 2.2, 0.5, 7.0], tau)
    assert cn.compatibility_gate([1.0, 2.2, 0.5, 7.0], tau, [1, 0, 0, 0]) == 1       # only the context dimension applies
