"""The cost-versus-memory-size experiment (Figure 1, Section 5.3) through the library's host entry
points: the values the paper prints for its worked example, and agreement with the oracle's
bounds on the benchmark shapes."""
import math

import pytest

from oracle import bounds as ob
from paper_1802_06905_b200 import curves
from paper_1802_06905_b200.synth import CONFIGS


def golden():
    vals = {}
    with open(__file__.rsplit("/", 1)[0] + "/golden/fig1_alexnet_layer.txt") as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    return vals


def test_fig1_layer_matches_the_printed_values():
    g = golden()
    dims = tuple(int(g[k]) for k in "B C K W H R S sw sh".split())
    assert dims == curves.FIG1_LAYER
    # "up to 11/4 times more communication" for matrix-multiply-style reuse
    assert curves.matmul_reuse_ratio(dims) == pytest.approx(g["matmul_reuse_ratio"], rel=1e-12)
    # "tight up to 17K words": the fifth term stops being the maximum at M = RS*sw*sh*(C/K)^2...
    # computed: B*C*K*W*H*sqrt(RS sw sh / M) = B*K*W*H  <=>  M = C^2 * R*S*sw*sh = 17 424
    m = curves.term5_tight_up_to(dims)
    assert m == pytest.approx(17424.0, rel=1e-6)
    assert round(m / 1000) == round(g["term5_tight_up_to_words"] / 1000)


@pytest.mark.parametrize("cfg", CONFIGS, ids=lambda c: c.name)
def test_curve_rows_agree_with_the_oracle_bounds(cfg):
    grid = curves.m_grid(per_decade=2)
    rows = curves.curve(cfg.dims(), grid)
    assert len(rows) == len(grid)
    for M, t1, t2, t3, t4, t5, bound, lp, mm in rows:
        exp = ob.theorem1_terms(*cfg.dims(), M)
        assert (t1, t2, t3, t4, t5) == pytest.approx(tuple(exp), rel=1e-12)
        assert bound == pytest.approx(max(exp), rel=1e-12)
        assert mm == pytest.approx(cfg.macs / math.sqrt(M), rel=1e-12)
        # the LP attains the bound wherever the bound is at least M (else everything fits: cost M)
        assert lp == pytest.approx(max(max(exp), M), rel=1e-6)


def test_measured_points_are_read_from_the_committed_summaries():
    pts = curves.measured_points()
    assert set(pts) == {c.name for c in CONFIGS}
    # DRAM traffic of the large 3x3 shape stays within 2x of the bound at the L2 level
    (m, words, _what), = [p for p in pts["cfg5_large_3x3"] if p[0] == curves.L2_WORDS]
    cfg = [c for c in CONFIGS if c.name == "cfg5_large_3x3"][0]
    assert words / max(ob.theorem1_terms(*cfg.dims(), m)) < 2.0
    text = curves.format_table(cfg.name, cfg.dims(), curves.curve(cfg.dims(), [1024.0, 1e6]),
                               pts[cfg.name])
    assert "measured: DRAM words per call" in text
