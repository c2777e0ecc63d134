"""Communication cost versus fast-memory size (the experiment behind Figure 1, Section 5.3).

For one convolution shape and a grid of fast-memory sizes M (in words) this tabulates, through the
library's host entry points `cconv_lower_bound` and `cconv_tiling_lp`:

  * the five terms of Theorem 1 and their maximum (the lower bound),
  * the words moved by the Section-5 blocked nest at the LP's optimum (`F*M/G`),
  * the cost of a blocking with matrix-multiply-style reuse, `B*C*K*W*H*R*S / sqrt(M)` (the dashed
    line of Figure 1), whose ratio to the fifth term is `sqrt(R*S/(sw*sh))` (11/4 in the figure),

and, for the benchmark shapes, where this machine's measured traffic sits: DRAM bytes at M = half
the L2 capacity in words, L2-to-shared-memory bytes at M = the shared memory of one CTA, both
taken from the ncu summaries under `profiles/`.

    python -m paper_1802_06905_b200.curves            # Figure 1's layer + the five benchmark shapes
    python -m paper_1802_06905_b200.curves --csv out.csv

Pure host arithmetic: no GPU is needed (the library loads without a driver).
"""
from __future__ import annotations

import argparse
import math
import os
import sys

from . import binding
from .synth import CONFIGS

FIG1_LAYER = (1000, 3, 96, 55, 55, 11, 11, 4, 4)  # B C K W H R S sw sh of the figure's caption
L2_WORDS = 126 * 1024 * 1024 // 2
CTA_SMEM_WORDS = 232448 // 2

_ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def macs(dims):
    B, C, K, W, H, R, S, _, _ = dims
    return float(B) * C * K * W * H * R * S


def curve(dims, m_grid):
    """Rows (M, term1..term5, bound, lp_words, matmul_reuse_words) for every M of the grid."""
    rows = []
    B, C, K, W, H, R, S, _, _ = dims
    for M in m_grid:
        terms = binding.lower_bound(*dims, float(M))
        _, _, lp_words = binding.tiling_lp(*dims, float(M))
        # matmul-style reuse: the fifth term of the same loop nest written as a matrix product
        # (C*R*S channels behind a 1x1 filter, unit strides), evaluated by the library
        matmul = binding.lower_bound(B, C * R * S, K, W, H, 1, 1, 1, 1, float(M))[4]
        rows.append((float(M), *terms, max(terms), lp_words, matmul))
    return rows


def m_grid(lo=64.0, hi=float(L2_WORDS), per_decade=8):
    n = int(math.ceil(math.log10(hi / lo) * per_decade))
    return [lo * (hi / lo) ** (i / n) for i in range(n + 1)]


def term5_tight_up_to(dims):
    """The largest M at which the fifth term is still the maximum of the five (bisection on M).
    Above it an array-size term takes over, i.e. one of the arrays should simply stay in cache."""
    def fifth_is_max(M):
        t = binding.lower_bound(*dims, float(M))
        return t[4] >= max(t[0], t[1], t[2], t[3])
    B, C, K, W, H, R, S, sw, sh = dims
    # below M = R*S/(sw*sh) the fourth term (no reuse at all) exceeds the fifth
    lo, hi = max(1.0, 1.0001 * R * S / (sw * sh)), 1e15
    if not fifth_is_max(lo):
        return 0.0
    for _ in range(200):
        mid = math.sqrt(lo * hi)
        if fifth_is_max(mid):
            lo = mid
        else:
            hi = mid
    return lo


def matmul_reuse_ratio(dims):
    """Cost of matrix-multiply-style reuse over the fifth term: sqrt(R*S/(sw*sh))."""
    M = 4096.0
    return (macs(dims) / math.sqrt(M)) / binding.lower_bound(*dims, M)[4]


def _read_table(name):
    out = {}
    path = os.path.join(_ROOT, "profiles", name)
    if os.path.exists(path):
        with open(path) as fh:
            for line in fh:
                parts = line.split()
                if len(parts) >= 2 and not parts[0].startswith("#"):
                    try:
                        out[parts[0]] = float(parts[1])
                    except ValueError:
                        pass
    return out


def measured_points():
    """{config name: [(M words, measured words, what)]} from the committed ncu summaries."""
    dram = _read_table("dram_traffic.txt")
    l2sm = _read_table("l2_to_sm_traffic.txt")
    pts = {}
    for c in CONFIGS:
        p = []
        if c.name in dram:
            p.append((float(L2_WORDS), dram[c.name] / 2.0, "DRAM words per call (ncu; Out still in L2 at kernel end is not counted)"))
        if c.name in l2sm:
            p.append((float(CTA_SMEM_WORDS), l2sm[c.name] / 2.0, "L2 -> shared-memory words per call (ncu)"))
        pts[c.name] = p
    return pts


def format_table(name, dims, rows, points=()):
    B, C, K, W, H, R, S, sw, sh = dims
    out = [f"# {name}: B={B} C={C} K={K} W={W} H={H} R={R} S={S} sw={sw} sh={sh}; "
           f"MACs={macs(dims):.4g}",
           f"# fifth term is the bound up to M = {term5_tight_up_to(dims):.0f} words; "
           f"matmul-style reuse costs {matmul_reuse_ratio(dims):.3f}x the fifth term",
           "#        M       bound    lp_tiling  matmul_reuse  argmax  lp/bound",
           "# (lp_tiling = M, marked 'fits': every array fits in M words and the blocked nest "
           "degenerates to loading them once)"]
    for M, t1, t2, t3, t4, t5, bound, lp, mm in rows:
        arg = 1 + max(range(5), key=lambda i: (t1, t2, t3, t4, t5)[i])
        ratio = "     fits" if lp <= M * (1 + 1e-9) else f"{lp / bound:9.3f}"
        out.append(f"{M:12.0f} {bound:11.4g} {lp:11.4g} {mm:13.4g} {arg:7d} {ratio}")
    for M, words, what in points:
        bound = max(binding.lower_bound(*dims, M))
        out.append(f"# measured: {what}: {words:.4g} at M = {M:.0f} words = {words / bound:.2f}x the bound there")
    return "\n".join(out)


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--csv", help="also write all rows to this CSV file")
    ap.add_argument("--per-decade", type=int, default=4)
    args = ap.parse_args(argv)
    grid = m_grid(per_decade=args.per_decade)
    shapes = [("fig1_alexnet_layer", FIG1_LAYER)] + [(c.name, c.dims()) for c in CONFIGS]
    pts = measured_points()
    csv_rows = []
    for name, dims in shapes:
        rows = curve(dims, grid)
        print(format_table(name, dims, rows, pts.get(name, ())))
        print()
        csv_rows += [(name, *r) for r in rows]
    if args.csv:
        with open(args.csv, "w") as fh:
            fh.write("shape,M,term1,term2,term3,term4,term5,bound,lp_words,matmul_reuse_words\n")
            for r in csv_rows:
                fh.write(",".join(str(x) for x in r) + "\n")
    return 0


if __name__ == "__main__":
    sys.exit(main())
