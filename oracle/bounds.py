"""TEST INFRASTRUCTURE ONLY -- oracle for the host-side planner's mathematics.

Plain restatements of
  * the five-term communication lower bound (Theorem 1, Section 4.1),
  * the tiling linear program over log-tile-sizes (Section 5, the LP that follows the tile
    constraints), solved with a library LP solver as one step,
  * the communication cost F*M/G of a tiling (Section 5.2 cost function; Appendix A cost formula),
  * the stride-1 decision tree (Theorem 2, Appendix A),
  * the small HBL linear program of Section 4.2 whose optimum is 2.
The CUDA product's planner has its own simplex and its own formulas; the two share nothing.

Pins (tests, "not gpu"): the values the paper prints for its worked AlexNet-layer example
(Figure 1 caption: crossover at C^2*R*S*sw*sh = 17 424 words, the 11/4 reuse ratio, the product of
the printed tile sizes at M = 1024), "LP cost equals the largest term whenever that term >= M"
(Section 5.2), term 5 > term 4 iff RS < M*sw*sh (Section 4.1), the R=S=1 reduction to the
matrix-multiply bound (Section 3), and the explicit tilings of the Appendix-A lemmas.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.optimize import linprog

VARS = ("b", "c", "k", "w", "h", "r1", "r2", "s1", "s2")  # r1=r', r2=r'', s1=s', s2=s''


def theorem1_terms(B, C, K, W, H, R, S, sw, sh, M):
    """The five expressions whose maximum is the lower bound of Theorem 1 (words moved)."""
    F = B * C * K * W * H
    return [
        float(B * K * W * H),                      # |Out|
        float(sw * sh * B * C * W * H),            # |Image| (asymptotic form used by the paper)
        float(C * K * R * S),                      # |Filter|
        F * R * S / M,                             # HBL term, Section 4.2
        F * math.sqrt(R * S * sw * sh / M),        # small-filter term, Section 4.3
    ]


def theorem1_bound(B, C, K, W, H, R, S, sw, sh, M):
    t = theorem1_terms(B, C, K, W, H, R, S, sw, sh, M)
    return max(t), int(np.argmax(t)) + 1


def pooling_terms(B, C, K, W, H, R, S, sw, sh, M):
    """The three expressions whose maximum bounds the words moved by pooling (Section 6):
    |Out|, |Image| (asymptotic form) and the HBL term of the nest without its Filter."""
    return [
        float(B * K * W * H),
        float(sw * sh * B * C * W * H),
        float(B * C * K * W * H) * R * S / M,
    ]


def parallel_terms(B, C, K, W, H, R, S, sw, sh, M, aB, aK, aH, aW):
    """The five terms of the bound for p processors behind one shared memory of M words when the
    output is cut into aB x aK x aH x aW equal blocks, one per processor (Section 8, "Parallel
    Algorithm"): p times Theorem 1 on the sub-problem B/aB, K/aK, H/aH, W/aW, which leaves terms
    1, 4 and 5 as they are, multiplies the Image term by aK and the Filter term by aB*aW*aH."""
    t = theorem1_terms(B, C, K, W, H, R, S, sw, sh, M)
    return [t[0], aK * t[1], aB * aW * aH * t[2], t[3], t[4]]


def parallel_partition(B, C, K, W, H, R, S, sw, sh, M, p):
    """Brute force over all (aB, aK, aH, aW) with aX <= X and product <= p.  Reading (the paper only
    says "choose those values in order to minimize"): use as many processors as the output allows
    (largest product first), then the smallest bound, then the least replicated traffic (terms 2+3),
    then the lexicographically smallest tuple.  Returns ((aB, aK, aH, aW), bound)."""
    best = None
    for aB in range(1, min(B, p) + 1):
        for aK in range(1, min(K, p // aB) + 1):
            for aH in range(1, min(H, p // (aB * aK)) + 1):
                for aW in range(1, min(W, p // (aB * aK * aH)) + 1):
                    t = parallel_terms(B, C, K, W, H, R, S, sw, sh, M, aB, aK, aH, aW)
                    key = (-(aB * aK * aH * aW), max(t), t[1] + t[2], (aB, aK, aH, aW))
                    if best is None or key < best:
                        best = key
    return best[3], best[1]


def tiling_lp(B, C, K, W, H, R, S, sw, sh, M, pooling=False):
    """Solve the Section-5 LP at the concrete parameters.

    Variables are log_M of the nine block sizes (b_b, b_c, b_k, b_w, b_h, b_r', b_r'', b_s', b_s'').
    Returns (tiles dict, G = product of block sizes, cost = F*M/G).
    ``pooling=True`` drops the Filter constraint (Section 6).
    """
    L = lambda x: math.log(x) / math.log(M)
    n = len(VARS)
    ix = {v: i for i, v in enumerate(VARS)}
    A, ub = [], []

    def row(names, rhs=1.0):
        a = [0.0] * n
        for v in names:
            a[ix[v]] = 1.0
        A.append(a)
        ub.append(rhs)

    row(["b", "k", "w", "h"])                              # Out block
    if not pooling:
        row(["c", "k", "r1", "r2", "s1", "s2"])            # Filter block
    row(["b", "c", "w", "h", "r2", "s2"])                  # Image block, four cross terms
    row(["b", "c", "w", "s1", "r2", "s2"])
    row(["b", "c", "r1", "h", "r2", "s2"])
    row(["b", "c", "r1", "s1", "r2", "s2"])
    bounds = [
        (0.0, L(B)), (0.0, L(C)), (0.0, L(K)), (0.0, L(W)), (0.0, L(H)),
        (0.0, max(0.0, L(R) - L(sw))), (0.0, L(sw)),
        (0.0, max(0.0, L(S) - L(sh))), (0.0, L(sh)),
    ]
    res = linprog([-1.0] * n, A_ub=A, b_ub=ub, bounds=bounds, method="highs")
    if res.status != 0:
        raise RuntimeError(res.message)
    logs = res.x
    tiles = {v: M ** logs[i] for i, v in enumerate(VARS)}
    G = M ** float(sum(logs))
    F = B * C * K * W * H * R * S
    return tiles, G, F * M / G


def tiling_cost(F, M, block_sizes):
    """Words moved by a tiling whose blocks fit in M: (F/G) outer iterations times M words each."""
    G = 1.0
    for b in block_sizes:
        G *= b
    return F * M / G


def theorem2_case(B, C, K, W, H, R, S, M):
    """Leaf of the stride-1 decision tree (Theorem 2) and its attainable-lower-bound expression."""
    CHWB, KCRS, KHWB = C * H * W * B, K * C * R * S, K * H * W * B
    if min(CHWB, KCRS, KHWB) <= M:
        return "1", float(max(CHWB, KCRS, KHWB))
    if R * S >= M:
        return "2.1", K * C * H * W * B * R * S / M
    if M * R * S >= (B * H * W) ** 2:
        return "2.2.1", float(KCRS)
    if min(C, K) >= math.sqrt(M / (R * S)):
        return "2.2.2.1", K * C * H * W * B * math.sqrt(R * S / M)
    return "2.2.2.2", float(max(KHWB, CHWB))


def hbl_lp_value():
    """min s1+s2+s3 subject to the four inequalities that close Section 4.2."""
    A = [[-1, -1, 0], [-1, 0, -1], [0, -1, -1], [-1, -1, -1]]
    b = [-1, -1, -1, -2]
    res = linprog([1, 1, 1], A_ub=A, b_ub=b, bounds=[(0, None)] * 3, method="highs")
    return float(res.fun)
