"""TEST INFRASTRUCTURE: hybrid-aware sequence chunking, written out from its definition (paper Section 3.2).

A sequence of T tokens is cut at boundaries 0 = c_0 < c_1 < ... < c_N = T; segment i has length s_i = c_{i+1} - c_i and

    Cost_i = W_tok * s_i + W_soft * (c_i * s_i + s_i^2 / 2)            (Eq. 9, W_tok = L_lin*C_lin + C_dense,
                                                                         W_soft = L_soft*C_soft)
The FLOP-balanced ("hybrid") boundaries make all Cost_i equal (Eq. 10).  Candidates interpolate between the equal-length
boundaries i*T/N and the hybrid ones,  c_i(alpha) = (1 - alpha) * i*T/N + alpha * c_i^hybrid  (Eq. 11), and are rounded
to the closest multiple of 128.

This file follows those three equations literally and slowly: the common cost is found by bisection, and each
boundary by another bisection on Eq. 9.  It uses no closed form.  Readings where the paper is silent: a tie in the
rounding goes up; c_N stays T; after rounding, boundaries are pushed apart so that every segment keeps at least one
multiple (forward pass, then backward pass); if that is impossible the partition is rejected.

Only tests may import this module.  Pinned in tests/test_partition.py (equal lengths for W_soft = 0 or alpha = 0,
equal costs, the N = 2 quadratic by hand, monotonicity).
"""
from __future__ import annotations

import math
from typing import List


def chunk_cost(c: float, s: float, w_tok: float, w_soft: float) -> float:
    """Eq. 9 for a segment that starts at token c and has s tokens."""
    return w_tok * s + w_soft * (c * s + 0.5 * s * s)


def _length_for_cost(c: float, kappa: float, w_tok: float, w_soft: float, hi: float) -> float:
    lo_s, hi_s = 0.0, hi
    for _ in range(200):
        mid = 0.5 * (lo_s + hi_s)
        if chunk_cost(c, mid, w_tok, w_soft) < kappa:
            lo_s = mid
        else:
            hi_s = mid
    return 0.5 * (lo_s + hi_s)


def hybrid_boundaries(T: float, N: int, w_tok: float, w_soft: float) -> List[float]:
    """Real-valued boundaries c_0..c_N with Cost_0 = ... = Cost_{N-1} (Eq. 10)."""
    if N < 1 or T <= 0 or w_tok < 0 or w_soft < 0 or (w_tok == 0 and w_soft == 0):
        raise ValueError("bad arguments")

    def end_of_walk(kappa: float) -> float:
        c = 0.0
        for _ in range(N):
            c += _length_for_cost(c, kappa, w_tok, w_soft, 2.0 * T)
        return c

    lo_k, hi_k = 0.0, chunk_cost(0.0, float(T), w_tok, w_soft)          # one segment holding everything
    for _ in range(200):
        mid = 0.5 * (lo_k + hi_k)
        if end_of_walk(mid) < T:
            lo_k = mid
        else:
            hi_k = mid
    kappa = 0.5 * (lo_k + hi_k)
    bounds = [0.0]
    for _ in range(N - 1):
        bounds.append(bounds[-1] + _length_for_cost(bounds[-1], kappa, w_tok, w_soft, 2.0 * T))
    bounds.append(float(T))
    return bounds


def candidate_boundaries(T: float, N: int, w_tok: float, w_soft: float, alpha: float) -> List[float]:
    """Eq. 11 before rounding."""
    hyb = hybrid_boundaries(T, N, w_tok, w_soft)
    return [(1.0 - alpha) * (i * T / N) + alpha * hyb[i] for i in range(N + 1)]


def round_boundaries(bounds: List[float], T: int, multiple: int) -> List[int]:
    """Closest multiple (ties up), c_0 = 0 and c_N = T kept, every segment at least one multiple long."""
    N = len(bounds) - 1
    r = [0] + [int(math.floor(b / multiple + 0.5)) * multiple for b in bounds[1:N]] + [int(T)]
    for i in range(1, N):
        r[i] = max(r[i], r[i - 1] + multiple)
    for i in range(N - 1, 0, -1):
        r[i] = min(r[i], r[i + 1] - multiple)
    if N > 1 and r[1] < multiple:
        raise ValueError("T is too short for N segments of at least one multiple")
    if N == 1 and T < multiple:
        raise ValueError("T is shorter than one multiple")
    return r


def partition(T: int, N: int, w_tok: float, w_soft: float, alpha: float, multiple: int = 128) -> List[int]:
    """Segment lengths s_0..s_{N-1} of the candidate partition (Eq. 9-11 with rounding)."""
    r = round_boundaries(candidate_boundaries(float(T), N, w_tok, w_soft, alpha), T, multiple)
    return [r[i + 1] - r[i] for i in range(N)]
