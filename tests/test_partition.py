"""Hybrid-aware sequence chunking (paper Section 3.2, Eq. 9-11): pins of the oracle (oracle/partition.py), then the
library's host function against the oracle.  CPU only."""
import ctypes
import math
import os
import random
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import partition as P  # noqa: E402


# ---- the oracle against what the equations fix -------------------------------------------------------------------

@pytest.mark.parametrize("N", [1, 2, 4, 6, 8, 16, 32])
def test_no_softmax_work_gives_equal_lengths(N):
    # Cost_i = W_tok * s_i when W_soft = 0: equal costs are equal lengths
    b = P.hybrid_boundaries(65536.0, N, 3.0, 0.0)
    for i, c in enumerate(b):
        assert abs(c - i * 65536.0 / N) < 1e-6
    if 65536 % (N * 128) == 0:
        assert P.partition(65536, N, 3.0, 0.0, 1.0) == [65536 // N] * N


@pytest.mark.parametrize("N", [2, 4, 8, 32])
def test_alpha_zero_is_the_equal_partition_whatever_the_costs(N):
    assert P.partition(131072, N, 1.0, 5e-4, 0.0) == [131072 // N] * N


def test_two_segments_by_hand():
    # N = 2: W_tok*c + W_soft*c^2/2 = (W_tok*T + W_soft*T^2/2) / 2 -- the quadratic solved here independently
    T, wt, ws = 1000.0, 2.0, 0.01
    half = 0.5 * (wt * T + 0.5 * ws * T * T)
    c1 = (-wt + math.sqrt(wt * wt + 2.0 * ws * half)) / ws
    b = P.hybrid_boundaries(T, 2, wt, ws)
    assert abs(b[1] - c1) < 1e-6
    # and the two costs of Eq. 9 agree
    assert abs(P.chunk_cost(0.0, c1, wt, ws) - P.chunk_cost(c1, T - c1, wt, ws)) < 1e-6


def test_pure_softmax_cost_has_square_root_boundaries():
    # W_tok = 0: the cost of a prefix is proportional to c^2, so c_i = T * sqrt(i / N)
    T, N = 4096.0, 8
    b = P.hybrid_boundaries(T, N, 0.0, 1.0)
    for i in range(N + 1):
        assert abs(b[i] - T * math.sqrt(i / N)) < 1e-6


@pytest.mark.parametrize("seed", range(5))
def test_costs_are_equal_and_lengths_decrease(seed):
    rng = random.Random(seed)
    T = float(rng.choice([32768, 65536, 262144]))
    N = rng.choice([2, 4, 6, 8, 16, 32])
    wt, ws = rng.uniform(0.5, 4.0), rng.uniform(1e-6, 1e-3)
    b = P.hybrid_boundaries(T, N, wt, ws)
    costs = [P.chunk_cost(b[i], b[i + 1] - b[i], wt, ws) for i in range(N)]
    assert max(costs) - min(costs) < 1e-7 * max(costs)
    lens = [b[i + 1] - b[i] for i in range(N)]
    assert all(lens[i] > lens[i + 1] for i in range(N - 1))          # later segments attend to longer prefixes
    assert abs(sum(lens) - T) < 1e-6
    # the total is the cost of the whole sequence as one segment
    assert abs(sum(costs) - P.chunk_cost(0.0, T, wt, ws)) < 1e-7 * sum(costs)


def test_interpolation_and_rounding():
    T, N = 65536, 8
    for alpha in (0.0, 0.3, 1.0, 1.25):
        lens = P.partition(T, N, 1.0, 2e-4, alpha)
        assert sum(lens) == T and all(s % 128 == 0 and s >= 128 for s in lens)
    # alpha = 1/2 lies halfway between the two boundary sets before rounding
    eq = [i * T / N for i in range(N + 1)]
    hy = P.hybrid_boundaries(float(T), N, 1.0, 2e-4)
    mid = P.candidate_boundaries(float(T), N, 1.0, 2e-4, 0.5)
    assert all(abs(mid[i] - 0.5 * (eq[i] + hy[i])) < 1e-9 for i in range(N + 1))
    # rounding: closest multiple, ties up
    assert P.round_boundaries([0.0, 191.9, 192.0, 600.0, 1024.0], 1024, 128) == [0, 128, 256, 640, 1024]


def test_rounding_keeps_every_segment_alive_or_rejects():
    # boundaries that collapse after rounding are pushed apart
    assert P.round_boundaries([0.0, 10.0, 20.0, 30.0, 1024.0], 1024, 128) == [0, 128, 256, 384, 1024]
    assert P.round_boundaries([0.0, 1000.0, 1010.0, 1020.0, 1024.0], 1024, 128) == [0, 640, 768, 896, 1024]
    with pytest.raises(ValueError):
        P.round_boundaries([0.0, 100.0, 200.0, 300.0, 384.0], 384, 128)


# ---- the library's host function against the oracle ---------------------------------------------------------------

@pytest.fixture(scope="module")
def binding():
    from paper_2608_06838_b200 import binding as b, build
    build.build()
    return b


def _near_tie(T, N, wt, ws, alpha, multiple):
    cand = P.candidate_boundaries(float(T), N, wt, ws, alpha)
    return any(abs((c / multiple) % 1.0 - 0.5) < 1e-6 for c in cand[1:N])


def test_library_matches_the_oracle_on_the_paper_grid(binding):
    # N and alpha values the paper profiles (Section 3.2), model-like weights
    for T in (65536, 262144):
        for N in (2, 4, 6, 8, 16, 32):
            for alpha in (0.0, 0.1, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 1.0, 1.25):
                for ws in (3e-5, 4e-4):
                    if _near_tie(T, N, 1.0, ws, alpha, 128):
                        continue
                    assert binding.sf_partition_hybrid(T, N, 1.0, ws, alpha, 128) == P.partition(T, N, 1.0, ws, alpha, 128), \
                        (T, N, alpha, ws)


@pytest.mark.parametrize("seed", range(40))
def test_library_matches_the_oracle_on_random_cases(binding, seed):
    rng = random.Random(1000 + seed)
    multiple = rng.choice([1, 64, 128, 256])
    N = rng.randint(1, 32)
    T = multiple * rng.randint(N, 40 * N) + (rng.randint(0, multiple - 1) if seed % 4 == 0 else 0)
    wt = rng.choice([0.0, rng.uniform(0.1, 5.0)])
    ws = rng.uniform(1e-6, 1e-2) if wt == 0.0 or seed % 3 else 0.0
    alpha = rng.choice([0.0, 1.0, 1.25, rng.uniform(-0.5, 2.0)])
    if _near_tie(T, N, wt, ws, alpha, multiple):
        pytest.skip("rounding tie within 1e-6: both neighbours are correct")
    try:
        ref = P.partition(T, N, wt, ws, alpha, multiple)
    except ValueError:
        with pytest.raises(binding.SfError):
            binding.sf_partition_hybrid(T, N, wt, ws, alpha, multiple)
        return
    got = binding.sf_partition_hybrid(T, N, wt, ws, alpha, multiple)
    assert got == ref
    assert sum(got) == T and min(got) >= multiple


def test_library_rejects_bad_arguments(binding):
    lib = binding.load()
    out = (ctypes.c_int32 * 8)()
    ok = dict(T=65536, N=8, w_tok=1.0, w_soft=1e-4, alpha=1.0, multiple=128)

    def call(**kw):
        a = dict(ok, **kw)
        return lib.sf_partition_hybrid(a["T"], a["N"], a["w_tok"], a["w_soft"], a["alpha"], a["multiple"], kw.get("out", out))

    assert call() == 0
    for bad in (dict(T=0), dict(N=0), dict(multiple=0), dict(w_tok=-1.0), dict(w_soft=-1e-3), dict(w_tok=0.0, w_soft=0.0),
                dict(alpha=float("nan")), dict(alpha=float("inf")), dict(w_tok=float("nan")), dict(T=512, N=8),
                dict(out=None)):
        assert call(**bad) == 1, bad


def test_partition_feeds_the_chain_driver(binding):
    # lengths are multiples of 128, hence of the chunk size: the chain driver accepts them as they are
    lens = binding.sf_partition_hybrid(65536, 8, 1.0, 2e-4, 1.0)
    from paper_2608_06838_b200.binding import SegDesc, SF_BF16
    d = SegDesc(1, 32, 128, 128, lens[0], 64, SF_BF16, 0, 32 * 128, 32 * 128, 32, 0, 0, 0)
    assert binding.sf_chain_workspace_bytes(d, lens, 0) > 0
    assert lens == sorted(lens, reverse=True) and sum(lens) == 65536
