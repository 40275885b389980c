"""bf16, d_k = d_v = 128, chunk 64 (the tcgen05 path) vs the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check(w, **kw):
    x = inputs.make_inputs(w, DEV)
    got, _ = run_chain(w, x, **kw)
    ref = oracle_reference(x)
    errs = compare(got, ref, tolerance(w), label=w.name)
    print(w.name, {k: "%.2e" % v for k, v in errs.items()})
    return errs


@pytest.mark.parametrize("g_scale", [1.0, 0.1, 0.01, 0.0])
def test_decay_regimes(g_scale):
    # several blocks per segment, a ragged last block (17 chunks with 4 per block), three segments
    w = Workload("bf16-128-g%g" % g_scale, 1, 3, 128, 128, [17 * 64, 8 * 64, 64], 64, g_scale=g_scale,
                 s_in_sigma=0.02, ds_out_sigma=0.02, seed=1)
    check(w, chunks_per_block=4)


def test_default_block_and_batch():
    w = Workload("bf16-128-b2", 2, 2, 128, 128, [2048, 1024], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=2)
    check(w)


def test_mixed_heads_strong_and_zero_decay():
    w = Workload("bf16-128-mixed", 1, 4, 128, 128, [1024, 1024], 64, seed=4, s_in_sigma=0.02)
    x = inputs.make_inputs(w, DEV)
    x["g"][:, :, 1] = 0.0
    x["g"][:, :, 3] *= 0.001
    x["g"][:, 700, 2] = -100.0          # one token that wipes the state of head 2
    got, _ = run_chain(w, x, chunks_per_block=8)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


def test_single_chunk_segments():
    w = Workload("bf16-128-1chunk", 1, 2, 128, 128, [64, 64, 128], 64, g_scale=0.05, s_in_sigma=0.1, ds_out_sigma=0.1, seed=6)
    check(w)


def test_chain_on_a_hybrid_aware_partition():
    # non-uniform, decreasing segment lengths as Section 3.2 (Eq. 9-11) produces them
    lens = binding.sf_partition_hybrid(4096, 4, 1.0, 1e-3, 1.0)
    assert sum(lens) == 4096 and lens == sorted(lens, reverse=True) and lens[0] > lens[-1]
    w = Workload("bf16-128-hybrid", 1, 2, 128, 128, lens, 64, g_scale=0.05, s_in_sigma=0.02, ds_out_sigma=0.02, seed=9)
    check(w)
