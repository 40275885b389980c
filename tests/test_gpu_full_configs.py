"""The benchmark configurations at full size, in the launch configuration bench.py times (overlap on,
saved block states, default block length), checked on sampled heads against the unsplit fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def sampled_check(w, heads):
    x = inputs.make_inputs(w, DEV)
    got, run = run_chain(w, x)
    ref = oracle_reference(x, heads=heads)
    errs = compare(got, ref, tolerance(w), heads=heads, label=w.name)
    print(w.name, "heads", heads, {k: "%.2e" % v for k, v in errs.items()})
    # properties that hold at any size: everything finite, and a rerun reproduces the same bits
    first = {n: t.clone() for n, t in got.items() if n in ("o", "dg", "dS_in")}
    for n, t in got.items():
        assert torch.isfinite(t.float()).all(), n
    run.forward(x["S_in"])
    run.backward(x["dS_out"])
    torch.cuda.synchronize()
    assert torch.equal(first["o"], run.o) and torch.equal(first["dg"], run.dg) and torch.equal(first["dS_in"], run.dS_init)
    del run, got, x
    torch.cuda.empty_cache()


def test_config2_32k():
    sampled_check(inputs.configs()[1], [0, 15])


def test_config3_64k_nonuniform():
    sampled_check(inputs.configs()[2], [3, 31])


def test_config4_256k():
    sampled_check(inputs.configs()[3], [17])


@pytest.mark.parametrize("seg_len", [512, 16384])
def test_config5_sweep_ends(seg_len):
    sampled_check(inputs.sweep_config(seg_len), [39])
