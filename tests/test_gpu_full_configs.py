"""The benchmark configurations at full size, in the launch configurations bench.py times, checked on sampled
heads against the unsplit fp64 oracle: direct launches with the library's block-length model, and - what the
benchmark's timed region runs - the chain recorded as a CUDA graph after profile-guided tuning of the block length,
replayed, with the default schedule and with the merged-launch schedule the schedule search may install."""
import numpy as np
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def graph_run(w, x):
    """The benchmark's way: tune the block length on the caller's buffers, record the chain as a graph, replay it."""
    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
    # the inputs were generated on the default stream; the side stream below does not wait for it by itself
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run.autotune(x["S_in"], x["dS_out"], [0, 22, 32, 64], reps=2)
        run.capture(x["S_in"], x["dS_out"])
        for t in (run.o, run.dq, run.dk, run.dv, run.dg, run.dS_init, run.S_bounds):
            t.zero_()
        run.replay()
    stream.synchronize()
    assert binding.sf_device_status() == 0
    got = dict(o=run.o, S_out=run.S_bounds[-1], dq=run.dq, dk=run.dk, dv=run.dv, dg=run.dg, dS_in=run.dS_init)
    return got, run


def sampled_check(w, heads, mode="direct"):
    if mode == "graph-merged":
        binding.sf_set_tuning(dict(merge_launches=1))
        try:
            sampled_check(w, heads, "graph")
        finally:
            binding.sf_set_tuning(None)
        return
    x = inputs.make_inputs(w, DEV)
    if mode == "graph":
        got, run = graph_run(w, x)
        ref = oracle_reference(x, heads=heads)
        errs = compare(got, ref, tolerance(w), heads=heads, label=w.name + "/graph")
        print(w.name, "graph, block length", int(run.desc.chunks_per_block), "heads", heads, {k: "%.2e" % v for k, v in errs.items()})
        first = {n: got[n].clone() for n in ("o", "dg", "dS_in")}
        with torch.cuda.stream(torch.cuda.Stream()):
            run.replay()
        torch.cuda.synchronize()
        assert torch.equal(first["o"], run.o) and torch.equal(first["dg"], run.dg) and torch.equal(first["dS_in"], run.dS_init)
        run.release()
        del run, got, x
        torch.cuda.empty_cache()
        return
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


@pytest.mark.parametrize("mode", ["direct", "graph", "graph-merged"])
def test_config2_32k(mode):
    sampled_check(inputs.configs()[1], [0, 15], mode)


@pytest.mark.parametrize("mode", ["direct", "graph", "graph-merged"])
def test_config3_64k_nonuniform(mode):
    sampled_check(inputs.configs()[2], [3, 31], mode)


@pytest.mark.parametrize("mode", ["direct", "graph", "graph-merged"])
def test_config4_256k(mode):
    sampled_check(inputs.configs()[3], [17], mode)


@pytest.mark.parametrize("mode", ["direct", "graph-merged"])
@pytest.mark.parametrize("seg_len", [512, 16384])
def test_config5_sweep_ends(seg_len, mode):
    sampled_check(inputs.sweep_config(seg_len), [39], mode)


@pytest.mark.parametrize("H,d", [(256, 128), (512, 64)])
def test_tensors_beyond_two_to_the_31_elements(H, d):
    """Maximum sizes: every [T, H, d] tensor holds more than 2^31 elements (4.4 GB in bf16), so element and byte
    offsets that were kept in 32 bits anywhere would wrap.  Many heads keep the per-head oracle run short; the last
    head sits at the largest offsets of every token row, the last segment at the largest of the sequence.  d = 128
    runs on the tensor-core kernels, d = 64 on the CUDA-core ones."""
    w = inputs.Workload("beyond-2^31-d%d" % d, 1, H, d, d, [16384, 16384, 16384, 16512], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=31)
    assert w.T * w.H * w.d_k > 2 ** 31
    heads = [0, H - 1]
    x = inputs.make_inputs(w, DEV)
    ref = oracle_reference(x, heads=heads)
    for merged in (0, 1):
        binding.sf_set_tuning(dict(merge_launches=merged))
        try:
            got, run = run_chain(w, x)
        finally:
            binding.sf_set_tuning(None)
        compare(got, ref, tolerance(w), heads=heads, label="%s/merged=%d" % (w.name, merged))
        for n in ("o", "dq", "dk", "dv"):
            tail = got[n][:, -4096:]                           # cheap whole-width look at the far end of the buffers
            assert torch.isfinite(tail.float()).all() and float(tail.float().abs().max()) > 0, n
        del run, got
        torch.cuda.empty_cache()
