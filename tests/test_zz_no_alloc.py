"""sf_segment_fwd_static: the forward entry point for callers that cannot allocate device memory.

Such callers (code inside a CUDA-graph capture or under an allocation-free memory pool, plug-ins that
are handed only input and output pointers, real-time loops) cannot provide a workspace, so the library
keeps a fixed scratch array of its own.  The test calls the entry point through the C ABI twice in a
row, with different inputs, and checks each result against sf_segment_fwd run with a caller-owned
workspace: the second call must not be disturbed by what the first one left in the shared scratch.
The two entry points run the same kernels, so their results must agree bit for bit (which also
satisfies the tolerance the parity tests use); one case is compared with the fp64 oracle as well, and
the free device memory must not change across a call.
This file sorts last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(w, x):
    q, k, v, g = x["q"], x["k"], x["v"], x["g"]
    desc = binding.make_desc(q, v, g, w.chunk)
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    ws = torch.empty(max(binding.sf_workspace_bytes(desc, 0), 256), dtype=torch.uint8, device=DEV)
    o_ref, S_ref = torch.empty_like(v), torch.empty(B, H, dk, dv, dtype=torch.float32, device=DEV)
    binding.sf_segment_fwd(desc, q, k, v, g, x["S_in"], o_ref, S_ref, ws)
    o, S = torch.empty_like(v), torch.empty_like(S_ref)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    binding.sf_segment_fwd_static(desc, q, k, v, g, x["S_in"], o, S)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
    assert binding.sf_device_status() == 0
    return (o, S), (o_ref, S_ref)


def _close(a, r, tol):
    a, r = a.double(), r.double()
    return float((a - r).abs().max() / r.abs().max().clamp_min(1e-30)) <= tol


@pytest.mark.parametrize("dtype,d,chunk,tol", [("bf16", 128, 64, 2e-2), ("f32", 64, 32, 1e-4)])
def test_two_calls_in_a_row_match_the_workspace_entry_point(dtype, d, chunk, tol):
    first = Workload("na-1", 1, 4, d, d, [32 * chunk], chunk, dtype=dtype, g_scale=0.05, s_in_sigma=0.1, seed=21)
    second = Workload("na-2", 2, 3, d, d, [19 * chunk], chunk, dtype=dtype, g_scale=1.0, seed=22)
    for w in (first, second):
        x = inputs.make_inputs(w, DEV)
        (o, S), (o_ref, S_ref) = _both(w, x)
        assert torch.isfinite(o.float()).all() and torch.isfinite(S).all()
        assert _close(o, o_ref, tol) and _close(S, S_ref, tol), w.name
        assert torch.equal(o, o_ref) and torch.equal(S, S_ref), w.name      # same kernels, same bits
        f = inputs.to_f64
        o_or, S_or = oracle.segment_fwd(f(x["q"]), f(x["k"]), f(x["v"]), f(x["g"]), f(x["S_in"]))
        for got, ref in ((o, o_or), (S, S_or)):
            err = np.abs(f(got) - ref).max() / max(np.abs(ref).max(), 1e-30)
            assert err <= tol, (w.name, err)


def test_shapes_beyond_the_static_scratch_are_rejected():
    w = Workload("na-big", 1, 64, 128, 128, [64 * 64], 64, seed=23)      # 64 heads x 4 blocks x 64 KB = 16 MiB + totals
    x = inputs.make_inputs(w, DEV)
    desc = binding.make_desc(x["q"], x["v"], x["g"], w.chunk, chunks_per_block=16)
    assert binding.sf_workspace_bytes(desc, 0) > binding.SF_STATIC_SCRATCH_BYTES
    o = torch.empty_like(x["v"])
    S = torch.empty(1, 64, 128, 128, dtype=torch.float32, device=DEV)
    with pytest.raises(binding.SfError) as e:
        binding.sf_segment_fwd_static(desc, x["q"], x["k"], x["v"], x["g"], None, o, S)
    assert e.value.code == 3


def test_a_call_recorded_in_a_stream_capture_replays_to_the_same_bits():
    # the use the entry point exists for: no allocation, no synchronisation, nothing the capture cannot record
    w = Workload("na-capture", 1, 4, 128, 128, [16 * 64], 64, g_scale=0.1, s_in_sigma=0.1, seed=24)
    x = inputs.make_inputs(w, DEV)
    (_, _), (o_ref, S_ref) = _both(w, x)          # a first call outside any capture resolves the scratch address
    desc = binding.make_desc(x["q"], x["v"], x["g"], w.chunk)
    o, S = torch.zeros_like(o_ref), torch.zeros_like(S_ref)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        binding.sf_segment_fwd_static(desc, x["q"], x["k"], x["v"], x["g"], x["S_in"], o, S)
    torch.cuda.synchronize()
    assert not o.any() and not S.any()            # recording runs nothing
    for _ in range(2):
        o.zero_()
        S.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(o, o_ref) and torch.equal(S, S_ref)
    assert binding.sf_device_status() == 0
