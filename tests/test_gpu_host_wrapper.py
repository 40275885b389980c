"""The host-memory entry point (inputs and results in host buffers, copies pipelined against the chain) vs the fp64
oracle, through the C ABI (one B200)."""
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_host(w, x, pinned=True, want_final=True, chunks_per_block=0):
    place = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    host = {n: (None if t is None else place(t.detach().to("cpu"))) for n, t in x.items()}
    outs = {n: place(torch.full_like(host[m], float("nan"))) for n, m in
            [("o", "v"), ("dq", "q"), ("dk", "k"), ("dv", "v"), ("dg", "g")]}
    S_final = place(torch.full((w.B, w.H, w.d_k, w.d_v), float("nan"), dtype=torch.float32)) if want_final else None
    dS_init = place(torch.full((w.B, w.H, w.d_k, w.d_v), float("nan"), dtype=torch.float32))
    desc = binding.make_desc(host["q"], host["v"], host["g"], w.chunk, chunks_per_block, seg_len=w.seg_lens[0])
    need = binding.sf_e2e_device_bytes(desc, w.seg_lens)
    assert need > 0
    scratch = torch.empty(need, dtype=torch.uint8, device=DEV)
    binding.sf_chain_fwd_bwd_host(desc, w.seg_lens, host["q"], host["k"], host["v"], host["g"], host["S_in"], host["dO"],
                                  host["dS_out"], outs["o"], S_final, outs["dq"], outs["dk"], outs["dv"], outs["dg"], dS_init,
                                  scratch)
    assert binding.sf_device_status() == 0
    return dict(o=outs["o"], S_out=S_final, dq=outs["dq"], dk=outs["dk"], dv=outs["dv"], dg=outs["dg"], dS_in=dS_init), desc


@pytest.mark.parametrize("pinned", [True, False])
def test_host_wrapper_fp32_batched_nonuniform_segments(pinned):
    # B = 2: a segment is two separate slices of every tensor
    w = Workload("host-f32", 2, 3, 32, 64, [128, 224, 32, 96], 32, dtype="f32", g_scale=0.2, s_in_sigma=0.4, ds_out_sigma=0.4, seed=21)
    x = inputs.make_inputs(w, DEV)
    got, _ = run_host(w, x, pinned=pinned)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


@pytest.mark.parametrize("segs", [[256, 640, 200], [1024], [64, 64, 64, 64, 64]])
def test_host_wrapper_bf16_tensor_core_path(segs):
    w = Workload("host-bf16-%d" % len(segs), 1, 2, 128, 128, segs, 64, g_scale=0.3, s_in_sigma=0.02, ds_out_sigma=0.02, seed=22)
    x = inputs.make_inputs(w, DEV)
    got, _ = run_host(w, x)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 32)])
def test_host_wrapper_segments_that_start_at_odd_tokens(dtype, d):
    # inner segments of 87, 1 and 15 tokens with one head: the later segments' g and dg start at addresses that are
    # only 4-byte aligned, as inside any chain
    w = Workload("host-odd-%s" % dtype, 2, 1, d, d, [512, 87, 1, 320, 15], 64, dtype=dtype, g_scale=0.1, s_in_sigma=0.3, ds_out_sigma=0.3, seed=26)
    x = inputs.make_inputs(w, DEV)
    got, _ = run_host(w, x)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


def test_host_wrapper_without_boundary_inputs_and_without_final_state():
    w = Workload("host-noinit", 1, 2, 64, 64, [192, 128], 32, dtype="f32", g_scale=0.1, seed=23)
    x = inputs.make_inputs(w, DEV)
    assert x["S_in"] is None and x["dS_out"] is None
    got, _ = run_host(w, x, want_final=False)
    ref = oracle_reference(x)
    got["S_out"] = torch.from_numpy(ref["S_out"]).float()         # not requested: nothing to compare
    compare(got, ref, tolerance(w), label=w.name)


def test_host_wrapper_equals_the_device_chain_run_segment_by_segment():
    # the wrapper runs every segment as a one-segment chain in order: the same launches as a chain without overlap,
    # hence the same bits, when the block length is given
    w = Workload("host-bits", 1, 2, 64, 64, [256, 128, 384], 32, dtype="f32", g_scale=0.1, s_in_sigma=0.3, ds_out_sigma=0.3, seed=24)
    x = inputs.make_inputs(w, DEV)
    base, _ = run_chain(w, x, chunks_per_block=2, overlap=False)
    got, _ = run_host(w, x, chunks_per_block=2)
    for n in base:
        assert torch.equal(base[n].cpu(), got[n]), n


def test_host_wrapper_rejects_short_scratch_before_copying():
    w = Workload("host-short", 1, 2, 64, 64, [128, 128], 32, dtype="f32", seed=25)
    x = inputs.make_inputs(w, DEV)
    host = {n: (None if t is None else t.detach().to("cpu")) for n, t in x.items()}
    o = torch.full_like(host["v"], 7.0)
    dq, dk, dv, dg = (torch.zeros_like(host[n]) for n in ("q", "k", "v", "g"))
    dS = torch.zeros(w.B, w.H, w.d_k, w.d_v)
    desc = binding.make_desc(host["q"], host["v"], host["g"], w.chunk, 0, seg_len=w.seg_lens[0])
    scratch = torch.empty(binding.sf_e2e_device_bytes(desc, w.seg_lens) - 256, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.SfError) as ei:
        binding.sf_chain_fwd_bwd_host(desc, w.seg_lens, host["q"], host["k"], host["v"], host["g"], None, host["dO"], None, o, None,
                                      dq, dk, dv, dg, dS, scratch)
    assert ei.value.code == 3          # SF_ERR_WORKSPACE
    assert bool((o == 7.0).all())
