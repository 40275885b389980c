"""The chain recorded as one CUDA graph gives bit-identical results to the direct calls."""
import numpy as np
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import NAMES, compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("overlap", [True, False])
def test_graph_replay_matches_direct_calls(overlap):
    w = Workload("graph", 1, 3, 128, 128, [1024, 512, 512, 256], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=11)
    x = inputs.make_inputs(w, DEV)
    direct, _ = run_chain(w, x, overlap=overlap)
    direct = {n: direct[n].clone() for n in NAMES}

    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        kernels = run.capture(x["S_in"], x["dS_out"], overlap=overlap)
        # per segment: aggregate, sweep; aggregate, dq, dk/dv, dg = 6 kernels, plus the scans (one per group of short
        # neighbouring segments when the streams overlap, one per segment otherwise)
        assert 6 * len(w.seg_lens) + 2 <= kernels <= 8 * len(w.seg_lens)
        for t in (run.o, run.dq, run.dk, run.dv, run.dg, run.dS_init, run.S_bounds):
            t.zero_()
        before = binding.sf_launch_count()
        run.replay()
        run.replay()
        assert binding.sf_launch_count() - before == 2 * kernels
    stream.synchronize()
    assert binding.sf_device_status() == 0
    got = dict(o=run.o, S_out=run.S_bounds[-1], dq=run.dq, dk=run.dk, dv=run.dv, dg=run.dg, dS_in=run.dS_init)
    for n in NAMES:
        assert torch.equal(got[n], direct[n]), n
    compare(got, oracle_reference(x), tolerance(w), label="graph")
    run.release()


def test_graph_needs_a_capturable_stream():
    w = Workload("graph-legacy", 1, 2, 128, 128, [256], 64, seed=12)
    x = inputs.make_inputs(w, DEV)
    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
    with pytest.raises(binding.SfError):
        run.capture(None, None, stream=torch.cuda.default_stream())


def test_autotune_picks_a_candidate_and_results_stay_correct():
    w = Workload("tune", 1, 4, 128, 128, [2048, 1024, 1024], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=13)
    x = inputs.make_inputs(w, DEV)
    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
    cands = [0, 4, 8, 16, 65]                      # 65 exceeds what the kernels support: skipped
    best, ms = run.autotune(x["S_in"], x["dS_out"], cands, reps=2)
    assert best in cands[:4] and run.desc.chunks_per_block == best
    assert ms[4] == -1.0 and all(t > 0 for t in ms[:4])
    assert ms[cands.index(best)] == min(t for t in ms if t > 0)
    run.forward(x["S_in"])
    run.backward(x["dS_out"])
    torch.cuda.synchronize()
    got = dict(o=run.o, S_out=run.S_bounds[-1], dq=run.dq, dk=run.dk, dv=run.dv, dg=run.dg, dS_in=run.dS_init)
    compare(got, oracle_reference(x), tolerance(w), label="autotuned")


@pytest.mark.parametrize("tuning", [dict(sweep_streams=1, agg_streams=1), dict(sweep_streams=2, agg_ahead=1),
                                    dict(agg_ahead=2, scan_group_tokens=0), dict(agg_inorder_ctas=1, agg_ahead=3),
                                    dict(scan_group_tokens=100000, sweep_streams=3)])
def test_every_schedule_gives_the_bits_of_the_default_one(tuning):
    # the schedule (streams, scan grouping, how far the aggregates run ahead) only orders independent work
    w = Workload("tuning", 1, 3, 128, 128, [1024, 512, 512, 256, 768], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=17)
    x = inputs.make_inputs(w, DEV)
    binding.sf_set_tuning(None)
    ref, _ = run_chain(w, x)
    ref = {n: ref[n].clone() for n in NAMES}
    try:
        binding.sf_set_tuning(tuning)
        got, _ = run_chain(w, x)
        for n in NAMES:
            assert torch.equal(got[n], ref[n]), n
        # and recorded as a graph
        run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
        torch.cuda.synchronize()
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            run.capture(x["S_in"], x["dS_out"])
            run.replay()
        stream.synchronize()
        assert torch.equal(run.o, ref["o"]) and torch.equal(run.dg, ref["dg"]) and torch.equal(run.dS_init, ref["dS_in"])
        run.release()
    finally:
        binding.sf_set_tuning(None)
    assert binding.sf_device_status() == 0
    compare(ref, oracle_reference(x), tolerance(w), label="tuning")


def test_schedule_search_installs_a_valid_choice_and_results_do_not_change():
    w = Workload("sched", 1, 4, 128, 128, [2048, 1024, 1024, 512], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=19)
    x = inputs.make_inputs(w, DEV)
    binding.sf_set_tuning(None)
    ref, _ = run_chain(w, x)
    ref = {n: ref[n].clone() for n in NAMES}
    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    try:
        with torch.cuda.stream(stream):
            t, ms, default_ms = run.autotune_schedule(x["S_in"], x["dS_out"], reps=2, margin=0.02)
        stream.synchronize()
        assert ms > 0 and default_ms > 0 and ms <= default_ms
        assert t.sweep_streams in (2, 4) and t.agg_ahead in (0, 1, 2) and t.agg_inorder_ctas in (1, 74)
        now = binding.sf_get_tuning()
        assert (now.sweep_streams, now.agg_ahead, now.agg_inorder_ctas) == (t.sweep_streams, t.agg_ahead, t.agg_inorder_ctas)
        assert t.merge_launches in (0, 1) and now.merge_launches == t.merge_launches
        if (t.sweep_streams, t.agg_ahead, t.agg_inorder_ctas, t.merge_launches) != (4, 0, 74, 0):
            assert ms < default_ms / 1.02                   # the default is only left for a clear win
        got, _ = run_chain(w, x)
        if t.merge_launches:                                # other blocks than the segments' own: equal to rounding
            compare(got, oracle_reference(x), tolerance(w), label="sched-merged")
        else:
            for n in NAMES:
                assert torch.equal(got[n], ref[n]), n
    finally:
        binding.sf_set_tuning(None)
    assert binding.sf_device_status() == 0


@pytest.mark.parametrize("dtype,d,chunk,segs,cpb", [
    ("bf16", 128, 64, [1024, 512, 512, 2048, 300], 8),        # blocks of 8 chunks divide every segment but the ragged last one
    ("bf16", 128, 64, [2048, 2048, 2048], 16),
    ("f32", 64, 32, [256, 128, 384, 77], 4),                  # CUDA-core path
])
@pytest.mark.parametrize("save_states", [True, False])
def test_merged_launches_give_the_bits_of_the_segment_by_segment_run(dtype, d, chunk, segs, cpb, save_states):
    # one launch per stage over the whole chain: with the same block length the blocks, the kernels and the arithmetic are
    # the same, so the bits are; fewer launches
    w = Workload("merged", 2 if dtype == "f32" else 1, 3, d, d, segs, chunk, dtype=dtype, g_scale=0.1, s_in_sigma=0.02,
                 ds_out_sigma=0.02, seed=61)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    binding.sf_set_tuning(None)
    n0 = binding.sf_launch_count()
    ref, run_ref = run_chain(w, x, chunks_per_block=cpb, save_states=save_states)
    per_segment = binding.sf_launch_count() - n0
    ref = {n: ref[n].clone() for n in NAMES}
    bounds_ref = run_ref.S_bounds.clone()
    try:
        binding.sf_set_tuning(dict(merge_launches=1))
        n0 = binding.sf_launch_count()
        got, run = run_chain(w, x, chunks_per_block=cpb, save_states=save_states)
        merged = binding.sf_launch_count() - n0
        for n in NAMES:
            assert torch.equal(got[n], ref[n]), n
        assert torch.equal(run.S_bounds, bounds_ref)            # every boundary state, not only the last
        # 3 forward + 5 backward kernels (+ 2 to replay the states, + 1 on the tensor-core path to mark the segment starts)
        assert merged < per_segment and merged == (8 if save_states else 10) + (1 if dtype == "bf16" else 0)
        if save_states:
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                run.capture(x["S_in"], x["dS_out"])
                run.o.zero_()
                run.dq.zero_()
                run.replay()
            stream.synchronize()
            assert torch.equal(run.o, ref["o"]) and torch.equal(run.dq, ref["dq"]) and torch.equal(run.dS_init, ref["dS_in"])
            run.release()
    finally:
        binding.sf_set_tuning(None)
    assert binding.sf_device_status() == 0
    compare(ref, oracle_reference(x), tolerance(w), label="merged")


def test_chains_that_cannot_be_merged_run_segment_by_segment():
    # a middle segment that is not a whole number of chunks: no common block grid
    w = Workload("unmerged", 1, 2, 128, 128, [512, 300, 512], 64, g_scale=0.1, s_in_sigma=0.02, ds_out_sigma=0.02, seed=62)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    binding.sf_set_tuning(None)
    ref, _ = run_chain(w, x)
    ref = {n: ref[n].clone() for n in NAMES}
    try:
        binding.sf_set_tuning(dict(merge_launches=1))
        got, _ = run_chain(w, x)
        for n in NAMES:
            assert torch.equal(got[n], ref[n]), n
    finally:
        binding.sf_set_tuning(None)


def test_merged_launches_with_the_library_s_own_block_length_match_the_oracle():
    # chunks_per_block = 0: the merged run picks the longest common block length, which may differ from the segments' own
    w = Workload("merged-auto", 1, 3, 128, 128, [1024, 512, 512, 2048, 300], 64, g_scale=0.1, s_in_sigma=0.02, ds_out_sigma=0.02,
                 seed=63)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    try:
        binding.sf_set_tuning(dict(merge_launches=1))
        n0 = binding.sf_launch_count()
        got, _ = run_chain(w, x)
        assert binding.sf_launch_count() - n0 == 9
        compare(got, oracle_reference(x), tolerance(w), label="merged-auto")
    finally:
        binding.sf_set_tuning(None)


@pytest.mark.parametrize("segs,cpb", [([512] * 24, 0), ([1024, 320, 64, 2048, 704, 128, 900], 0), ([640, 1216, 192], 7)])
def test_merged_launches_with_blocks_across_segment_boundaries(segs, cpb):
    # tensor-core path: the blocks ignore the segment boundaries; the forward sweep writes the boundary states itself
    import oracle
    w = Workload("merged-free", 1, 3, 128, 128, segs, 64, g_scale=0.1, s_in_sigma=0.02, ds_out_sigma=0.02, seed=64)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    try:
        binding.sf_set_tuning(dict(merge_launches=1))
        n0 = binding.sf_launch_count()
        got, run = run_chain(w, x, chunks_per_block=cpb)
        assert binding.sf_launch_count() - n0 == 9
        compare(got, oracle_reference(x), tolerance(w), label="merged-free")
        # every boundary state against the oracle's chained run
        f = inputs.to_f64
        _, _, S_ins = oracle.chain_fwd(f(x["q"]), f(x["k"]), f(x["v"]), f(x["g"]), segs, f(x["S_in"]))
        for i, ref in enumerate(S_ins):
            a = f(run.S_bounds[i])
            assert np.abs(a - ref).max() <= tolerance(w) * max(np.abs(ref).max(), 1e-30), i
    finally:
        binding.sf_set_tuning(None)
    assert binding.sf_device_status() == 0
