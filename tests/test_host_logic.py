"""CPU-only checks: exported symbols, argument validation before any launch, workspace arithmetic,
the golden regression pin of the oracle, and the multi-rank (replica) bookkeeping on gloo."""
import ctypes
import os
import re
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2608_06838_b200 import binding, build  # noqa: E402
from paper_2608_06838_b200.binding import SegDesc  # noqa: E402


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "stateflow.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sf_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert {"sf_segment_fwd", "sf_segment_bwd", "sf_state_scan", "sf_chain_fwd", "sf_chain_bwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def desc(**kw):
    d = dict(B=1, H=2, d_k=128, d_v=128, seg_len=1024, chunk=64, dtype=binding.SF_BF16, chunks_per_block=0)
    d.update(kw)
    H, dk, dv = d["H"], d["d_k"], d["d_v"]
    return SegDesc(d["B"], H, dk, dv, d["seg_len"], d["chunk"], d["dtype"], d["chunks_per_block"],
                   H * dk, H * dv, H, 0, 0, 0)


P = ctypes.c_void_p(0x10000)        # never dereferenced: every call below must fail validation first


def fwd(lib, d, q=P, k=P, v=P, g=P, S_in=None, o=P, S_out=ctypes.c_void_p(0x20000), ws=ctypes.c_void_p(0x30000), nbytes=1 << 40):
    return lib.sf_segment_fwd(ctypes.byref(d), q, k, v, g, S_in, o, S_out, ws, nbytes, None)


def test_forward_validation_happens_before_any_launch(lib):
    assert fwd(lib, desc(), q=None) == 1
    assert fwd(lib, desc(), S_out=None) == 1
    assert fwd(lib, desc(seg_len=0)) == 1 and fwd(lib, desc(seg_len=-64)) == 1     # empty or negative segment
    assert fwd(lib, desc(B=0)) == 1
    assert fwd(lib, desc(d_k=96, d_v=96)) == 2                      # unsupported head width
    assert fwd(lib, desc(chunk=32)) == 2                            # bf16 d=128 needs chunk 64
    assert fwd(lib, desc(chunks_per_block=65)) == 1
    assert fwd(lib, desc(), q=ctypes.c_void_p(0x10004)) == 1        # misaligned
    assert fwd(lib, desc(), S_in=ctypes.c_void_p(0x20000)) == 1     # S_in aliases S_out
    assert fwd(lib, desc(), nbytes=16) == 3
    assert fwd(lib, desc(), ws=None) == 3
    assert fwd(lib, desc(), ws=ctypes.c_void_p(0x30010)) == 1       # workspace not 256-byte aligned


def test_backward_and_scan_validation(lib):
    d = desc()
    args = [P] * 4 + [None, P, None] + [P] * 4 + [ctypes.c_void_p(0x40000)]
    assert lib.sf_segment_bwd(ctypes.byref(d), *args, None, ctypes.c_void_p(0x30000), 16, None) == 3
    bad = list(args)
    bad[5] = None                                                   # dO missing
    assert lib.sf_segment_bwd(ctypes.byref(d), *bad, None, ctypes.c_void_p(0x30000), 1 << 40, None) == 1
    alias = list(args)
    alias[6] = ctypes.c_void_p(0x40000)                             # dS_out aliases dS_in
    assert lib.sf_segment_bwd(ctypes.byref(d), *alias, None, ctypes.c_void_p(0x30000), 1 << 40, None) == 1
    assert lib.sf_state_scan(ctypes.byref(d), 0, 0, None, P, None, P, P, None) == 1
    assert lib.sf_state_scan(ctypes.byref(d), 0, 0, P, P, P, P, P, None) == 1       # in aliases out
    assert lib.sf_segment_fwd_static(ctypes.byref(desc(H=64, seg_len=4096, chunks_per_block=16)), P, P, P, P, None, P, P, None) == 3


def test_workspace_arithmetic(lib):
    d = desc(H=32, seg_len=8192, chunks_per_block=16)
    assert binding.sf_num_blocks(d) == 8
    state = 128 * 128 * 4
    f = binding.sf_workspace_bytes(d, 0)
    assert f == 32 * 8 * state + 1024                               # block states + 32*8 block totals (256-byte padded)
    b1 = binding.sf_workspace_bytes(d, 1)
    assert b1 == 32 * 8 * state + 2 * 32 * 8192 * 4
    assert binding.sf_workspace_bytes(d, 2) == b1 + f + 32 * state
    assert binding.sf_num_blocks(desc(seg_len=17 * 64, chunks_per_block=4)) == 5
    assert binding.sf_workspace_bytes(desc(seg_len=0), 0) == 0
    # a ragged segment counts its partial last chunk: 1000 tokens = 16 chunks of 64
    assert binding.sf_workspace_bytes(desc(seg_len=1000, chunks_per_block=16), 0) == binding.sf_workspace_bytes(desc(seg_len=1024, chunks_per_block=16), 0)
    segs = [12288, 10240, 8192]
    tot = sum(binding.sf_workspace_bytes(desc(H=32, seg_len=s, chunks_per_block=16), 0) for s in segs)
    # plus, for the merged-launch mode, one int per chunk of the whole chain (480 chunks, 256-byte padded)
    assert binding.sf_chain_workspace_bytes(d, segs, 0) == tot + 2048
    tot_b = sum(binding.sf_workspace_bytes(desc(H=32, seg_len=s, chunks_per_block=16), 1) for s in segs)
    assert binding.sf_chain_workspace_bytes(d, segs, 1) == tot_b + 3 * 32 * state
    # left open, the block length is chosen per shape (148 SMs assumed without a device): one wave where possible
    auto = desc(H=32, seg_len=8192)
    assert binding.sf_num_blocks(auto) == 4                          # 32 chunks per block: 128 CTAs, one wave
    assert binding.sf_num_blocks(desc(H=16, seg_len=4096)) == 8      # 8 chunks per block: 128 CTAs
    assert 1 <= binding.sf_num_blocks(desc(H=1, seg_len=64)) <= 1
    assert binding.sf_chain_workspace_bytes(d, [0], 0) == 0 and binding.sf_chain_workspace_bytes(d, [100], 0) > 0


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(3)
    assert binding.sf_launch_count() == 0                            # nothing above launched a kernel


def test_oracle_reproduces_the_golden_case():
    import oracle
    vals = {}
    with open(os.path.join(ROOT, "tests", "golden", "tiny_case.txt")) as f:
        lines = [ln for ln in f.read().splitlines() if not ln.startswith("#")]
    for head, data in zip(lines[0::2], lines[1::2]):
        name, *shape = head.split()
        vals[name] = np.array([float(t) for t in data.split()]).reshape([int(s) for s in shape])
    o, S_out = oracle.segment_fwd(vals["q"], vals["k"], vals["v"], vals["g"], vals["S_in"])
    grads = oracle.segment_bwd(vals["q"], vals["k"], vals["v"], vals["g"], vals["S_in"], vals["dO"], vals["dS_out"])
    for name, a in zip(["o", "S_out", "dq", "dk", "dv", "dg", "dS_in"], (o, S_out) + tuple(grads)):
        np.testing.assert_allclose(a, vals[name], rtol=1e-13, atol=1e-13, err_msg=name)
    # the first output row can be checked by hand: o_0 = q_0 (e^{g_0} S_in + k_0^T v_0)
    S1 = np.exp(vals["g"][0, 0, 0]) * vals["S_in"][0, 0] + np.outer(vals["k"][0, 0, 0], vals["v"][0, 0, 0])
    np.testing.assert_allclose(vals["o"][0, 0, 0], vals["q"][0, 0, 0] @ S1, atol=1e-12)


def _replica_rank(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")          # rank 1 is the slow one
    dist.barrier()
    if rank == 0:
        out.put((ms, bench.replica_throughput(1000, world, ms)))
    dist.destroy_process_group()


def test_replica_timing_takes_the_slowest_rank_on_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_replica_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, value = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert ms == 15.0
    assert abs(value - 2 * 1000 / 15e-3) < 1e-6


def test_graph_create_rejects_bad_arguments_before_any_cuda_call(lib):
    d = desc()
    segs = (ctypes.c_int32 * 1)(1024)
    handle = ctypes.c_void_p(0x1)
    args = [ctypes.byref(d), segs, 1] + [P] * 7 + [P, 1 << 40] + [P] * 7 + [P, 1 << 40, 1]
    # no place for the handle; then the legacy default stream, which cannot be captured
    assert lib.sf_chain_graph_create(*args, ctypes.c_void_p(0x40), None) == 1
    assert lib.sf_chain_graph_create(*args, None, ctypes.byref(handle)) == 1
    assert handle.value is None                      # cleared on error
    assert lib.sf_chain_graph_launch(None, None) == 1
    assert lib.sf_chain_graph_kernels(None) == 0
    lib.sf_chain_graph_destroy(None)                 # a no-op


def test_autotune_rejects_bad_arguments_before_any_cuda_call(lib):
    d = desc()
    segs = (ctypes.c_int32 * 1)(1024)
    cands = (ctypes.c_int32 * 2)(0, 16)
    best = ctypes.c_int32(-7)
    head = [ctypes.byref(d), segs, 1] + [P] * 7 + [P, 1 << 40] + [P] * 7 + [P, 1 << 40]
    assert lib.sf_chain_autotune(*head, None, 2, 3, 1, None, ctypes.byref(best), None) == 1        # no candidates
    assert lib.sf_chain_autotune(*head, cands, 0, 3, 1, None, ctypes.byref(best), None) == 1
    assert lib.sf_chain_autotune(*head, cands, 2, 0, 1, None, ctypes.byref(best), None) == 1       # no repetitions
    assert lib.sf_chain_autotune(*head, cands, 2, 3, 1, None, None, None) == 1                     # nowhere to report
    bad = (ctypes.c_int32 * 1)(0)                                                                  # an empty segment
    assert lib.sf_chain_autotune(ctypes.byref(d), bad, 1, *head[3:], cands, 2, 3, 1, None, ctypes.byref(best), None) == 1
    assert best.value == -7


def test_tuning_is_validated_and_restored(lib):
    from paper_2608_06838_b200.binding import SfError, Tuning
    binding.sf_set_tuning(None)
    d = binding.sf_get_tuning()
    assert (d.sweep_streams, d.agg_streams, d.scan_group_tokens, d.agg_inorder_ctas, d.agg_ahead, d.merge_launches) == (4, 4, 4096, 74, 0, 0)
    binding.sf_set_tuning(dict(sweep_streams=2, agg_ahead=1))
    t = binding.sf_get_tuning()
    assert (t.sweep_streams, t.agg_streams, t.agg_ahead) == (2, 4, 1)
    for bad in (dict(sweep_streams=0), dict(sweep_streams=5), dict(agg_streams=0), dict(agg_streams=9),
                dict(scan_group_tokens=-1), dict(agg_inorder_ctas=0), dict(agg_ahead=-1), dict(merge_launches=2), dict(merge_launches=-1)):
        with pytest.raises(SfError) as e:
            binding.sf_set_tuning(bad)
        assert e.value.code == 1
        t2 = binding.sf_get_tuning()                      # a rejected tuning changes nothing
        assert (t2.sweep_streams, t2.agg_streams, t2.agg_ahead) == (2, 4, 1)
    binding.sf_set_tuning(None)
    assert binding.sf_get_tuning().sweep_streams == 4


def test_extension_operators_validate_before_any_launch(lib):
    f32 = dict(dtype=binding.SF_F32, d_k=64, d_v=64, seg_len=100)
    d = desc(**f32)
    S1, S2 = ctypes.c_void_p(0x20000), ctypes.c_void_p(0x30000)
    assert lib.sf_recurrent_workspace_bytes(ctypes.byref(d)) == 1 * 2 * (7 + 16) * 64 * 64 * 4   # ceil(100/16) + 16 states
    assert lib.sf_recurrent_workspace_bytes(ctypes.byref(desc())) == 0                          # d_k = 128: not offered
    cf = lambda dd, q=P, S_in=None, S_out=S1: lib.sf_channel_segment_fwd(ctypes.byref(dd), q, P, P, P, S_in, P, S_out, None)
    assert cf(desc()) == 2 and cf(desc(**dict(f32, d_k=128))) == 2 and cf(desc(**dict(f32, d_v=48))) == 2
    assert cf(d, q=None) == 1 and cf(d, S_out=None) == 1 and cf(d, S_in=S1) == 1
    assert cf(desc(**dict(f32, seg_len=0))) == 1 and cf(desc(**dict(f32, B=70000))) == 1
    df = lambda dd, beta=P: lib.sf_delta_segment_fwd(ctypes.byref(dd), P, P, P, P, beta, None, P, S1, None)
    assert df(d, beta=None) == 1 and df(desc()) == 2
    bargs = [P] * 4 + [None, P, None] + [P] * 4 + [S2]
    assert lib.sf_channel_segment_bwd(ctypes.byref(d), *bargs, ctypes.c_void_p(0x40000), 16, None) == 3
    assert lib.sf_channel_segment_bwd(ctypes.byref(d), *bargs, None, 1 << 40, None) == 3
    assert lib.sf_channel_segment_bwd(ctypes.byref(d), *bargs, ctypes.c_void_p(0x40010), 1 << 40, None) == 3
    dargs = [P] * 5 + [None, P, None] + [P] * 4 + [None, S2]                # dbeta missing
    assert lib.sf_delta_segment_bwd(ctypes.byref(d), *dargs, ctypes.c_void_p(0x40000), 1 << 40, None) == 1
    conv = lambda B=1, L=8, C=4, W=4, x=P, tail_out=S1: lib.sf_conv_segment_fwd(B, L, C, W, x, P, None, P, tail_out, None)
    assert conv(L=0) == 1 and conv(W=0) == 1 and conv(W=9) == 2 and conv(x=None) == 1 and conv(tail_out=None) == 1
    assert conv(B=65536) == 2                                                              # B is a grid dimension
    assert lib.sf_conv_segment_bwd(1, 8, 4, 4, P, P, None, P, S1, P, P, S1, None) == 1       # dtail_out aliases dtail_in
    assert lib.sf_conv_segment_bwd(1, 8, 4, 4, P, P, None, None, None, P, P, S1, None) == 1  # dy missing


def test_chunked_delta_rule_validates_before_any_launch(lib):
    f32 = dict(dtype=binding.SF_F32, d_k=64, d_v=64, seg_len=100, chunk=32)
    d = desc(**f32)
    lib.sf_delta_chunked_workspace_bytes.restype = ctypes.c_size_t
    per_bh_fwd = 100 * 64 + 100 * 64 + 3 * 4 * 64 * 64 + 3 * 64 * 64   # U, Wk per token; Phi, Psi, one state per chunk (4 chunks); the same per block of 16 chunks
    assert lib.sf_delta_chunked_workspace_bytes(ctypes.byref(d), 0) == 2 * per_bh_fwd * 4
    # the backward adds Z0 per token, Theta and one state gradient per chunk and two chunk x chunk matrices per chunk
    assert lib.sf_delta_chunked_workspace_bytes(ctypes.byref(d), 1) == 2 * (per_bh_fwd + 100 * 64 + 2 * 4 * 64 * 64 + 2 * 4 * 32 * 32) * 4
    S1, S2, W = ctypes.c_void_p(0x20000), ctypes.c_void_p(0x30000), ctypes.c_void_p(0x40000)
    cf = lambda dd, q=P, beta=P, S_in=None, ws=W, n=1 << 40: lib.sf_delta_chunked_fwd(ctypes.byref(dd), q, P, P, P, beta, S_in, P, S1, ws, n, None)
    assert cf(d, q=None) == 1 and cf(d, beta=None) == 1 and cf(d, S_in=S1) == 1
    assert cf(d, ws=None) == 3 and cf(d, n=16) == 3 and cf(d, ws=ctypes.c_void_p(0x40010)) == 3
    assert cf(desc(**dict(f32, chunk=64))) == 2 and cf(desc(**dict(f32, d_v=128))) == 2 and cf(desc(**dict(f32, d_k=128, d_v=128))) == 2
    assert lib.sf_delta_chunked_workspace_bytes(ctypes.byref(desc(**dict(f32, d_k=128, d_v=128, chunk=16))), 1) > 0   # 128-wide heads fit at chunk 16
    assert cf(desc(**dict(f32, chunk=0))) == 1 and cf(desc(**dict(f32, seg_len=0))) == 1
    bargs = [P] * 5 + [None, P, None] + [P] * 5 + [S2]
    assert lib.sf_delta_chunked_bwd(ctypes.byref(d), *bargs, W, 16, None) == 3
    bad = list(bargs)
    bad[12] = None                                                  # dbeta missing
    assert lib.sf_delta_chunked_bwd(ctypes.byref(d), *bad, W, 1 << 40, None) == 1


def test_chunked_diagonal_decay_validates_before_any_launch(lib):
    f32 = dict(dtype=binding.SF_F32, d_k=64, d_v=32, seg_len=100, chunk=32)
    d = desc(**f32)
    lib.sf_channel_chunked_workspace_bytes.restype = ctypes.c_size_t
    per_bh = 4 * 64 * 32 + 4 * 64 + 5 * 64 * 32                     # Psi and gam_n per chunk, NC + 1 states (4 chunks)
    assert lib.sf_channel_chunked_workspace_bytes(ctypes.byref(d), 0) == 2 * per_bh * 4
    assert lib.sf_channel_chunked_workspace_bytes(ctypes.byref(d), 1) == 2 * (per_bh + 2 * 4 * 64 * 32) * 4
    S1, S2, W = ctypes.c_void_p(0x20000), ctypes.c_void_p(0x30000), ctypes.c_void_p(0x40000)
    cf = lambda dd, q=P, S_in=None, ws=W, n=1 << 40: lib.sf_channel_chunked_fwd(ctypes.byref(dd), q, P, P, P, S_in, P, S1, ws, n, None)
    assert cf(d, q=None) == 1 and cf(d, S_in=S1) == 1 and cf(d, ws=None) == 3 and cf(d, n=16) == 3
    assert cf(desc(**dict(f32, chunk=64))) == 2 and cf(desc(**dict(f32, seg_len=0))) == 1
    wide = dict(f32, d_k=128, d_v=128)
    assert cf(desc(**wide)) == 2                                     # 128-wide heads do not fit at chunk 32 ...
    assert lib.sf_channel_chunked_workspace_bytes(ctypes.byref(desc(**dict(wide, chunk=16))), 1) > 0   # ... but do at chunk 16
    bargs = [P] * 4 + [None, P, None] + [P] * 4 + [S2]
    assert lib.sf_channel_chunked_bwd(ctypes.byref(d), *bargs, W, 16, None) == 3
    bad = list(bargs)
    bad[5] = None                                                    # dO missing
    assert lib.sf_channel_chunked_bwd(ctypes.byref(d), *bad, W, 1 << 40, None) == 1


def test_host_wrapper_scratch_size_and_validation(lib):
    d = desc()
    segs = (ctypes.c_int32 * 3)(1024, 512, 2048)
    T = 3584
    need = lib.sf_e2e_device_bytes(ctypes.byref(d), segs, 3)
    # eight [T, H, 128] bf16 tensors, g and dg, four + three boundary-state buffers, per-segment forward workspaces
    # kept for the backward, one backward workspace (the largest segment's)
    state = 2 * 128 * 128 * 4
    one = lambda i, bwd: lib.sf_chain_workspace_bytes(ctypes.byref(d), (ctypes.c_int32 * 1)(segs[i]), 1, bwd)
    up = lambda n: (n + 255) // 256 * 256
    want = 8 * T * 2 * 128 * 2 + 2 * T * 2 * 4 + 7 * state + sum(up(one(i, 0)) for i in range(3)) + max(up(one(i, 1)) for i in range(3))
    assert need == want
    assert lib.sf_e2e_device_bytes(ctypes.byref(d), segs, 0) == 0
    call = lambda dev, nbytes, dq=P: lib.sf_chain_fwd_bwd_host(ctypes.byref(d), segs, 3, P, P, P, P, None, P, None, P, None, dq, P, P, P,
                                                              P, dev, nbytes, None)
    assert call(ctypes.c_void_p(0x40000), need - 1) == 3          # SF_ERR_WORKSPACE
    assert call(None, need) == 3
    assert call(ctypes.c_void_p(0x40000), need, dq=None) == 1     # SF_ERR_INVALID_ARG
    assert call(ctypes.c_void_p(0x40010), need) == 1              # scratch not 256-byte aligned
    strided = desc()
    strided.tok_stride_qk = 2 * 2 * 128                            # the wrapper wants densely packed host tensors
    assert lib.sf_chain_fwd_bwd_host(ctypes.byref(strided), segs, 3, P, P, P, P, None, P, None, P, None, P, P, P, P, P,
                                     ctypes.c_void_p(0x40000), 1 << 40, None) == 1
