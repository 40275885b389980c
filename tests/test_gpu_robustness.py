"""Checks that stand in for a race detector and a memory checker: run-to-run bit determinism with the stream overlap
on, guard regions around every output and workspace buffer, and every block length against the oracle."""
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import NAMES, compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 4096          # bytes on each side


def guarded(nbytes, fill=0xA5):
    """A byte buffer of nbytes between two guard regions; returns (whole, middle view, 256-byte aligned)."""
    pad = (GUARD + 255) // 256 * 256
    whole = torch.full((pad + (nbytes + 255) // 256 * 256 + pad,), fill, dtype=torch.uint8, device=DEV)
    return whole, whole[pad:pad + nbytes]


def guards_intact(whole, nbytes, fill=0xA5):
    pad = (GUARD + 255) // 256 * 256
    return bool((whole[:pad] == fill).all()) and bool((whole[pad + nbytes:] == fill).all())


@pytest.mark.parametrize("dtype,d,chunk", [("bf16", 128, 64), ("f32", 64, 32)])
def test_nothing_is_written_outside_the_buffers(dtype, d, chunk):
    w = Workload("guards", 2, 3, d, d, [5 * chunk, 3 * chunk, 8 * chunk], chunk, dtype=dtype, g_scale=0.1, s_in_sigma=0.05,
                 ds_out_sigma=0.05, seed=21)
    x = inputs.make_inputs(w, DEV)
    B, T, H = w.B, w.T, w.H
    esz = 2 if dtype == "bf16" else 4
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    desc = binding.make_desc(x["q"], x["v"], x["g"], chunk, 2, seg_len=w.seg_lens[0])
    sizes = dict(o=B * T * H * d * esz, dq=B * T * H * d * esz, dk=B * T * H * d * esz, dv=B * T * H * d * esz,
                 dg=B * T * H * 4, S_bounds=(len(w.seg_lens) + 1) * B * H * d * d * 4, dS_init=B * H * d * d * 4,
                 ws_f=binding.sf_chain_workspace_bytes(desc, w.seg_lens, 0),
                 ws_b=binding.sf_chain_workspace_bytes(desc, w.seg_lens, 1))
    whole, mid = {}, {}
    for n, sz in sizes.items():
        whole[n], mid[n] = guarded(sz)
    view = lambda n, dt, shape: mid[n].view(dt).view(*shape)
    o, dv = view("o", tdt, (B, T, H, d)), view("dv", tdt, (B, T, H, d))
    dq, dk = view("dq", tdt, (B, T, H, d)), view("dk", tdt, (B, T, H, d))
    dg = view("dg", torch.float32, (B, T, H))
    S_bounds = view("S_bounds", torch.float32, (len(w.seg_lens) + 1, B, H, d, d))
    dS_init = view("dS_init", torch.float32, (B, H, d, d))
    for overlap in (False, True):
        binding.sf_chain_fwd(desc, w.seg_lens, x["q"], x["k"], x["v"], x["g"], x["S_in"], o, S_bounds, mid["ws_f"], overlap)
        binding.sf_chain_bwd(desc, w.seg_lens, x["q"], x["k"], x["v"], x["g"], S_bounds, x["dO"], x["dS_out"], dq, dk, dv, dg,
                             dS_init, mid["ws_f"], mid["ws_b"], overlap)
        torch.cuda.synchronize()
        assert binding.sf_device_status() == 0
        for n, sz in sizes.items():
            assert guards_intact(whole[n], sz), "guard region of %s was overwritten (overlap=%s)" % (n, overlap)
    got = dict(o=o, S_out=S_bounds[-1], dq=dq, dk=dk, dv=dv, dg=dg, dS_in=dS_init)
    compare(got, oracle_reference(x), tolerance(w), label="guards")


def test_repeated_runs_with_overlap_are_bit_identical():
    # a race between the streams or inside a kernel would show as run-to-run differences
    w = Workload("determinism", 1, 8, 128, 128, [2048, 1024, 512, 512], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=22)
    x = inputs.make_inputs(w, DEV)
    first, _ = run_chain(w, x, overlap=True)
    first = {n: first[n].clone() for n in NAMES}
    for _ in range(5):
        again, _ = run_chain(w, x, overlap=True)
        for n in NAMES:
            assert torch.equal(first[n], again[n]), n


@pytest.mark.parametrize("cpb", [1, 2, 3, 5, 7, 8, 13, 16, 31, 32, 33, 47, 64])
def test_every_block_length_matches_the_oracle(cpb):
    # 37 chunks (or 131 for the block lengths beyond 32): most block lengths leave a ragged last block
    nc = 37 if cpb <= 32 else 131
    w = Workload("blocks-%d" % cpb, 1, 2, 128, 128, [nc * 64], 64, g_scale=0.05, s_in_sigma=0.02, ds_out_sigma=0.02, seed=23)
    x = inputs.make_inputs(w, DEV)
    got, _ = run_chain(w, x, chunks_per_block=cpb)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


@pytest.mark.parametrize("dtype,d,chunk,segs", [
    ("f32", 64, 32, [100, 37, 200]),
    ("f32", 32, 16, [5]),
    ("bf16", 128, 64, [1000, 70, 300, 65]),
    ("bf16", 128, 64, [17]),
    ("bf16", 64, 64, [130, 63]),
])
def test_segments_that_are_not_whole_chunks(dtype, d, chunk, segs):
    # the last chunk of a segment may be partial; the next segment then starts in the middle of a chunk-sized stretch
    w = Workload("ragged-%s-%d" % (dtype, sum(segs)), 2, 3, d, d, segs, chunk, dtype=dtype, g_scale=0.1, s_in_sigma=0.05,
                 ds_out_sigma=0.05, seed=31)
    x = inputs.make_inputs(w, DEV)
    for cpb in (2, 0):
        got, _ = run_chain(w, x, chunks_per_block=cpb)
        compare(got, oracle_reference(x), tolerance(w), label=w.name)
    got = {n: got[n].clone() for n in NAMES}                  # the run with the library's own block length
    # and nothing beyond the last token is touched: the same run on views of tensors with `chunk` more tokens per batch
    T, pad = w.T, chunk
    def padded(t, fill):
        shape = list(t.shape)
        shape[1] = T + pad
        big = torch.full(shape, fill, dtype=t.dtype, device=DEV)
        big[:, :T] = t
        return big
    xin = {n: padded(x[n], 3.0) for n in ("q", "k", "v", "g", "dO")}
    run = binding.ChainRun(xin["q"][:, :T], xin["k"][:, :T], xin["v"][:, :T], xin["g"][:, :T], xin["dO"][:, :T], w.seg_lens, w.chunk)
    outs = {n: padded(getattr(run, n), 7.0) for n in ("o", "dq", "dk", "dv", "dg")}
    for n in outs:
        setattr(run, n, outs[n][:, :T])
    run.forward(x["S_in"])
    run.backward(x["dS_out"])
    torch.cuda.synchronize()
    assert binding.sf_device_status() == 0
    for n in outs:
        assert bool((outs[n][:, T:] == 7.0).all()), "%s was written beyond the last token" % n
    padded_got = dict(o=run.o, S_out=run.S_bounds[-1], dq=run.dq, dk=run.dk, dv=run.dv, dg=run.dg, dS_in=run.dS_init)
    for n in NAMES:
        assert torch.equal(padded_got[n], got[n]), n          # the padding's content (3.0, not zero) must not leak in


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # failure detection without a fault: a self-test kernel waits (about a millisecond) on a barrier nothing completes;
    # the bounded wait gives up, the status word says so, and after clearing it a normal chain runs and is correct
    binding.sf_device_status_clear()
    assert binding.sf_device_check() == 0
    assert binding.sf_selftest_bounded_wait(2_000_000) == 5            # SF_ERR_TIMEOUT
    assert binding.sf_device_status() == 3 and binding.sf_device_check() == 5
    binding.sf_device_status_clear()
    assert binding.sf_device_status() == 0
    assert binding.sf_selftest_bounded_wait(0) == 1 and binding.sf_selftest_bounded_wait(10 ** 9) == 1   # limit out of range
    w = Workload("after-timeout", 1, 2, 128, 128, [640, 320], 64, s_in_sigma=0.02, ds_out_sigma=0.02, seed=31)
    x = inputs.make_inputs(w, DEV)
    got, _ = run_chain(w, x)
    compare(got, oracle_reference(x), tolerance(w), label=w.name)


def test_two_host_threads_on_two_streams_give_the_bits_of_the_serial_run():
    # Calls without side streams (overlap = 0) may come from any thread; ctypes drops the GIL during a call, so the two
    # threads really are inside the library at the same time.  Each thread has its own stream, buffers and workspaces.
    import threading
    ws = [Workload("thr-%d" % i, 1, 4, 128, 128, [1024, 640, 2048], 64, g_scale=0.1, s_in_sigma=0.1, ds_out_sigma=0.1, seed=40 + i)
          for i in range(2)]
    xs = [inputs.make_inputs(w, DEV) for w in ws]
    serial = [run_chain(w, x, overlap=False)[0] for w, x in zip(ws, xs)]
    torch.cuda.synchronize()
    out, errors = [None, None], []

    def work(i):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                for _ in range(3):
                    out[i] = run_chain(ws[i], xs[i], overlap=False)[0]
        except Exception as e:                   # surfaced below: an exception in a thread would otherwise be lost
            errors.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for i in range(2):
        for n in NAMES:
            assert torch.equal(out[i][n], serial[i][n]), (i, n)
    assert binding.sf_device_status() == 0
