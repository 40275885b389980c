"""Shared test helpers: run the CUDA chain on a workload and compare with the fp64 oracle."""
import numpy as np
import torch

import oracle
from paper_2608_06838_b200 import binding, inputs

NAMES = ["o", "S_out", "dq", "dk", "dv", "dg", "dS_in"]


def tolerance(w):
    # float32 mode: max relative error <= 1e-4; bf16 storage with float32 accumulation: <= 2e-2
    # (both as max |x - ref| / max |ref| per output tensor over the whole chained sequence)
    return 1e-4 if w.dtype == "f32" else 2e-2


def norm_err(a, r):
    return float(np.abs(a - r).max() / max(np.abs(r).max(), 1e-30))


def floored_rel_err(a, r):
    """Largest element-wise relative error with the denominator floored at 1e-3 of the tensor's largest magnitude
    (a plain relative error is undefined at the zeros of the reference).  Reported, not gated."""
    m = max(np.abs(r).max(), 1e-30)
    return float((np.abs(a - r) / np.maximum(np.abs(r), 1e-3 * m)).max())


def rms_err(a, r):
    """RMS of the error over the RMS of the reference.  Reported, not gated."""
    return float(np.sqrt(np.mean((a - r) ** 2)) / max(np.sqrt(np.mean(r ** 2)), 1e-30))


def oracle_reference(x, heads=None):
    """Unsplit oracle run on the same bits; optionally on a subset of heads."""
    f = inputs.to_f64
    sl = slice(None) if heads is None else heads
    q, k, v, g, dO = (f(x[n][:, :, sl]) for n in ("q", "k", "v", "g", "dO"))
    S_in = None if x["S_in"] is None else f(x["S_in"][:, sl])
    dS_out = None if x["dS_out"] is None else f(x["dS_out"][:, sl])
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    dq, dk, dv, dg, dS_in = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    return dict(o=o, S_out=S_out, dq=dq, dk=dk, dv=dv, dg=dg, dS_in=dS_in)


def run_chain(w, x, chunks_per_block=0, save_states=True, overlap=True):
    run = binding.ChainRun(x["q"], x["k"], x["v"], x["g"], x["dO"], w.seg_lens, w.chunk, chunks_per_block, save_states)
    run.forward(x["S_in"], overlap=overlap)
    run.backward(x["dS_out"], overlap=overlap)
    torch.cuda.synchronize()
    assert binding.sf_device_status() == 0
    return dict(o=run.o, S_out=run.S_bounds[-1], dq=run.dq, dk=run.dk, dv=run.dv, dg=run.dg, dS_in=run.dS_init), run


def compare(got, ref, tol, heads=None, label=""):
    errs = {}
    for n in NAMES:
        a = got[n]
        if heads is not None:
            a = a[:, heads] if n in ("S_out", "dS_in") else a[:, :, heads]
        a = inputs.to_f64(a)
        assert np.isfinite(a).all(), "%s %s has non-finite values" % (label, n)
        errs[n] = norm_err(a, ref[n])
        # the gate is the normalised max error; the other two figures are printed for the reader (pytest -s shows them)
        print("[parity] %-28s %-6s normalised-max %.2e  floored-relative %.2e  rms %.2e"
              % (label, n, errs[n], floored_rel_err(a, ref[n]), rms_err(a, ref[n])))
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, "%s: normalised max error above %.1e: %s (all: %s)" % (label, tol, bad, errs)
    return errs
