"""Writes tests/golden/tiny_case.txt from the fp64 oracle alone (no CUDA code is imported or run).

The paper prints no worked numeric example for this recurrence, so this fixture is a regression pin:
it freezes the oracle's output on one tiny hand-checkable case (Eq. 1 with F_t = exp(g_t) I, Eq. 4 and
Eq. 6 boundary semantics) so that an accidental edit of the oracle shows up as a diff here.
Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle  # noqa: E402


def case():
    r = np.random.default_rng(20260806)
    B, T, H, dk, dv = 1, 6, 1, 2, 3
    q = np.round(r.standard_normal((B, T, H, dk)), 3)
    k = np.round(r.standard_normal((B, T, H, dk)), 3)
    v = np.round(r.standard_normal((B, T, H, dv)), 3)
    g = -np.round(np.abs(r.standard_normal((B, T, H))), 3)
    S_in = np.round(r.standard_normal((B, H, dk, dv)), 3)
    dO = np.round(r.standard_normal((B, T, H, dv)), 3)
    dS_out = np.round(r.standard_normal((B, H, dk, dv)), 3)
    return dict(q=q, k=k, v=v, g=g, S_in=S_in, dO=dO, dS_out=dS_out)


def main():
    x = case()
    o, S_out = oracle.segment_fwd(x["q"], x["k"], x["v"], x["g"], x["S_in"])
    dq, dk, dv, dg, dS_in = oracle.segment_bwd(x["q"], x["k"], x["v"], x["g"], x["S_in"], x["dO"], x["dS_out"])
    out = dict(x, o=o, S_out=S_out, dq=dq, dk=dk, dv=dv, dg=dg, dS_in=dS_in)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_case.txt")
    with open(path, "w") as f:
        f.write("# Regression pin written by tests/golden/make_golden.py from oracle/ only.\n")
        f.write("# Gated linear recurrence, paper Eq. 1 (F_t = exp(g_t) I), segment semantics Eq. 4 / Eq. 6.\n")
        for name, a in out.items():
            f.write("%s %s\n" % (name, " ".join(str(d) for d in a.shape)))
            f.write(" ".join(repr(float(t)) for t in a.ravel()) + "\n")
    print(path)


if __name__ == "__main__":
    main()
