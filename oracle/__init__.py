"""TEST INFRASTRUCTURE: numpy front end of the fp64 CPU oracle (sf_oracle.c).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library and never imports it.

Functions mirror the paper's segment semantics:
  segment_fwd  - Fwd(C_in, S_in) -> (C_out, S_out)            (Eq. 4)
  segment_bwd  - Bwd(C_in, S_in, dC_out, dS_out) -> (dC_in, dS_in)   (Eq. 6)
  chain_fwd / chain_bwd - segments run in order with S_{i+1}^in = S_i^out
                          and dS_i^out = dS_{i+1}^in          (Eq. 5, Eq. 7)
  state_scan   - the ST stage alone over block aggregates     (Eq. 2)

Every function is pinned by tests marked "not gpu" (closed forms, brute
force, finite differences, split invariance); none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sf_oracle.c")
_LIB = os.path.join(_HERE, "libsf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile sf_oracle.c with gcc (-O2 -fopenmp) into libsf_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("B", "T", "H", "dk", "dv", "tok_qk", "tok_v", "tok_g", "bat_qk", "bat_v", "bat_g")]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.sfo_segment_fwd.restype = ctypes.c_int
        _lib.sfo_segment_bwd.restype = ctypes.c_int
        _lib.sfo_state_scan.restype = None
        _lib.sfo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().sfo_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _shape(q, v):
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    return _Shape(B, T, H, dk, dv, H * dk, H * dv, H, T * H * dk, T * H * dv, T * H)


def segment_fwd(q, k, v, g, S_in=None):
    """q,k [B,T,H,dk]; v [B,T,H,dv]; g [B,T,H]; S_in [B,H,dk,dv] or None.
    Returns (o [B,T,H,dv], S_out [B,H,dk,dv]) in float64."""
    q, k, v, g, S_in = map(_f64, (q, k, v, g, S_in))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    o = np.zeros((B, T, H, dv))
    S_out = np.zeros((B, H, dk, dv))
    sh = _shape(q, v)
    rc = _load().sfo_segment_fwd(ctypes.byref(sh), _p(q), _p(k), _p(v), _p(g), _p(S_in), _p(o), _p(S_out))
    if rc != 0:
        raise MemoryError("oracle forward")
    return o, S_out


def segment_bwd(q, k, v, g, S_in, dO, dS_out=None):
    """Returns (dq, dk, dv, dg, dS_in) in float64."""
    q, k, v, g, S_in, dO, dS_out = map(_f64, (q, k, v, g, S_in, dO, dS_out))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    dq = np.zeros_like(q)
    dk_ = np.zeros_like(k)
    dv_ = np.zeros_like(v)
    dg = np.zeros_like(g)
    dS_in = np.zeros((B, H, dk, dv))
    sh = _shape(q, v)
    rc = _load().sfo_segment_bwd(ctypes.byref(sh), _p(q), _p(k), _p(v), _p(g), _p(S_in), _p(dO), _p(dS_out),
                                 _p(dq), _p(dk_), _p(dv_), _p(dg), _p(dS_in))
    if rc != 0:
        raise MemoryError("oracle backward")
    return dq, dk_, dv_, dg, dS_in


def _bounds(seg_lens, T):
    b = np.concatenate([[0], np.cumsum(np.asarray(seg_lens, dtype=np.int64))])
    if b[-1] != T:
        raise ValueError("segment lengths must sum to T")
    return b


def chain_fwd(q, k, v, g, seg_lens, S_init=None):
    """Run the segments in order, S_{i+1}^in = S_i^out.  Returns (o, S_final, [S_i^in])."""
    c = _bounds(seg_lens, q.shape[1])
    outs, S, S_ins = [], S_init, []
    for i in range(len(seg_lens)):
        sl = slice(c[i], c[i + 1])
        S_ins.append(None if S is None else np.array(S))
        o_i, S = segment_fwd(q[:, sl], k[:, sl], v[:, sl], g[:, sl], S)
        outs.append(o_i)
    return np.concatenate(outs, axis=1), S, S_ins


def chain_bwd(q, k, v, g, seg_lens, S_ins, dO, dS_final=None):
    """Run the segments in reverse, dS_i^out = dS_{i+1}^in.  Returns (dq, dk, dv, dg, dS_init)."""
    c = _bounds(seg_lens, q.shape[1])
    n = len(seg_lens)
    parts, dS = [None] * n, dS_final
    for i in range(n - 1, -1, -1):
        sl = slice(c[i], c[i + 1])
        dq, dk_, dv_, dg, dS = segment_bwd(q[:, sl], k[:, sl], v[:, sl], g[:, sl], S_ins[i], dO[:, sl], dS)
        parts[i] = (dq, dk_, dv_, dg)
    cat = lambda j: np.concatenate([p[j] for p in parts], axis=1)
    return cat(0), cat(1), cat(2), cat(3), dS


def state_scan(log_decay, U, init=None, reverse=False):
    """log_decay [lanes,n]; U [lanes,n,m]; init [lanes,m] or None.
    Returns (states [lanes,n,m], final [lanes,m])."""
    ld, U, init = map(_f64, (log_decay, U, init))
    lanes, n, m = U.shape
    states = np.zeros_like(U)
    final = np.zeros((lanes, m))
    _load().sfo_state_scan(ctypes.c_int64(lanes), ctypes.c_int64(n), ctypes.c_int64(m), ctypes.c_int(int(reverse)),
                           _p(ld), _p(U), _p(init), _p(states), _p(final))
    return states, final
