"""TEST INFRASTRUCTURE: fp64 oracles of the three extensions of the segment operator, written token by token in numpy.

Only tests may import this module.  It shares nothing with the CUDA library.  Loops are plain Python: small cases only.

  channel_fwd / channel_bwd   diagonal transition (Section 2.1: structured F_t, diagonal family): one log-decay per
                              key channel,  S_t = diag(exp(g_t)) S_{t-1} + k_t^T v_t ,  o_t = q_t S_t
  delta_fwd / delta_bwd       scalar + low-rank transition (Section 2.1; the gated delta rule of the paper's experiments,
                              Eq. 2 with V_new != empty), in this library's orientation (S is d_k x d_v, o = q S):
                                  u_t = k_t S_{t-1} ;  w_t = beta_t (v_t - a_t u_t) ;  S_t = a_t S_{t-1} + k_t^T w_t ;  a_t = exp(g_t)
                              which is S_t = a_t (I - beta_t k_t^T k_t) S_{t-1} + beta_t k_t^T v_t
  conv_fwd / conv_bwd         causal depthwise short convolution whose last W-1 inputs travel with the boundary state
                              from one segment to the next (Section 3.1, footnote on auxiliary boundary states)

All follow the segment semantics of Eq. 4-7: a forward takes the incoming boundary state and returns the outgoing
one; a backward takes the gradient of the outgoing boundary state and returns that of the incoming one.  The
backward sweeps are derived by hand from the token recurrences (the paper prints none) and are pinned by finite
differences, by the special cases that reduce to the scalar-decay oracle, by split invariance and by the defining
property of the delta rule (tests/test_oracle_variants.py).  None is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def _z(x, shape):
    return np.zeros(shape) if x is None else np.array(x, dtype=np.float64)


# ------------------------------------------------------------------------------------------ diagonal decay ---

def channel_fwd(q, k, v, g, S_in=None, keep_states=False):
    """q,k,g [B,T,H,dk]; v [B,T,H,dv]; S_in [B,H,dk,dv] or None -> (o [B,T,H,dv], S_out)."""
    q, k, v, g = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    S = _z(S_in, (B, H, dk, dv))
    o = np.zeros((B, T, H, dv))
    states = [S.copy()] if keep_states else None
    for t in range(T):
        S = np.exp(g[:, t])[..., None] * S + k[:, t][..., :, None] * v[:, t][..., None, :]
        o[:, t] = np.einsum("bhi,bhij->bhj", q[:, t], S)
        if keep_states:
            states.append(S.copy())
    return (o, S, states) if keep_states else (o, S)


def channel_bwd(q, k, v, g, S_in, dO, dS_out=None):
    """-> (dq, dk, dv, dg [B,T,H,dk], dS_in)."""
    q, k, v, g, dO = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g, dO))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    _, _, st = channel_fwd(q, k, v, g, S_in, keep_states=True)          # st[t] = S_{t-1}, st[t+1] = S_t
    G = _z(dS_out, (B, H, dk, dv))
    dq, dk_, dv_, dg = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v), np.zeros_like(g)
    for t in range(T - 1, -1, -1):
        G = G + q[:, t][..., :, None] * dO[:, t][..., None, :]          # o_t = q_t S_t reads S_t
        dq[:, t] = np.einsum("bhj,bhij->bhi", dO[:, t], st[t + 1])
        dk_[:, t] = np.einsum("bhij,bhj->bhi", G, v[:, t])              # S_t contains k_t^T v_t
        dv_[:, t] = np.einsum("bhi,bhij->bhj", k[:, t], G)
        a = np.exp(g[:, t])
        dg[:, t] = a * np.sum(G * st[t], axis=-1)                       # S_t contains diag(exp(g_t)) S_{t-1}
        G = a[..., None] * G
    return dq, dk_, dv_, dg, G


# ---------------------------------------------------------------------------------------------- delta rule ---

def delta_fwd(q, k, v, g, beta, S_in=None, keep_states=False):
    """q,k [B,T,H,dk]; v [B,T,H,dv]; g, beta [B,T,H]; S_in [B,H,dk,dv] or None -> (o, S_out)."""
    q, k, v, g, beta = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g, beta))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    S = _z(S_in, (B, H, dk, dv))
    o = np.zeros((B, T, H, dv))
    states = [S.copy()] if keep_states else None
    for t in range(T):
        a = np.exp(g[:, t])[..., None]                                   # [B,H,1]
        u = np.einsum("bhi,bhij->bhj", k[:, t], S)                       # what the state returns for this key
        w = beta[:, t][..., None] * (v[:, t] - a * u)                    # V_new of Eq. 2: the correction that is written
        S = a[..., None] * S + k[:, t][..., :, None] * w[..., None, :]
        o[:, t] = np.einsum("bhi,bhij->bhj", q[:, t], S)
        if keep_states:
            states.append(S.copy())
    return (o, S, states) if keep_states else (o, S)


def delta_bwd(q, k, v, g, beta, S_in, dO, dS_out=None):
    """-> (dq, dk, dv, dg [B,T,H], dbeta [B,T,H], dS_in)."""
    q, k, v, g, beta, dO = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g, beta, dO))
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    _, _, st = delta_fwd(q, k, v, g, beta, S_in, keep_states=True)
    G = _z(dS_out, (B, H, dk, dv))
    dq, dk_, dv_ = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dg, dbeta = np.zeros_like(g), np.zeros_like(beta)
    for t in range(T - 1, -1, -1):
        Sp, St = st[t], st[t + 1]
        a = np.exp(g[:, t])                                              # [B,H]
        b = beta[:, t]
        u = np.einsum("bhi,bhij->bhj", k[:, t], Sp)
        w = b[..., None] * (v[:, t] - a[..., None] * u)
        G = G + q[:, t][..., :, None] * dO[:, t][..., None, :]
        dq[:, t] = np.einsum("bhj,bhij->bhi", dO[:, t], St)
        # S_t = a S_{t-1} + k^T w
        dw = np.einsum("bhi,bhij->bhj", k[:, t], G)
        dk_t = np.einsum("bhij,bhj->bhi", G, w)
        da = np.sum(G * Sp, axis=(-1, -2))
        # w = beta (v - a u)
        dbeta[:, t] = np.sum(dw * (v[:, t] - a[..., None] * u), axis=-1)
        dv_[:, t] = b[..., None] * dw
        da = da - b * np.sum(dw * u, axis=-1)
        du = -(a * b)[..., None] * dw
        # u = k S_{t-1}
        dk_t = dk_t + np.einsum("bhj,bhij->bhi", du, Sp)
        dk_[:, t] = dk_t
        dg[:, t] = a * da
        G = a[..., None, None] * G + k[:, t][..., :, None] * du[..., None, :]
    return dq, dk_, dv_, dg, dbeta, G


# ------------------------------------------------------------------------------------- short convolution ---

def conv_fwd(x, w, tail_in=None):
    """x [B,L,C]; w [W,C] (w[j] multiplies the input j tokens back); tail_in [B,W-1,C] = the W-1 inputs before the
    segment (None: zeros).  -> (y [B,L,C], tail_out [B,W-1,C] = the last W-1 inputs seen so far)."""
    x, w = np.asarray(x, dtype=np.float64), np.asarray(w, dtype=np.float64)
    B, L, C = x.shape
    W = w.shape[0]
    tail = _z(tail_in, (B, W - 1, C))
    ext = np.concatenate([tail, x], axis=1)                              # ext[:, W-1+t] = x_t
    y = np.zeros((B, L, C))
    for t in range(L):
        for j in range(W):
            y[:, t] += w[j] * ext[:, W - 1 + t - j]
    return y, ext[:, ext.shape[1] - (W - 1):].copy()


def conv_bwd(x, w, tail_in, dy, dtail_out=None):
    """-> (dx [B,L,C], dw [W,C], dtail_in [B,W-1,C])."""
    x, w, dy = (np.asarray(a, dtype=np.float64) for a in (x, w, dy))
    B, L, C = x.shape
    W = w.shape[0]
    tail = _z(tail_in, (B, W - 1, C))
    ext = np.concatenate([tail, x], axis=1)
    dext = np.zeros_like(ext)
    if dtail_out is not None:
        dext[:, ext.shape[1] - (W - 1):] += np.asarray(dtail_out, dtype=np.float64)
    dw = np.zeros((W, C))
    for t in range(L):
        for j in range(W):
            dext[:, W - 1 + t - j] += w[j] * dy[:, t]
            dw[j] += np.sum(dy[:, t] * ext[:, W - 1 + t - j], axis=0)
    return dext[:, W - 1:].copy(), dw, dext[:, :W - 1].copy()
