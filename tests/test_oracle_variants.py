"""Pins of the extension oracles (oracle/variants.py): diagonal decay, gated delta rule, short convolution.

Each pin is something other than the oracle's own formula: central differences of a scalar loss, the special case
that collapses to the scalar-decay oracle (a separate C program), split invariance of the boundary state (Eq. 5, 7),
the retrieval property that defines the delta rule, an explicit matrix-product form, and numpy's own convolution.
"""
import numpy as np
import pytest

import oracle
from oracle import variants as V


def rnd(seed, *shape, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def make(seed, B=1, T=9, H=2, dk=3, dv=4, channel=False):
    q, k = rnd(seed, B, T, H, dk), rnd(seed + 1, B, T, H, dk)
    v = rnd(seed + 2, B, T, H, dv)
    gshape = (B, T, H, dk) if channel else (B, T, H)
    g = -np.abs(rnd(seed + 3, *gshape, scale=0.3))
    beta = 1.0 / (1.0 + np.exp(-rnd(seed + 4, B, T, H)))
    S = rnd(seed + 5, B, H, dk, dv, scale=0.5)
    return q, k, v, g, beta, S


def fd(loss, x, idx, eps=1e-6):
    xp, xm = x.copy(), x.copy()
    xp[idx] += eps
    xm[idx] -= eps
    return (loss(xp) - loss(xm)) / (2 * eps)


def sample_idx(rng, shape, n=6):
    return [tuple(int(rng.integers(0, s)) for s in shape) for _ in range(n)]


# ------------------------------------------------------------------------------------------ diagonal decay ---

def test_channel_reduces_to_scalar_decay_when_all_channels_agree():
    q, k, v, g, _, S = make(10, B=2, T=33, H=2, dk=4, dv=3)
    gc = np.repeat(g[..., None], 4, axis=-1)
    o_ref, S_ref = oracle.segment_fwd(q, k, v, g, S)
    o, S_out = V.channel_fwd(q, k, v, gc, S)
    np.testing.assert_allclose(o, o_ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(S_out, S_ref, rtol=1e-12, atol=1e-12)
    dO, dS = rnd(20, *o.shape), rnd(21, *S.shape)
    r = oracle.segment_bwd(q, k, v, g, S, dO, dS)
    c = V.channel_bwd(q, k, v, gc, S, dO, dS)
    for a, b in zip((c[0], c[1], c[2], c[3].sum(-1), c[4]), r):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-11)


def test_channel_matches_independent_rows():
    # with a diagonal transition row i of S never meets row j: each row is a scalar-decay recurrence with d_k = 1
    q, k, v, g, _, S = make(11, T=17, H=1, dk=3, dv=2, channel=True)
    o, S_out = V.channel_fwd(q, k, v, g, S)
    acc = np.zeros_like(o)
    for i in range(3):
        oi, Si = oracle.segment_fwd(q[..., i:i + 1], k[..., i:i + 1], v, g[..., i], S[:, :, i:i + 1])
        acc += oi
        np.testing.assert_allclose(S_out[:, :, i:i + 1], Si, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(o, acc, rtol=1e-12, atol=1e-12)


def test_channel_gradients_match_central_differences():
    q, k, v, g, _, S = make(12, T=7, H=2, dk=3, dv=2, channel=True)
    dO, dS = rnd(30, 1, 7, 2, 2), rnd(31, *S.shape)
    names = ["q", "k", "v", "g", "S"]
    x = dict(q=q, k=k, v=v, g=g, S=S)
    grads = dict(zip(names, V.channel_bwd(q, k, v, g, S, dO, dS)))

    def loss_of(name):
        def f(val):
            a = dict(x)
            a[name] = val
            o, So = V.channel_fwd(a["q"], a["k"], a["v"], a["g"], a["S"])
            return np.sum(o * dO) + np.sum(So * dS)
        return f

    rng = np.random.default_rng(5)
    for n in names:
        for idx in sample_idx(rng, x[n].shape):
            assert grads[n][idx] == pytest.approx(fd(loss_of(n), x[n], idx), rel=1e-6, abs=1e-8), (n, idx)


def test_channel_split_invariance():
    q, k, v, g, _, S = make(13, T=21, channel=True)
    o, S_out = V.channel_fwd(q, k, v, g, S)
    dO, dS = rnd(40, *o.shape), rnd(41, *S.shape)
    full = V.channel_bwd(q, k, v, g, S, dO, dS)
    for cut in (1, 8, 20):
        a, b = slice(0, cut), slice(cut, None)
        o1, S1 = V.channel_fwd(q[:, a], k[:, a], v[:, a], g[:, a], S)
        o2, S2 = V.channel_fwd(q[:, b], k[:, b], v[:, b], g[:, b], S1)
        np.testing.assert_allclose(np.concatenate([o1, o2], 1), o, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(S2, S_out, rtol=1e-12, atol=1e-12)
        g2 = V.channel_bwd(q[:, b], k[:, b], v[:, b], g[:, b], S1, dO[:, b], dS)
        g1 = V.channel_bwd(q[:, a], k[:, a], v[:, a], g[:, a], S, dO[:, a], g2[4])
        for i in range(4):
            np.testing.assert_allclose(np.concatenate([g1[i], g2[i]], 1), full[i], rtol=1e-11, atol=1e-11)
        np.testing.assert_allclose(g1[4], full[4], rtol=1e-11, atol=1e-11)


# ---------------------------------------------------------------------------------------------- delta rule ---

def test_delta_with_beta_zero_is_pure_decay_and_beta_path_vanishes():
    q, k, v, g, _, S = make(50, T=12)
    o, S_out = V.delta_fwd(q, k, v, g, np.zeros(g.shape), S)
    # nothing is written: the state only decays, o_t = exp(cumsum g) q_t S_in
    c = np.exp(np.cumsum(g, axis=1))
    np.testing.assert_allclose(S_out, c[:, -1][..., None, None] * S, rtol=1e-12)
    np.testing.assert_allclose(o, c[..., None] * np.einsum("bthi,bhij->bthj", q, S), rtol=1e-12, atol=1e-13)


def test_delta_with_orthogonal_state_matches_scalar_decay_oracle():
    # if every key is orthogonal to everything already stored (u_t = 0) the correction is beta*v: the recurrence
    # is the plain one with values beta_t v_t.  Keys are distinct unit vectors, S_in = 0.
    B, T, H, dk, dv = 1, 5, 2, 5, 3
    q, _, v, g, beta, _ = make(51, B, T, H, dk, dv)
    k = np.zeros((B, T, H, dk))
    for t in range(T):
        k[:, t, :, t] = 1.0
    o, S_out = V.delta_fwd(q, k, v, g, beta, None)
    o_ref, S_ref = oracle.segment_fwd(q, k, beta[..., None] * v, g, None)
    np.testing.assert_allclose(o, o_ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(S_out, S_ref, rtol=1e-12, atol=1e-13)


def test_delta_rule_retrieval_property():
    # beta = 1, no decay, unit-norm key: after the write the state returns exactly v for that key
    q, k, v, g, _, S = make(52, T=6, H=1, dk=4, dv=3)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    o, _ = V.delta_fwd(k, k, v, np.zeros(g.shape), np.ones(g.shape), S)
    np.testing.assert_allclose(o, v, rtol=1e-12, atol=1e-12)


def test_delta_matches_explicit_transition_matrices():
    # S_t = a_t (I - beta_t k_t^T k_t) S_{t-1} + beta_t k_t^T v_t, unrolled as matrix products for one head
    q, k, v, g, beta, S = make(53, T=6, H=1, dk=3, dv=2)
    o, S_out = V.delta_fwd(q, k, v, g, beta, S)
    M = S[0, 0].copy()
    for t in range(6):
        kt, vt = k[0, t, 0][None, :], v[0, t, 0][None, :]
        F = np.exp(g[0, t, 0]) * (np.eye(3) - beta[0, t, 0] * kt.T @ kt)
        M = F @ M + beta[0, t, 0] * kt.T @ vt
        np.testing.assert_allclose(o[0, t, 0], (q[0, t, 0][None, :] @ M)[0], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(S_out[0, 0], M, rtol=1e-12, atol=1e-13)


def test_delta_gradients_match_central_differences():
    q, k, v, g, beta, S = make(54, T=7, H=2, dk=3, dv=2)
    dO, dS = rnd(60, 1, 7, 2, 2), rnd(61, *S.shape)
    names = ["q", "k", "v", "g", "beta", "S"]
    x = dict(q=q, k=k, v=v, g=g, beta=beta, S=S)
    grads = dict(zip(names, V.delta_bwd(q, k, v, g, beta, S, dO, dS)))

    def loss_of(name):
        def f(val):
            a = dict(x)
            a[name] = val
            o, So = V.delta_fwd(a["q"], a["k"], a["v"], a["g"], a["beta"], a["S"])
            return np.sum(o * dO) + np.sum(So * dS)
        return f

    rng = np.random.default_rng(6)
    for n in names:
        for idx in sample_idx(rng, x[n].shape, n=8):
            assert grads[n][idx] == pytest.approx(fd(loss_of(n), x[n], idx), rel=1e-6, abs=1e-8), (n, idx)


def test_delta_split_invariance():
    q, k, v, g, beta, S = make(55, T=19)
    o, S_out = V.delta_fwd(q, k, v, g, beta, S)
    dO, dS = rnd(70, *o.shape), rnd(71, *S.shape)
    full = V.delta_bwd(q, k, v, g, beta, S, dO, dS)
    for cut in (1, 7, 18):
        a, b = slice(0, cut), slice(cut, None)
        o1, S1 = V.delta_fwd(q[:, a], k[:, a], v[:, a], g[:, a], beta[:, a], S)
        o2, S2 = V.delta_fwd(q[:, b], k[:, b], v[:, b], g[:, b], beta[:, b], S1)
        np.testing.assert_allclose(np.concatenate([o1, o2], 1), o, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(S2, S_out, rtol=1e-12, atol=1e-12)
        g2 = V.delta_bwd(q[:, b], k[:, b], v[:, b], g[:, b], beta[:, b], S1, dO[:, b], dS)
        g1 = V.delta_bwd(q[:, a], k[:, a], v[:, a], g[:, a], beta[:, a], S, dO[:, a], g2[5])
        for i in range(5):
            np.testing.assert_allclose(np.concatenate([g1[i], g2[i]], 1), full[i], rtol=1e-11, atol=1e-11)
        np.testing.assert_allclose(g1[5], full[5], rtol=1e-11, atol=1e-11)


# ------------------------------------------------------------------------------------- short convolution ---

def test_conv_matches_numpy_convolve_and_carries_its_tail():
    B, L, C, W = 2, 23, 3, 4
    x, w = rnd(80, B, L, C), rnd(81, W, C)
    y, tail = V.conv_fwd(x, w, None)
    for b in range(B):
        for c in range(C):
            np.testing.assert_allclose(y[b, :, c], np.convolve(x[b, :, c], w[:, c])[:L], rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(tail, x[:, L - (W - 1):])
    for cut in (1, 2, 3, 11, 22):                       # a first part shorter than the tail included
        y1, t1 = V.conv_fwd(x[:, :cut], w, None)
        y2, t2 = V.conv_fwd(x[:, cut:], w, t1)
        np.testing.assert_allclose(np.concatenate([y1, y2], 1), y, rtol=1e-12, atol=1e-13)
        np.testing.assert_array_equal(t2, tail)


def test_conv_gradients_match_central_differences_and_split():
    B, L, C, W = 2, 9, 2, 4
    x, w, tail = rnd(90, B, L, C), rnd(91, W, C), rnd(92, B, W - 1, C)
    dy, dt = rnd(93, B, L, C), rnd(94, B, W - 1, C)
    arrs = dict(x=x, w=w, tail=tail)
    grads = dict(zip(["x", "w", "tail"], V.conv_bwd(x, w, tail, dy, dt)))

    def loss_of(name):
        def f(val):
            a = dict(arrs)
            a[name] = val
            y, to = V.conv_fwd(a["x"], a["w"], a["tail"])
            return np.sum(y * dy) + np.sum(to * dt)
        return f

    for n in arrs:
        for idx in np.ndindex(*arrs[n].shape):
            assert grads[n][idx] == pytest.approx(fd(loss_of(n), arrs[n], idx), rel=1e-6, abs=1e-8), (n, idx)
    for cut in (1, 2, 5):                               # gradient of the tail links the two halves (Eq. 7)
        _, t1 = V.conv_fwd(x[:, :cut], w, tail)
        dx2, dw2, dt1 = V.conv_bwd(x[:, cut:], w, t1, dy[:, cut:], dt)
        dx1, dw1, dt0 = V.conv_bwd(x[:, :cut], w, tail, dy[:, :cut], dt1)
        np.testing.assert_allclose(np.concatenate([dx1, dx2], 1), grads["x"], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(dw1 + dw2, grads["w"], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(dt0, grads["tail"], rtol=1e-12, atol=1e-13)


# ---- the chunkwise (UT transform) form of the delta rule, written out in numpy: a second algorithm for the same operator ----

def _chunk_fwd(Q, K, Vv, g, beta, H):
    C = Q.shape[0]
    b = np.cumsum(g)
    gam = np.exp(b)
    M = np.tril(np.exp(b[:, None] - b[None, :]))
    Ms = np.tril(M, -1)
    Kk = K @ K.T
    KH = K @ H
    # (I + L) W = beta*V - beta*gam*(K H),  L = diag(beta) (Ms * K K^T): the tokens of a chunk solved together
    W = np.linalg.solve(np.eye(C) + beta[:, None] * (Ms * Kk), beta[:, None] * Vv - (beta * gam)[:, None] * KH)
    QK = Q @ K.T
    A = M * QK
    om = np.exp(b[-1] - b)
    O = A @ W + gam[:, None] * (Q @ H)
    Hn = gam[-1] * H + K.T @ (om[:, None] * W)
    return O, Hn, dict(b=b, gam=gam, M=M, Ms=Ms, Kk=Kk, KH=KH, W=W, QK=QK, A=A, om=om, H=H)


def _chunk_bwd(Q, K, Vv, beta, c, dO, dHn):
    C = Q.shape[0]
    b, gam, M, Ms, Kk, KH, W, QK, A, om, H = (c[n] for n in ("b", "gam", "M", "Ms", "Kk", "KH", "W", "QK", "A", "om", "H"))
    KdH = K @ dHn
    dW = A.T @ dO + om[:, None] * KdH
    dA = dO @ W.T
    dQK = dA * M
    Z = np.linalg.solve((np.eye(C) + beta[:, None] * (Ms * Kk)).T, dW)
    dL = -np.tril(Z @ W.T, -1)
    bgZ = (beta * gam)[:, None] * Z
    P = beta[:, None] * dL * Ms
    dQ = dQK @ K + gam[:, None] * (dO @ H.T)
    dK = dQK.T @ Q + om[:, None] * (W @ dHn.T) - bgZ @ H.T + P @ K + P.T @ K
    dV = beta[:, None] * Z
    dbeta = np.sum(Z * Vv, axis=1) - gam * np.sum(Z * KH, axis=1) + np.sum(dL * Ms * Kk, axis=1)
    dH = gam[-1] * dHn + Q.T @ (gam[:, None] * dO) - K.T @ bgZ
    dgam = np.sum(dO * (Q @ H), axis=1) - beta * np.sum(Z * KH, axis=1)
    dom = np.sum(W * KdH, axis=1)
    E = (dA * QK * np.tril(np.ones((C, C))) + beta[:, None] * dL * Kk) * M
    db = E.sum(axis=1) - E.sum(axis=0) + dgam * gam - dom * om
    db[-1] += np.sum(dom * om) + np.sum(dHn * H) * gam[-1]
    return dQ, dK, dV, np.cumsum(db[::-1])[::-1], dbeta, dH


@pytest.mark.parametrize("T,C,dk,dv", [(50, 16, 5, 4), (64, 64, 8, 8), (33, 32, 3, 6)])
def test_delta_oracle_equals_the_chunkwise_ut_form(T, C, dk, dv):
    # Eq. 2 with V_new: Pre / ST / Out per chunk and their adjoints, against the token-by-token oracle (forward and backward)
    q, k, v, g, beta, S = make(56, T=T, H=1, dk=dk, dv=dv)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    dO, dS = rnd(80, *v.shape), rnd(81, *S.shape)
    o_ref, S_ref = V.delta_fwd(q, k, v, g, beta, S)
    ref = V.delta_bwd(q, k, v, g, beta, S, dO, dS)
    sl = [slice(t0, min(T, t0 + C)) for t0 in range(0, T, C)]
    H, caches, o = S[0, 0].copy(), [], np.zeros((T, dv))
    for s in sl:
        o[s], H, c = _chunk_fwd(q[0, s, 0], k[0, s, 0], v[0, s, 0], g[0, s, 0], beta[0, s, 0], H)
        caches.append(c)
    np.testing.assert_allclose(o, o_ref[0, :, 0], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(H, S_ref[0, 0], rtol=1e-11, atol=1e-12)
    dH = dS[0, 0].copy()
    got = [np.zeros((T, dk)), np.zeros((T, dk)), np.zeros((T, dv)), np.zeros(T), np.zeros(T)]
    for s, c in zip(sl[::-1], caches[::-1]):
        res = _chunk_bwd(q[0, s, 0], k[0, s, 0], v[0, s, 0], beta[0, s, 0], c, dO[0, s, 0], dH)
        for a, x in zip(got, res[:5]):
            a[s] = x
        dH = res[5]
    for a, r in zip(got, ref[:5]):
        np.testing.assert_allclose(a, r[0, :, 0], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dH, ref[5][0, 0], rtol=1e-9, atol=1e-11)


# ---- the chunkwise form of the diagonal decay in numpy: a second algorithm for the same operator --------------------

def _dchunk_fwd(Q, K, Vv, g, H):
    b = np.cumsum(g, axis=0)
    gam = np.exp(b)
    D = np.exp(b[:, None, :] - b[None, :, :])
    A = np.tril(np.einsum("ti,si,tsi->ts", Q, K, D))
    Kw = K * np.exp(b[-1][None, :] - b)
    Hn = gam[-1][:, None] * H + Kw.T @ Vv
    return A @ Vv + (Q * gam) @ H, Hn, dict(b=b, gam=gam, D=D, A=A, Kw=Kw, H=H, Hn=Hn)


def _dchunk_bwd(Q, K, Vv, c, dO, dHn):
    b, gam, D, A, Kw, H, Hn = (c[n] for n in ("b", "gam", "D", "A", "Kw", "H", "Hn"))
    dA = np.tril(dO @ Vv.T)
    dQ = np.einsum("ts,si,tsi->ti", dA, K, D) + gam * (dO @ H.T)
    dK = np.einsum("ts,ti,tsi->si", dA, Q, D) + np.exp(b[-1][None, :] - b) * (Vv @ dHn.T)
    dV = A.T @ dO + Kw @ dHn
    # rows of S are independent scalar recurrences: dg_t = dg_{t+1} + q dq - k dk per channel, anchored at the chunk end
    dg = np.cumsum((Q * dQ - K * dK)[::-1], axis=0)[::-1] + np.sum(dHn * Hn, axis=1)[None, :]
    return dQ, dK, dV, dg, gam[-1][:, None] * dHn + (Q * gam).T @ dO


@pytest.mark.parametrize("T,C,dk,dv", [(50, 16, 5, 4), (33, 32, 3, 6)])
def test_channel_oracle_equals_the_chunkwise_form(T, C, dk, dv):
    q, k, v, g, _, S = make(57, T=T, H=1, dk=dk, dv=dv, channel=True)
    dO, dS = rnd(90, *v.shape), rnd(91, *S.shape)
    o_ref, S_ref = V.channel_fwd(q, k, v, g, S)
    ref = V.channel_bwd(q, k, v, g, S, dO, dS)
    sl = [slice(t0, min(T, t0 + C)) for t0 in range(0, T, C)]
    H, caches, o = S[0, 0].copy(), [], np.zeros((T, dv))
    for s in sl:
        o[s], H, c = _dchunk_fwd(q[0, s, 0], k[0, s, 0], v[0, s, 0], g[0, s, 0], H)
        caches.append(c)
    np.testing.assert_allclose(o, o_ref[0, :, 0], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(H, S_ref[0, 0], rtol=1e-11, atol=1e-12)
    dH = dS[0, 0].copy()
    got = [np.zeros((T, dk)), np.zeros((T, dk)), np.zeros((T, dv)), np.zeros((T, dk))]
    for s, c in zip(sl[::-1], caches[::-1]):
        res = _dchunk_bwd(q[0, s, 0], k[0, s, 0], v[0, s, 0], c, dO[0, s, 0], dH)
        for a, x in zip(got, res[:4]):
            a[s] = x
        dH = res[4]
    for a, r in zip(got, ref[:4]):
        np.testing.assert_allclose(a, r[0, :, 0], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dH, ref[4][0, 0], rtol=1e-9, atol=1e-11)
