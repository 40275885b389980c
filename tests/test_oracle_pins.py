"""Pins of the fp64 oracle against things the paper and the mathematics fix.

None of these tests re-types the oracle's token loop: each compares it with an
independent statement of the same result (a matrix closed form, brute force,
a geometric series, finite differences, an adjoint identity, split invariance).
"""
import itertools

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(1234)


def rand_case(B, H, dk, dv, T, decay="config", s_in=True, ds_out=True, rng=RNG):
    q = rng.standard_normal((B, T, H, dk)) / np.sqrt(dk)
    k = rng.standard_normal((B, T, H, dk)) / np.sqrt(dk)
    v = rng.standard_normal((B, T, H, dv))
    z = rng.standard_normal((B, T, H))
    sp = np.log1p(np.exp(z))
    if decay == "zero":
        g = np.zeros((B, T, H))
    elif decay == "config":
        g = -sp
    elif decay == "weak":
        g = -0.01 * sp
    elif decay == "spike":
        g = -0.1 * sp
        g[:, T // 2] = -40.0
    else:
        raise ValueError(decay)
    dO = rng.standard_normal((B, T, H, dv))
    S_in = rng.standard_normal((B, H, dk, dv)) * 0.5 if s_in else None
    dS_out = rng.standard_normal((B, H, dk, dv)) * 0.5 if ds_out else None
    return q, k, v, g, S_in, dO, dS_out


SHAPES = [(1, 1, 1, 1, 8), (1, 1, 2, 3, 5), (2, 2, 4, 3, 16), (1, 2, 8, 8, 64)]
DECAYS = ["zero", "config", "weak", "spike"]


# ---------------------------------------------------------------- forward ---

def brute_force_fwd(q, k, v, g, S_in):
    """o = M V + diag(e^B) Q S_in with M[t,s] = e^{B_t - B_s} (q_t.k_s) for s <= t, B = cumsum(g)
    (the fully materialised decay-masked attention matrix)."""
    B_, T, H, dk = q.shape
    dv = v.shape[-1]
    o = np.zeros((B_, T, H, dv))
    S_out = np.zeros((B_, H, dk, dv))
    for b in range(B_):
        for h in range(H):
            Bc = np.cumsum(g[b, :, h])
            M = np.tril(np.exp(Bc[:, None] - Bc[None, :]) * (q[b, :, h] @ k[b, :, h].T))
            S0 = np.zeros((dk, dv)) if S_in is None else S_in[b, h]
            o[b, :, h] = M @ v[b, :, h] + np.exp(Bc)[:, None] * (q[b, :, h] @ S0)
            w = np.exp(Bc[-1] - Bc)
            S_out[b, h] = np.exp(Bc[-1]) * S0 + (w[:, None] * k[b, :, h]).T @ v[b, :, h]
    return o, S_out


@pytest.mark.parametrize("shape", SHAPES + [(1, 2, 32, 32, 256)])
@pytest.mark.parametrize("decay", DECAYS)
@pytest.mark.parametrize("s_in", [False, True])
def test_forward_matches_materialised_attention(shape, decay, s_in):
    q, k, v, g, S_in, _, _ = rand_case(*shape, decay=decay, s_in=s_in)
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    o_ref, S_ref = brute_force_fwd(q, k, v, g, S_in)
    np.testing.assert_allclose(o, o_ref, rtol=0, atol=1e-12 * max(1.0, np.abs(o_ref).max()))
    np.testing.assert_allclose(S_out, S_ref, rtol=0, atol=1e-12 * max(1.0, np.abs(S_ref).max()))


def test_zero_decay_is_causal_linear_attention():
    q, k, v, g, _, _, _ = rand_case(1, 2, 8, 5, 40, decay="zero", s_in=False)
    o, S_out = oracle.segment_fwd(q, k, v, g, None)
    for h in range(2):
        A = np.tril(q[0, :, h] @ k[0, :, h].T)
        np.testing.assert_allclose(o[0, :, h], A @ v[0, :, h], atol=1e-12)
        np.testing.assert_allclose(S_out[0, h], k[0, :, h].T @ v[0, :, h], atol=1e-12)


def test_scalar_geometric_series():
    # d_k = d_v = 1, q = k = v = 1, constant decay gamma: S_t = (1 - gamma^t) / (1 - gamma), o_t = S_t
    T, gamma = 50, 0.9
    one = np.ones((1, T, 1, 1))
    g = np.full((1, T, 1), np.log(gamma))
    o, S_out = oracle.segment_fwd(one, one, one, g, None)
    t = np.arange(1, T + 1)
    np.testing.assert_allclose(o[0, :, 0, 0], (1 - gamma ** t) / (1 - gamma), rtol=1e-13)
    np.testing.assert_allclose(S_out[0, 0, 0, 0], (1 - gamma ** T) / (1 - gamma), rtol=1e-13)


def test_single_token_by_hand():
    q = np.array([1.0, 2.0]).reshape(1, 1, 1, 2)
    k = np.array([3.0, -1.0]).reshape(1, 1, 1, 2)
    v = np.array([0.5, 4.0, -2.0]).reshape(1, 1, 1, 3)
    g = np.array([np.log(0.5)]).reshape(1, 1, 1)
    S_in = np.arange(6, dtype=float).reshape(1, 1, 2, 3)
    # S_1 = 0.5*S_in + k^T v
    S1 = 0.5 * S_in[0, 0] + np.array([[1.5, 12.0, -6.0], [-0.5, -4.0, 2.0]])
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    np.testing.assert_allclose(S_out[0, 0], S1, atol=1e-15)
    np.testing.assert_allclose(o[0, 0, 0], np.array([1.0, 2.0]) @ S1, atol=1e-15)
    # the token sees itself with weight 1 (decay applies to the old state only)
    o0, _ = oracle.segment_fwd(q, k, v, g, None)
    np.testing.assert_allclose(o0[0, 0, 0], (q.ravel() @ k.ravel()) * v.ravel(), atol=1e-15)


def test_linear_in_v_and_state():
    q, k, v, g, S_in, _, _ = rand_case(1, 2, 4, 3, 24)
    q2, k2, v2, g2, S2, _, _ = rand_case(1, 2, 4, 3, 24)
    oa, Sa = oracle.segment_fwd(q, k, v, g, S_in)
    ob, Sb = oracle.segment_fwd(q, k, v2, g, S2)
    oc, Sc = oracle.segment_fwd(q, k, 2 * v - 3 * v2, g, 2 * S_in - 3 * S2)
    np.testing.assert_allclose(oc, 2 * oa - 3 * ob, atol=1e-11)
    np.testing.assert_allclose(Sc, 2 * Sa - 3 * Sb, atol=1e-11)


def test_infinite_decay_forgets_everything_but_the_current_token():
    q, k, v, g, S_in, _, _ = rand_case(1, 1, 4, 3, 12)
    g = np.full_like(g, -800.0)          # exp underflows to exactly 0 in fp64
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    ref = np.einsum("btha,btha->bth", q, k)[..., None] * v
    np.testing.assert_allclose(o, ref, atol=1e-14)
    np.testing.assert_allclose(S_out[0, 0], np.outer(k[0, -1, 0], v[0, -1, 0]), atol=1e-14)


# --------------------------------------------------------------- backward ---

def loss(q, k, v, g, S_in, dO, dS_out):
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    val = np.sum(o * dO)
    if dS_out is not None:
        val += np.sum(S_out * dS_out)
    return val


@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 8), (1, 1, 2, 3, 5), (2, 2, 4, 3, 16)])
@pytest.mark.parametrize("decay", DECAYS)
@pytest.mark.parametrize("ds_out", [False, True])
def test_gradients_match_central_differences(shape, decay, ds_out):
    q, k, v, g, S_in, dO, dS_out = rand_case(*shape, decay=decay, ds_out=ds_out)
    if decay == "spike":
        g = np.maximum(g, -3.0)          # keep the spike differentiable at step 1e-6
    grads = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    args = [q, k, v, g, S_in]
    h = 1e-6
    for idx, (x, gx) in enumerate(zip(args, grads)):
        fd = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + h
            lp = loss(*args, dO, dS_out)
            x[i] = old - h
            lm = loss(*args, dO, dS_out)
            x[i] = old
            fd[i] = (lp - lm) / (2 * h)
        scale = max(np.abs(fd).max(), 1e-3)
        assert np.abs(fd - gx).max() / scale < 2e-7, "input %d" % idx


@pytest.mark.parametrize("decay", DECAYS)
def test_adjoint_identity(decay):
    # <dO, J d> + <dS_out, J_S d> == <J^T(dO, dS_out), d> for a random direction d of the linear inputs (v, S_in),
    # and a first-order check for the nonlinear ones (q, k, g) with a tiny step
    q, k, v, g, S_in, dO, dS_out = rand_case(1, 2, 8, 8, 64, decay=decay)
    dq, dk, dv, dg, dS_in = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    r = np.random.default_rng(7)
    d_v, d_S = r.standard_normal(v.shape), r.standard_normal(S_in.shape)
    o1, S1 = oracle.segment_fwd(q, k, d_v, g, d_S)        # linear in (v, S_in): J applied exactly
    lhs = np.sum(dO * o1) + np.sum(dS_out * S1)
    rhs = np.sum(dv * d_v) + np.sum(dS_in * d_S)
    assert abs(lhs - rhs) <= 1e-11 * max(1.0, abs(lhs))
    eps = 1e-6
    d_q, d_k, d_g = r.standard_normal(q.shape), r.standard_normal(k.shape), r.standard_normal(g.shape)
    lp = loss(q + eps * d_q, k + eps * d_k, v, g + eps * d_g, S_in, dO, dS_out)
    lm = loss(q - eps * d_q, k - eps * d_k, v, g - eps * d_g, S_in, dO, dS_out)
    rhs = np.sum(dq * d_q) + np.sum(dk * d_k) + np.sum(dg * d_g)
    assert abs((lp - lm) / (2 * eps) - rhs) <= 1e-6 * max(1.0, abs(rhs))


# The reverse sweep of the oracle replays states from checkpoints taken every clamp(floor(sqrt(T)), 16, 512) tokens and
# walks the windows backwards; the last window is shorter when T is not a multiple of the interval.  The shapes above
# have a single window (T <= 16) or only whole ones.  These have several windows and a short last one:
# T = 37 -> 16, 16, 5 ; T = 300 -> seventeen windows of 17 and one of 11.  d_k != d_v throughout.
@pytest.mark.parametrize("decay", DECAYS)
@pytest.mark.parametrize("ds_out", [False, True])
def test_gradients_match_central_differences_across_checkpoint_windows(decay, ds_out):
    q, k, v, g, S_in, dO, dS_out = rand_case(1, 1, 2, 3, 37, decay=decay, ds_out=ds_out, rng=np.random.default_rng(37))
    if decay == "spike":
        g = np.maximum(g, -3.0)
    grads = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    args = [q, k, v, g, S_in]
    h = 1e-6
    for idx, (x, gx) in enumerate(zip(args, grads)):
        fd = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + h
            lp = loss(*args, dO, dS_out)
            x[i] = old - h
            lm = loss(*args, dO, dS_out)
            x[i] = old
            fd[i] = (lp - lm) / (2 * h)
        scale = max(np.abs(fd).max(), 1e-3)
        assert np.abs(fd - gx).max() / scale < 2e-7, "input %d" % idx


@pytest.mark.parametrize("T", [37, 300])
@pytest.mark.parametrize("decay", DECAYS)
@pytest.mark.parametrize("ds_out", [False, True])
def test_adjoint_and_directional_derivatives_across_checkpoint_windows(T, decay, ds_out):
    q, k, v, g, S_in, dO, dS_out = rand_case(1, 2, 3, 5, T, decay=decay, ds_out=ds_out, rng=np.random.default_rng(T))
    if decay == "spike":
        g = np.maximum(g, -3.0)
    dq, dk, dv, dg, dS_in = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    r = np.random.default_rng(T + 1)
    # exact in the linear inputs (v, S_in)
    d_v, d_S = r.standard_normal(v.shape), r.standard_normal(S_in.shape)
    o1, S1 = oracle.segment_fwd(q, k, d_v, g, d_S)
    lhs = np.sum(dO * o1) + (np.sum(dS_out * S1) if ds_out else 0.0)
    rhs = np.sum(dv * d_v) + np.sum(dS_in * d_S)
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
    # several random directions of every input, one input at a time (so that an error in one gradient cannot hide
    # behind another), and directions confined to the last window and to the first one
    eps = 1e-6
    ckpt = min(max(int(np.floor(np.sqrt(T))), 16), 512)
    last0 = (T - 1) // ckpt * ckpt
    for name, x, gx in (("q", q, dq), ("k", k, dk), ("v", v, dv), ("g", g, dg)):
        for where in ("all", "last", "first"):
            d = r.standard_normal(x.shape)
            if where == "last":
                d[:, :last0] = 0.0
            elif where == "first":
                d[:, ckpt:] = 0.0
            a = dict(q=q, k=k, v=v, g=g)
            ap, am = dict(a), dict(a)
            ap[name] = x + eps * d
            am[name] = x - eps * d
            lp = loss(ap["q"], ap["k"], ap["v"], ap["g"], S_in, dO, dS_out)
            lm = loss(am["q"], am["k"], am["v"], am["g"], S_in, dO, dS_out)
            want = np.sum(gx * d)
            assert abs((lp - lm) / (2 * eps) - want) <= 2e-6 * max(1.0, abs(want)), (name, where)


def test_zero_decay_backward_closed_form():
    q, k, v, g, _, dO, _ = rand_case(1, 1, 6, 4, 32, decay="zero", s_in=False, ds_out=False)
    dq, dk, dv, dg, dS_in = oracle.segment_bwd(q, k, v, g, None, dO, None)
    Q, K, V, D = q[0, :, 0], k[0, :, 0], v[0, :, 0], dO[0, :, 0]
    dA = np.tril(D @ V.T)
    np.testing.assert_allclose(dq[0, :, 0], dA @ K, atol=1e-12)
    np.testing.assert_allclose(dk[0, :, 0], dA.T @ Q, atol=1e-12)
    np.testing.assert_allclose(dv[0, :, 0], np.tril(Q @ K.T).T @ D, atol=1e-12)
    np.testing.assert_allclose(dS_in[0, 0], Q.T @ D, atol=1e-12)


@pytest.mark.parametrize("decay", DECAYS)
def test_dg_telescoping_identity(decay):
    # dg_t - dg_{t+1} = q_t.dq_t - k_t.dk_t and dg_T = <dS_out, S_out> + (q_T.dq_T - k_T.dk_T):
    # an independent consequence of the recurrence that the token loop does not use
    q, k, v, g, S_in, dO, dS_out = rand_case(1, 2, 5, 7, 48, decay=decay)
    _, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    dq, dk, dv, dg, _ = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    x = np.sum(q * dq, -1) - np.sum(k * dk, -1)                       # [B,T,H]
    tail = np.einsum("bhij,bhij->bh", dS_out, S_out)
    ref = np.cumsum(x[:, ::-1], axis=1)[:, ::-1] + tail[:, None, :]
    np.testing.assert_allclose(dg, ref, atol=1e-10 * max(1.0, np.abs(ref).max()))
    # and k.dk == v.dv token by token (both equal k_t G v_t^T)
    np.testing.assert_allclose(np.sum(k * dk, -1), np.sum(v * dv, -1), atol=1e-11)


# ----------------------------------------------------- segment boundaries ---

def compositions(n):
    for mask in itertools.product([0, 1], repeat=n - 1):
        parts, run = [], 1
        for m in mask:
            if m:
                parts.append(run)
                run = 1
            else:
                run += 1
        parts.append(run)
        yield parts


def run_chain(case, seg_lens):
    q, k, v, g, S_in, dO, dS_out = case
    o, S_fin, S_ins = oracle.chain_fwd(q, k, v, g, seg_lens, S_in)
    return (o, S_fin) + tuple(oracle.chain_bwd(q, k, v, g, seg_lens, S_ins, dO, dS_out))


@pytest.mark.parametrize("decay", ["config", "weak"])
def test_every_split_of_a_short_sequence_equals_the_unsplit_run(decay):
    case = rand_case(1, 1, 2, 3, 6, decay=decay)
    ref = run_chain(case, [6])
    for parts in compositions(6):
        got = run_chain(case, parts)
        for a, b in zip(got, ref):
            np.testing.assert_allclose(a, b, atol=1e-12)


@pytest.mark.parametrize("decay", DECAYS)
def test_random_splits_equal_the_unsplit_run(decay):
    T, unit = 256, 32
    case = rand_case(1, 2, 32, 32, T, decay=decay)
    ref = run_chain(case, [T])
    r = np.random.default_rng(3)
    for _ in range(6):
        cuts = sorted(r.choice(np.arange(1, T // unit), size=r.integers(1, 5), replace=False) * unit)
        parts = list(np.diff([0] + list(cuts) + [T]))
        got = run_chain(case, parts)
        for a, b in zip(got, ref):
            np.testing.assert_allclose(a, b, atol=1e-11 * max(1.0, np.abs(b).max()))


def test_wrong_boundary_state_changes_the_result():
    # weak decay so that the incoming state matters for the whole segment
    case = list(rand_case(1, 1, 4, 4, 32, decay="weak"))
    q, k, v, g, S_in, dO, dS_out = case
    o_good, _, _ = oracle.chain_fwd(q, k, v, g, [16, 16], S_in)
    oa, Sa = oracle.segment_fwd(q[:, :16], k[:, :16], v[:, :16], g[:, :16], S_in)
    ob, _ = oracle.segment_fwd(q[:, 16:], k[:, 16:], v[:, 16:], g[:, 16:], None)     # state dropped
    assert np.abs(np.concatenate([oa, ob], 1) - o_good).max() > 1e-2


def test_batch_and_heads_are_independent():
    q, k, v, g, S_in, dO, dS_out = rand_case(2, 3, 4, 5, 20)
    o, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    grads = oracle.segment_bwd(q, k, v, g, S_in, dO, dS_out)
    b, h = 1, 2
    sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
    st = (slice(b, b + 1), slice(h, h + 1))
    o1, S1 = oracle.segment_fwd(q[sl], k[sl], v[sl], g[sl], S_in[st])
    np.testing.assert_allclose(o1, o[sl], atol=1e-14)
    np.testing.assert_allclose(S1, S_out[st], atol=1e-14)
    g1 = oracle.segment_bwd(q[sl], k[sl], v[sl], g[sl], S_in[st], dO[sl], dS_out[st])
    for a, full in zip(g1[:4], grads[:4]):
        np.testing.assert_allclose(a, full[sl], atol=1e-13)
    np.testing.assert_allclose(g1[4], grads[4][st], atol=1e-13)


# ------------------------------------------------------------------- scan ---

def test_scan_matches_textbook_recurrence_and_closed_form():
    r = np.random.default_rng(5)
    lanes, n, m = 3, 7, 5
    ld = -np.abs(r.standard_normal((lanes, n)))
    U = r.standard_normal((lanes, n, m))
    init = r.standard_normal((lanes, m))
    states, final = oracle.state_scan(ld, U, init)
    for l in range(lanes):
        x = init[l].copy()
        for j in range(n):
            np.testing.assert_allclose(states[l, j], x, atol=1e-14)
            x = np.exp(ld[l, j]) * x + U[l, j]
        np.testing.assert_allclose(final[l], x, atol=1e-14)
    # constant decay a, constant input u, zero start: X_j = u (1 - a^j) / (1 - a)
    a, u = 0.7, 2.0
    states, final = oracle.state_scan(np.full((1, n), np.log(a)), np.full((1, n, 1), u), None)
    j = np.arange(n)
    np.testing.assert_allclose(states[0, :, 0], u * (1 - a ** j) / (1 - a), rtol=1e-13)
    np.testing.assert_allclose(final[0, 0], u * (1 - a ** n) / (1 - a), rtol=1e-13)


def test_reverse_scan_is_forward_scan_on_reversed_blocks():
    r = np.random.default_rng(6)
    lanes, n, m = 2, 6, 4
    ld = -np.abs(r.standard_normal((lanes, n)))
    U = r.standard_normal((lanes, n, m))
    init = r.standard_normal((lanes, m))
    s_rev, f_rev = oracle.state_scan(ld, U, init, reverse=True)
    s_fwd, f_fwd = oracle.state_scan(ld[:, ::-1], U[:, ::-1], init)
    np.testing.assert_allclose(s_rev, s_fwd[:, ::-1], atol=1e-14)
    np.testing.assert_allclose(f_rev, f_fwd, atol=1e-14)


def test_scan_over_block_aggregates_reproduces_the_segment_state():
    # Aggregates U_j = S_out of block j run from a zero state, beta_j = sum of g over the block:
    # scanning them must give the token-level states at the block starts and S_out (Eq. 2's ST stage, Eq. 5).
    q, k, v, g, S_in, dO, dS_out = rand_case(1, 2, 4, 3, 48, decay="weak")
    blk = 16
    U, ld = [], []
    for j in range(3):
        sl = slice(j * blk, (j + 1) * blk)
        _, Uj = oracle.segment_fwd(q[:, sl], k[:, sl], v[:, sl], g[:, sl], None)
        U.append(Uj.reshape(2, -1))
        ld.append(g[0, sl].sum(0))
    states, final = oracle.state_scan(np.stack(ld, 1), np.stack(U, 1), S_in.reshape(2, -1))
    _, S_out = oracle.segment_fwd(q, k, v, g, S_in)
    np.testing.assert_allclose(final, S_out.reshape(2, -1), atol=1e-12)
    _, S_mid = oracle.segment_fwd(q[:, :blk], k[:, :blk], v[:, :blk], g[:, :blk], S_in)
    np.testing.assert_allclose(states[:, 1], S_mid.reshape(2, -1), atol=1e-12)


def test_oracle_runs_clean_under_the_address_and_undefined_behaviour_sanitizers(tmp_path):
    # the C oracle with exactly-sized buffers, several checkpoint windows with a short last one, with and without boundary
    # states, and the scan in both directions: any out-of-range index or undefined operation aborts the driver
    import os
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("gcc not available")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    exe = str(tmp_path / "oracle_san")
    build = subprocess.run(["gcc", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fopenmp", "-std=c11",
                            "-o", exe, os.path.join(root, "tests", "oracle_sanitizer_main.c"),
                            os.path.join(root, "oracle", "sf_oracle.c"), "-lm"], capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr.lower():
        pytest.skip("sanitizer runtime not installed: " + build.stderr[-200:])
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0 and "clean" in run.stdout, run.stdout + run.stderr
