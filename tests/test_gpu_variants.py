"""Extension operators (diagonal decay, gated delta rule, short convolution with a carried tail) through the C ABI
against their fp64 oracles, element by element, on chains of segments that hand the boundary state on (one B200)."""
import numpy as np
import pytest
import torch

from oracle import variants as V
from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import norm_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-4          # float32 kernels: max |x - ref| / max |ref| per output tensor
f64 = inputs.to_f64


def bounds(seg_lens):
    t = 0
    for n in seg_lens:
        yield t, t + n
        t += n


def run_recurrent(kind, w, x):
    """Chain of segments through sf_{channel,delta}_segment_{fwd,bwd}; returns the outputs over the whole sequence."""
    q, k, v, dO = x["q"], x["k"], x["v"], x["dO"]
    g = x["g_channel"] if kind.startswith("channel") else x["g"]
    beta = x["beta"]
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    o = torch.zeros_like(v)
    dq, dk_, dv_, dg = torch.zeros_like(q), torch.zeros_like(k), torch.zeros_like(v), torch.zeros_like(g)
    dbeta = torch.zeros_like(beta)
    S = [x["S_in"]]
    segs = list(bounds(w.seg_lens))
    for a, b in segs:
        d = binding.make_desc(q[:, a:b], v[:, a:b], x["g"][:, a:b], w.chunk)
        S_out = torch.empty(B, H, dk, dv, device=DEV)
        if kind == "channel":
            binding.sf_channel_segment_fwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], S[-1], o[:, a:b], S_out)
        elif kind == "channel_chunked":
            ws = torch.empty(binding.sf_channel_chunked_workspace_bytes(d, 0), dtype=torch.uint8, device=DEV)
            binding.sf_channel_chunked_fwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], S[-1], o[:, a:b], S_out, ws)
        elif kind == "delta_chunked":
            ws = torch.empty(binding.sf_delta_chunked_workspace_bytes(d, 0), dtype=torch.uint8, device=DEV)
            binding.sf_delta_chunked_fwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], beta[:, a:b], S[-1], o[:, a:b], S_out, ws)
        else:
            binding.sf_delta_segment_fwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], beta[:, a:b], S[-1], o[:, a:b], S_out)
        S.append(S_out)
    G = x["dS_out"]
    for i in range(len(segs) - 1, -1, -1):
        a, b = segs[i]
        d = binding.make_desc(q[:, a:b], v[:, a:b], x["g"][:, a:b], w.chunk)
        nws = (binding.sf_delta_chunked_workspace_bytes(d, 1) if kind == "delta_chunked" else
               binding.sf_channel_chunked_workspace_bytes(d, 1) if kind == "channel_chunked" else binding.sf_recurrent_workspace_bytes(d))
        ws = torch.empty(nws, dtype=torch.uint8, device=DEV)
        dS_in = torch.empty(B, H, dk, dv, device=DEV)
        if kind == "delta_chunked":
            binding.sf_delta_chunked_bwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], beta[:, a:b], S[i], dO[:, a:b], G,
                                         dq[:, a:b], dk_[:, a:b], dv_[:, a:b], dg[:, a:b], dbeta[:, a:b], dS_in, ws)
        elif kind == "channel_chunked":
            binding.sf_channel_chunked_bwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], S[i], dO[:, a:b], G,
                                           dq[:, a:b], dk_[:, a:b], dv_[:, a:b], dg[:, a:b], dS_in, ws)
        elif kind == "channel":
            binding.sf_channel_segment_bwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], S[i], dO[:, a:b], G,
                                           dq[:, a:b], dk_[:, a:b], dv_[:, a:b], dg[:, a:b], dS_in, ws)
        else:
            binding.sf_delta_segment_bwd(d, q[:, a:b], k[:, a:b], v[:, a:b], g[:, a:b], beta[:, a:b], S[i], dO[:, a:b], G,
                                         dq[:, a:b], dk_[:, a:b], dv_[:, a:b], dg[:, a:b], dbeta[:, a:b], dS_in, ws)
        G = dS_in
    torch.cuda.synchronize()
    out = dict(o=o, S_out=S[-1], dq=dq, dk=dk_, dv=dv_, dg=dg, dS_in=G)
    if kind.startswith("delta"):
        out["dbeta"] = dbeta
    return out


def oracle_recurrent(kind, x):
    q, k, v, dO = (f64(x[n]) for n in ("q", "k", "v", "dO"))
    S_in, dS_out = f64(x["S_in"]), f64(x["dS_out"])
    if kind == "channel":
        g = f64(x["g_channel"])
        o, S_out = V.channel_fwd(q, k, v, g, S_in)
        dq, dk, dv, dg, dS_in = V.channel_bwd(q, k, v, g, S_in, dO, dS_out)
        return dict(o=o, S_out=S_out, dq=dq, dk=dk, dv=dv, dg=dg, dS_in=dS_in)
    g, beta = f64(x["g"]), f64(x["beta"])                 # "delta" and "delta_chunked": the same operator
    o, S_out = V.delta_fwd(q, k, v, g, beta, S_in)
    dq, dk, dv, dg, dbeta, dS_in = V.delta_bwd(q, k, v, g, beta, S_in, dO, dS_out)
    return dict(o=o, S_out=S_out, dq=dq, dk=dk, dv=dv, dg=dg, dbeta=dbeta, dS_in=dS_in)


def check(got, ref, label, tol=TOL):
    errs = {}
    for n, r in ref.items():
        a = f64(got[n])
        assert np.isfinite(a).all(), "%s %s has non-finite values" % (label, n)
        errs[n] = norm_err(a, r)
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, "%s: normalised max error above %.0e: %s (all %s)" % (label, tol, bad, errs)


@pytest.mark.parametrize("kind", ["channel", "delta"])
@pytest.mark.parametrize("dk,dv", [(32, 32), (64, 64), (32, 128), (64, 32), (32, 64), (64, 128)])
def test_chained_segments_match_the_oracle(kind, dk, dv):
    # segment lengths: several 16-token tiles with a ragged tail, exactly one tile, shorter than a tile, one token
    w = Workload("%s-%d-%d" % (kind, dk, dv), 2, 3, dk, dv, [37, 16, 100, 5, 1], 64, dtype="f32", qk_norm="l2", g_scale=0.3,
                 s_in_sigma=0.5, ds_out_sigma=0.5, seed=21)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent(kind, w, x), oracle_recurrent(kind, x), w.name)


@pytest.mark.parametrize("kind", ["channel", "delta"])
@pytest.mark.parametrize("dk,dv", [(64, 64), (32, 128)])
def test_bf16_storage_matches_the_oracle_on_the_same_bits(kind, dk, dv):
    # bf16 q, k, v, dO in and o, dq, dk, dv out; arithmetic, decays, beta and states stay float32.  The oracle gets the
    # bf16 values widened to fp64, so only the rounding of the stored outputs and float32 arithmetic separate the two.
    w = Workload("%s-bf16-%d-%d" % (kind, dk, dv), 2, 3, dk, dv, [37, 16, 100, 5, 1], 64, dtype="bf16", qk_norm="l2", g_scale=0.3,
                 s_in_sigma=0.5, ds_out_sigma=0.5, seed=27)
    x = inputs.make_variant_inputs(w, DEV)
    assert x["q"].dtype == torch.bfloat16
    check(run_recurrent(kind, w, x), oracle_recurrent(kind, x), w.name, tol=2e-2)


@pytest.mark.parametrize("kind", ["channel", "delta"])
@pytest.mark.parametrize("g_scale", [1.0, 0.01, 0.0])
def test_decay_regimes_and_absent_boundary_states(kind, g_scale):
    w = Workload("%s-g%g" % (kind, g_scale), 1, 2, 64, 64, [64, 200], 64, dtype="f32", qk_norm="l2", g_scale=g_scale, seed=22)
    x = inputs.make_variant_inputs(w, DEV)
    assert x["S_in"] is None and x["dS_out"] is None
    check(run_recurrent(kind, w, x), oracle_recurrent(kind, x), w.name)


@pytest.mark.parametrize("kind", ["channel", "delta"])
def test_long_segment_and_bit_reproducibility(kind):
    w = Workload("%s-long" % kind, 1, 4, 64, 64, [2048], 64, dtype="f32", qk_norm="l2", g_scale=0.1, s_in_sigma=0.3,
                 ds_out_sigma=0.3, seed=23)
    x = inputs.make_variant_inputs(w, DEV)
    a = run_recurrent(kind, w, x)
    b = run_recurrent(kind, w, x)
    for n in a:
        assert torch.equal(a[n], b[n]), n
    check(a, oracle_recurrent(kind, x), w.name)


def test_delta_rule_with_beta_zero_only_decays():
    # beta = 0: nothing is written, so o_t = exp(cumsum g) q_t S_in; compared with the fp64 closed form
    w = Workload("delta-b0", 1, 2, 32, 32, [48], 64, dtype="f32", g_scale=0.2, s_in_sigma=1.0, seed=24)
    x = inputs.make_variant_inputs(w, DEV)
    x["beta"] = torch.zeros_like(x["beta"])
    got = run_recurrent("delta", w, x)
    c = np.exp(np.cumsum(f64(x["g"]), axis=1))
    ref_o = c[..., None] * np.einsum("bthi,bhij->bthj", f64(x["q"]), f64(x["S_in"]))
    assert norm_err(f64(got["o"]), ref_o) <= TOL
    assert norm_err(f64(got["S_out"]), c[:, -1][..., None, None] * f64(x["S_in"])) <= TOL


# channel counts: 96 and 260 (16-byte accesses, the second with a partly filled last group of threads), 7 (scalar path)
@pytest.mark.parametrize("H,dv", [(3, 32), (5, 52), (1, 7)])
@pytest.mark.parametrize("W,seg_lens", [(4, [37, 2, 1, 88]), (2, [5, 123]), (1, [64, 64]), (8, [3, 300, 7]), (4, [700, 257, 32])])
def test_conv_chain_matches_the_oracle(W, seg_lens, H, dv):
    w = Workload("conv-%d" % W, 2, H, 32, dv, seg_lens, 64, dtype="f32", seed=25)
    x = inputs.make_variant_inputs(w, DEV, conv_width=W)
    X, Wt, dY = x["conv_x"], x["conv_w"], x["conv_dy"]
    B, T, C = X.shape
    tail0 = x["conv_tail"] if W > 1 else None
    dtail = x["conv_dtail"] if W > 1 else None
    y = torch.zeros_like(X)
    tails = [tail0]
    segs = list(bounds(seg_lens))
    for a, b in segs:
        t_out = torch.empty(B, W - 1, C, device=DEV) if W > 1 else None
        y_seg = torch.empty(B, b - a, C, device=DEV)
        binding.sf_conv_segment_fwd(X[:, a:b].contiguous(), Wt, tails[-1], y_seg, t_out)
        y[:, a:b] = y_seg
        tails.append(t_out)
    dx = torch.zeros_like(X)
    dw = torch.zeros(W, C, dtype=torch.float64, device=DEV)
    G = dtail
    for i in range(len(segs) - 1, -1, -1):
        a, b = segs[i]
        dx_seg, dw_seg = torch.empty(B, b - a, C, device=DEV), torch.empty(W, C, device=DEV)
        dt_in = torch.empty(B, W - 1, C, device=DEV) if W > 1 else None
        binding.sf_conv_segment_bwd(X[:, a:b].contiguous(), Wt, tails[i], dY[:, a:b].contiguous(), G, dx_seg, dw_seg, dt_in)
        dx[:, a:b] = dx_seg
        dw += dw_seg.double()
        G = dt_in
    torch.cuda.synchronize()
    ry, rt = V.conv_fwd(f64(X), f64(Wt), f64(tail0))
    rdx, rdw, rdt = V.conv_bwd(f64(X), f64(Wt), f64(tail0), f64(dY), f64(dtail))
    assert norm_err(f64(y), ry) <= TOL
    assert norm_err(f64(dx), rdx) <= TOL
    assert norm_err(f64(dw), rdw) <= TOL
    if W > 1:
        assert np.array_equal(f64(tails[-1]), rt)           # a copy: exact
        assert norm_err(f64(G), rdt) <= TOL


def test_launches_are_counted():
    w = Workload("count", 1, 1, 32, 32, [16], 64, dtype="f32", seed=26)
    x = inputs.make_variant_inputs(w, DEV)
    n0 = binding.sf_launch_count()
    run_recurrent("delta", w, x)
    assert binding.sf_launch_count() - n0 == 2


# ---- chunkwise (UT transform) form of the delta rule: same operator, same oracle -------------------------------------

@pytest.mark.parametrize("chunk", [16, 32])
@pytest.mark.parametrize("dk,dv", [(32, 32), (64, 64), (32, 64), (64, 32)])
def test_chunked_delta_rule_matches_the_oracle(chunk, dk, dv):
    # segments of several chunks with a ragged last one, exactly one chunk, shorter than a chunk, one token
    w = Workload("chunked-%d-%d-%d" % (chunk, dk, dv), 2, 3, dk, dv, [3 * chunk + 5, chunk, 100, 5, 1], chunk, dtype="f32",
                 qk_norm="l2", g_scale=0.3, s_in_sigma=0.5, ds_out_sigma=0.5, seed=31)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent("delta_chunked", w, x), oracle_recurrent("delta", x), w.name)


@pytest.mark.parametrize("g_scale", [1.0, 0.01, 0.0])
def test_chunked_delta_rule_decay_regimes_and_absent_boundary_states(g_scale):
    w = Workload("chunked-g%g" % g_scale, 1, 2, 64, 64, [64, 200], 32, dtype="f32", qk_norm="l2", g_scale=g_scale, seed=32)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent("delta_chunked", w, x), oracle_recurrent("delta", x), w.name)


def test_chunked_delta_rule_long_segment_bf16_and_agreement_with_the_token_kernel():
    w = Workload("chunked-long", 1, 4, 64, 64, [2048], 32, dtype="f32", qk_norm="l2", g_scale=0.1, s_in_sigma=0.3,
                 ds_out_sigma=0.3, seed=33)
    x = inputs.make_variant_inputs(w, DEV)
    a = run_recurrent("delta_chunked", w, x)
    b = run_recurrent("delta_chunked", w, x)
    for n in a:
        assert torch.equal(a[n], b[n]), n                      # deterministic
    check(a, oracle_recurrent("delta", x), w.name)
    t = run_recurrent("delta", w, x)                           # the token-recurrent kernel: same operator, other algorithm
    for n in a:
        assert norm_err(f64(a[n]), f64(t[n])) <= 2 * TOL, n
    wb = Workload("chunked-bf16", 2, 3, 64, 32, [37, 16, 100, 5, 1], 16, dtype="bf16", qk_norm="l2", g_scale=0.3, s_in_sigma=0.5,
                  ds_out_sigma=0.5, seed=34)
    xb = inputs.make_variant_inputs(wb, DEV)
    check(run_recurrent("delta_chunked", wb, xb), oracle_recurrent("delta", xb), wb.name, tol=2e-2)


# ---- chunkwise form of the diagonal decay: same operator, same oracle -------------------------------------------------

@pytest.mark.parametrize("chunk", [16, 32])
@pytest.mark.parametrize("dk,dv", [(32, 32), (64, 64), (32, 64), (64, 32)])
def test_chunked_diagonal_decay_matches_the_oracle(chunk, dk, dv):
    w = Workload("dchunk-%d-%d-%d" % (chunk, dk, dv), 2, 3, dk, dv, [3 * chunk + 5, chunk, 100, 5, 1], chunk, dtype="f32",
                 qk_norm="l2", g_scale=0.3, s_in_sigma=0.5, ds_out_sigma=0.5, seed=41)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent("channel_chunked", w, x), oracle_recurrent("channel", x), w.name)


@pytest.mark.parametrize("g_scale", [1.0, 0.01, 0.0])
def test_chunked_diagonal_decay_regimes_and_absent_boundary_states(g_scale):
    w = Workload("dchunk-g%g" % g_scale, 1, 2, 64, 64, [64, 200], 32, dtype="f32", qk_norm="l2", g_scale=g_scale, seed=42)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent("channel_chunked", w, x), oracle_recurrent("channel", x), w.name)


def test_chunked_diagonal_decay_long_segment_bf16_and_agreement_with_the_token_kernel():
    w = Workload("dchunk-long", 1, 4, 64, 64, [2048], 32, dtype="f32", qk_norm="l2", g_scale=0.1, s_in_sigma=0.3,
                 ds_out_sigma=0.3, seed=43)
    x = inputs.make_variant_inputs(w, DEV)
    a = run_recurrent("channel_chunked", w, x)
    b = run_recurrent("channel_chunked", w, x)
    for n in a:
        assert torch.equal(a[n], b[n]), n
    check(a, oracle_recurrent("channel", x), w.name)
    t = run_recurrent("channel", w, x)
    for n in a:
        assert norm_err(f64(a[n]), f64(t[n])) <= 2 * TOL, n
    wb = Workload("dchunk-bf16", 2, 3, 64, 32, [37, 16, 100, 5, 1], 16, dtype="bf16", qk_norm="l2", g_scale=0.3, s_in_sigma=0.5,
                  ds_out_sigma=0.5, seed=44)
    xb = inputs.make_variant_inputs(wb, DEV)
    check(run_recurrent("channel_chunked", wb, xb), oracle_recurrent("channel", xb), wb.name, tol=2e-2)


@pytest.mark.parametrize("kind", ["delta_chunked", "channel_chunked"])
def test_chunked_operators_with_128_wide_heads(kind):
    # the head width of the paper's models; the tiles fit into shared memory with 16-token chunks
    w = Workload("%s-128" % kind, 1, 2, 128, 128, [53, 16, 7], 16, dtype="f32", qk_norm="l2", g_scale=0.3, s_in_sigma=0.5,
                 ds_out_sigma=0.5, seed=51)
    x = inputs.make_variant_inputs(w, DEV)
    check(run_recurrent(kind, w, x), oracle_recurrent("delta" if kind == "delta_chunked" else "channel", x), w.name)
    wb = Workload("%s-128-bf16" % kind, 2, 2, 128, 128, [40, 9], 16, dtype="bf16", qk_norm="l2", g_scale=0.3, s_in_sigma=0.5,
                  ds_out_sigma=0.5, seed=52)
    xb = inputs.make_variant_inputs(wb, DEV)
    check(run_recurrent(kind, wb, xb), oracle_recurrent("delta" if kind == "delta_chunked" else "channel", xb), wb.name, tol=2e-2)
