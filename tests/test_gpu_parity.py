"""CUDA path vs the fp64 oracle, element by element, through the C ABI (one B200)."""
import numpy as np
import pytest
import torch

from paper_2608_06838_b200 import binding, inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check(w, **kw):
    x = inputs.make_inputs(w, DEV)
    got, _ = run_chain(w, x, **kw)
    ref = oracle_reference(x)
    return compare(got, ref, tolerance(w), label=w.name)


def test_config1_tiny_fp32():
    check(inputs.configs()[0])


@pytest.mark.parametrize("dk,dv,chunk", [(32, 32, 16), (64, 64, 32), (32, 64, 64), (128, 128, 64), (64, 64, 64)])
@pytest.mark.parametrize("g_scale", [1.0, 0.01, 0.0])
def test_fp32_shapes_and_decay_regimes(dk, dv, chunk, g_scale):
    w = Workload("f32-%d-%d-%d-g%g" % (dk, dv, chunk, g_scale), 2, 3, dk, dv, [4 * chunk, 7 * chunk, chunk], chunk,
                 dtype="f32", qk_norm="l2", g_scale=g_scale, s_in_sigma=0.5, ds_out_sigma=0.5, seed=3)
    check(w, chunks_per_block=3)


@pytest.mark.parametrize("dk,dv,chunk", [(32, 32, 32), (64, 64, 64), (32, 64, 16)])
def test_bf16_small_heads(dk, dv, chunk):
    w = Workload("bf16-%d-%d-%d" % (dk, dv, chunk), 1, 4, dk, dv, [8 * chunk, 3 * chunk], chunk, g_scale=0.1,
                 s_in_sigma=0.1, ds_out_sigma=0.1, seed=5)
    check(w, chunks_per_block=4)


@pytest.mark.parametrize("save_states", [True, False])
@pytest.mark.parametrize("overlap", [True, False])
def test_replay_and_overlap_modes_agree_bitwise(save_states, overlap):
    w = Workload("modes", 1, 2, 64, 64, [256, 128, 384], 32, dtype="f32", g_scale=0.1, s_in_sigma=0.3, ds_out_sigma=0.3, seed=9)
    x = inputs.make_inputs(w, DEV)
    base, _ = run_chain(w, x, chunks_per_block=2, save_states=True, overlap=False)
    got, _ = run_chain(w, x, chunks_per_block=2, save_states=save_states, overlap=overlap)
    for n in base:
        assert torch.equal(base[n], got[n]), n


def test_state_scan_matches_oracle_scan():
    import oracle
    B, H, d, n = 2, 3, 32, 5
    gen = torch.Generator(device=DEV).manual_seed(11)
    ld = -torch.rand(B, H, n, generator=gen, device=DEV)
    U = torch.randn(B, H, n, d, d, generator=gen, device=DEV)
    init = torch.randn(B, H, d, d, generator=gen, device=DEV)
    q = torch.empty(B, n * 32, H, d, device=DEV)
    g = torch.empty(B, n * 32, H, device=DEV)
    desc = binding.make_desc(q, q, g, 32, 1)
    for reverse in (False, True):
        for use_init in (True, False):
            states = torch.empty_like(U)
            fin = torch.empty_like(init)
            binding.sf_state_scan(desc, 1, reverse, ld, U, init if use_init else None, states, fin)
            torch.cuda.synchronize()
            s_ref, f_ref = oracle.state_scan(inputs.to_f64(ld).reshape(B * H, n), inputs.to_f64(U).reshape(B * H, n, d * d),
                                             inputs.to_f64(init).reshape(B * H, d * d) if use_init else None, reverse)
            assert np.abs(inputs.to_f64(states).reshape(B * H, n, d * d) - s_ref).max() <= 1e-5 * np.abs(s_ref).max()
            assert np.abs(inputs.to_f64(fin).reshape(B * H, d * d) - f_ref).max() <= 1e-5 * np.abs(f_ref).max()


def test_dropping_the_boundary_state_is_detected():
    # weak decay: the incoming state matters for the whole second segment
    w = Workload("neg", 1, 2, 32, 32, [128, 128], 32, dtype="f32", g_scale=0.01, s_in_sigma=0.5, seed=2)
    x = inputs.make_inputs(w, DEV)
    ref = oracle_reference(x)
    x_bad = dict(x)
    x_bad["S_in"] = None
    got, _ = run_chain(w, x_bad)
    with pytest.raises(AssertionError):
        compare(got, ref, tolerance(w), label="dropped state")
