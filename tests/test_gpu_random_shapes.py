"""Seeded random shapes through the chain driver against the fp64 oracle (one B200): batch, heads, segment lists with ragged
lengths, block lengths, overlap and replay modes drawn at random, on both kernel families."""
import random

import pytest
import torch

from paper_2608_06838_b200 import inputs
from paper_2608_06838_b200.inputs import Workload

from helpers import compare, oracle_reference, run_chain, tolerance

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def draw(seed):
    r = random.Random(seed)
    bf16 = r.random() < 0.5
    if bf16:
        d_k = d_v = 128
        chunk = 64
    else:
        d_k, d_v = r.choice([(32, 32), (64, 64), (32, 64), (128, 128)])
        chunk = r.choice([16, 32, 64])
    n_seg = r.randint(1, 5)
    seg_lens = [r.choice([1, r.randint(2, 90), r.randint(64, 700), chunk * r.randint(1, 9)]) for _ in range(n_seg)]
    w = Workload("rnd-%d" % seed, r.randint(1, 2), r.randint(1, 5), d_k, d_v, seg_lens, chunk, dtype="bf16" if bf16 else "f32",
                 qk_norm=r.choice(["l2", "scaled"]), g_scale=r.choice([1.0, 0.1, 0.01, 0.0]),
                 s_in_sigma=r.choice([None, 0.02, 0.5]), ds_out_sigma=r.choice([None, 0.02, 0.5]), seed=seed)
    kw = dict(chunks_per_block=r.choice([0, 0, 1, 2, 3, 5, 8, 13]), save_states=r.random() < 0.6, overlap=r.random() < 0.6)
    return w, kw


@pytest.mark.parametrize("seed", list(range(100, 124)))
def test_random_chain_matches_the_oracle(seed):
    w, kw = draw(seed)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    got, _ = run_chain(w, x, **kw)
    compare(got, oracle_reference(x), tolerance(w), label="%s %s %s" % (w.name, w.seg_lens, kw))


def draw_merged(seed):
    r = random.Random(seed)
    bf16 = r.random() < 0.6
    d, chunk = (128, 64) if bf16 else (r.choice([32, 64]), r.choice([16, 32, 64]))
    n_seg = r.randint(2, 7)
    # whole chunks except for the last segment: the chains the merged-launch schedule takes
    seg_lens = [chunk * r.randint(1, 12) for _ in range(n_seg - 1)] + [r.choice([chunk * r.randint(1, 9), r.randint(1, 500)])]
    w = Workload("rndm-%d" % seed, r.randint(1, 2), r.randint(1, 4), d, d, seg_lens, chunk, dtype="bf16" if bf16 else "f32",
                 qk_norm="l2", g_scale=r.choice([1.0, 0.1, 0.01, 0.0]), s_in_sigma=r.choice([None, 0.02, 0.5]),
                 ds_out_sigma=r.choice([None, 0.02]), seed=seed)
    kw = dict(chunks_per_block=r.choice([0, 0, 1, 3, 7, 16, 64]), save_states=r.random() < 0.6, overlap=r.random() < 0.6)
    return w, kw


@pytest.mark.parametrize("seed", list(range(500, 516)))
def test_random_chain_with_merged_launches_matches_the_oracle(seed):
    import numpy as np
    import oracle
    from paper_2608_06838_b200 import binding
    w, kw = draw_merged(seed)
    x = inputs.make_inputs(w, DEV)
    torch.cuda.synchronize()
    binding.sf_set_tuning(dict(merge_launches=1))
    try:
        got, run = run_chain(w, x, **kw)
    finally:
        binding.sf_set_tuning(None)
    compare(got, oracle_reference(x), tolerance(w), label="%s %s %s" % (w.name, w.seg_lens, kw))
    f = inputs.to_f64                                      # every boundary state against the oracle's chained run
    _, _, S_ins = oracle.chain_fwd(f(x["q"]), f(x["k"]), f(x["v"]), f(x["g"]), w.seg_lens, f(x["S_in"]))
    for i, ref in enumerate(S_ins):
        a = f(run.S_bounds[i])
        ref = np.zeros_like(a) if ref is None else ref
        assert np.abs(a - ref).max() <= tolerance(w) * max(np.abs(ref).max(), 1e-6), i
