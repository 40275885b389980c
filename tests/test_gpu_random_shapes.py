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
