"""Reduced slices of the full-size configurations: 1.5B-shape draft and PRM with the 7B-shape
target, bf16, full depth and vocabulary, teacher-forced on the oracle's tokens.  The scope of the
claim: a few rows, short prompts, short steps (the oracle's cost bounds it), every layer and every
logit column compared."""
import numpy as np
import pytest

import rsd_inputs as ri
from helpers import build_pair, parity_step, compare_counters

pytestmark = [pytest.mark.gpu, pytest.mark.slow]

TOL16 = dict(tol_logits=3e-2, tol_reward=1e-2, margin_tok=5e-2, margin_gate=1e-2)


def test_config2_shapes_reduced_slice():
    shapes = (ri.SHAPES["1.5b"], ri.SHAPES["1.5b"], ri.SHAPES["7b"])
    prompts = ri.prompts(1, 3, 9, 14, shapes[0].vocab)
    base = dict(max_step_tokens=4, max_steps=2, max_seq_tokens=32, step_end_id=13, temperature=0.7, seed=0)
    eng, loop = build_pair(shapes, bf16=True, prompts=prompts, loop_kwargs=base)
    stats = {}
    g, o = parity_step(eng, loop, 0.0, stats=stats, **TOL16)          # all accepted (delta = 0)
    r_first = o["rewards"].copy()
    delta = float(np.sort(r_first)[1]) + 0.02                          # next step: expect a mix
    g, o = parity_step(eng, loop, delta, stats=stats, **TOL16)
    compare_counters(eng, loop)
    print("config-2 shapes, 3 rows x 2 steps x <=4 tokens:", stats, "rejected:", o["rej_idx"])
    assert stats["tokens"] >= 12
