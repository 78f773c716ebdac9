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
    g, o = parity_step(eng, loop, 0.0, stats=stats, **TOL16)          # delta = 0: every draft step accepted
    assert g["accept"].all()
    # delta above the PRM's range: every row is rejected, so the target first catches up on the
    # prompt and the accepted step, then writes the step itself
    g, o = parity_step(eng, loop, 1.5, stats=stats, **TOL16)
    assert not g["accept"].any() and o["rej_idx"] == [0, 1, 2]
    compare_counters(eng, loop)
    print("config-2 shapes, 3 rows x 2 steps x <=4 tokens:", stats)
    assert stats["tokens"] >= 30
