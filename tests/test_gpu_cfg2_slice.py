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


def test_config3_shapes_prm_at_target_shape():
    """Config-3 slice: 1.5B-shape draft, 7B-shape PRM and 7B-shape target, full depth and vocabulary; four rows,
    three steps of at most 3 tokens, one step at each threshold of the configuration's sweep (delta = 0.5, 0.7,
    0.9).  The gate is left to the GPU wherever the oracle's reward is more than 1e-2 away from delta: a random-init
    7B-shape PRM spreads its rewards over most of [0, 1], so the sweep accepts fewer and fewer rows."""
    import os
    if os.sysconf("SC_PAGE_SIZE") * os.sysconf("SC_PHYS_PAGES") < 90e9:
        pytest.skip("the oracle needs ~65 GB of host memory for two 7B-shape fp32 weight sets")
    shapes = (ri.SHAPES["1.5b"], ri.SHAPES["7b"], ri.SHAPES["7b"])
    prompts = ri.prompts(2, 4, 5, 8, shapes[0].vocab)
    base = dict(max_step_tokens=3, max_steps=3, max_seq_tokens=24, step_end_id=13, temperature=0.7, seed=3)
    eng, loop = build_pair(shapes, bf16=True, prompts=prompts, loop_kwargs=base)
    stats = {}
    accepted = []
    for delta in (0.5, 0.7, 0.9):
        g, o = parity_step(eng, loop, delta, stats=stats, **TOL16)
        accepted.append(int(g["accept"].sum()))
        assert np.all(o["rewards"] >= 0) and np.all(o["rewards"] <= 1)
    compare_counters(eng, loop)
    c = eng.counters()
    assert c["accepted_steps"] == sum(accepted) and c["rejected_steps"] == 12 - sum(accepted)
    assert c["rejected_steps"] > 0                      # the target ran (catch-up over prompt and accepted steps)
    print("config-3 shapes, 4 rows x 3 steps x <=3 tokens, delta 0.5 / 0.7 / 0.9: accepted", accepted, stats)
    eng.close()


def test_config4_width_loop_level():
    """Config 4 at the loop level: batch 8, a target of the 72B shape's width (d 8192, 64 / 8 heads, ffn 29568,
    vocabulary 152064 -- larger than the draft's and the PRM's 151936, so sampling is confined to the shared ids)
    with the 1.5B-width draft and PRM, all cut to two layers so that the oracle can hold them; the full depth of
    the 72B shape is covered by the layer-major test below.  Mixed accept / reject steps with the gate left to
    the GPU: logits, rewards, tokens, the rejected-row list, cursors and page tables against the oracle."""
    import dataclasses
    small = dataclasses.replace(ri.SHAPES["1.5b"], n_layers=2)
    wide = dataclasses.replace(ri.SHAPES["72b"], n_layers=2)
    shapes = (small, small, wide)
    prompts = ri.prompts(4, 8, 5, 20, small.vocab)
    base = dict(max_step_tokens=3, max_steps=3, max_seq_tokens=40, step_end_id=13, temperature=0.7, seed=11)
    eng, loop = build_pair(shapes, bf16=True, prompts=prompts, loop_kwargs=base)
    assert loop.v_limit == small.vocab < wide.vocab
    delta = float(np.sort(loop.step(0.0)["rewards"])[2])          # the quantile rule: about 70 % accepted
    eng, loop = build_pair(shapes, bf16=True, prompts=prompts, loop_kwargs=base)
    stats, seen = {}, set()
    for _ in range(3):
        g, o = parity_step(eng, loop, delta, stats=stats, **TOL16)
        seen |= set(int(a) for a, n in zip(o["accept"], o["step_len"]) if n)
    assert seen == {0, 1}
    compare_counters(eng, loop)
    print("config-4 width (two layers), 8 rows x 3 steps x <=3 tokens:", stats)
    eng.close()


def test_config4_shape_target_layer_major():
    """Config-4 slice: the 72B-shape target (80 layers, d 8192, vocab 152064) cannot be held by the
    oracle, so the oracle runs layer-major: weights of one layer at a time are generated, all tokens
    of a forced trace are pushed through it, and the layer is dropped.  The GPU is forced onto the
    same tokens; compared are the target's logits of every decode iteration (catch-up over the prompt
    included) for one row, full depth and full vocabulary."""
    import os
    import torch
    import oracle
    from oracle import OracleModel
    from paper_2501_19324_b200 import Engine, Model, RSD_DEBUG_KEEP_LOGITS, RSD_DRAFT, RSD_TARGET
    free, total = torch.cuda.mem_get_info()
    if total < 170e9:
        pytest.skip("needs a 180 GB GPU for the 72B-shape weights")
    sd, st = ri.SHAPES["1.5b"], ri.SHAPES["72b"]
    heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
    models = [Model(sh, ri.gpu_model_tensors(sh, slot, 0, True, hk), hk) for slot, (sh, hk) in enumerate(zip((sd, sd, st), heads))]
    rng = np.random.default_rng(5)
    prompt = rng.integers(0, sd.vocab, size=7).astype(np.int32)
    draft_step = rng.integers(0, sd.vocab, size=4).tolist()
    target_step = rng.integers(0, sd.vocab, size=4).tolist()
    got = {}
    for ext in (2, 0):          # plain 16-bit cache forced, and the library's default for an 80-layer model (hi + lo pairs)
        eng = Engine(*models, max_batch=1, max_seq_tokens=32, max_step_tokens=4, max_steps=2, step_end_id=13,
                     temperature=0.0, seed=0, debug_flags=RSD_DEBUG_KEEP_LOGITS, max_chunk_tokens=64, kv_extended=ext)
        eng.prefill(prompt, np.array([0, 7], np.int32))
        eng.force_tokens(RSD_DRAFT, [draft_step])
        eng.force_tokens(RSD_TARGET, [target_step])
        eng.force_accept([0])
        g = eng.step(0.5)
        assert g["accept"][0] == 0 and g["step_tokens"][0].tolist() == target_step
        got[ext] = eng.logits(RSD_TARGET)[0].copy()       # [4, V]: logits that chose step tokens 0..3
        eng.close()
    del models
    torch.cuda.empty_cache()
    # oracle, layer-major over the forced sequence prompt + target step (the last token is not fed)
    seq = prompt.tolist() + target_step[:-1]
    w = ri.cpu_model_weights(st, ri.SLOT_TARGET, 0, True, ri.HEAD_LM, with_layers=False)
    om = OracleModel(w, 2)
    x = om.embed(seq)
    cache = oracle.KVCache(1, len(seq), st.n_kv_heads * st.head_dim)
    for l in range(st.n_layers):
        lw = ri.cpu_layer_weights(st, ri.SLOT_TARGET, l, 0, True)
        ls = OracleModel._layer_struct(lw)
        oracle.lib().orc_layer_forward(om._cshape, ls, x.ctypes.data, len(seq), 0, cache.k[0].ctypes.data,
                                       cache.v[0].ctypes.data)
    errs = {2: [], 0: []}
    for j in range(4):
        want = om.logits(x[len(prompt) - 1 + j])
        for ext in (2, 0):
            errs[ext].append(float(np.abs(got[ext][j].astype(np.float64) - want).max()))
    print("config-4 target shape, 1 row, 7-token prompt + 4-token step: max logit errors, plain 16-bit KV", errs[2],
          "default (hi + lo pairs at this depth)", errs[0])
    # With keys, values, queries and softmax weights all at 11-bit mantissas (fp16) the residual stream
    # picks up about 5e-4 of relative error per layer, most of it from the rounded keys; over 80 layers
    # and 152 K logits of standard deviation 1.8 that is about 5e-2 at the worst logit, above the 3e-2
    # asked of bf16 arithmetic (28 layers: 1.5e-2).  kv_extended = 1 keeps keys and values as hi + lo
    # pairs and splits queries and softmax weights: the attention is then exact to fp32 rounding and
    # this shape lands near 2e-3, at twice the KV bytes.  The library therefore picks the pairs by itself for
    # models deeper than 48 layers (kv_extended = 0): the default configuration, which is also the one the
    # benchmark times for this shape, meets the bound asked of bf16 arithmetic.  The plain cache, which a
    # caller has to force (kv_extended = 2), is characterised only.
    assert max(errs[0]) <= 1e-2
    assert max(errs[2]) <= 1e-1 and max(errs[2]) > 3e-2 > max(errs[0])      # measured: 5e-2 to 7e-2 against 2e-3
