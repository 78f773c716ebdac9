"""Configs 2, 3 and 4 at their full sizes, in the launch configuration bench.py times (batch 32 / 64 / 8, prompts of
128-512 / 256 / 256 tokens, steps of up to 128 / 256 / 256 tokens, CUDA graphs): properties that hold at any size,
and for config 2 the one output the oracle can afford to compute on its own -- the first draft logits of the row with
the shortest prompt; plus the 7B-shape target against the oracle in the bucketed launch configuration."""
import numpy as np
import pytest

import rsd_inputs as ri

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


@pytest.mark.parametrize("config", ["cfg2", "cfg2-pairs", "cfg3", "cfg4"])
def test_full_size_properties_and_sampled_output(config):
    import torch
    from oracle import OracleModel
    from paper_2501_19324_b200 import Engine, Model, RSD_DEBUG_KEEP_LOGITS, RSD_DRAFT
    from paper_2501_19324_b200.binding import RSD_DEBUG_NO_F16_DENSE
    # "-pairs": the passes of more than 128 tokens keep bf16 weights x bf16 hi + lo operand pairs (the form the
    # 72B-shape target always takes) instead of the fp16 weight copies x one fp16 operand
    pairs = RSD_DEBUG_NO_F16_DENSE if config.endswith("-pairs") else 0
    config = config.split("-")[0]
    names, B, lo, hi, cap = {"cfg2": (("1.5b", "1.5b", "7b"), 32, 128, 512, 128),
                             "cfg3": (("1.5b", "7b", "7b"), 64, 256, 256, 256),
                             "cfg4": (("1.5b", "1.5b", "72b"), 8, 256, 256, 256)}[config]
    if config == "cfg4" and torch.cuda.mem_get_info()[1] < 170e9:
        pytest.skip("needs a 180 GB GPU for the 72B-shape weights")
    shapes = [ri.SHAPES[n] for n in names]
    heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
    models = [Model(sh, ri.gpu_model_tensors(sh, slot, 0, True, hk), hk) for slot, (sh, hk) in enumerate(zip(shapes, heads))]
    tokens, offsets = ri.prompts(1, B, lo, hi, shapes[0].vocab)
    lens = np.diff(offsets)

    def run(debug):
        eng = Engine(*models, max_batch=B, max_seq_tokens=hi + 3 * cap, max_step_tokens=cap, max_steps=3,
                     step_end_id=13, temperature=0.7, seed=0, debug_flags=debug | pairs)
        eng.prefill(tokens, offsets)
        r0 = eng.step(0.0)                                  # delta = 0: draft-only decoding
        delta = float(np.sort(r0["rewards"])[int(0.3 * B)])
        r1 = eng.step(delta)
        return eng, r0, r1, delta

    # the logits of every iteration are kept only where the oracle looks at them (config 2)
    eng, r0, r1, delta = run(RSD_DEBUG_KEEP_LOGITS if config == "cfg2" else 0)
    c = eng.counters()
    # delta = 0 accepted every row and never touched the target
    assert r0["accept"].all() and (r0["step_len"] == cap).sum() >= B - 2
    # rewards lie in [0, 1]; the gate is the threshold; the rejected list is the ascending complement
    for r in (r0, r1):
        assert np.all(r["rewards"] >= 0) and np.all(r["rewards"] <= 1)
    assert np.array_equal(r1["accept"], (r1["rewards"] >= np.float32(delta)).astype(np.uint8))
    st = eng.state()
    assert st["rej_idx"] == [b for b in range(B) if not r1["accept"][b]]
    assert np.array_equal(st["z_len"], lens + r0["step_len"] + r1["step_len"])
    assert np.array_equal(st["kv_len"][0][r1["accept"] == 1], st["z_len"][r1["accept"] == 1] - 1)
    for w in range(3):                                       # every page is owned by exactly one row
        pages = [p for row in st["pages"][w] for p in row]
        assert sorted(pages) == list(range(st["next_page"][w]))
    assert c["gen_tokens"][2] == int(r1["step_len"][r1["accept"] == 0].sum())
    assert c["gen_tokens"][0] == int(r0["step_len"].sum()) + int(c["score_tokens"] - r0["step_len"].sum())
    assert c["rejected_steps"] == int((r1["accept"] == 0).sum()) > 0 and c["accepted_steps"] == B + int(r1["accept"].sum())
    if config != "cfg2":
        eng.close()
        eng2, q0, q1, delta2 = run(0)                        # determinism of the whole run
        assert delta2 == delta and np.array_equal(q0["step_tokens"], r0["step_tokens"])
        assert np.array_equal(q1["step_tokens"], r1["step_tokens"]) and np.array_equal(q1["accept"], r1["accept"])
        eng2.close()
        print(f"full-size {config}: accepted {int(r1['accept'].sum())}/{B}, delta {delta:.4f}")
        return
    # sampled output: first draft logits of the shortest prompt against the oracle's full recompute
    b = int(np.argmin(lens))
    got = eng.logits(RSD_DRAFT)[b, 0]                        # logits of step 2's first token ... of the last step
    eng.close()
    om = OracleModel(ri.cpu_model_weights(shapes[0], 0, 0, True, ri.HEAD_LM), 0)
    seq = tokens[offsets[b]:offsets[b + 1]].tolist() + r0["step_tokens"][b, :r0["step_len"][b]].tolist()
    want = om.logits(om.forward_full(seq)[-1])               # context = prompt + the accepted first step
    err = float(np.abs(got.astype(np.float64) - want).max())
    print(f"full-size config 2: row {b} ({lens[b]}-token prompt + {r0['step_len'][b]}-token step), "
          f"max logit error of the next draft token {err:.4f}; accepted {int(r1['accept'].sum())}/{B}")
    assert err <= 3e-2
    # determinism: the same run again gives the same tokens and gate decisions
    eng2, q0, q1, delta2 = run(0)
    assert delta2 == delta and np.array_equal(q0["step_tokens"], r0["step_tokens"])
    assert np.array_equal(q1["step_tokens"], r1["step_tokens"]) and np.array_equal(q1["accept"], r1["accept"])
    eng2.close()



def test_target_decode_in_the_benchmarked_launch_configuration():
    """The else-branch of Algorithm 1 (y_i <- M(x, y_{1:i-1})) batched the way the benchmark runs it: a context of
    32 rows, the rejected rows compacted into the first slots, the target's decode iteration captured once per
    power-of-two bucket of their number (5 rows -> the 8-slot graph, 9 -> 16 slots, 17 -> 32 slots) and replayed
    from the second token on; the three patterns run one after the other on ONE context, as the buckets alternate
    in a benchmark run.  The target has the full 7B shape (28 layers, d 3584, vocabulary 151936); draft and PRM
    keep the 1.5B width at two layers, since they are not the subject and the oracle's time is better spent on
    the target.  Two of the rejected rows carry 9- to 14-token prompts (a real catch-up pass), the others 2-token
    prompts, which keeps the oracle affordable while every slot of the bucket is occupied.  Compared: every logit
    column of every target (and draft) iteration of every row at 3e-2, rewards, tokens, the rejected-row list,
    cursors and page tables bit for bit."""
    import dataclasses
    from helpers import build_pair, parity_step, compare_counters, compare_state
    from oracle.rsd_loop import OracleRSD
    small = dataclasses.replace(ri.SHAPES["1.5b"], n_layers=2)
    shapes = (small, small, ri.SHAPES["7b"])
    B, cap = 32, 3
    kw = dict(max_step_tokens=cap, max_steps=2, max_seq_tokens=32, step_end_id=13, temperature=0.7, seed=3)
    eng = loop = None
    for n_rejected in (5, 17, 9):
        rng = np.random.default_rng(100 + n_rejected)
        rejected = sorted(rng.choice(B, size=n_rejected, replace=False).tolist())
        long_rows = [rejected[0], rejected[-1]]                  # first and last slot of the compacted list
        lens = np.full(B, 2, dtype=np.int32)
        lens[long_rows] = rng.integers(9, 15, size=2)
        offsets = np.zeros(B + 1, dtype=np.int32)
        offsets[1:] = np.cumsum(lens)
        tokens = rng.integers(0, small.vocab, size=int(offsets[-1])).astype(np.int32)
        if eng is None:
            eng, loop = build_pair(shapes, bf16=True, prompts=(tokens, offsets), loop_kwargs=kw)
        else:
            eng.prefill(tokens, offsets)                         # drops the previous pattern's rows
            loop = OracleRSD(*loop.models, loop.cfg)
            loop.prefill([tokens[offsets[b]:offsets[b + 1]].tolist() for b in range(B)])
        compare_state(eng, loop)
        pattern = [0 if b in rejected else 1 for b in range(B)]
        stats = {}
        g, o = parity_step(eng, loop, 0.5, stats=stats, accept_pattern=pattern, tol_logits=3e-2, tol_reward=1e-2,
                           margin_tok=5e-2, margin_gate=1e-2)
        assert o["rej_idx"] == rejected and eng.state()["rej_idx"] == rejected
        assert not g["accept"][rejected].any() and g["accept"].sum() == B - n_rejected
        compare_counters(eng, loop)
        assert eng.counters()["gen_tokens"][2] == int(g["step_len"][rejected].sum())
        assert eng.counters()["ingest_tokens"][2] == int((lens[rejected] - 1).sum())
        print(f"7B-shape target, 32-row context, {n_rejected} rejected rows:", stats)
    eng.close()


def test_dense_pass_on_fp16_weight_copies_at_the_7b_shape():
    """Passes of more than 128 tokens run on fp16 copies of the layer matrices with ONE fp16 activation operand
    (instead of bf16 weights x bf16 hi + lo pairs).  A 150-token prompt beside a 3-token one makes the prefill of
    every model such a pass; PRM and target have the full 7B shape (28 layers, d 3584), the draft the 1.5B width at
    two layers.  Row 0's first step is rejected, so the target decodes from the cache the fp16 pass wrote: every
    logit column of every draft and target iteration within 3e-2 of the oracle, the 7B-shape PRM's rewards (read
    over the cache its fp16 prefill wrote) within 1e-2, tokens, cursors and page tables bit for bit."""
    import dataclasses
    import os
    from helpers import build_pair, parity_step, compare_counters, compare_state
    if os.sysconf("SC_PAGE_SIZE") * os.sysconf("SC_PHYS_PAGES") < 90e9:
        pytest.skip("the oracle needs ~65 GB of host memory for two 7B-shape fp32 weight sets")
    small = dataclasses.replace(ri.SHAPES["1.5b"], n_layers=2)
    shapes = (small, ri.SHAPES["7b"], ri.SHAPES["7b"])
    rng = np.random.default_rng(77)
    lens = np.array([150, 3], dtype=np.int32)
    offsets = np.zeros(3, dtype=np.int32)
    offsets[1:] = np.cumsum(lens)
    tokens = rng.integers(0, small.vocab, size=int(offsets[-1])).astype(np.int32)
    kw = dict(max_step_tokens=3, max_steps=2, max_seq_tokens=176, step_end_id=13, temperature=0.7, seed=5)
    eng, loop = build_pair(shapes, bf16=True, prompts=(tokens, offsets), loop_kwargs=kw)
    compare_state(eng, loop)
    stats = {}
    g, o = parity_step(eng, loop, 0.5, stats=stats, accept_pattern=[0, 1], tol_logits=3e-2, tol_reward=1e-2,
                       margin_tok=5e-2, margin_gate=1e-2)
    assert o["rej_idx"] == [0] and eng.state()["rej_idx"] == [0]
    compare_counters(eng, loop)
    print("fp16 dense passes, 7B-shape PRM and target after a 150-token prompt:", stats)
    eng.close()
