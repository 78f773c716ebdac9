"""Config 2 at its full size, in the launch configuration bench.py times (batch 32, prompts of 128 to 512
tokens, steps of up to 128 tokens, CUDA graphs): properties that hold at any size, and the one output
the oracle can afford to compute on its own -- the first draft logits of the row with the shortest
prompt."""
import numpy as np
import pytest

import rsd_inputs as ri

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


def test_config2_full_size_properties_and_sampled_output():
    from oracle import OracleModel
    from paper_2501_19324_b200 import Engine, Model, RSD_DEBUG_KEEP_LOGITS, RSD_DRAFT
    shapes = [ri.SHAPES["1.5b"], ri.SHAPES["1.5b"], ri.SHAPES["7b"]]
    heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
    models = [Model(sh, ri.gpu_model_tensors(sh, slot, 0, True, hk), hk) for slot, (sh, hk) in enumerate(zip(shapes, heads))]
    B, cap = 32, 128
    tokens, offsets = ri.prompts(1, B, 128, 512, shapes[0].vocab)
    lens = np.diff(offsets)

    def run(debug):
        eng = Engine(*models, max_batch=B, max_seq_tokens=512 + 3 * cap, max_step_tokens=cap, max_steps=3,
                     step_end_id=13, temperature=0.7, seed=0, debug_flags=debug)
        eng.prefill(tokens, offsets)
        r0 = eng.step(0.0)                                  # delta = 0: draft-only decoding
        delta = float(np.sort(r0["rewards"])[int(0.3 * B)])
        r1 = eng.step(delta)
        return eng, r0, r1, delta

    eng, r0, r1, delta = run(RSD_DEBUG_KEEP_LOGITS)
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
