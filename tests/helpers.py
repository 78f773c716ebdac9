"""Shared pieces of the GPU parity tests: build the same three models for the CUDA library and for
the oracle from the seeded generators, then walk the step loop with the GPU teacher-forced on the
oracle's tokens and compare everything the step returns plus the integer state."""
from __future__ import annotations

import numpy as np

import rsd_inputs as ri
from oracle import OracleModel
from oracle.rsd_loop import OracleRSD, LoopConfig, DRAFT, PRM, TARGET


def build_pair(shapes, *, bf16, seed=0, prompts, loop_kwargs, engine_kwargs=None):
    """shapes = (draft, prm, target) ModelShape.  Returns (engine, oracle_loop)."""
    from paper_2501_19324_b200 import Engine, Model, RSD_DEBUG_KEEP_LOGITS
    heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
    merged = bool(loop_kwargs.get("prm_shares_draft"))     # the PRM is its head on the draft's trunk
    gpu_models = [Model(sh, ri.gpu_model_tensors(sh, slot, seed, bf16, hk), hk, head_only=merged and slot == PRM)
                  for slot, (sh, hk) in enumerate(zip(shapes, heads))]
    cpu_models = [OracleModel(ri.cpu_model_weights(sh, slot, seed, bf16, hk, with_layers=not (merged and slot == PRM)), slot)
                  for slot, (sh, hk) in enumerate(zip(shapes, heads))]
    tokens, offsets = prompts
    B = len(offsets) - 1
    kw = dict(max_batch=B, debug_flags=RSD_DEBUG_KEEP_LOGITS)
    kw.update({k: loop_kwargs[k] for k in ("max_seq_tokens", "max_step_tokens", "max_steps", "step_end_id",
                                           "eos_id", "step_end_mod", "temperature", "seed", "sd_tokens") if k in loop_kwargs})
    # loop_kwargs may also carry oracle-only settings (omega_kind, omega_b); the engine takes its own
    if merged:
        kw["prm_shares_draft"] = 1
    kw.update(engine_kwargs or {})
    eng = Engine(*gpu_models, **kw)
    loop = OracleRSD(*cpu_models, LoopConfig(keep_logits=True, **loop_kwargs))
    eng.prefill(tokens, offsets)
    loop.prefill([tokens[offsets[b]:offsets[b + 1]].tolist() for b in range(B)])
    return eng, loop


def compare_state(eng, loop):
    g, o = eng.state(), loop.state()
    assert np.array_equal(g["z_len"], o["z_len"])
    assert np.array_equal(g["kv_len"], o["kv_len"]), (g["kv_len"], o["kv_len"])
    assert np.array_equal(g["n_pages"], o["n_pages"])
    assert g["pages"] == o["pages"]
    assert g["next_page"] == o["next_page"]


def parity_step(eng, loop, delta, *, tol_logits, tol_reward, margin_tok, margin_gate, stats=None, min_target_rows=1,
                accept_pattern=None):
    """One step on both sides.  The GPU is forced onto the oracle's tokens; its own samples and its
    own gate decisions are checked wherever the oracle's margins are clear.  accept_pattern (per row
    0 / 1 / None) imposes gate decisions on BOTH sides, to steer how many rows the target serves."""
    B = len(loop.rows)
    o = loop.step(delta, min_target_rows=min_target_rows, forced_accept=accept_pattern)
    eng.force_tokens(DRAFT, o["draft_tokens"])
    eng.force_tokens(TARGET, o["target_tokens"])
    # the gate is left to the GPU except where the oracle's reward sits within the margin of delta
    amb = [None] * B
    for b in range(B):
        if o["drafted"][b] and abs(o["rewards"][b] - delta) <= margin_gate:
            amb[b] = int(o["accept"][b])
        if accept_pattern is not None and accept_pattern[b] is not None:
            amb[b] = int(accept_pattern[b])
    eng.force_accept(amb)
    if loop.cfg.sd_tokens > 0 and any(r is not None for r in o["sd_rounds"]):
        # speculative decoding of rejected steps: the draft's proposals are imposed too, so that the rounds (and
        # their counters) are the oracle's even where a proposal was a near tie
        eng.force_sd_proposals([None if r is None else [rd["props"] for rd in r] for r in o["sd_rounds"]])
    g = eng.step(delta, min_target_rows)
    live_before = (o["step_len"] > 0) | (o["drafted"] > 0) | (o["waiting"] > 0)
    # rewards, gate, outputs
    err_r = np.abs(g["rewards"].astype(np.float64) - o["rewards"])[live_before]
    assert err_r.size == 0 or err_r.max() <= tol_reward, f"reward error {err_r.max()}"
    assert np.array_equal(g["accept"], o["accept"])
    assert np.array_equal(g["step_len"], o["step_len"])
    assert np.array_equal(g["live"], o["live"])
    if min_target_rows > 1:
        assert np.array_equal(g["waiting"], o["waiting"])
    for b in range(B):
        n = o["step_len"][b]
        assert g["step_tokens"][b, :n].tolist() == list(o["step_tokens"][b])
        assert not g["step_tokens"][b, n:].any()
    assert eng.state()["rej_idx"] == o["rej_idx"]
    # rewards of steps the target wrote in an earlier call, read when the PRM cached them in this one
    fresh = ~np.isnan(o["target_rewards"])
    if fresh.any():
        got_t = eng.target_step_rewards()
        err_t = np.abs(got_t[fresh].astype(np.float64) - o["target_rewards"][fresh])
        assert err_t.max() <= tol_reward, f"target-step reward error {err_t.max()}"
        if stats is not None:
            stats["target_step_rewards"] = stats.get("target_step_rewards", 0) + int(fresh.sum())
    # logits and free samples of both decode phases
    max_err = 0.0
    n_tok = n_cmp = 0
    for which, key in ((DRAFT, "draft_trace"), (TARGET, "target_trace")):
        rows = [b for b in range(B) if o[key][b] is not None and len(o[key][b]["sampled"])]
        if not rows:
            continue
        lg = eng.logits(which)
        smp = eng.sampled(which)
        for b in rows:
            tr = o[key][b]
            for j, want in enumerate(tr["logits"]):
                err = np.abs(lg[b, j].astype(np.float64) - want).max()
                max_err = max(max_err, err)
                n_tok += 1
                if tr["margin"][j] > margin_tok:
                    n_cmp += 1
                    assert smp[b, j] == tr["sampled"][j], (which, b, j, smp[b, j], tr["sampled"][j], tr["margin"][j])
    assert max_err <= tol_logits, f"logit error {max_err}"
    compare_state(eng, loop)
    if stats is not None:
        stats.setdefault("max_logit_err", 0.0)
        stats["max_logit_err"] = max(stats["max_logit_err"], max_err)
        stats["max_reward_err"] = max(stats.get("max_reward_err", 0.0), float(err_r.max()) if err_r.size else 0.0)
        stats["tokens"] = stats.get("tokens", 0) + n_tok
        stats["tokens_compared"] = stats.get("tokens_compared", 0) + n_cmp
    return g, o


def compare_counters(eng, loop):
    g, o = eng.counters(), loop.counters
    for k in ("gen_tokens", "ingest_tokens"):
        assert list(g[k]) == list(o[k]), (k, g[k], o[k])
    for k in ("score_tokens", "steps", "accepted_steps", "rejected_steps", "discarded_draft_tokens",
              "sd_rounds", "sd_proposed", "sd_matched", "sd_verified"):
        assert g[k] == o[k], (k, g[k], o[k])
    assert abs(g["flops_paper"] - loop.flops_paper()) <= 1e-9 * max(1.0, loop.flops_paper())
