"""Pins for the oracle's step loop (Algorithm 1 batched over rows) and its book-keeping."""
import math

import numpy as np
import pytest

import oracle
import rsd_inputs as ri
from oracle import OracleModel
from oracle.rsd_loop import OracleRSD, LoopConfig, DRAFT, PRM, TARGET


def tiny_models(tiny_weights):
    d, p, t = tiny_weights
    return OracleModel(d, DRAFT), OracleModel(p, PRM), OracleModel(t, TARGET)


def plain_decode(model, which, row, prompt, n_tokens, cfg, v_limit):
    """Decoding straight from the definition: every token from a full-sequence recompute."""
    seq = list(prompt)
    for _ in range(n_tokens):
        h = model.forward_full(seq)
        tok, _ = oracle.sample(model.logits(h[-1]), v_limit, cfg.temperature, cfg.seed, which, row, len(seq))
        seq.append(tok)
    return seq[len(prompt):]


def chunk_steps(tokens, cfg):
    steps, cur = [], []
    for t in tokens:
        cur.append(t)
        end = (t % cfg.step_end_mod == cfg.step_end_id % cfg.step_end_mod) if cfg.step_end_mod else t == cfg.step_end_id
        if end or len(cur) == cfg.max_step_tokens:
            steps.append(cur); cur = []
    return steps, cur


@pytest.mark.parametrize("temperature", [0.0, 0.7])
def test_delta_limits_reproduce_draft_only_and_target_only(tiny_weights, temperature):
    """delta = 0 accepts every step (draft-only decoding); delta above the PRM's range rejects every
    step (target-only decoding cut into steps) -- Appendix B, per-level analysis of delta."""
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=6, max_steps=3, max_seq_tokens=64, step_end_id=5, step_end_mod=4,
                     temperature=temperature, seed=11)
    tok, off = ri.prompts(3, 3, 5, 9, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(3)]
    for delta, model, which in [(0.0, dm, DRAFT), (1.5, tm, TARGET)]:
        loop = OracleRSD(dm, pm, tm, cfg)
        loop.prefill(prompts)
        got = [[] for _ in prompts]
        for _ in range(cfg.max_steps):
            r = loop.step(delta)
            assert np.all(r["accept"][r["step_len"] > 0] == (1 if delta == 0.0 else 0))
            for b in range(3):
                got[b].append(list(r["step_tokens"][b]))
        for b, p in enumerate(prompts):
            n = sum(len(s) for s in got[b])
            want = plain_decode(model, which, b, p, n, cfg, 1024)
            steps, rest = chunk_steps(want, cfg)
            assert rest == [] and steps == got[b]


def test_rollback_and_mixed_accept_match_plain_decoding(tiny_weights):
    """With forced gate decisions each committed step must equal what the chosen model would
    write from the committed context alone, whatever was cached or discarded before."""
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=5, max_steps=4, max_seq_tokens=64, step_end_id=1, step_end_mod=3,
                     temperature=0.7, seed=3)
    tok, off = ri.prompts(4, 2, 4, 7, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(2)]
    loop = OracleRSD(dm, pm, tm, cfg)
    loop.prefill(prompts)
    pattern = [[1, 0], [0, 0], [1, 1], [0, 1]]
    ctx = [list(p) for p in prompts]
    for i in range(4):
        r = loop.step(0.5, forced_accept=pattern[i])
        for b in range(2):
            model, which = (dm, DRAFT) if pattern[i][b] else (tm, TARGET)
            want = plain_decode(model, which, b, ctx[b], len(r["step_tokens"][b]), cfg, 1024)
            assert want == list(r["step_tokens"][b])
            # the reward is that of the draft's step given the committed context
            seq = ctx[b] + list(r["draft_tokens"][b])
            assert abs(pm.reward(pm.forward_full(seq)[-1]) - r["rewards"][b]) < 1e-9
            # the reward of a step the target wrote is read one call later, when the PRM caches that step:
            # the PRM's score at the last token of the context as it stood after the target's step
            if i > 0 and not pattern[i - 1][b]:
                assert abs(pm.reward(pm.forward_full(ctx[b])[-1]) - r["target_rewards"][b]) < 1e-9
            else:
                assert np.isnan(r["target_rewards"][b])
            ctx[b] += list(r["step_tokens"][b])
        st = loop.state()
        assert np.array_equal(st["z_len"], [len(c) for c in ctx])
        assert np.all(st["kv_len"][DRAFT] <= st["z_len"] - 1) and np.all(st["kv_len"][PRM] <= st["z_len"])
        assert np.all(st["kv_len"][TARGET] <= st["z_len"] - 1)


def toy_loop(seed, temperature=1.0, omega_kind=1, omega_b=0.0):
    """Vocabulary-8 models with one-token steps, so a step's law is a categorical distribution."""
    shape = ri.ModelShape(1, 16, 2, 1, 8, 24, 8)
    ws = []
    for slot, hk in [(0, ri.HEAD_LM), (1, ri.HEAD_REWARD_SIGMOID), (2, ri.HEAD_LM)]:
        w = ri.cpu_model_weights(shape, slot, 21, False, hk)
        w["head"] = w["head"] * (20.0 if hk == ri.HEAD_LM else 40.0)
        w["tok_embed"] = w["tok_embed"] * 50.0
        ws.append(w)
    models = [OracleModel(w, i) for i, w in enumerate(ws)]
    cfg = LoopConfig(max_step_tokens=1, max_steps=1, max_seq_tokens=8, step_end_id=0, temperature=temperature,
                     seed=seed, omega_kind=omega_kind, omega_b=omega_b)
    return models, cfg


def toy_laws(models, prompt, temperature):
    dm, pm, tm = models
    def law(m):
        lg = m.logits(m.forward_full(prompt)[-1]) / temperature
        p = np.exp(lg - lg.max()); return p / p.sum()
    rewards = np.array([pm.reward(pm.forward_full(prompt + [v])[-1]) for v in range(8)])
    return law(dm), law(tm), rewards


@pytest.mark.parametrize("omega_kind,a,b", [(1, None, 0.0), (2, 0.0, 0.0), (4, None, 12.0)])
def test_mixture_distribution_of_one_step(omega_kind, a, b):
    """Proposition 2.1: P_RSD = omega_r P_m + nu P_M with nu = 1 - E_{P_m}[omega_r]; Proposition 2.2:
    E_RSD[r] >= E_m[r] when omega is non-decreasing and E_M[r] >= E_m[r]."""
    prompt = [2, 7, 1]
    models, cfg = toy_loop(0, omega_kind=omega_kind, omega_b=b)
    pm_, pM_, rew = toy_laws(models, prompt, cfg.temperature)
    delta = float(np.median(rew)) if a is None else a
    w = np.array([oracle.omega(omega_kind, r, delta, b) for r in rew])
    nu = 1.0 - float(pm_ @ w)
    want = w * pm_ + nu * pM_
    assert abs(want.sum() - 1.0) < 1e-12 and 0.05 < nu < 0.95

    # exact part: force each draft token in turn and read the gate's decision
    if omega_kind == 1:
        for v in range(8):
            loop = OracleRSD(*models, cfg); loop.prefill([prompt])
            r = loop.step(delta, forced_draft=[[v]])
            assert r["accept"][0] == (1 if rew[v] >= delta else 0)
            assert abs(r["rewards"][0] - rew[v]) < 1e-12
    # statistical part: the loop's output law over seeds
    n = 3000
    counts = np.zeros(8)
    for s in range(n):
        cfg_s = LoopConfig(**{**cfg.__dict__, "seed": 1000 + s})
        loop = OracleRSD(*models, cfg_s); loop.prefill([prompt])
        counts[loop.step(delta)["step_tokens"][0][0]] += 1
    keep = want * n >= 5
    chi2 = ((counts[keep] - n * want[keep]) ** 2 / (n * want[keep])).sum()
    assert chi2 < 26.1      # chi-square, <= 8 degrees of freedom, p = 0.001
    if pM_ @ rew >= pm_ @ rew:
        assert want @ rew >= pm_ @ rew - 1e-12


def test_threshold_at_reward_quantile_meets_budget():
    """Proposition 2.3: under a budget nu <= gamma the best omega is the step at the largest feasible
    threshold, i.e. a reward quantile; on a batch, delta = k-th smallest reward accepts B - k rows."""
    models, cfg = toy_loop(5)
    cfg = LoopConfig(**{**cfg.__dict__, "max_steps": 2})
    prompts = [[i % 8, (3 * i + 1) % 8, (5 * i + 2) % 8] for i in range(10)]
    loop = OracleRSD(*models, cfg); loop.prefill(prompts)
    r0 = loop.step(0.0)["rewards"]
    k = 3
    delta = float(np.sort(r0)[k])
    loop = OracleRSD(*models, cfg); loop.prefill(prompts)
    r = loop.step(delta)
    assert np.array_equal(r["rewards"], r0)
    assert int(r["accept"].sum()) == int((r0 >= delta).sum()) >= 10 - k
    assert r["rej_idx"] == [b for b in range(10) if r0[b] < delta]
    # among all masks that reject k rows, the threshold mask keeps the largest total draft reward
    assert r0[r["accept"] == 1].sum() >= np.sort(r0)[k:].sum() - 1e-12


def test_counters_pages_and_dead_rows(tiny_weights):
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=4, max_steps=2, max_seq_tokens=40, step_end_id=9999, temperature=0.0, seed=0)
    prompts = [list(range(10, 10 + n)) for n in (17, 16, 33)]
    # all accepted: draft writes 2 steps x 4 tokens per row, PRM sees prompt + those tokens
    loop = OracleRSD(dm, pm, tm, cfg); loop.prefill(prompts)
    st = loop.state()
    assert st["pages"][DRAFT] == [[0], [1], [2, 3]] and st["pages"][PRM] == [[0, 1], [2], [3, 4, 5]]
    assert st["pages"][TARGET] == [[], [], []]
    r1 = loop.step(0.0)
    assert list(r1["step_len"]) == [4, 4, 4] and list(r1["live"]) == [1, 1, 0]   # row 2: 37+4 > 40
    r2 = loop.step(0.0)
    assert list(r2["step_len"]) == [4, 4, 0] and list(r2["accept"]) == [1, 1, 0] and r2["rewards"][2] == 0.0
    assert list(r2["live"]) == [0, 0, 0]
    c = loop.counters
    assert c["gen_tokens"] == [20, 0, 0] and c["score_tokens"] == 20 and c["ingest_tokens"] == [63, 66, 0]
    assert c["steps"] == 5 and c["accepted_steps"] == 5 and c["discarded_draft_tokens"] == 0
    n_d, n_p = ri.SHAPES["tiny_draft"].n_params(0), ri.SHAPES["tiny_draft"].n_params(1)
    assert loop.flops_paper() == 2.0 * n_d * 20 + 2.0 * n_p * (20 + 66)
    st = loop.state()
    # draft needs |z|-1+cap slots at step start: row 0: 16+4 -> 2 pages, then 20+4 -> 2 pages
    assert st["pages"][DRAFT] == [[0, 4], [1, 5], [2, 3, 6]]
    assert st["pages"][PRM][0] == [0, 1] and st["pages"][PRM][2] == [3, 4, 5]
    # all rejected: target generates everything, draft tokens are discarded
    loop = OracleRSD(dm, pm, tm, cfg); loop.prefill(prompts)
    loop.step(2.0); loop.step(2.0)
    c = loop.counters
    assert c["gen_tokens"] == [20, 0, 20] and c["discarded_draft_tokens"] == 20 and c["rejected_steps"] == 5
    # target ingested, lazily, everything but each row's newest token (16+15+32); afterwards it has
    # cached its own step while decoding it, so nothing is left to catch up on
    assert c["ingest_tokens"][TARGET] == 63
    # draft re-ingests the target's step of the two rows that lived on (4 tokens each)
    assert c["ingest_tokens"][DRAFT] == 63 + 8
    assert loop.flops_paper() == 2.0 * n_d * 20 + 2.0 * ri.SHAPES["tiny_target"].n_params(0) * 20 \
        + 2.0 * n_p * (20 + 66 + 8)
    st = loop.state()
    assert st["pages"][TARGET] == [[0, 1], [2, 3], [4, 5, 6]]
    all_pages = [p for row in st["pages"][TARGET] for p in row]
    assert sorted(all_pages) == list(range(st["next_page"][TARGET]))


def test_eos_stops_a_row_and_row_independence(tiny_weights):
    dm, pm, tm = tiny_models(tiny_weights)
    base = dict(max_step_tokens=8, max_steps=3, max_seq_tokens=64, step_end_id=7, step_end_mod=5,
                temperature=0.7, seed=2)
    tok, off = ri.prompts(9, 4, 6, 12, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(4)]
    loop = OracleRSD(dm, pm, tm, LoopConfig(**base)); loop.prefill(prompts)
    first = loop.step(0.5)
    eos = int(first["step_tokens"][1][-1])            # make row 1's first step end with "EOS"
    loop = OracleRSD(dm, pm, tm, LoopConfig(**base, eos_id=eos)); loop.prefill(prompts)
    r = loop.step(0.5)
    assert eos in r["step_tokens"][1] and r["live"][1] == 0
    assert r["step_tokens"][1][-1] == eos and eos not in r["step_tokens"][1][:-1]
    r2 = loop.step(0.5)
    assert r2["step_len"][1] == 0 and r2["accept"][1] == 0
    # a row's results do not depend on which other rows share the batch (noise is keyed by row id,
    # so compare row 0 alone with row 0 inside the batch)
    solo = OracleRSD(dm, pm, tm, LoopConfig(**base)); solo.prefill(prompts[:1])
    s = solo.step(0.5)
    assert list(s["step_tokens"][0]) == list(first["step_tokens"][0]) and s["rewards"][0] == first["rewards"][0]


def run_to_end(loop, delta, min_target_rows, max_calls=200):
    """Calls step until no row is live; returns per row the list of (tokens, accepted) in commit order."""
    B = len(loop.rows)
    hist = [[] for _ in range(B)]
    flushes = calls = 0
    for _ in range(max_calls):
        if not any(r.live for r in loop.rows):
            break
        r = loop.step(delta, min_target_rows=min_target_rows)
        calls += 1
        flushes += int(r["flushed"])
        for b in range(B):
            if r["step_len"][b] > 0:
                hist[b].append((list(r["step_tokens"][b]), int(r["accept"][b])))
            else:
                assert r["accept"][b] == 0
        # a row that waits stays live, took no step, and keeps its reward
        for b in range(B):
            if r["waiting"][b]:
                assert r["live"][b] == 1 and r["step_len"][b] == 0
    assert not any(r.live for r in loop.rows)
    return hist, flushes, calls


@pytest.mark.parametrize("min_rows", [2, 3, 100])
def test_queued_rejections_leave_every_rows_sequence_unchanged(tiny_weights, min_rows):
    """Rows are independent in Algorithm 1, so letting rejected rows wait for a fuller target batch
    changes when a step is written, never what is written: every row's committed steps, gate
    decisions, final context and the token counters equal those of the lock-step loop; only the
    number of target passes drops."""
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=5, max_steps=5, max_seq_tokens=80, step_end_id=2, step_end_mod=4,
                     temperature=0.7, seed=21)
    tok, off = ri.prompts(9, 5, 4, 9, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(5)]
    # a threshold near the median reward of the first step mixes accepted and rejected rows
    probe = OracleRSD(dm, pm, tm, cfg)
    probe.prefill(prompts)
    delta = float(np.median(probe.step(0.0)["rewards"]))
    lock = OracleRSD(dm, pm, tm, cfg)
    lock.prefill(prompts)
    want, flushes_lock, calls_lock = run_to_end(lock, delta, 1)
    assert any(a for h in want for _, a in h) and any(not a for h in want for _, a in h)
    queued = OracleRSD(dm, pm, tm, cfg)
    queued.prefill(prompts)
    got, flushes_q, calls_q = run_to_end(queued, delta, min_rows)
    assert got == want
    assert [r.z for r in queued.rows] == [r.z for r in lock.rows]
    for key in ("gen_tokens", "score_tokens", "steps", "accepted_steps", "rejected_steps", "discarded_draft_tokens"):
        assert queued.counters[key] == lock.counters[key], key
    assert flushes_q <= flushes_lock and calls_q >= calls_lock


def test_queued_flush_rule_and_cursors(tiny_weights):
    """Forced gate decisions: rejected rows wait with their draft and PRM cursors rolled back and the
    target untouched; the target pass happens in the call in which the number of waiting rows reaches
    min_target_rows (or every live row waits), serves all of them in ascending order and hands out
    their pages in that order."""
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=4, max_steps=6, max_seq_tokens=64, step_end_id=900, temperature=0.0, seed=2)
    tok, off = ri.prompts(5, 4, 6, 6, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(4)]
    loop = OracleRSD(dm, pm, tm, cfg)
    loop.prefill(prompts)
    # call 1: row 2 rejected -> waits (1 < 3)
    r = loop.step(0.5, forced_accept=[1, 1, 0, 1], min_target_rows=3)
    assert not r["flushed"] and list(r["waiting"]) == [0, 0, 1, 0] and r["rej_idx"] == [2]
    assert list(r["step_len"]) == [4, 4, 0, 4] and list(r["drafted"]) == [1, 1, 1, 1]
    st = loop.state()
    assert st["kv_len"][DRAFT][2] == 5 and st["kv_len"][PRM][2] == 6 and st["kv_len"][TARGET][2] == 0
    assert st["n_pages"][TARGET].sum() == 0 and st["n_steps"][2] == 0
    # call 2: row 0 rejected -> two wait (2 < 3); row 2 does not draft
    r = loop.step(0.5, forced_accept=[0, 1, None, 1], min_target_rows=3)
    assert not r["flushed"] and list(r["waiting"]) == [1, 0, 1, 0] and r["rej_idx"] == [0, 2]
    assert list(r["drafted"]) == [1, 1, 0, 1] and list(r["step_len"]) == [0, 4, 0, 4]
    assert r["draft_tokens"][2] == []
    # call 3: row 3 rejected -> three wait: the target writes the step of rows 0, 2 and 3
    r = loop.step(0.5, forced_accept=[None, 1, None, 0], min_target_rows=3)
    assert r["flushed"] and r["rej_idx"] == [0, 2, 3] and list(r["waiting"]) == [0, 0, 0, 0]
    assert list(r["step_len"]) == [4, 4, 4, 4] and list(r["accept"]) == [0, 1, 0, 0]
    st = loop.state()
    # target pages in ascending row order: rows 0, 2, 3 need ceil((z - 1 + 4) / 16) pages each
    assert st["pages"][TARGET][0] == [0] and st["pages"][TARGET][1] == []
    assert st["pages"][TARGET][2] == [1] and st["pages"][TARGET][3] == [2, 3]
    assert list(st["n_steps"]) == [2, 3, 1, 3]
    # each committed target step is what the target writes from the committed context alone
    for b, ctx_len in ((0, 6 + 4), (2, 6), (3, 6 + 8)):
        ctx = loop.rows[b].z[:ctx_len]
        want = plain_decode(tm, TARGET, b, ctx, 4, cfg, 1024)
        assert want == list(r["step_tokens"][b])
    # every live row waits -> flush although fewer than min_target_rows wait
    r = loop.step(0.5, forced_accept=[0, 0, 0, 0], min_target_rows=100)
    assert r["flushed"] and r["rej_idx"] == [0, 1, 2, 3]


def test_merged_prm_equals_a_separate_prm_with_the_drafts_trunk(tiny_weights):
    """A PRM that is a reward head on the draft's trunk (Appendix B.3: a projection layer on top of the
    final transformer layer) scored from the draft's own cache plus one single-token forward must give
    the rewards of a separately cached PRM whose trunk weights are the draft's -- and with them the same
    gate decisions, tokens, draft / target cursors and pages -- while the PRM keeps no cache and bills
    one processed token per scored step."""
    d, p, t = tiny_weights
    dm, tm = OracleModel(d, DRAFT), OracleModel(t, TARGET)
    twin = dict(d)                      # the draft's trunk ...
    twin["head"], twin["head_kind"], twin["final_norm"] = p["head"], p["head_kind"], p["final_norm"]   # ... the PRM's head
    pm_twin = OracleModel(twin, PRM)
    pm_head_only = OracleModel(dict(p, layers=[]), PRM)      # merged mode never touches PRM layers
    cfg = dict(max_step_tokens=5, max_steps=4, max_seq_tokens=64, step_end_id=2, step_end_mod=4, temperature=0.7, seed=8)
    tok, off = ri.prompts(12, 4, 4, 9, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(4)]
    sep = OracleRSD(dm, pm_twin, tm, LoopConfig(**cfg))
    sep.prefill(prompts)
    delta = float(np.median(sep.step(0.0)["rewards"]))
    sep = OracleRSD(dm, pm_twin, tm, LoopConfig(**cfg))
    mrg = OracleRSD(dm, pm_head_only, tm, LoopConfig(prm_shares_draft=True, **cfg))
    sep.prefill(prompts)
    mrg.prefill(prompts)
    saw = set()
    for _ in range(cfg["max_steps"]):
        a, b = sep.step(delta), mrg.step(delta)
        assert np.allclose(a["rewards"], b["rewards"], rtol=0, atol=1e-12)
        assert np.array_equal(a["accept"], b["accept"]) and np.array_equal(a["live"], b["live"])
        assert [list(x) for x in a["step_tokens"]] == [list(x) for x in b["step_tokens"]]
        saw |= set(int(x) for x, n in zip(a["accept"], a["step_len"]) if n)
        sa, sb = sep.state(), mrg.state()
        for w in (DRAFT, TARGET):
            assert np.array_equal(sa["kv_len"][w], sb["kv_len"][w])
        assert sa["pages"][TARGET] == sb["pages"][TARGET]
        assert not sb["kv_len"][PRM].any() and not sb["n_pages"][PRM].any()
    assert saw == {0, 1}
    for key in ("gen_tokens", "steps", "accepted_steps", "rejected_steps", "discarded_draft_tokens"):
        assert sep.counters[key] == mrg.counters[key]
    assert mrg.counters["ingest_tokens"][PRM] == 0
    assert mrg.counters["score_tokens"] == mrg.counters["steps"]     # one token per scored step (lock-step)


# ---------------------------------------------------------------------------------------------------------
# RSD combined with speculative decoding for the rejected steps (Section 4, "Combine RSD with SD")
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("temperature,k", [(0.0, 1), (0.0, 4), (0.7, 3), (0.7, 8)])
def test_speculative_rejected_steps_equal_plain_target_decoding(tiny_weights, temperature, k):
    """However many tokens the draft proposes per round and whatever it proposes, the step a rejected row
    receives is the target's own: every committed step equals plain full-recompute decoding with the
    target from the committed context, and the whole run equals the loop without speculative decoding."""
    dm, pm, tm = tiny_models(tiny_weights)
    base = dict(max_step_tokens=7, max_steps=3, max_seq_tokens=64, step_end_id=2, step_end_mod=5,
                temperature=temperature, seed=13)
    tok, off = ri.prompts(6, 3, 4, 9, 1024)
    prompts = [tok[off[b]:off[b + 1]].tolist() for b in range(3)]
    sd = OracleRSD(dm, pm, tm, LoopConfig(sd_tokens=k, **base))
    ref = OracleRSD(dm, pm, tm, LoopConfig(**base))
    sd.prefill(prompts); ref.prefill(prompts)
    pattern = [[0, 1, 0], [0, 0, 1], [1, 0, 0]]
    ctx = [list(p) for p in prompts]
    for i in range(3):
        a = sd.step(0.5, forced_accept=pattern[i])
        r = ref.step(0.5, forced_accept=pattern[i])
        for b in range(3):
            assert list(a["step_tokens"][b]) == list(r["step_tokens"][b])
            if not pattern[i][b]:
                want = plain_decode(tm, TARGET, b, ctx[b], len(a["step_tokens"][b]), sd.cfg, 1024)
                assert want == list(a["step_tokens"][b])
                rounds = a["sd_rounds"][b]
                assert sum(rd["emitted"] for rd in rounds) == len(want)
                assert all(1 <= rd["emitted"] <= len(rd["props"]) <= k for rd in rounds)
                # a round writes its matching prefix and, unless the step or the round ended there, one more token
                for rd in rounds:
                    assert rd["emitted"] in (rd["matched"], rd["matched"] + 1)
                # the same logits chose the tokens: traces agree with the plain loop's
                assert a["target_trace"][b]["sampled"] == r["target_trace"][b]["sampled"]
            ctx[b] += list(a["step_tokens"][b])
        sa, sr = sd.state(), ref.state()
        assert np.array_equal(sa["z_len"], sr["z_len"]) and np.array_equal(sa["kv_len"][PRM], sr["kv_len"][PRM])
        assert np.array_equal(sa["kv_len"][TARGET], sr["kv_len"][TARGET])
        for b in range(3):
            if not pattern[i][b]:        # the draft proposed along: it has cached the step, the plain loop's draft has not
                assert sa["kv_len"][DRAFT][b] == sa["z_len"][b] - 1 and sr["kv_len"][DRAFT][b] < sa["kv_len"][DRAFT][b]
        assert sa["pages"] == sr["pages"]
    cs, cr = sd.counters, ref.counters
    assert cs["gen_tokens"] == cr["gen_tokens"] and cs["steps"] == cr["steps"]
    assert cs["sd_verified"] == cs["sd_proposed"] >= cs["gen_tokens"][TARGET] >= cs["sd_rounds"] > 0
    # the draft never has to catch up on a step it proposed along with
    assert cs["ingest_tokens"][DRAFT] < cr["ingest_tokens"][DRAFT]


def test_speculative_rounds_accept_exactly_the_matching_prefix(tiny_weights):
    """Proposals planted around the target's true continuation: a round keeps the proposals up to the
    first one that differs from the target's choice and writes the target's token there; rounds, matches
    and evaluated positions follow by hand."""
    dm, pm, tm = tiny_models(tiny_weights)
    cfg = LoopConfig(max_step_tokens=9, max_steps=1, max_seq_tokens=32, step_end_id=1 << 20, temperature=0.7, seed=5,
                     sd_tokens=4)
    prompt = ri.prompts(9, 1, 6, 6, 1024)[0].tolist()
    truth = plain_decode(tm, TARGET, 0, prompt, 9, cfg, 1024)
    bad = lambda t: (t + 1) % 1024
    # round 1 at offset 0: all four right -> 4 written; round 2 at offset 4: wrong at once -> 1 written;
    # round 3 at offset 5: two right, third wrong -> 3 written; round 4 at offset 8: one slot left, right -> 1 written
    planted = [truth[0:4], [bad(truth[4]), 7, 7, 7], [truth[5], truth[6], bad(truth[7]), truth[8]], [truth[8]]]
    loop = OracleRSD(dm, pm, tm, cfg)
    loop.prefill([prompt])
    r = loop.step(0.5, forced_accept=[0], forced_sd_props=[planted])
    assert list(r["step_tokens"][0]) == truth
    assert [(rd["emitted"], rd["matched"]) for rd in r["sd_rounds"][0]] == [(4, 4), (1, 0), (3, 2), (1, 1)]
    assert [len(rd["props"]) for rd in r["sd_rounds"][0]] == [4, 4, 4, 1]
    c = loop.counters
    assert (c["sd_rounds"], c["sd_proposed"], c["sd_verified"], c["sd_matched"]) == (4, 13, 13, 7)
    assert c["gen_tokens"][TARGET] == 9 and c["gen_tokens"][DRAFT] == 9
    st = loop.state()
    assert st["kv_len"][TARGET][0] == st["kv_len"][DRAFT][0] == len(prompt) + 9 - 1
    # Section 3.3 accounting: the draft is billed its step and its proposals, the target every evaluated position
    nd, npr, nt = (m.n_params for m in (dm, pm, tm))
    want = 2.0 * nd * (9 + 13) + 2.0 * nt * 13 + 2.0 * npr * (c["score_tokens"] + c["ingest_tokens"][PRM])
    assert loop.flops_paper() == want


def test_speculative_rounds_with_an_agreeing_draft(tiny_weights):
    """When the draft IS the target (same weights) and decoding is greedy, every proposal matches: a step of
    n tokens takes ceil(n / k) rounds and as many target passes instead of n."""
    d, p, t = tiny_weights
    dm, pm = OracleModel(d, DRAFT), OracleModel(p, PRM)
    tm = OracleModel(d, TARGET)                       # the draft's weights under the target's id
    cfg = LoopConfig(max_step_tokens=10, max_steps=1, max_seq_tokens=40, step_end_id=1 << 20, temperature=0.0, seed=0,
                     sd_tokens=4)
    prompt = ri.prompts(12, 1, 8, 8, 1024)[0].tolist()
    loop = OracleRSD(dm, pm, tm, cfg)
    loop.prefill([prompt])
    r = loop.step(0.5, forced_accept=[0])
    assert list(r["step_tokens"][0]) == list(r["draft_tokens"][0]) == plain_decode(tm, TARGET, 0, prompt, 10, cfg, 1024)
    assert [(rd["emitted"], rd["matched"]) for rd in r["sd_rounds"][0]] == [(4, 4), (4, 4), (2, 2)]
