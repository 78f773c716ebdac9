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
