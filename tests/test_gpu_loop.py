"""Step-loop parity of the CUDA library against the oracle (Algorithm 1 batched over rows)."""
import numpy as np
import pytest

import rsd_inputs as ri
from helpers import build_pair, parity_step, compare_counters, compare_state

pytestmark = pytest.mark.gpu

TINY = (ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_target"])
MINI = (ri.SHAPES["mini_draft"], ri.SHAPES["mini_draft"], ri.SHAPES["mini_target"])
# fp32 path: fp32 sums against fp64 sums; 16-bit path: the bounds asked of bf16 arithmetic
TOL32 = dict(tol_logits=2e-4, tol_reward=1e-5, margin_tok=1e-3, margin_gate=1e-4)
TOL16 = dict(tol_logits=3e-2, tol_reward=1e-2, margin_tok=5e-2, margin_gate=1e-2)


def test_tiny_fp32_config_all_deltas():
    """Tiny fp32 models, batch 4, 64-token prompts, step ends at id 13 or after 32 tokens, 4 steps,
    greedy; delta = 0.7 as configured, plus the median reward (both branches) and the two limits."""
    prompts = ri.prompts(0, 4, 64, 64, 1024)
    base = dict(max_step_tokens=32, max_steps=4, max_seq_tokens=64 + 4 * 32, step_end_id=13, temperature=0.0, seed=0)
    eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=base)
    compare_state(eng, loop)
    r0 = loop.step(0.0)["rewards"]
    median = float(np.median(r0))
    for delta in (0.7, median, 0.0, 1.5):
        eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=base)
        stats = {}
        n_acc = 0
        for _ in range(4):
            g, o = parity_step(eng, loop, delta, stats=stats, **TOL32)
            n_acc += int(g["accept"].sum())
        compare_counters(eng, loop)
        assert stats["tokens_compared"] >= 0.9 * stats["tokens"]
        if delta == 0.0:
            assert n_acc == 16 and eng.counters()["gen_tokens"][2] == 0
        if delta == 1.5:
            assert n_acc == 0 and eng.counters()["gen_tokens"][2] == eng.counters()["gen_tokens"][0]
        assert not g["live"].any()          # four steps were the budget
        eng.close()


def test_tiny_free_running_equals_oracle_when_margins_are_clear():
    """Without forcing, wherever every margin of the oracle's trace is clear the GPU must walk the
    same path by itself: same tokens, gate decisions and integer state."""
    prompts = ri.prompts(5, 3, 9, 30, 1024)
    base = dict(max_step_tokens=12, max_steps=3, max_seq_tokens=96, step_end_id=3, step_end_mod=7,
                temperature=0.7, seed=4)
    eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=base)
    delta = 0.5
    for _ in range(3):
        o = loop.step(delta)
        margins = [m for key in ("draft_trace", "target_trace") for tr in o[key] if tr for m in tr["margin"]]
        gate_margin = np.abs(o["rewards"][o["step_len"] > 0] - delta).min() if (o["step_len"] > 0).any() else 1.0
        if min(margins) < 1e-3 or gate_margin < 1e-4:
            pytest.skip("a margin of the oracle trace is too small for a free-running comparison")
        g = eng.step(delta)
        assert np.array_equal(g["accept"], o["accept"]) and np.array_equal(g["step_len"], o["step_len"])
        for b in range(3):
            assert g["step_tokens"][b, :o["step_len"][b]].tolist() == list(o["step_tokens"][b])
        compare_state(eng, loop)
    compare_counters(eng, loop)


def test_ragged_steps_eos_and_dead_rows():
    """Ragged prompts, steps of different lengths (delimiter by residue), an EOS id, a row that has
    no room to start, and rows that stop at different times."""
    tokens, offsets = ri.prompts(7, 6, 3, 40, 1024)
    base = dict(max_step_tokens=9, max_steps=5, max_seq_tokens=72, step_end_id=2, step_end_mod=5, eos_id=77,
                temperature=0.7, seed=9)
    # row 5 gets a prompt that leaves no room for a step
    long = np.arange(64, dtype=np.int32)
    tokens = np.concatenate([tokens[:offsets[5]], long]).astype(np.int32)
    offsets = offsets.copy(); offsets[6] = offsets[5] + 64
    eng, loop = build_pair(TINY, bf16=False, prompts=(tokens, offsets), loop_kwargs=base)
    r0 = loop.step(0.0)["rewards"]
    delta = float(np.median(r0[r0 > 0]))
    eng, loop = build_pair(TINY, bf16=False, prompts=(tokens, offsets), loop_kwargs=base)
    lens = set()
    for _ in range(5):
        g, o = parity_step(eng, loop, delta, **TOL32)
        lens.update(g["step_len"].tolist())
        assert g["step_len"][5] == 0 and g["live"][5] == 0
    assert len(lens) > 3
    compare_counters(eng, loop)


@pytest.mark.parametrize("kv_extended", [0, 1])
def test_mini_bf16_models(kv_extended):
    """16-bit weights, head_dim 128, Gumbel-max at T = 0.7, chunked multi-token passes; with the
    16-bit KV cache and with the extended one (values as hi + lo pairs)."""
    prompts = ri.prompts(2, 5, 20, 70, 4096)
    base = dict(max_step_tokens=10, max_steps=3, max_seq_tokens=112, step_end_id=1, step_end_mod=6,
                temperature=0.7, seed=21)
    eng, loop = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=base)
    r0 = loop.step(0.0)["rewards"]
    delta = float(np.sort(r0)[1])
    eng, loop = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=base,
                           engine_kwargs=dict(max_chunk_tokens=64, kv_extended=kv_extended))
    stats = {}
    for _ in range(3):
        parity_step(eng, loop, delta, stats=stats, **TOL16)
    compare_counters(eng, loop)
    print("mini bf16 parity, kv_extended =", kv_extended, stats)


def test_page_pool_exhaustion_is_an_error_not_a_fault():
    from paper_2501_19324_b200 import RsdError
    prompts = ri.prompts(0, 4, 64, 64, 1024)
    base = dict(max_step_tokens=32, max_steps=4, max_seq_tokens=192, step_end_id=13, temperature=0.0, seed=0)
    sh = ri.SHAPES["tiny_draft"]
    page_bytes = sh.n_layers * 2 * sh.n_kv_heads * 16 * sh.head_dim * 4
    with pytest.raises(RsdError) as e:
        build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=base,
                   engine_kwargs=dict(kv_bytes=[page_bytes * 10, page_bytes * 400, page_bytes * 800]))
    assert e.value.code == -3


@pytest.mark.parametrize("omega_kind,delta,alpha", [(0, 0.6, 0.0), (2, 0.0, 0.0), (3, 0.0, 0.0), (4, 0.5, 30.0)])
def test_general_acceptance_criterion_on_gpu(omega_kind, delta, alpha):
    """Algorithm 2 with the other weighting functions of Table 1 (constant, clip, r/(1+r), logistic):
    the GPU draws the same Philox uniform per (row, |z_i|) and takes the same decision as the oracle."""
    prompts = ri.prompts(11, 8, 10, 24, 1024)
    base = dict(max_step_tokens=6, max_steps=4, max_seq_tokens=64, step_end_id=3, step_end_mod=4,
                temperature=0.7, seed=17, omega_kind=omega_kind, omega_b=alpha)
    eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=base,
                           engine_kwargs=dict(omega_kind=omega_kind, omega_alpha=alpha))
    seen = set()
    for _ in range(4):
        tol = dict(TOL32, margin_gate=0.0)            # never force the gate: it must agree by itself
        g, o = parity_step(eng, loop, delta, **tol)
        seen.update(g["accept"][g["step_len"] > 0].tolist())
    assert seen == {0, 1}                             # both outcomes occurred
    compare_counters(eng, loop)


def test_reset_and_new_batch_sizes_reuse_one_context():
    """rsd_reset / a second rsd_prefill with another batch size on the same context: pages return to the
    pool, the captured decode graphs are rebuilt for the new slot count, results match a fresh oracle."""
    from oracle.rsd_loop import OracleRSD
    base = dict(max_step_tokens=6, max_steps=3, max_seq_tokens=64, step_end_id=5, step_end_mod=9, temperature=0.7, seed=8)
    p4 = ri.prompts(21, 4, 8, 20, 4096)
    eng, loop = build_pair(MINI, bf16=True, prompts=p4, loop_kwargs=base, engine_kwargs=dict(max_batch=6))
    for _ in range(2):
        parity_step(eng, loop, 0.45, **TOL16)
    for seed, B in ((22, 6), (23, 2)):
        tokens, offsets = ri.prompts(seed, B, 8, 20, 4096)
        eng.prefill(tokens, offsets)                     # drops the old rows
        assert eng.counters()["steps"] == 0
        loop = OracleRSD(*loop.models, loop.cfg)
        loop.prefill([tokens[offsets[b]:offsets[b + 1]].tolist() for b in range(B)])
        compare_state(eng, loop)
        for _ in range(2):
            parity_step(eng, loop, 0.45, **TOL16)
        compare_counters(eng, loop)


def test_call_order_and_argument_errors():
    from paper_2501_19324_b200 import Engine, Model, RsdError
    sh = ri.SHAPES["tiny_draft"]
    models = [Model(sh, ri.gpu_model_tensors(sh, slot, 0, False, hk), hk)
              for slot, hk in enumerate((ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM))]
    eng = Engine(*models, max_batch=2, max_seq_tokens=48, max_step_tokens=8, max_steps=2, step_end_id=13)
    eng.B = 2
    with pytest.raises(RsdError) as e:
        eng.step(0.5)                                    # step before prefill
    assert e.value.code == -2
    with pytest.raises(RsdError) as e:
        eng.prefill(np.array([1, 2, 5000], np.int32), np.array([0, 2, 3], np.int32))    # id beyond the vocabulary
    assert e.value.code == -1
    with pytest.raises(RsdError) as e:
        eng.prefill(np.arange(6, dtype=np.int32), np.array([0, 2, 4, 6], np.int32))      # more rows than max_batch
    assert e.value.code == -1
    eng.prefill(np.array([1, 2, 3, 4], np.int32), np.array([0, 2, 4], np.int32))          # still usable afterwards
    r = eng.step(0.0)
    assert r["accept"].all() and (r["step_len"] > 0).all()
    with pytest.raises(RsdError):                        # a PRM must not carry an lm head, and vice versa
        Engine(models[0], models[0], models[2], max_batch=2, max_seq_tokens=48, max_step_tokens=8, max_steps=2, step_end_id=13)
    # models are loaded once per context: the captured decode graphs hold their pointers
    from paper_2501_19324_b200 import lib
    assert lib().rsd_load_models(eng.ctx, models[0].desc, models[1].desc, models[2].desc) == -2
    assert b"once per context" in lib().rsd_last_error(eng.ctx)
    r = eng.step(0.0)                                    # the refusal left the context as it was
    assert (r["step_len"] > 0).all()
    with pytest.raises(RsdError) as e:                   # kv_extended takes 0 (by depth), 1 or 2
        Engine(*models, max_batch=2, max_seq_tokens=48, max_step_tokens=8, max_steps=2, step_end_id=13, kv_extended=3)
    assert e.value.code == -1


@pytest.mark.parametrize("delta,min_rows", [(0.47, 3), (0.49, 4)])
def test_queued_rejections_match_the_oracle(delta, min_rows):
    """rsd_step_queued: rejected rows wait until min_rows wait, then one target pass serves all of
    them.  Compared call by call with the oracle under the same rule (tokens, rewards, gate, waiting
    flags, cursors, page tables, the list of waiting rows, counters), and at the end every row's
    sequence equals the one the lock-step oracle loop writes."""
    shapes = (ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_target"])
    prompts = ri.prompts(31, 6, 5, 20, 1024)
    # thresholds just under the tiny PRM's reward range (0.5 +- 0.08): a rejection every few steps
    kw = dict(max_step_tokens=6, max_steps=6, max_seq_tokens=96, step_end_id=3, step_end_mod=5, temperature=0.7, seed=4)
    eng, loop = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=kw)
    _, lock = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=kw)
    stats = {}
    waited = flushed = 0
    for _ in range(40):
        if not any(r.live for r in loop.rows):
            break
        g, o = parity_step(eng, loop, delta, tol_logits=2e-4, tol_reward=1e-5, margin_tok=1e-3, margin_gate=1e-4,
                           stats=stats, min_target_rows=min_rows)
        waited += int(o["waiting"].sum())
        flushed += int(o["flushed"])
    assert not any(r.live for r in loop.rows)
    assert waited > 0 and flushed > 0
    compare_counters(eng, loop)
    while any(r.live for r in lock.rows):
        lock.step(delta)
    assert [r.z for r in loop.rows] == [r.z for r in lock.rows]
    print("queued rejections, min_rows", min_rows, stats)


def test_queued_with_min_rows_one_is_rsd_step_and_bad_arguments():
    from paper_2501_19324_b200 import lib
    shapes = (ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_draft"], ri.SHAPES["tiny_target"])
    prompts = ri.prompts(32, 4, 5, 12, 1024)
    kw = dict(max_step_tokens=5, max_steps=3, max_seq_tokens=64, step_end_id=3, temperature=0.7, seed=5)
    a, _ = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=kw)
    b, _ = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=kw)
    for _ in range(3):
        ra = a.step(0.5)
        out = {k: np.zeros_like(v) for k, v in ra.items()}
        ptr = [out[k].ctypes.data for k in ("step_tokens", "step_len", "rewards", "accept", "live", "waiting")]
        assert lib().rsd_step_queued(b.ctx, 0.5, 1, None, *ptr) == 0
        for k in ("step_tokens", "step_len", "rewards", "accept", "live"):
            assert np.array_equal(ra[k], out[k]), k
        assert not out["waiting"].any()
    assert lib().rsd_step_queued(b.ctx, 0.5, 0, None, *ptr) == -1
    assert b"min_target_rows" in lib().rsd_last_error(b.ctx)


@pytest.mark.parametrize("shapes,bf16,tol", [(TINY, False, TOL32), (MINI, True, TOL16)])
def test_merged_prm_on_the_drafts_trunk(shapes, bf16, tol):
    """prm_shares_draft: the reward comes from one more single-token pass of the draft and the PRM's head;
    step-by-step parity with the oracle in the same mode (rewards, gate, tokens, cursors -- the PRM's stay
    at zero -- pages, counters)."""
    prompts = ri.prompts(41, 5, 6, 30, shapes[0].vocab)
    kw = dict(max_step_tokens=6, max_steps=4, max_seq_tokens=96, step_end_id=3, step_end_mod=5, temperature=0.7,
              seed=6, prm_shares_draft=True)
    eng, loop = build_pair(shapes, bf16=bf16, prompts=prompts, loop_kwargs=kw)
    probe = loop.step(0.0)["rewards"]
    delta = float(np.median(probe))
    eng, loop = build_pair(shapes, bf16=bf16, prompts=prompts, loop_kwargs=kw)
    stats, seen = {}, set()
    for _ in range(4):
        g, o = parity_step(eng, loop, delta, stats=stats, **tol)
        seen |= set(int(a) for a, n in zip(o["accept"], o["step_len"]) if n)
    assert seen == {0, 1}
    st = eng.state()
    assert not st["kv_len"][1].any() and not st["n_pages"][1].any()
    compare_counters(eng, loop)
    print("merged PRM", "bf16" if bf16 else "fp32", stats)


@pytest.mark.parametrize("B,ext", [(5, 0), (20, 0), (40, 0), (6, 1)])
def test_persistent_decode_kernel_against_the_oracle_and_the_separate_kernels(B, ext):
    """RSD_DEBUG_PERSISTENT_DECODE: bf16 models at up to 64 rows decode with one persistent kernel per iteration
    (all layers, grid barriers between the phases).  It must meet the oracle like the default kernel-by-kernel
    path, agree with that path far inside the bf16 bound, and launch far fewer kernels.  Batch sizes cover the 16-, 32- and 64-row
    operand tiles; ext = hi + lo KV cache."""
    from paper_2501_19324_b200 import lib, RSD_DEBUG_KEEP_LOGITS, RSD_DEBUG_PERSISTENT_DECODE
    from oracle.rsd_loop import DRAFT, TARGET
    prompts = ri.prompts(50 + B, B, 5, 40, MINI[0].vocab)
    kw = dict(max_step_tokens=5, max_steps=3, max_seq_tokens=80, step_end_id=3, step_end_mod=5, temperature=0.7, seed=8)
    probe_eng, probe = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=kw,
                                  engine_kwargs=dict(debug_flags=RSD_DEBUG_KEEP_LOGITS))
    delta = float(np.median(probe.step(0.0)["rewards"]))
    probe_eng.close()
    runs = {}
    for name, flags in (("mega", RSD_DEBUG_KEEP_LOGITS | RSD_DEBUG_PERSISTENT_DECODE), ("separate", RSD_DEBUG_KEEP_LOGITS)):
        eng, loop = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=kw,
                               engine_kwargs=dict(debug_flags=flags, kv_extended=ext))
        before = lib().rsd_debug_launch_count()
        stats, logits, seen = {}, [], set()
        for _ in range(3):
            g, o = parity_step(eng, loop, delta, stats=stats, **TOL16)
            seen |= set(int(a) for a, n in zip(o["accept"], o["step_len"]) if n)
            logits.append((eng.logits(DRAFT).copy(), eng.logits(TARGET).copy(), o))
        compare_counters(eng, loop)
        runs[name] = dict(stats=stats, logits=logits, launches=lib().rsd_debug_launch_count() - before, seen=seen)
        eng.close()
    assert runs["mega"]["seen"] == {0, 1}                      # both models decoded
    assert runs["mega"]["launches"] < 0.6 * runs["separate"]["launches"]
    worst = 0.0
    for (d0, t0, o), (d1, t1, _) in zip(runs["mega"]["logits"], runs["separate"]["logits"]):
        for key, a, b in (("draft_trace", d0, d1), ("target_trace", t0, t1)):
            for r in range(B):
                if o[key][r] is not None:
                    n = len(o[key][r]["logits"])
                    worst = max(worst, float(np.abs(a[r, :n] - b[r, :n]).max()))
    assert worst <= 2e-3, worst
    print("persistent decode kernel", B, ext, runs["mega"]["stats"], "vs separate kernels", worst,
          "launches", runs["mega"]["launches"], runs["separate"]["launches"])


def test_persistent_decode_kernel_phase_timeline():
    """rsd_debug_mega_profile: with RSD_DEBUG_MEGA_PROFILE the persistent kernel's first CTA stamps the global timer
    at its start, before and after each of its 7 * layers grid barriers and at its end, in order; without the flag
    the call is refused."""
    from paper_2501_19324_b200 import RSD_DEBUG_KEEP_LOGITS, RSD_DEBUG_PERSISTENT_DECODE, RSD_DEBUG_MEGA_PROFILE
    from paper_2501_19324_b200.binding import RsdError
    from oracle.rsd_loop import DRAFT, TARGET
    prompts = ri.prompts(77, 4, 5, 20, MINI[0].vocab)
    kw = dict(max_step_tokens=3, max_steps=2, max_seq_tokens=48, step_end_id=3, temperature=0.7, seed=2)
    eng, loop = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=kw,
                           engine_kwargs=dict(debug_flags=RSD_DEBUG_KEEP_LOGITS | RSD_DEBUG_PERSISTENT_DECODE | RSD_DEBUG_MEGA_PROFILE))
    parity_step(eng, loop, 2.0, **TOL16)                   # delta above the reward range: both models decode
    for which, shape in ((DRAFT, MINI[0]), (TARGET, MINI[2])):
        st = eng.mega_profile(which).astype(np.int64)
        assert len(st) == 14 * shape.n_layers + 2, len(st)
        assert (np.diff(st) >= 0).all() and st[-1] > st[0]
        assert st[-1] - st[0] < 50_000_000                 # one launch of a two- or three-layer model: far below 50 ms
    eng.close()
    eng, loop = build_pair(MINI, bf16=True, prompts=prompts, loop_kwargs=kw)
    with pytest.raises(RsdError):
        eng.mega_profile(DRAFT)
    eng.close()


@pytest.mark.parametrize("shapes,bf16,tol,k", [(TINY, False, TOL32, 3), (MINI, True, TOL16, 4), (TINY, False, TOL32, 1)])
def test_speculative_decoding_of_rejected_steps(shapes, bf16, tol, k):
    """sd_tokens = k (the paper's discussion of combining RSD with speculative decoding): the steps of rejected rows
    are written in rounds of k draft proposals and one target pass.  Step by step against the oracle in the same
    mode: logits of every written token, tokens, cursors of all three caches (the draft's now follow the target's),
    pages, the rounds' counters; and the committed sequences equal those of the plain loop."""
    prompts = ri.prompts(61, 6, 6, 30, shapes[0].vocab)
    kw = dict(max_step_tokens=7, max_steps=4, max_seq_tokens=96, step_end_id=3, step_end_mod=5, temperature=0.7,
              seed=6, sd_tokens=k)
    eng, loop = build_pair(shapes, bf16=bf16, prompts=prompts, loop_kwargs=kw)
    delta = float(np.median(loop.step(0.0)["rewards"]))
    eng, loop = build_pair(shapes, bf16=bf16, prompts=prompts, loop_kwargs=kw)
    _, plain = build_pair(shapes, bf16=bf16, prompts=prompts, loop_kwargs=dict(kw, sd_tokens=0))
    stats, seen = {}, set()
    for _ in range(4):
        g, o = parity_step(eng, loop, delta, stats=stats, **tol)
        seen |= set(int(a) for a, n in zip(o["accept"], o["step_len"]) if n)
        plain.step(delta)
    assert seen == {0, 1}
    assert [r.z for r in loop.rows] == [r.z for r in plain.rows]
    compare_counters(eng, loop)
    c = eng.counters()
    assert c["sd_rounds"] > 0 and c["sd_verified"] == c["sd_proposed"] >= c["gen_tokens"][2]
    print("speculative decoding of rejected steps, k =", k, stats, {q: c[q] for q in c if q.startswith("sd_")})
    eng.close()


@pytest.mark.parametrize("extra,min_rows", [(dict(), 3), (dict(prm_shares_draft=True), 1)])
def test_speculative_decoding_with_queued_rows_and_with_a_merged_prm(extra, min_rows):
    """sd_tokens together with the other two scheduling modes: rejected rows that wait for a shared target pass
    (rsd_step_queued), and a PRM that is a head on the draft's trunk (its scoring pass leaves one more position in
    the draft's cache beyond the cursor, which the proposals then overwrite)."""
    prompts = ri.prompts(63, 6, 5, 20, 1024)
    kw = dict(max_step_tokens=6, max_steps=5, max_seq_tokens=96, step_end_id=3, step_end_mod=5, temperature=0.7,
              seed=12, sd_tokens=3, **extra)
    eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=kw)
    delta = float(np.median(loop.step(0.0)["rewards"]))
    eng, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=kw)
    served = 0
    for _ in range(12):
        if not any(r.live for r in loop.rows):
            break
        g, o = parity_step(eng, loop, delta, min_target_rows=min_rows, **TOL32)
        served += sum(1 for r in o["sd_rounds"] if r)
    assert served > 0
    compare_counters(eng, loop)
    eng.close()


def test_speculative_rounds_keep_the_matching_prefix_on_gpu():
    """Proposals planted around the target's true continuation (known from a first, plain run of the oracle): all
    right, wrong at once, right-right-wrong, a short last round.  The GPU must write the matching prefix plus the
    target's own token, round by round: tokens, cursors and the round counters against the oracle's."""
    from oracle.rsd_loop import OracleRSD, LoopConfig
    shapes = TINY
    prompts = ri.prompts(62, 3, 5, 12, shapes[0].vocab)
    kw = dict(max_step_tokens=9, max_steps=1, max_seq_tokens=40, step_end_id=1 << 20, temperature=0.7, seed=5, sd_tokens=4)
    _, probe = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=dict(kw, sd_tokens=0))
    truth = [list(y) for y in probe.step(2.0)["step_tokens"]]          # delta above the range: the target's steps
    bad = lambda t: (t + 1) % 1024
    planted = []
    for b in range(3):
        t = truth[b]
        planted.append([t[0:4], [bad(t[4]), 7, 7, 7], [t[5], t[6], bad(t[7]), t[8]], [t[8]]])
    planted[2] = None                                                   # row 2 keeps the draft's own proposals
    eng, loop = build_pair(shapes, bf16=False, prompts=prompts, loop_kwargs=kw)
    o = loop.step(2.0, forced_sd_props=planted)
    eng.force_tokens(0, o["draft_tokens"])
    eng.force_tokens(2, o["target_tokens"])
    eng.force_sd_proposals([None if r is None else [rd["props"] for rd in r] for r in o["sd_rounds"]])
    g = eng.step(2.0)
    for b in range(3):
        assert g["step_tokens"][b].tolist() == truth[b] == list(o["step_tokens"][b])
    for b in range(2):
        assert [(rd["emitted"], rd["matched"]) for rd in o["sd_rounds"][b]] == [(4, 4), (1, 0), (3, 2), (1, 1)]
    from helpers import compare_state
    compare_state(eng, loop)
    compare_counters(eng, loop)
    smp = eng.sampled(2)
    for b in range(3):                                   # the target's own choices were the truth everywhere
        clear = [j for j in range(9) if o["target_trace"][b]["margin"][j] > 1e-3]
        assert [smp[b, j] for j in clear] == [truth[b][j] for j in clear]
    eng.close()


def test_device_outputs_and_target_step_rewards():
    """rsd_step_device fills device arrays with what rsd_step returns on the host, and the reward of a step the
    target wrote shows up one call later (the PRM caches that step before it scores the next draft step): NaN
    before, equal to the oracle's value afterwards."""
    prompts = ri.prompts(71, 5, 6, 20, 1024)
    kw = dict(max_step_tokens=6, max_steps=4, max_seq_tokens=64, step_end_id=3, step_end_mod=5, temperature=0.7, seed=9)
    a, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=kw)
    b, _ = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=kw)
    assert np.isnan(a.target_step_rewards()).all()
    delta = float(np.median(loop.step(0.0)["rewards"]))
    _, loop = build_pair(TINY, bf16=False, prompts=prompts, loop_kwargs=kw)
    seen = 0
    for i in range(4):
        o = loop.step(delta)
        host = a.step(delta)
        dev = b.step_device(delta)
        for k in ("step_tokens", "step_len", "rewards", "accept", "live"):
            assert np.array_equal(host[k], dev[k].cpu().numpy()), k
        fresh = ~np.isnan(o["target_rewards"])
        got = a.target_step_rewards()
        if fresh.any():
            assert np.abs(got[fresh] - o["target_rewards"][fresh]).max() <= 1e-5
            seen += int(fresh.sum())
        if i == 0:
            assert np.isnan(got).all()                                   # nothing the target wrote has been scored yet
    assert seen > 0
    a.close(); b.close()
