"""TEST INFRASTRUCTURE -- Algorithm 1 (RSD) of the paper, batched over independent rows.

For every live row and step i (Algorithm 1, loop body):
    draft step   y^_i <- m(x, y_{1:i-1})
    reward       r_i  <- r(y^_i | x, y_{1:i-1})          (the listing prints y_i; the prose around
                                                           it scores the draft step)
    if A_omega(r_i):  y_i <- y^_i                          (Algorithm 2, Table 1)
    else:             y_i <- M(x, y_{1:i-1})
    stop the row when the EOS token s is in y_i, or after N steps.

A "step" is a run of tokens that ends with the step delimiter (Section 3, "Default Setting": a
generation ending in a blank line is one reasoning step), with EOS, or at a token cap.

Besides the token-level results the loop keeps the integer book-keeping a paged implementation
needs, under one deterministic policy, so it can be compared bit for bit:
  * per model a cursor kv_len[b] = number of positions whose keys/values are cached.  The newest
    committed token may be un-cached; it is the first input of the next decode;
  * 16-token pages handed out by a bump counter, in ascending row order, when a phase needs
    capacity: draft (live rows) up to |z_i|-1+cap at step start, PRM (live rows) up to
    |z_i|+len(y^_i) before scoring, target (rejected rows) up to |z_i|-1+cap after the gate;
    pages stay with their row until reset;
  * the ascending list of rejected rows, and token / FLOPs counters (Section 3.3: 2N FLOPs per
    inference token of an N-parameter model, PRM included).

Merged PRM (`prm_shares_draft`).  Appendix B.3 builds the PRM as a projection layer on top of the
final transformer layer of a language model, and the discussion of model merging (Section 4, "PRM
overhead") asks for one model that is both policy and PRM.  When the PRM's trunk IS the draft's
trunk, the reward of y^_i needs no second pass over (z_i, y^_i): the draft's cache already covers
everything but the last token of y^_i, so one more single-token forward of the draft at that token
gives the hidden state the reward head reads.  The draft cursor is not advanced by it (the token
is fed again as the first input of the next decode), so the cursors and every token are exactly
those of the loop with a separate PRM whose trunk weights equal the draft's; the PRM keeps no
cache at all.

Queued rejections (`min_target_rows` > 1).  Rows never interact, so nothing in Algorithm 1 says that
all rows must take their i-th step together.  The paper counts the cost of the target by the tokens
it generates (Section 3.3), but a batched target pass reads all of M's weights whether one row or
the whole batch was rejected; to turn the saved FLOPs into saved time a rejected row may WAIT, its
draft step dropped, while the accepted rows go on drafting, until `min_target_rows` rows wait (or
nothing else is left to run); then the target writes y_i for all of them in one pass.  Each row's
own sequence of steps is the one Algorithm 1 gives it: only the order in time changes.

RSD combined with speculative decoding (`sd_tokens` = k > 0; Section 4, the discussion item on combining
RSD with SD: the target need not write a rejected step alone, draft + target speculative decoding can).  The step
of a rejected row is then written in rounds.  In a round the draft proposes up to k tokens after the
tokens written so far; the target evaluates, in ONE pass over the last written token and all but the
last proposal, its own choice at each of those positions; the choices are taken one by one while every
earlier one equalled the draft's proposal, so a round writes the matching prefix plus the target's first
differing (or, after k matches nothing more: at most k) token.  A token's sampling noise depends only on
(model, row, position), so the target's choice at a position is a function of the context alone and the
step equals, token for token, the one the target would have decoded by itself: only the number of target
passes changes.  Both caches keep the positions whose input tokens were written; what the draft and the
target cached beyond them is overwritten later.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import OracleModel, sample, accept as _accept, uniform as _uniform

DRAFT, PRM, TARGET = 0, 1, 2
STREAM_ACCEPT = 3  # Philox stream of the acceptance uniform of Algorithm 2


@dataclass
class LoopConfig:
    max_step_tokens: int
    max_steps: int
    max_seq_tokens: int
    step_end_id: int
    eos_id: int = -1
    step_end_mod: int = 0          # >0: a token ends a step iff id % mod == step_end_id % mod
    temperature: float = 0.0
    seed: int = 0
    page_tokens: int = 16
    omega_kind: int = 1            # Table 1 row: 0 constant, 1 binary step, 2 clip, 3 r/(1+r), 4 logistic
    omega_b: float = 0.0           # alpha of the logistic; the first parameter is the delta of each step
    prm_shares_draft: bool = False  # the PRM is a reward head on the draft's trunk (merged serving, see below)
    sd_tokens: int = 0             # k > 0: rejected steps are rewritten by draft + target speculative decoding
    pool_pages: tuple = (1 << 30, 1 << 30, 1 << 30)
    keep_logits: bool = False


@dataclass
class Row:
    z: list                         # committed tokens: prompt x followed by y_{1:i-1}
    live: bool = True
    waiting: bool = False           # the row's draft step was rejected and the target has not written y_i yet
    reward: float = 0.0             # reward of the row's latest draft step
    n_steps: int = 0
    kv_len: list = field(default_factory=lambda: [0, 0, 0])
    caches: list = field(default_factory=lambda: [None, None, None])
    pages: list = field(default_factory=lambda: [[], [], []])


class OracleRSD:
    def __init__(self, draft: OracleModel, prm: OracleModel, target: OracleModel, cfg: LoopConfig):
        self.models = [draft, prm, target]
        self.cfg = cfg
        self.v_limit = min(m.shape.vocab for m in self.models)  # ids valid for all three embeddings
        self.rows: list[Row] = []
        self.next_page = [0, 0, 0]
        self.counters = dict(gen_tokens=[0, 0, 0], ingest_tokens=[0, 0, 0], score_tokens=0, steps=0,
                             accepted_steps=0, rejected_steps=0, discarded_draft_tokens=0,
                             sd_rounds=0, sd_proposed=0, sd_matched=0, sd_verified=0)

    # -- book-keeping ---------------------------------------------------------------------
    def _reserve(self, which: int, b: int, need_tokens: int):
        row = self.rows[b]
        pt = self.cfg.page_tokens
        while len(row.pages[which]) * pt < need_tokens:
            if self.next_page[which] >= self.cfg.pool_pages[which]:
                raise MemoryError("page pool exhausted")
            row.pages[which].append(self.next_page[which])
            self.next_page[which] += 1

    def _ends_step(self, tok: int) -> bool:
        c = self.cfg
        if c.eos_id >= 0 and tok == c.eos_id:
            return True
        if c.step_end_mod > 0:
            return tok % c.step_end_mod == c.step_end_id % c.step_end_mod
        return tok == c.step_end_id

    def _ingest(self, which: int, b: int, upto: int, tokens: list) -> np.ndarray | None:
        """Cache positions [kv_len, upto) of `tokens` in model `which`; returns their hidden states."""
        row = self.rows[b]
        start = row.kv_len[which]
        if upto <= start:
            return None
        h = self.models[which].forward(row.caches[which], tokens[start:upto], start)
        row.kv_len[which] = upto
        return h

    # -- entry points -----------------------------------------------------------------------
    def prefill(self, prompts: list):
        """Rows start with z_1 = x.  The draft caches x without its last token, the PRM all of x;
        the target is left untouched until a row is first rejected."""
        self.rows = []
        for b, p in enumerate(prompts):
            row = Row(z=[int(t) for t in p])
            for which in (DRAFT, PRM, TARGET):
                row.caches[which] = self.models[which].new_cache(self.cfg.max_seq_tokens)
            self.rows.append(row)
        for row in self.rows:
            if len(row.z) + self.cfg.max_step_tokens > self.cfg.max_seq_tokens:
                row.live = False        # no room for even one step: the row never starts
        live_rows = [b for b, row in enumerate(self.rows) if row.live]
        shared = self.cfg.prm_shares_draft
        for b in live_rows:
            self._reserve(DRAFT, b, len(self.rows[b].z) - 1)
        for b in live_rows:
            if not shared:
                self._reserve(PRM, b, len(self.rows[b].z))
        for b in live_rows:
            row = self.rows[b]
            n = len(row.z)
            self._ingest(DRAFT, b, n - 1, row.z)
            self.counters["ingest_tokens"][DRAFT] += n - 1
            if not shared:
                self._ingest(PRM, b, n, row.z)
                self.counters["ingest_tokens"][PRM] += n

    def _generate_step(self, which: int, b: int, forced=None, trace=None) -> list:
        """One step from model `which` given the row's context z (Algorithm 1: m(x, y_{1:i-1}) or
        M(x, y_{1:i-1})): cache what of z is missing, then decode token by token."""
        row, cfg, model = self.rows[b], self.cfg, self.models[which]
        z = row.z
        before = row.kv_len[which]
        self._ingest(which, b, len(z) - 1, z)
        self.counters["ingest_tokens"][which] += (len(z) - 1) - before
        out, cur, pos = [], z[-1], len(z) - 1
        for j in range(cfg.max_step_tokens):
            h = model.forward(row.caches[which], [cur], pos)
            row.kv_len[which] = pos + 1
            logits = model.logits(h[0])
            tok, margin = sample(logits, self.v_limit, cfg.temperature, cfg.seed, which, b, pos + 1)
            if trace is not None:
                trace["sampled"].append(tok)
                trace["margin"].append(margin)
                if cfg.keep_logits:
                    trace["logits"].append(logits.copy())
            if forced is not None:
                tok = int(forced[j])
            out.append(tok)
            self.counters["gen_tokens"][which] += 1
            if self._ends_step(tok) or (forced is not None and j + 1 == len(forced)):
                break
            cur, pos = tok, pos + 1
        return out

    def _generate_step_sd(self, b: int, forced=None, trace=None, sd_trace=None, forced_props=None) -> list:
        """The step of a rejected row by speculative decoding: rounds of (draft proposes, target checks)."""
        row, cfg = self.rows[b], self.cfg
        draft, target = self.models[DRAFT], self.models[TARGET]
        z = row.z
        before = row.kv_len[TARGET]
        self._ingest(TARGET, b, len(z) - 1, z)
        self.counters["ingest_tokens"][TARGET] += (len(z) - 1) - before
        before = row.kv_len[DRAFT]
        self._ingest(DRAFT, b, len(z) - 1, z)          # nothing to do after a rollback; kept for generality
        self.counters["ingest_tokens"][DRAFT] += (len(z) - 1) - before
        out, cur, pos = [], z[-1], len(z) - 1
        limit = len(forced) if forced is not None else cfg.max_step_tokens
        done = False
        while not done:
            kk = min(cfg.sd_tokens, cfg.max_step_tokens - len(out))   # a round never reaches beyond the step cap
            # the draft proposes kk tokens for positions pos + 1 .. pos + kk
            props, c, p = [], cur, pos
            for i in range(kk):
                h = draft.forward(row.caches[DRAFT], [c], p)
                tok, _ = sample(draft.logits(h[0]), self.v_limit, cfg.temperature, cfg.seed, DRAFT, b, p + 1)
                if forced_props is not None:
                    tok = int(forced_props[len(sd_trace) if sd_trace is not None else 0][i])
                props.append(tok)
                c, p = tok, p + 1
            # the target's choices at the same positions, from one pass over (cur, props[:-1])
            hs = target.forward(row.caches[TARGET], [cur] + props[:kk - 1], pos)
            n_emit = n_match = 0
            for i in range(kk):
                logits = target.logits(hs[i])
                tok, margin = sample(logits, self.v_limit, cfg.temperature, cfg.seed, TARGET, b, pos + 1 + i)
                if trace is not None:
                    trace["sampled"].append(tok)
                    trace["margin"].append(margin)
                    if cfg.keep_logits:
                        trace["logits"].append(logits.copy())
                if forced is not None:
                    tok = int(forced[len(out)])
                out.append(tok)
                n_emit += 1
                if self._ends_step(tok) or len(out) == limit:
                    done = True
                if tok == props[i]:
                    n_match += 1
                if done or tok != props[i]:
                    break
            # both caches now hold the positions whose input tokens were written: cur and all written but the last
            row.kv_len[TARGET] = pos + n_emit
            row.kv_len[DRAFT] = pos + n_emit
            self.counters["gen_tokens"][TARGET] += n_emit
            self.counters["sd_rounds"] += 1
            self.counters["sd_proposed"] += kk
            self.counters["sd_matched"] += n_match
            self.counters["sd_verified"] += kk
            if sd_trace is not None:
                sd_trace.append(dict(props=list(props), emitted=n_emit, matched=n_match))
            cur, pos = out[-1], pos + n_emit
        return out

    def step(self, delta: float, forced_draft=None, forced_target=None, forced_accept=None,
             min_target_rows: int = 1, forced_sd_props=None) -> dict:
        """One pass of the loop body of Algorithm 1 over the rows.  `forced_*` (per-row lists, or
        None entries) replace sampled tokens / gate decisions; what was sampled is still reported.

        min_target_rows = 1: every live row takes one step (draft, score, gate, target for the
        rejected rows).  min_target_rows > 1: rows whose step is rejected wait until that many rows
        wait, or until all live rows do; waiting rows take no part in the draft phase and report
        step_len 0 until the target has written their step."""
        cfg, B = self.cfg, len(self.rows)
        res = dict(step_tokens=[[] for _ in range(B)], step_len=np.zeros(B, np.int32),
                   rewards=np.zeros(B, np.float64), accept=np.zeros(B, np.uint8), live=np.zeros(B, np.uint8),
                   draft_tokens=[[] for _ in range(B)], target_tokens=[[] for _ in range(B)],
                   draft_trace=[None] * B, target_trace=[None] * B, rej_idx=[], z_len_before=np.zeros(B, np.int32),
                   drafted=np.zeros(B, np.uint8), waiting=np.zeros(B, np.uint8), flushed=False,
                   sd_rounds=[None] * B, target_rewards=np.full(B, np.nan))
        run_rows = [b for b in range(B) if self.rows[b].live and not self.rows[b].waiting]
        for b in range(B):
            res["z_len_before"][b] = len(self.rows[b].z)
        for b in run_rows:
            res["drafted"][b] = 1

        # draft step y^_i for every live row that is not waiting for the target (with a merged PRM the
        # draft also caches the step's last token when it scores it: one more position)
        shared = cfg.prm_shares_draft
        for b in run_rows:
            self._reserve(DRAFT, b, len(self.rows[b].z) - 1 + cfg.max_step_tokens + (1 if shared else 0))
        for b in run_rows:
            tr = dict(sampled=[], margin=[], logits=[])
            f = forced_draft[b] if forced_draft is not None else None
            res["draft_tokens"][b] = self._generate_step(DRAFT, b, f, tr)
            res["draft_trace"][b] = tr

        # reward r_i = r(y^_i | z_i), read at the last token of the draft step
        for b in run_rows:
            if not shared:
                self._reserve(PRM, b, len(self.rows[b].z) + len(res["draft_tokens"][b]))
        for b in run_rows:
            row = self.rows[b]
            if shared:
                # the draft's cache holds z_i and all of y^_i but its last token: push that token
                # through the draft's trunk, read the reward head, leave the cursor where it was
                pos = row.kv_len[DRAFT]
                assert pos == len(row.z) + len(res["draft_tokens"][b]) - 1
                h = self.models[DRAFT].forward(row.caches[DRAFT], [res["draft_tokens"][b][-1]], pos)
                row.reward = self.models[PRM].reward(h[0])
                self.counters["score_tokens"] += 1
                continue
            seq = row.z + res["draft_tokens"][b]
            n_known = len(row.z) - row.kv_len[PRM]      # committed tokens the PRM has not cached yet
            h = self._ingest(PRM, b, len(seq), seq)
            row.reward = self.models[PRM].reward(h[-1])
            if n_known > 0:
                # the row's previous step was written by the target: the PRM caches it only now, and the hidden
                # state at its last token gives that step's reward r(y_{i-1} | z_{i-1}) on the way (the paper's
                # comparison of draft-step and target-step rewards inside RSD reads such values); not used by the gate
                res["target_rewards"][b] = self.models[PRM].reward(h[n_known - 1])
            self.counters["ingest_tokens"][PRM] += n_known
            self.counters["score_tokens"] += len(res["draft_tokens"][b])

        # acceptance criterion A_omega(r_i)  (Algorithm 2; binary step: accept iff r_i >= delta)
        for b in run_rows:
            row = self.rows[b]
            u = _uniform(cfg.seed, STREAM_ACCEPT, b, len(row.z), 0)
            a = _accept(cfg.omega_kind, row.reward, float(delta), cfg.omega_b, u)
            if forced_accept is not None and forced_accept[b] is not None:
                a = int(forced_accept[b])
            res["accept"][b] = a
            if not a:
                # drop the draft step from the draft and PRM caches; the target will write y_i
                row.waiting = True
                row.kv_len[DRAFT] = len(row.z) - 1
                if not shared:
                    row.kv_len[PRM] = len(row.z)
                self.counters["discarded_draft_tokens"] += len(res["draft_tokens"][b])
        wait_rows = [b for b in range(B) if self.rows[b].live and self.rows[b].waiting]
        res["rej_idx"] = wait_rows
        n_live = sum(1 for r in self.rows if r.live)
        flush = len(wait_rows) > 0 and len(wait_rows) >= min(max(1, int(min_target_rows)), n_live)
        res["flushed"] = flush

        if flush:
            for b in wait_rows:
                self._reserve(TARGET, b, len(self.rows[b].z) - 1 + cfg.max_step_tokens)
            for b in wait_rows:
                tr = dict(sampled=[], margin=[], logits=[])
                f = forced_target[b] if forced_target is not None else None
                if cfg.sd_tokens > 0:
                    res["sd_rounds"][b] = []
                    fp = forced_sd_props[b] if forced_sd_props is not None else None
                    res["target_tokens"][b] = self._generate_step_sd(b, f, tr, res["sd_rounds"][b], fp)
                else:
                    res["target_tokens"][b] = self._generate_step(TARGET, b, f, tr)
                res["target_trace"][b] = tr

        # commit y_i, stop rows that produced EOS or ran out of steps / room
        for b in range(B):
            row = self.rows[b]
            if not row.live:
                continue
            res["rewards"][b] = row.reward
            if res["accept"][b]:
                y = res["draft_tokens"][b]
            elif row.waiting and flush:
                y = res["target_tokens"][b]
                row.waiting = False
            else:
                continue                # waits for a later target pass
            row.z = row.z + y
            row.n_steps += 1
            res["step_tokens"][b] = y
            res["step_len"][b] = len(y)
            self.counters["steps"] += 1
            self.counters["accepted_steps" if res["accept"][b] else "rejected_steps"] += 1
            if (cfg.eos_id >= 0 and cfg.eos_id in y) or row.n_steps >= cfg.max_steps \
                    or len(row.z) + cfg.max_step_tokens > cfg.max_seq_tokens:
                row.live = False
        for b in range(B):
            res["live"][b] = 1 if self.rows[b].live else 0
            res["waiting"][b] = 1 if (self.rows[b].live and self.rows[b].waiting) else 0
        return res

    # -- reporting --------------------------------------------------------------------------
    def flops_paper(self) -> float:
        """2N per inference token (Section 3.3): every token the draft or the target generated
        (discarded draft tokens included) and every token the PRM processed.  With speculative decoding of the
        rejected steps the draft is billed its proposals as well and the target every position it evaluated."""
        c = self.counters
        n = [m.n_params for m in self.models]
        target_tokens = c["sd_verified"] if self.cfg.sd_tokens > 0 else c["gen_tokens"][TARGET]
        return 2.0 * n[DRAFT] * (c["gen_tokens"][DRAFT] + c["sd_proposed"]) + 2.0 * n[TARGET] * target_tokens \
            + 2.0 * n[PRM] * (c["score_tokens"] + c["ingest_tokens"][PRM])

    def state(self) -> dict:
        B = len(self.rows)
        return dict(z_len=np.array([len(r.z) for r in self.rows], np.int32),
                    kv_len=np.array([[r.kv_len[w] for r in self.rows] for w in range(3)], np.int32),
                    n_pages=np.array([[len(r.pages[w]) for r in self.rows] for w in range(3)], np.int32),
                    pages=[[list(r.pages[w]) for r in self.rows] for w in range(3)],
                    next_page=list(self.next_page),
                    live=np.array([r.live for r in self.rows], np.uint8),
                    waiting=np.array([r.live and r.waiting for r in self.rows], np.uint8),
                    n_steps=np.array([r.n_steps for r in self.rows], np.int32))
