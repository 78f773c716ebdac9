#!/usr/bin/env python
"""Benchmark of the RSD step loop on B200: tokens committed per second by rsd_step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2|mini]

A "step" is one rsd_step: draft decode of one reasoning step for every live row, PRM scoring, the
threshold gate, target re-decode of the rejected rows, commit.  The default workload is the
1.5B-shape draft and PRM with the 7B-shape target in bf16, batch 32, prompts of 128..512 uniform
random tokens, steps of at most 128 tokens, Gumbel-max sampling at temperature 0.7, delta set on a
calibration pass to the reward quantile that accepts about 70 % of the draft steps.  All inputs are
seeded and synthetic (random-init weights, random prompts).

With N > 1 (torchrun) every rank runs an independent replica of the workload on its own GPU with its
own prompts; there is no collective on the data path.  `--impl reference` times the CPU oracle on a
bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import rsd_inputs as ri  # noqa: E402

METRIC = "rsd_step_tokens_per_sec"
UNIT = "tokens/s"

WORKLOADS = {
    # name: (draft, prm, target shapes, batch, prompt lo, hi, step cap)
    "cfg2": ("1.5b", "1.5b", "7b", 32, 128, 512, 128),
    "mini": ("mini_draft", "mini_draft", "mini_target", 8, 32, 96, 16),
    # PRM at the target's shape, batch 64, 256-token prompts, steps of up to 256 tokens (delta sweep via --delta)
    "cfg3": ("1.5b", "7b", "7b", 64, 256, 256, 256),
    # 72B-shape target (about 145 GB of bf16 weights), batch 8, 256-token prompts, steps of up to 256 tokens
    "cfg4": ("1.5b", "1.5b", "72b", 8, 256, 256, 256),
}


TRAFFIC_SOURCES = ("gemm_tc.cu", "tc_ptx.cuh", "attn_decode.cu", "kernels_math.cu", "kernels_state.cu", "common.cuh")


def kernel_sources_sha() -> str:
    """One hash over the sources of every kernel of a decode iteration."""
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2501_19324_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def iteration_traffic_ratio():
    """DRAM traffic / algorithmic bytes of one target decode iteration from the committed ncu capture (taken at a
    step cap of 8 tokens, where the iteration's kernels are those of the full-size step; traffic grows with the
    weights and the KV read, as the algorithmic bytes do), or None when a kernel source has changed since."""
    try:
        d = json.load(open(os.path.join(ROOT, "profiles", "target_decode_iteration_traffic.json")))
        return d["ratio"] if kernel_sources_sha() == d["sha256"] else None
    except (OSError, KeyError, ValueError):
        return None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["hbm_gbs"], d["bf16_tflops_sustained"], "measured"
    return 6650.0, 1400.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def mark(self) -> int:
        """Number of samples taken so far; two marks bracket a region for summary()."""
        return len(self.rows)

    def summary(self, lo: int = 0, hi: int | None = None) -> dict:
        """Median SM clock, maximum clock and the throttle reasons seen in samples [lo, hi)."""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[lo:hi]:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self.summary()


def cpu_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def mem_available_gb() -> float:
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) / 1e6
    except OSError:
        pass
    return 0.0


# ------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample of the workload
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """One row of the workload pushed through the oracle's step loop for one short step.

    level 0: 24-token prompt, 6-token step, forced rejection, so draft, PRM and target all run (about 10 s of
    host time at the 1.5B / 1.5B / 7B shapes);
    level 1: 4-token prompt, 1-token step, accepted (draft and PRM only) -- used when many steps are
    requested or the host has too little memory for the target's fp32 weights."""

    def __init__(self, workload: str, level: int):
        from oracle import OracleModel
        d, p, t, _, _, _, _ = WORKLOADS[workload]
        self.level = level
        self.shapes = [ri.SHAPES[d], ri.SHAPES[p], ri.SHAPES[t]]
        heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
        self.models = []
        for slot, (sh, hk) in enumerate(zip(self.shapes, heads)):
            with_layers = not (slot == 2 and level == 1)
            self.models.append(OracleModel(ri.cpu_model_weights(sh, slot, 0, True, hk, with_layers=with_layers), slot))
        self.prompt_len, self.cap = (24, 6) if level == 0 else (4, 1)
        self.delta = 2.0 if level == 0 else 0.0
        self.desc = (f"1 row, {self.prompt_len}-token prompt, one step of {self.cap} token(s), "
                     + ("delta above the PRM range so the target re-decodes it" if level == 0 else
                        "delta 0 so the step is accepted (target not run)")
                     + "; full depth and vocabulary, bf16-rounded weights, fp64 arithmetic")

    def run_once(self, seed: int) -> tuple:
        from oracle.rsd_loop import OracleRSD, LoopConfig
        tokens, offsets = ri.prompts(100 + seed, 1, self.prompt_len, self.prompt_len, self.shapes[0].vocab)
        cfg = LoopConfig(max_step_tokens=self.cap, max_steps=1, max_seq_tokens=self.prompt_len + self.cap,
                         step_end_id=13, temperature=0.7, seed=seed)
        loop = OracleRSD(*self.models, cfg)
        t0 = time.perf_counter()
        loop.prefill([tokens.tolist()])
        r = loop.step(self.delta)
        dt = time.perf_counter() - t0
        return int(r["step_len"].sum()), dt


def run_reference(args, rank: int):
    if rank != 0:
        return
    level = 0 if (args.steps + args.warmup) <= 10 and mem_available_gb() > 60 else 1
    if args.workload == "mini":
        level = 0
    if args.workload in ("cfg3", "cfg4"):
        level = 1          # two 7B-shape or one 72B-shape fp32 weight set do not fit the host: draft + PRM only
    sample = OracleSample(args.workload, level)
    for i in range(args.warmup):
        sample.run_once(i)
    toks, secs = 0, 0.0
    for i in range(args.steps):
        n, dt = sample.run_once(args.warmup + i)
        toks += n
        secs += dt
    value = toks / secs
    out = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic", "config": workload_config(args),
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": sample.desc},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def kv_extended(args) -> int:
    """rsd_config.kv_extended: 0 lets the library decide per model by depth (the 80-layer target of cfg4 gets
    the hi + lo KV cache that keeps its logits within 3e-2 of the fp64 definition), 1 forces the pairs, 2 the
    plain fp16 cache."""
    v = getattr(args, "kv_extended", None)
    return int(v) if v is not None else 0


def chunk_tokens(args) -> int:
    """max_chunk_tokens of the run: configs 2 and 3 score more than 4096 tokens per step (32 x 128 draft tokens plus the
    target-written steps the PRM still has to cache; 64 x 256), so their passes take 8192-token chunks instead of
    the library's 4096 (one dense pass instead of a full one and a thin one); 0 = the library's default."""
    if getattr(args, "chunk", 0):
        return args.chunk
    return 8192 if args.workload in ("cfg2", "cfg3") else 0


def kv_cache_label(args) -> str:
    setting = kv_extended(args)
    names = WORKLOADS[args.workload][:3]
    ext = [setting == 1 or (setting == 0 and ri.SHAPES[n].n_layers > 48) for n in names]
    if all(ext):
        return "fp16 hi+lo pairs"
    if not any(ext):
        return "fp16"
    return "fp16; fp16 hi+lo pairs for " + ", ".join(r for r, e in zip(("draft", "PRM", "target"), ext) if e)


def workload_config(args) -> dict:
    d, p, t, B, lo, hi, cap = WORKLOADS[args.workload]
    return {"workload": f"{args.workload}: draft {d} / PRM {p} / target {t} shapes, batch {B}, prompts {lo}-{hi} tokens, "
                        f"step <= {cap} tokens, Gumbel-max T=0.7, "
                        + (f"delta {args.delta}" if getattr(args, "delta", None) is not None else "delta at the 70% accept quantile"),
            "batch": B, "max_step_tokens": args.cap or cap, "replicas": args.gpus,
            "kv_cache": kv_cache_label(args), "max_chunk_tokens": chunk_tokens(args) or 4096,
            "dense_operands": "bf16 hi + lo pairs" if getattr(args, "no_f16_dense", False) else
                              "passes of more than 128 tokens: fp16 copies of the layer weights (made at load, models up to 20 GB) "
                              "x one fp16 activation; decode and the 72B-shape target: bf16 weights x bf16 hi + lo pairs",
            "prm": "head on the draft's trunk (prm_shares_draft)" if getattr(args, "merged_prm", False) else "separate model",
            "schedule": "lock-step rsd_step" if getattr(args, "queue", 1) == 1 else
                        f"rsd_step_queued, target pass once {args.queue} rows wait",
            "rejected_steps": "target decoding" if not getattr(args, "sd", 0) else
                              f"speculative decoding, {args.sd} draft proposals per target pass",
            "l2": "weights and KV read per decode iteration exceed the 126 MB L2 (no flush needed)"}


def combine_ranks(ms, e2e_ms, tokens, e2e_tokens, world, device):
    """Whole-job figures of N independent replicas: the slowest rank's time, the sum of the tokens."""
    if world <= 1:
        return ms, e2e_ms, float(tokens), float(e2e_tokens)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms, e2e_ms], dtype=torch.float64, device=device)
    n = torch.tensor([float(tokens), float(e2e_tokens)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(n[0]), float(n[1])


def debug_flags(args) -> int:
    from paper_2501_19324_b200 import RSD_DEBUG_PERSISTENT_DECODE, RSD_DEBUG_MEGA_PROFILE
    from paper_2501_19324_b200.binding import RSD_DEBUG_NO_F16_DENSE
    return ((RSD_DEBUG_PERSISTENT_DECODE if (args.mega or args.mega_profile) else 0) | (RSD_DEBUG_MEGA_PROFILE if args.mega_profile else 0)
            | (RSD_DEBUG_NO_F16_DENSE if getattr(args, "no_f16_dense", False) else 0))


def mega_phase_table(eng, which: int, n_layers: int) -> dict:
    """Mean duration (us) of each phase of the persistent decode kernel's last launch, work and barrier wait
    apart, as seen by its first CTA."""
    st = eng.mega_profile(which).astype(np.int64)
    names = ["qkv", "attention", "wo", "resid_norm_1", "gate_up_swiglu", "down", "resid_norm_2"]
    out = {"total_us": float(st[-1] - st[0]) / 1e3, "embed_us": float(st[1] - st[0]) / 1e3}
    work = {n: [] for n in names}
    wait = {n: [] for n in names}
    # stamps: [start, (work end, barrier end) of the embedding phase, then of every layer phase ..., kernel end]
    i = 3
    for l in range(n_layers):
        for n in names:
            if i >= len(st):
                break
            work[n].append(st[i] - st[i - 1])
            if i + 1 < len(st) and not (l == n_layers - 1 and n == names[-1]):
                wait[n].append(st[i + 1] - st[i])
            i += 2
    for n in names:
        out[n] = {"work_us": float(np.mean(work[n])) / 1e3 if work[n] else None,
                  "barrier_us": float(np.mean(wait[n])) / 1e3 if wait[n] else None}
    return out


def decode_iteration_roofline(phases, iters, kv_bytes, steps, shapes, hbm, queue, sd=0):
    """Whole decode iterations against the HBM roofline.  One iteration of model X is one replay of its captured
    graph (every layer, the lm head, sampling).  Algorithmic bytes of an iteration: every layer's weights and the
    lm head once (the embedding table is gathered, not streamed) plus the keys and values of every attended
    position (kv_bytes: summed on the host from the rows' context lengths).  Time: the phase's device time from
    CUDA events on the launching stream over the timed steps / the iterations it ran (a phase runs until its
    longest row ends; a rejected row's draft step ran to the cap before it was dropped).  Only meaningful for the
    lock-step schedule."""
    if queue != 1:
        return None
    out = {}
    for name, slot, key in (("draft", 0, "draft_decode"), ("target", 2, "target_decode")):
        sh = shapes[slot]
        weight_bytes = 2.0 * (sh.n_params() - sh.vocab * sh.d_model)       # bf16; the embedding table is not streamed
        n = iters[name]
        if n <= 0 or phases.get(key, 0) <= 0 or (sd and name == "target"):   # rounds of speculative decoding are not iterations
            out[name] = None
            continue
        ms = phases[key] * steps / n
        per_iter = weight_bytes + kv_bytes[name] / n
        gbs = per_iter / (ms * 1e-3) / 1e9
        out[name] = {"ms": ms, "weight_gb": weight_bytes / 1e9, "kv_gb": kv_bytes[name] / n / 1e9, "gbs": gbs,
                     "frac_of_hbm": gbs / hbm, "frac_of_hbm_weights_only": weight_bytes / (ms * 1e-3) / 1e9 / hbm,
                     "iterations": n}
    return out


def rank_prompts(rank, B, lo, hi, vocab):
    """Every replica works on its own prompts (seed 1 + rank)."""
    return ri.prompts(1 + rank, B, lo, hi, vocab)


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def run_ours(args, rank: int, world: int):
    import torch
    import torch.distributed as dist
    from paper_2501_19324_b200 import Engine, Model, lib

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    d, p, t, B, lo, hi, cap = WORKLOADS[args.workload]
    if args.cap:
        cap = args.cap          # profiling aid: shorter steps (recorded in the config line)
    shapes = [ri.SHAPES[d], ri.SHAPES[p], ri.SHAPES[t]]
    heads = (ri.HEAD_LM, ri.HEAD_REWARD_SIGMOID, ri.HEAD_LM)
    merged = bool(args.merged_prm)
    if merged and shapes[1] != shapes[0]:
        raise SystemExit("--merged-prm needs a PRM of the draft's shape")
    models = [Model(sh, ri.gpu_model_tensors(sh, slot, 0, True, hk), hk, head_only=merged and slot == 1)
              for slot, (sh, hk) in enumerate(zip(shapes, heads))]
    if merged:                      # only the PRM's embedding row count, final norm and head are read
        for k in ("wqkv", "wo", "wgu", "wdown", "norm1", "norm2"):
            models[1].t[k] = []
        torch.cuda.empty_cache()
    n_steps = args.warmup + args.steps + 1        # + one untimed step in which single GEMM launches are timed
    S = hi + n_steps * cap
    eng = Engine(*models, max_batch=B, max_seq_tokens=S, max_step_tokens=cap, max_steps=n_steps + 1,
                 step_end_id=13, temperature=0.7, seed=0, kv_extended=kv_extended(args),
                 prm_shares_draft=int(merged), debug_flags=debug_flags(args), sd_tokens=args.sd,
                 max_chunk_tokens=chunk_tokens(args))
    tokens, offsets = rank_prompts(rank, B, lo, hi, shapes[0].vocab)
    pinned_tokens = torch.from_numpy(tokens).pin_memory()

    # calibration pass: rewards of the first step decide delta (30th percentile -> ~70 % accepted)
    eng.prefill(tokens, offsets)
    r0 = eng.step(0.0)["rewards"]
    delta = float(np.sort(r0)[int(0.3 * B)])
    if args.delta is not None:
        delta = args.delta         # fixed threshold (config 3 sweeps 0.5 / 0.7 / 0.9)
    eng.reset()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # host-side book-keeping of context lengths, for the algorithmic bytes and flops of the phases
    z = np.diff(offsets).astype(np.int64)          # committed tokens per row
    prm_len = z.copy()                             # positions the PRM has cached
    kv_tok = [sh.kv_bytes_per_token(2) for sh in shapes]
    kv_bytes = {"draft": 0.0, "target": 0.0}
    prm_ctx_sum = 0                                # sum over the PRM's processed tokens of the positions each attends

    def account(r, timed):
        nonlocal prm_ctx_sum
        took = r["step_len"] > 0
        acc = took & (r["accept"] == 1)
        rej = took & (r["accept"] == 0)
        for b in np.nonzero(took)[0]:
            n_draft = int(r["step_len"][b]) if acc[b] else cap      # a rejected draft step ran to the cap
            if timed:
                kv_bytes["draft"] += kv_tok[0] * (n_draft * int(z[b]) + n_draft * (n_draft - 1) // 2)
                lo_p, hi_p = int(prm_len[b]), int(z[b]) + n_draft   # PRM: positions [lo_p, hi_p), token p attends p + 1
                prm_ctx_sum += (hi_p * (hi_p + 1) - lo_p * (lo_p + 1)) // 2
            if rej[b] and timed:
                n = int(r["step_len"][b])
                kv_bytes["target"] += kv_tok[2] * (n * int(z[b]) + n * (n - 1) // 2)
            if acc[b]:
                prm_len[b] = z[b] + r["step_len"][b]
            z[b] += r["step_len"][b]

    sampler = ClockSampler(local)
    launches0 = lib().rsd_debug_launch_count()
    barrier()
    sampler.start()
    e2e_t0 = time.perf_counter()
    e2e_start = torch.cuda.Event(enable_timing=True); e2e_end = torch.cuda.Event(enable_timing=True)
    e2e_start.record()
    eng.prefill(pinned_tokens.numpy(), offsets)          # host prompts -> device inside the call
    e2e_tokens = 0
    accepted = live_steps = 0
    for _ in range(args.warmup):
        r = eng.step(delta, args.queue)
        e2e_tokens += int(r["step_len"].sum())
        account(r, False)
    eng.gemm_timing(0)                                   # no event records inside the timed steps: every decode
    eng.phase_ms(True)                                   # iteration replays its captured graph
    c0 = eng.counters()
    barrier()
    launches1 = lib().rsd_debug_launch_count()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    clk_lo = sampler.mark()
    t_start.record()
    timed_tokens = 0
    iters = {"draft": 0, "target": 0}
    for _ in range(args.steps):
        r = eng.step(delta, args.queue)                    # host outputs: D2H inside the call
        timed_tokens += int(r["step_len"].sum())
        accepted += int(r["accept"].sum())
        live_steps += int((r["step_len"] > 0).sum())
        # decode iterations of the step: a phase runs until its longest row ends
        took = r["step_len"] > 0
        rejected = took & (r["accept"] == 0)
        if took.any():
            iters["draft"] += cap if rejected.any() else int(r["step_len"][took].max())
        if rejected.any():
            iters["target"] += int(r["step_len"][rejected].max())
        account(r, True)
    t_end.record()
    barrier()
    e2e_end.record()
    torch.cuda.synchronize()
    launches2 = lib().rsd_debug_launch_count()
    clocks = sampler.summary(clk_lo, sampler.mark())
    c1 = eng.counters()
    phases = {k: v / args.steps for k, v in eng.phase_ms(False).items()}
    # one more step, outside every timed region: single GEMM launches bracketed by CUDA events (decode
    # iterations chosen for it run kernel by kernel instead of replaying their graph)
    gt = {"ms": 0.0, "bytes": 0.0, "launches": 0}
    gd = {}
    if args.time_stride > 0:
        eng.gemm_timing(args.time_stride)
        eng.gemm_timing_dense()
        eng.step(delta, args.queue)
        gd = eng.gemm_timing_dense()
        gt = eng.gemm_timing(0)
    sampler.stop()
    e2e_tokens += timed_tokens
    ms = t_start.elapsed_time(t_end)
    e2e_ms = e2e_start.elapsed_time(e2e_end)
    ms, e2e_ms, timed_tokens, e2e_tokens = combine_ranks(ms, e2e_ms, timed_tokens, e2e_tokens, world, "cuda")
    counters = c1
    mega_tables = None
    if args.mega_profile and rank == 0:
        mega_tables = {}
        for name, which in (("draft", 0), ("target", 2)):
            try:
                mega_tables[name] = mega_phase_table(eng, which, shapes[which].n_layers)
            except Exception as e:       # the model does not run the persistent kernel
                mega_tables[name] = str(e)

    if rank == 0:
        hbm, tf, how = peaks()
        dec = decode_iteration_roofline(phases, iters, kv_bytes, args.steps, shapes, hbm, args.queue, args.sd)
        gemm_gbs = gt["bytes"] / (gt["ms"] * 1e-3) / 1e9 if gt["ms"] > 0 else None
        ratio = iteration_traffic_ratio()
        gemm_sub = {"what": "single weight-GEMM launches (decode, scoring, catch-up) in one extra, untimed step: CUDA events "
                            f"around every {args.time_stride}th launch; the decode iterations picked for it run kernel by kernel",
                    "GBps": gemm_gbs, "frac_of_hbm": (gemm_gbs / hbm) if gemm_gbs else None, "timed_launches": gt["launches"],
                    "algorithmic_bytes_per_launch": (gt["bytes"] / gt["launches"]) if gt["launches"] else None}
        # dominant phase: the target's decode iterations
        tgt = dec["target"] if dec else None
        if tgt:
            roofline = {"bound": "hbm", "kernel": "target decode iteration: one replay of the captured graph (28 layers of qkv / "
                        "attention / wo / gate-up + SwiGLU / down, lm head, sampling)",
                        "achieved": tgt["gbs"], "peak": hbm, "unit": "GB/s", "frac": tgt["frac_of_hbm"],
                        "traffic": (ratio * (tgt["weight_gb"] + tgt["kv_gb"]) * 1e9) if ratio else None,
                        "algorithmic_bytes_per_launch": (tgt["weight_gb"] + tgt["kv_gb"]) * 1e9,
                        "launches": tgt["iterations"], "avg_launch_ms": tgt["ms"],
                        "traffic_source": ("ncu dram__bytes_read + dram__bytes_write summed over the kernels of one iteration at a "
                                           f"step cap of 8 (profiles/), traffic / algorithmic = {ratio:.4f}, scaled to this "
                                           "run's bytes per iteration") if ratio else
                                          "none: a kernel source changed since the counters were taken",
                        "peak_source": how, "timing": "CUDA events on the launching stream around the phase, inside the timed steps",
                        "gemm": gemm_sub}
        else:
            roofline = {"bound": "hbm", "kernel": "weight GEMM launches (no target decode phase ran, or queued schedule)",
                        "achieved": gemm_gbs, "peak": hbm, "unit": "GB/s", "frac": (gemm_gbs / hbm) if gemm_gbs else None,
                        "traffic": None, "peak_source": how, "gemm": gemm_sub}
        # dense regime: the PRM's scoring pass (one ragged multi-token pass per step)
        prm = shapes[1]
        prm_tokens = (c1["score_tokens"] + c1["ingest_tokens"][1]) - (c0["score_tokens"] + c0["ingest_tokens"][1])
        prm_layer_params = prm.n_params(ri.HEAD_REWARD_SIGMOID) - prm.vocab * prm.d_model
        prm_flops = 2.0 * prm_layer_params * prm_tokens + 4.0 * prm.n_layers * prm.n_heads * prm.head_dim * prm_ctx_sum
        prm_ms = phases["prm_scoring"] * args.steps
        dense = None
        if not merged and prm_ms > 0 and prm_tokens > 0:
            tfs = prm_flops / (prm_ms * 1e-3) / 1e12
            dense = {"bound": "tensor", "kernel": "PRM scoring phase (page reservation, pass list, every layer's GEMMs, chunk "
                     "attention, norms, reward head)", "achieved": tfs, "peak": tf, "unit": "TFLOP/s", "frac": tfs / tf,
                     "flops": "algorithmic: 2 * layer parameters * tokens + 4 * L * H * hd * attended positions (no factor "
                              "for split-precision operands)",
                     "tokens_per_step": prm_tokens / args.steps, "ms_per_step": phases["prm_scoring"],
                     "peak_source": how + " (sustained bf16)"}
            dense["gemm"] = {"what": "the dense weight-GEMM launches (more than 128 rows: scoring, sync and catch-up passes) of "
                                     "the extra, untimed step, CUDA events around single launches; algorithmic flops 2 M N K; "
                                     "'plain' = one 16-bit operand per activation (bf16 for the narrow PRM; fp16 against fp16 "
                                     "weight copies for the models that otherwise use pairs), 'split' = bf16 hi + lo pair (twice "
                                     "the tensor-core work per algorithmic flop: --no-f16-dense, or models too large for copies)"}
            for k, v in gd.items():
                if v["launches"]:
                    g_tfs = v["flops"] / (v["ms"] * 1e-3) / 1e12
                    dense["gemm"][k] = {"TFLOPs": g_tfs, "frac": g_tfs / tf, "timed_launches": v["launches"]}
        out = {"metric": METRIC, "value": timed_tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
               "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
               "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
               "data": "synthetic", "config": workload_config(args),
               "accept_rate": accepted / max(1, live_steps), "delta": delta,
               "e2e": {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(tokens.nbytes + offsets.nbytes) // (args.warmup + args.steps),
                       "d2h_bytes_per_step": B * (cap * 4 + 4 + 4 + 1 + 1) + 3 * 32,
                       "covers": "prefill from host prompts + all warm-up and timed steps"},
               "gpu_launches": int(launches2 - launches1),
               "roofline": roofline, "roofline_dense": dense,
               "phase_ms_per_step": phases,
               "decode_iteration": dec,
               "flops_paper": counters["flops_paper"], "clocks": clocks,
               "gen_tokens": counters["gen_tokens"]}
        if args.sd:
            # speculative decoding of the rejected steps: what the rounds did (random-init draft and target agree on
            # next to no token, so a round writes about one token: the figure shows the mechanism's cost, not its gain)
            d_sd = {k: c1[k] - c0[k] for k in ("sd_rounds", "sd_proposed", "sd_matched", "sd_verified")}
            d_sd["target_tokens"] = c1["gen_tokens"][2] - c0["gen_tokens"][2]
            d_sd["tokens_per_round"] = d_sd["target_tokens"] / max(1, d_sd["sd_rounds"])
            out["speculative_decoding"] = d_sd
        if mega_tables is not None:
            out["mega_profile"] = mega_tables
        if world == 1 and args.queue == 1 and not args.sd and not args.no_alt:
            # the same rows under the queued schedule (rejected rows wait until half the batch does, then one target
            # pass serves them all): every row's sequence of steps is unchanged, the target's weight passes are
            # shared by more rows.  Reported beside the headline, which stays the lock-step rsd_step.
            q_rows = max(2, B // 2)
            calls_w, calls_t = 3, max(1, min(args.steps, n_steps - 4))
            eng.prefill(tokens, offsets)
            for _ in range(calls_w):
                eng.step(delta, q_rows)
            qs, qe = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            qs.record()
            q_tokens = 0
            for _ in range(calls_t):
                q_tokens += int(eng.step(delta, q_rows)["step_len"].sum())
            qe.record()
            torch.cuda.synchronize()
            q_ms = qs.elapsed_time(qe)
            out["other_schedules"] = {f"rsd_step_queued(min_target_rows={q_rows})": {
                "value": q_tokens / (q_ms * 1e-3), "unit": UNIT, "calls": calls_t, "warmup_calls": calls_w,
                "ms_per_call": q_ms / calls_t}}
        if world == 1 and not args.no_cpu_baseline:
            level = 0 if (args.workload == "mini" or (args.workload == "cfg2" and mem_available_gb() > 60)) else 1
            smp = OracleSample(args.workload, level)
            n, dt = smp.run_once(0)
            out["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle",
                                   "sample": smp.desc, "seconds": dt}
        print(json.dumps(out), flush=True)
    eng.close()
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# Kernel sweeps: each point is one JSON line with its fraction of the HBM or bf16 roofline
# ------------------------------------------------------------------------------------------------
def _graph_time_us(fn, variants, iters=20, sampler=None, min_seconds=0.3):
    """Device time per call of fn(v), v cycling over `variants` (distinct buffers, so that repeated calls do not
    hit L2): a CUDA graph of `iters` calls is replayed at least seven times and for at least `min_seconds`, each
    replay timed by its own pair of CUDA events; the result is the MEDIAN replay.  Returns (us per call, detail)
    where detail carries the number of replays, the fastest replay and -- when a ClockSampler is given -- the SM
    clocks and throttle reasons sampled while this point ran."""
    import torch
    torch.cuda.synchronize()          # inputs were filled on the default stream: finish before the side stream reads them
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        for v in variants:
            fn(v)
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            for i in range(iters):
                fn(variants[i % len(variants)])
    torch.cuda.synchronize()
    for _ in range(3):                # warm-up replays
        g.replay()
    torch.cuda.synchronize()
    lo = sampler.mark() if sampler is not None else 0
    times = []
    t0 = time.perf_counter()
    while len(times) < 7 or (time.perf_counter() - t0 < min_seconds and len(times) < 20000):
        batch = []
        for _ in range(7 if not times else 32):
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record(); g.replay(); e.record()
            batch.append((s, e))
        torch.cuda.synchronize()
        times += [a.elapsed_time(b) for a, b in batch]
    detail = {"replays": len(times), "us_min": min(times) * 1e3 / iters, "calls_per_replay": iters}
    if sampler is not None:
        detail["clocks"] = sampler.summary(lo, sampler.mark())
    return float(np.median(times)) * 1e3 / iters, detail


def _sweep_sampler():
    import torch
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    time.sleep(0.5)
    return sampler


def sweep_gemm(args):
    import torch
    from paper_2501_19324_b200 import binding as rb
    hbm, tf, how = peaks()
    if args.only:
        # one point, launched plainly (no graph): the form an ncu capture of the GEMM kernel uses
        vals = [int(v) for v in args.only.split(",")]
        M, K, N = vals[:3]
        if len(vals) > 3 and vals[3] == 16:
            # M,K,N,16: the dense fp16 form (fp16 weights x one fp16 activation operand, rsd_k_gemm impl 4)
            Ws = [(torch.randn(N, K, device="cuda") * 0.02).to(torch.float16) for _ in range(3)]
            x16 = torch.randn(M, K, device="cuda").to(torch.float16)
            for W in Ws + Ws:
                rb.k_gemm(W, x16, impl=4)
            torch.cuda.synchronize()
            print(json.dumps({"sweep": "gemm_f16_dense", "only": [M, K, N], "flops": 2.0 * M * N * K}))
            return
        Ws = [(torch.randn(N, K, device="cuda") * 0.02).to(torch.bfloat16) for _ in range(3)]
        x = torch.randn(M, K, device="cuda")
        hi = x.to(torch.bfloat16)
        lo = (x - hi.float()).to(torch.bfloat16)
        for W in Ws + Ws:
            rb.k_gemm(W, hi, x_lo=lo)
        torch.cuda.synchronize()
        print(json.dumps({"sweep": "gemm", "only": [M, K, N], "algorithmic_bytes": N * K * 2 + 2 * M * K * 2 + M * N * 4}))
        return
    sampler = _sweep_sampler()
    for K, N in ((1536, 8960), (3584, 18944)):
        nbuf = max(2, int(400e6 // (N * K * 2)))
        Ws = [(torch.randn(N, K, device="cuda") * 0.02).to(torch.bfloat16) for _ in range(nbuf)]
        for M in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512):
            x = torch.randn(M, K, device="cuda")
            hi = x.to(torch.bfloat16)
            lo = (x - hi.float()).to(torch.bfloat16)
            y = torch.zeros(M, N, device="cuda")
            nbytes = rb.lib().rsd_k_gemm_scratch_bytes(M, N, K)
            scratch = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")

            def call(W):
                rb._check(rb.lib().rsd_k_gemm(rb._ptr(W), rb._ptr(hi), rb._ptr(lo), rb._ptr(y), M, N, K, 1, 0, 0,
                                              rb._ptr(scratch), nbytes, rb._stream()))
            us, detail = _graph_time_us(call, Ws, sampler=sampler)
            byts = N * K * 2 + 2 * M * K * 2 + M * N * 4
            flops = 2.0 * M * N * K              # the contraction itself; the hi + lo operand rows double the tensor-core work
            print(json.dumps({"sweep": "gemm", "M": M, "K": K, "N": N, "us": us, "GBps": byts / us * 1e-3,
                              "hbm_frac": byts / us * 1e-3 / hbm, "TFLOPs_algorithmic": flops / us * 1e-6,
                              "bf16_frac_algorithmic": flops / us * 1e-6 / tf, "TFLOPs_mma": 2 * flops / us * 1e-6,
                              "peak_source": how, **detail}), flush=True)
        # the dense form of the long passes: fp16 weights x one fp16 activation operand (rsd_k_gemm impl 4)
        W16 = [(torch.randn(N, K, device="cuda") * 0.02).to(torch.float16) for _ in range(nbuf)]
        for M in (256, 512, 1024, 4096, 8192):
            x16 = torch.randn(M, K, device="cuda").to(torch.float16)
            y = torch.zeros(M, N, device="cuda")
            nbytes = rb.lib().rsd_k_gemm_scratch_bytes(M, N, K)
            scratch = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")

            def call16(W):
                rb._check(rb.lib().rsd_k_gemm(rb._ptr(W), rb._ptr(x16), None, rb._ptr(y), M, N, K, 1, 0, 4,
                                              rb._ptr(scratch), nbytes, rb._stream()))
            us, detail = _graph_time_us(call16, W16, sampler=sampler)
            byts = N * K * 2 + M * K * 2 + M * N * 4
            flops = 2.0 * M * N * K
            print(json.dumps({"sweep": "gemm_f16_dense", "M": M, "K": K, "N": N, "us": us, "GBps": byts / us * 1e-3,
                              "hbm_frac": byts / us * 1e-3 / hbm, "TFLOPs_algorithmic": flops / us * 1e-6,
                              "bf16_frac_algorithmic": flops / us * 1e-6 / tf, "TFLOPs_mma": flops / us * 1e-6,
                              "peak_source": how, **detail}), flush=True)
        del W16
    sampler.stop()


def sweep_attn(args):
    import torch
    from paper_2501_19324_b200 import binding as rb
    hbm, _, how = peaks()
    hd = 128
    points = [(H, KV, ctx, B) for (H, KV) in ((12, 2), (28, 4)) for ctx in (512, 1024, 2048, 4096, 8192, 16384)
              for B in (1, 2, 4, 8, 16, 32, 64, 128, 256)]
    only = bool(args.only)
    if only:          # --only batch,ctx,H,KV: a single point with plain launches (the form an ncu capture uses)
        B, ctx, H, KV = (int(v) for v in args.only.split(","))
        points = [(H, KV, ctx, B)]
    sampler = None if only else _sweep_sampler()
    for H, KV, ctx, B in points:
        n_pages = B * (ctx // 16)
        pool_bytes = n_pages * 2 * KV * 16 * hd * 2
        if pool_bytes > 24e9:
            continue
        reps = max(1, min(4, int(300e6 // pool_bytes) + 1))
        pools = [torch.randn(n_pages * 2 * KV * 16 * hd, device="cuda", dtype=torch.float16) for _ in range(reps)]
        table = torch.randperm(n_pages, device="cuda", dtype=torch.int32).view(B, ctx // 16).contiguous()
        q = torch.randn(B, H, hd, device="cuda")
        ctx_len = torch.full((B,), ctx, dtype=torch.int32, device="cuda")
        out = torch.empty_like(q)
        nbytes = rb.lib().rsd_k_attn_decode_scratch_bytes(B, H, hd, ctx)
        scratch = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")

        def call(pool):
            rb._check(rb.lib().rsd_k_attn_decode(rb._ptr(q), rb._ptr(pool), rb._ptr(table), rb._ptr(ctx_len),
                                                 rb._ptr(out), B, H, KV, hd, ctx // 16, 2, rb._ptr(scratch),
                                                 nbytes, rb._stream()))
        if only:
            for i in range(6):
                call(pools[i % len(pools)])
            torch.cuda.synchronize()
            print(json.dumps({"sweep": "attn_decode", "only": [B, ctx, H, KV], "kv_bytes": pool_bytes}))
            return
        us, detail = _graph_time_us(call, pools, iters=10, sampler=sampler)
        print(json.dumps({"sweep": "attn_decode", "H": H, "KV": KV, "ctx": ctx, "batch": B, "us": us,
                          "GBps": pool_bytes / us * 1e-3, "hbm_frac": pool_bytes / us * 1e-3 / hbm,
                          "pages": "randomly permuted", "peak_source": how, **detail}), flush=True)
        del pools
    if sampler is not None:
        sampler.stop()


def sweep_chunk(args):
    """Causal chunk attention (prefill / scoring / catch-up) over a paged prefix: `rows` rows, each with `new` query
    tokens after `prefix` cached positions, fp16 cache, pages randomly permuted.  --only rows,new,prefix,H,KV runs a
    single point with plain launches (the form an ncu capture uses)."""
    import torch
    from paper_2501_19324_b200 import binding as rb
    _, tf, how = peaks()
    hd = 128
    points = [(H, KV, B, new, prefix) for (H, KV) in ((12, 2), (28, 4))
              for (B, new, prefix) in ((32, 128, 256), (32, 128, 1024), (16, 256, 2048), (16, 256, 3072), (8, 512, 0))]
    only = None
    if args.only:
        B, new, prefix, H, KV = (int(v) for v in args.only.split(","))
        points, only = [(H, KV, B, new, prefix)], True
    sampler = None if only else _sweep_sampler()
    for H, KV, B, new, prefix in points:
        ctx = prefix + new
        n_pages_row = (ctx + 15) // 16
        n_pages = B * n_pages_row
        pool = torch.randn(n_pages * 2 * KV * 16 * hd, device="cuda", dtype=torch.float16)
        table = torch.randperm(n_pages, device="cuda", dtype=torch.int32).view(B, n_pages_row).contiguous()
        rows = torch.arange(B, device="cuda", dtype=torch.int32).repeat_interleave(new)
        pos = (torch.arange(new, device="cuda", dtype=torch.int32) + prefix).repeat(B)
        T = B * new
        q = torch.randn(T, H, hd, device="cuda")
        out = torch.zeros_like(q)

        def call(_):
            rb._check(rb.lib().rsd_k_attn_chunk(rb._ptr(q), rb._ptr(pool), rb._ptr(table), rb._ptr(rows), rb._ptr(pos),
                                                rb._ptr(out), T, H, KV, hd, n_pages_row, 2, rb._stream()))
        flops = 4.0 * H * hd * B * (new * prefix + new * (new + 1) // 2)
        kv_bytes = B * ctx * 2 * KV * hd * 2
        if only:
            for _ in range(4):
                call(0)
            torch.cuda.synchronize()
            print(json.dumps({"sweep": "chunk_attn", "only": [B, new, prefix, H, KV], "flops": flops, "kv_bytes": kv_bytes}))
            return
        us, detail = _graph_time_us(call, [0], iters=5, sampler=sampler)
        print(json.dumps({"sweep": "chunk_attn", "H": H, "KV": KV, "rows": B, "new_tokens": new, "prefix": prefix, "us": us,
                          "TFLOPs": flops / us * 1e-6, "bf16_frac": flops / us * 1e-6 / tf, "kv_bytes": kv_bytes,
                          "peak_source": how, **detail}), flush=True)
    if sampler is not None:
        sampler.stop()


def sweep_gate(args):
    import torch
    from paper_2501_19324_b200 import binding as rb
    hbm, _, how = peaks()
    sampler = _sweep_sampler()
    for B in (256, 1 << 20):
        for p in (0.1, 0.3, 0.5, 0.7, 0.9):
            r = torch.rand(B, device="cuda")
            live = torch.ones(B, dtype=torch.uint8, device="cuda")
            acc = torch.empty(B, dtype=torch.uint8, device="cuda")
            rej = torch.empty(B, dtype=torch.int32, device="cuda")
            n = torch.zeros(1, dtype=torch.int32, device="cuda")
            scratch = torch.zeros(4 * ((B + 1023) // 1024) + 16, dtype=torch.uint8, device="cuda")

            def call(_):
                rb._check(rb.lib().rsd_k_gate_compact(rb._ptr(r), rb._ptr(live), float(1 - p), rb._ptr(acc), rb._ptr(rej),
                                                      rb._ptr(n), B, rb._ptr(scratch), scratch.numel(), rb._stream()))
            us, detail = _graph_time_us(call, [0], sampler=sampler)
            byts = B * (4 + 1 + 1) + int(B * (1 - p)) * 4
            print(json.dumps({"sweep": "gate_compact", "rows": B, "accept_p": p, "us": us, "GBps": byts / us * 1e-3,
                              "hbm_frac": byts / us * 1e-3 / hbm, "bound": "latency" if B <= 1024 else "hbm",
                              "peak_source": how, **detail}), flush=True)
    sampler.stop()


def sweep_score(args):
    """PRM scoring of 128-token steps: the 1.5B-shape PRM behind small draft / target models; the time is
    the PRM-scoring phase of one rsd_step."""
    import torch
    from paper_2501_19324_b200 import Engine, Model
    from paper_2501_19324_b200 import lib as rb_lib
    _, tf, how = peaks()
    small_d, small_t = ri.SHAPES["mini_draft"], ri.SHAPES["mini_target"]
    prm = ri.SHAPES[args.prm_shape]
    models = [Model(small_d, ri.gpu_model_tensors(small_d, 0, 0, True, ri.HEAD_LM), ri.HEAD_LM),
              Model(prm, ri.gpu_model_tensors(prm, 1, 0, True, ri.HEAD_REWARD_SIGMOID), ri.HEAD_REWARD_SIGMOID),
              Model(small_t, ri.gpu_model_tensors(small_t, 2, 0, True, ri.HEAD_LM), ri.HEAD_LM)]
    layer_params = prm.n_params(ri.HEAD_REWARD_SIGMOID) - prm.vocab * prm.d_model
    sampler = _sweep_sampler()
    n_rep = 15                                   # at least 7 timed steps, more while they take under half a second
    batches = (1, 2, 4, 8, 16, 32, 64, 128)
    prompt_len = 256
    if args.only:
        # one point, one timed step (the form a launch-list capture of the scoring pass uses): "batch" or "batch,prompt"
        v = [int(x) for x in args.only.split(",")]
        batches, n_rep = (v[0],), 1
        prompt_len = v[1] if len(v) > 1 else 256
    for B in batches:
        eng = Engine(*models, max_batch=B, max_seq_tokens=prompt_len + (n_rep + 2) * 128, max_step_tokens=128, max_steps=n_rep + 2,
                     step_end_id=13, temperature=0.7, seed=0)
        tokens, offsets = ri.prompts(3, B, prompt_len, prompt_len, small_d.vocab)
        eng.prefill(tokens, offsets)
        eng.step(0.0)
        eng.phase_ms(True)
        lo = sampler.mark()
        ms_all, flops_all = [], []
        t_begin = time.perf_counter()
        for i in range(n_rep):
            if i >= min(7, n_rep) and time.perf_counter() - t_begin > 0.5:
                break
            r = eng.step(0.0)
            ms_all.append(eng.phase_ms(True)["prm_scoring"])
            # scored tokens sit at positions z .. z + len - 1 of their rows: contraction flops of the layers plus the
            # attention products (QK^T and PV: 4 * H * hd flops per attended position and layer)
            z0 = prompt_len + (i + 1) * 128
            T = int(r["step_len"].sum())
            ctx_sum = sum(int(n) * z0 + int(n) * (int(n) + 1) // 2 for n in r["step_len"])
            flops_all.append(2.0 * layer_params * T + 4.0 * prm.n_layers * prm.n_heads * prm.head_dim * ctx_sum)
        eng.phase_ms(False)
        k = int(np.argsort(ms_all)[len(ms_all) // 2])
        ms, flops = ms_all[k], flops_all[k]
        print(json.dumps({"sweep": "prm_scoring", "batch": B, "step_tokens": 128, "ms": ms, "ms_min": min(ms_all),
                          "steps_timed": len(ms_all), "TFLOPs_algorithmic": flops / ms * 1e-9,
                          "bf16_frac_algorithmic": flops / ms * 1e-9 / tf,
                          "note": "median step; algorithmic flops = 2 * layer parameters * tokens + attention products",
                          "peak_source": how, "clocks": sampler.summary(lo, sampler.mark()),
                          "library_launches_so_far": int(rb_lib().rsd_debug_launch_count())}), flush=True)
        eng.close()
    sampler.stop()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(WORKLOADS))
    ap.add_argument("--time-stride", type=int, default=16, dest="time_stride")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-alt", action="store_true", dest="no_alt", help="skip the extra measurement of the queued schedule")
    ap.add_argument("--delta", type=float, default=None, help="fixed threshold instead of the 70 %% accept quantile")
    ap.add_argument("--cap", type=int, default=0, help="override the step cap (profiling aid)")
    ap.add_argument("--merged-prm", action="store_true", dest="merged_prm",
                    help="prm_shares_draft: the PRM is a head on the draft's trunk (not the headline configuration)")
    ap.add_argument("--mega", action="store_true",
                    help="decode with the persistent decode kernel instead of kernel by kernel (not the headline path)")
    ap.add_argument("--mega-profile", action="store_true", dest="mega_profile",
                    help="record and print the phase timeline of the persistent decode kernel's last launches")
    ap.add_argument("--chunk", type=int, default=0,
                    help="max_chunk_tokens: tokens per multi-token pass (default: 8192 for cfg2 / cfg3, else the library's 4096)")
    ap.add_argument("--no-f16-dense", action="store_true", dest="no_f16_dense",
                    help="keep bf16 hi + lo operand pairs in the dense passes (no fp16 weight copies)")
    ap.add_argument("--sd", type=int, default=0,
                    help="sd_tokens: rejected steps by speculative decoding with this many proposals per round (0 = off, the headline)")
    ap.add_argument("--queue", type=int, default=1,
                    help="min_target_rows of rsd_step_queued (1 = rsd_step, the headline configuration)")
    ap.add_argument("--kv-extended", type=int, default=None, choices=[0, 1, 2], dest="kv_extended",
                    help="KV cache: 0 by model depth (default: hi+lo pairs beyond 48 layers), 1 fp16 hi+lo pairs, 2 plain fp16")
    ap.add_argument("--only", default="", help="with --sweep gemm: a single M,K,N point, plain launches; with --sweep score: "
                                               "a single batch[,prompt length], one timed step; with --sweep attn: batch,ctx,H,KV; "
                                               "with --sweep chunk: rows,new,prefix,H,KV (plain launches)")
    ap.add_argument("--prm-shape", default="1.5b", dest="prm_shape", choices=["1.5b", "7b"],
                    help="with --sweep score: shape of the PRM")
    ap.add_argument("--sweep", default="", choices=["", "gemm", "attn", "chunk", "gate", "score"],
                    help="kernel sweep on config-2 shapes instead of the step-loop benchmark")
    args = ap.parse_args()
    if args.sweep:
        {"gemm": sweep_gemm, "attn": sweep_attn, "chunk": sweep_chunk, "gate": sweep_gate, "score": sweep_score}[args.sweep](args)
        return
    args.warmup = max(args.warmup, 0)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    run_ours(args, rank, world)


if __name__ == "__main__":
    main()
