"""The N > 1 path of bench.py on CPU: two gloo ranks run the replica bookkeeping (own prompts per
rank, slowest rank's time, summed tokens) and the reference arm stays silent on ranks other than 0."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [100.0, 140.0][rank]
    res = bench.combine_ranks(ms, ms + 50.0, 1000 + rank, 3000 + 10 * rank, world, "cpu")
    tok, off = bench.rank_prompts(rank, 4, 8, 16, 1024)
    gathered = [None] * world
    dist.all_gather_object(gathered, (res, tok.tolist(), off.tolist()))
    if rank == 0:
        out.put(gathered)
    dist.destroy_process_group()


def test_two_replicas_combine_and_use_own_prompts():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (res0, tok0, off0), (res1, tok1, off1) = gathered
    assert res0 == res1 == (140.0, 190.0, 2001.0, 6010.0)      # max of the times, sum of the tokens
    assert tok0 != tok1                                         # replicas do not share prompts
    import bench
    assert bench.combine_ranks(5.0, 6.0, 7, 8, 1, "cpu") == (5.0, 6.0, 7.0, 8.0)


def test_reference_arm_only_rank_zero_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mini",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mini",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2


def test_decode_iteration_roofline_arithmetic():
    """bench.py's whole-iteration roofline: weight bytes of the model (embedding table excluded) over the measured
    time of one decode iteration, by hand for the 1.5B shape."""
    sys.path.insert(0, ROOT)
    import bench
    import rsd_inputs as ri
    shapes = [ri.SHAPES["1.5b"], ri.SHAPES["1.5b"], ri.SHAPES["7b"]]
    phases = {"draft_decode": 256.0, "target_decode": 448.0}          # ms per step
    kv = {"draft": 3 * 128 * 1.0e9, "target": 0.0}                    # KV bytes read over all iterations of the phase
    r = bench.decode_iteration_roofline(phases, {"draft": 3 * 128, "target": 2 * 128}, kv, 3, shapes, 6538.0, 1)
    # 28 layers x 46,792,704 matrix parameters + norm gains + lm head of 151936 x 1536, two bytes each
    want_bytes = 2.0 * (28 * (46_792_704 + 2 * 1536) + 1536 + 151936 * 1536)
    assert abs(r["draft"]["weight_gb"] * 1e9 - want_bytes) < 1.0
    assert abs(r["draft"]["ms"] - 2.0) < 1e-12 and abs(r["target"]["ms"] - 5.25) < 1e-12
    # an iteration's bytes: the weights once plus its share of the KV reads (1 GB per draft iteration here)
    assert abs(r["draft"]["kv_gb"] - 1.0) < 1e-12 and r["target"]["kv_gb"] == 0.0
    assert abs(r["draft"]["frac_of_hbm"] - (want_bytes + 1.0e9) / 2.0e-3 / 1e9 / 6538.0) < 1e-9
    assert abs(r["draft"]["frac_of_hbm_weights_only"] - want_bytes / 2.0e-3 / 1e9 / 6538.0) < 1e-9
    none = {"draft": 0.0, "target": 0.0}
    assert bench.decode_iteration_roofline(phases, {"draft": 1, "target": 0}, none, 3, shapes, 6538.0, 1)["target"] is None
    assert bench.decode_iteration_roofline(phases, {"draft": 1, "target": 1}, none, 3, shapes, 6538.0, 8) is None
    # rounds of speculative decoding are not decode iterations: no target figure in that mode
    assert bench.decode_iteration_roofline(phases, {"draft": 1, "target": 1}, none, 3, shapes, 6538.0, 1, sd=4)["target"] is None
