"""The allocation-free gate + compaction entry point, for hosts of the library that cannot call
cudaMalloc (memory handed out once at start-up, a fixed per-tenant budget, or a section where an
allocation may not stall the device): it must give exactly what rsd_k_gate_compact gives, on two
calls in a row that share the library's built-in scratch, and must refuse batches the scratch
cannot cover.  Collected last on purpose, so a run that stops at the first failure has already run
every other test; it passes alone in a fresh process as well."""
import numpy as np
import pytest
import torch

from paper_2501_19324_b200 import binding as rb

pytestmark = pytest.mark.gpu


def run_both(B, p_reject, seed):
    rng = np.random.default_rng(seed)
    rewards = torch.from_numpy(rng.random(B).astype(np.float32)).cuda()
    live = torch.from_numpy((rng.random(B) < 0.9).astype(np.uint8)).cuda()
    delta = float(np.float32(p_reject))
    want_acc, want_rej, want_n = rb.k_gate_compact(rewards, live, delta)
    # every buffer of the allocation-free call exists before it is made
    acc = torch.full((B,), 7, dtype=torch.uint8, device="cuda")
    rej = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    n = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    rc = rb.k_gate_compact_static(rewards, live, delta, acc, rej, n)
    torch.cuda.synchronize()
    assert rc == 0, rb.lib().rsd_k_gate_compact_static_error()
    assert torch.cuda.memory_allocated() == before
    k = int(want_n.item())
    assert int(n.item()) == k                                   # integer work: bit-exact
    assert torch.equal(rej[:k], want_rej[:k])
    assert torch.equal(acc, want_acc)
    return k


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    # a large batch first, then a smaller one that reuses (and does not clear) the same scratch
    k1 = run_both(300_001, 0.6, seed=1)
    k2 = run_both(4_100, 0.2, seed=2)
    k3 = run_both(1 << 20, 0.5, seed=3)
    assert k1 > 0 and k2 > 0 and k3 > 0


def test_static_scratch_rejects_oversized_batches():
    B = (1 << 20) + 1
    rewards = torch.zeros(B, dtype=torch.float32, device="cuda")
    live = torch.ones(B, dtype=torch.uint8, device="cuda")
    acc = torch.zeros(B, dtype=torch.uint8, device="cuda")
    rej = torch.zeros(B, dtype=torch.int32, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert rb.k_gate_compact_static(rewards, live, 0.5, acc, rej, n) == -1
    msg = rb.lib().rsd_k_gate_compact_static_error().decode()
    assert "1048577" in msg and "1048576" in msg
