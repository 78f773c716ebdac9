"""Each CUDA kernel against the oracle's function for the same operation, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import rsd_inputs as ri
from paper_2501_19324_b200 import binding as rb

pytestmark = pytest.mark.gpu


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def test_input_generators_agree_bit_for_bit():
    sh = ri.SHAPES["tiny_draft"]
    for bf16 in (False, True):
        g = ri.gpu_model_tensors(sh, 1, 3, bf16, ri.HEAD_REWARD_SIGMOID)
        c = ri.cpu_model_weights(sh, 1, 3, bf16, ri.HEAD_REWARD_SIGMOID)
        assert np.array_equal(g["tok_embed"].float().cpu().numpy(), c["tok_embed"])
        assert np.array_equal(g["head"].float().cpu().numpy(), c["head"])
        l = c["layers"][1]
        assert np.array_equal(g["wqkv"][1].float().cpu().numpy(), np.concatenate([l["wq"], l["wk"], l["wv"]]))
        assert np.array_equal(g["wgu"][1].float().cpu().numpy(), np.concatenate([l["wgate"], l["wup"]]))
        assert np.array_equal(g["wo"][1].float().cpu().numpy(), l["wo"])
        assert np.array_equal(g["wdown"][1].float().cpu().numpy(), l["wdown"])
        for k in ("norm1", "norm2"):
            assert np.array_equal(g[k][1].float().cpu().numpy(), l[k]) and np.abs(l[k] - 1).max() > 0.1
        assert np.array_equal(g["final_norm"].float().cpu().numpy(), c["final_norm"])


def philox_numpy(ctr, key):
    """Philox4x32-10 over an array of counters [n, 4] (uint32), written out with numpy integer arithmetic: ten rounds of
    two 32 x 32 -> 64-bit products whose halves are mixed with the other words and the key, the key advancing by the
    two Weyl constants.  A third statement of the algorithm beside the oracle's and the kernel's; the test checks it
    against the oracle before using it on every counter."""
    c = [ctr[:, i].astype(np.uint64) for i in range(4)]
    k0, k1 = np.uint64(key[0]), np.uint64(key[1])
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(0xD2511F53) * c[0]
        p1 = np.uint64(0xCD9E8D57) * c[2]
        c = [(p1 >> np.uint64(32)) ^ c[1] ^ k0, p1 & mask, (p0 >> np.uint64(32)) ^ c[3] ^ k1, p0 & mask]
        k0 = (k0 + np.uint64(0x9E3779B9)) & mask
        k1 = (k1 + np.uint64(0xBB67AE85)) & mask
    return np.stack(c, axis=1).astype(np.uint32)


def test_philox_matches_oracle_on_many_counters():
    """2^20 random counters (plus all-zero and all-one words): every block of the kernel against the numpy
    restatement, which itself is checked against the oracle's C implementation on 512 of them."""
    rng = np.random.default_rng(0)
    n = 1 << 20
    ctr = rng.integers(0, 2 ** 32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0
    ctr[1] = 0xFFFFFFFF
    key = np.array([0x12345678, 0x9ABCDEF0], dtype=np.uint32)
    want = philox_numpy(ctr, key)
    for i in list(range(64)) + list(rng.integers(0, n, size=448)):
        assert np.array_equal(want[i], oracle.philox4x32_10(ctr[i], key))
    got = rb.k_philox(dev(ctr.view(np.int32)), dev(key.view(np.int32))).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want)
    zero = rb.k_philox(dev(np.zeros((1, 4), np.int32)), dev(np.zeros(2, np.int32))).cpu().numpy().view(np.uint32)
    assert [hex(v) for v in zero[0]] == ["0x6627e8d5", "0xe169c58d", "0xbc57ac4c", "0x9b00dbd8"]


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("M,N,K", [(1, 1024, 256), (4, 688 * 2, 256), (7, 256, 688), (33, 1000, 512), (130, 257, 1024)])
def test_gemm_simt(M, N, K, bf16):
    rng = np.random.default_rng(M * 1000 + N)
    W = ri.cpu_tensor(1, 77, N, K, bf16)
    x = rng.normal(size=(M, K)).astype(np.float32)
    dt = torch.bfloat16 if bf16 else torch.float32
    xd = dev(x, dt)
    want = oracle.matmul(W, xd.float().cpu().numpy())
    y0 = rng.normal(size=(M, N)).astype(np.float32)
    got = rb.k_gemm(dev(W, dt), xd, impl=1).cpu().numpy()
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-5 * np.sqrt(K))
    acc = rb.k_gemm(dev(W, dt), xd, y=dev(y0), accumulate=True, impl=1).cpu().numpy()
    np.testing.assert_allclose(acc, want + y0, rtol=0, atol=2e-5 * np.sqrt(K))


@pytest.mark.parametrize("M,N,K", [(16, 128, 64), (5, 256, 512), (17, 1536, 1536), (32, 2048, 1536), (33, 1000, 520),
                                   (64, 1536, 8960), (100, 384, 1408), (128, 640, 768), (129, 256, 2048),
                                   (300, 4096, 512), (1000, 1280, 768), (8, 17920, 1536), (200, 384, 520), (2500, 1024, 192)])
def test_gemm_tcgen05(M, N, K):
    """Tensor-core path: ragged M, N not a multiple of the 128-row tile, K not a multiple of 64,
    split-K with the last-arriver reduction, several x tiles (more than 128 rows with a split operand take the
    persistent kernel: several tiles per CTA, more row tiles than one group of eight), accumulate into y."""
    rng = np.random.default_rng(M * 7 + N)
    W = ri.cpu_tensor(2, 5, N, K, True)
    x = rng.normal(size=(M, K)).astype(np.float32)
    xd = dev(x, torch.bfloat16)
    want = oracle.matmul(W, xd.float().cpu().numpy())
    Wd = dev(W, torch.bfloat16)
    got = rb.k_gemm(Wd, xd, impl=2).cpu().numpy()
    tol = 3e-5 * np.sqrt(K)
    np.testing.assert_allclose(got, want, rtol=0, atol=tol)
    y0 = rng.normal(size=(M, N)).astype(np.float32)
    acc = rb.k_gemm(Wd, xd, y=dev(y0), accumulate=True, impl=2).cpu().numpy()
    np.testing.assert_allclose(acc, want + y0, rtol=0, atol=tol)
    again = rb.k_gemm(Wd, xd, impl=2).cpu().numpy()
    assert np.array_equal(again, got)          # deterministic, whatever order the split CTAs finish in
    # split-precision activations: x = hi + lo, both bf16, both multiplied on the tensor cores
    xf = dev(x)
    hi = xf.to(torch.bfloat16)
    lo = (xf - hi.float()).to(torch.bfloat16)
    want2 = oracle.matmul(W, (hi.float() + lo.float()).cpu().numpy())
    got2 = rb.k_gemm(Wd, hi, impl=2, x_lo=lo).cpu().numpy()
    np.testing.assert_allclose(got2, want2, rtol=0, atol=tol)
    assert np.abs(want2 - oracle.matmul(W, x)).max() < 1e-3 * np.sqrt(K) * 0.02 + 1e-4   # hi + lo ~ x
    got3 = rb.k_gemm(Wd, hi, impl=1, x_lo=lo).cpu().numpy()                    # SIMT path, same operands
    np.testing.assert_allclose(got3, want2, rtol=0, atol=tol)


def test_rmsnorm_rope_swiglu():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5, 1536)).astype(np.float32) * 3
    g = (1 + 0.1 * rng.normal(size=1536)).astype(np.float32)
    got = rb.k_rmsnorm(dev(x), dev(g), 1e-6).cpu().numpy()
    want = np.stack([oracle.rmsnorm(x[i], g, 1e-6) for i in range(5)])
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6 * np.abs(want).max())
    got16 = rb.k_rmsnorm(dev(x), dev(g, torch.bfloat16), 1e-6).float().cpu().numpy()
    g16 = dev(g, torch.bfloat16).float().cpu().numpy()
    want16 = np.stack([oracle.rmsnorm(x[i], g16, 1e-6) for i in range(5)])
    np.testing.assert_allclose(got16, want16, rtol=2 ** -8, atol=0)

    for hd in (64, 128):
        v = rng.normal(size=(6, 3, hd)).astype(np.float32)
        pos = np.array([0, 1, 17, 255, 4095, 16383], dtype=np.int32)
        got = rb.k_rope(dev(v.copy()), dev(pos), 1e4).cpu().numpy()
        want = np.stack([[oracle.rope(v[t, h], pos[t], 1e4) for h in range(3)] for t in range(6)])
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)

    gu = rng.normal(size=(4, 2 * 688)).astype(np.float32) * 2
    got = rb.k_swiglu(dev(gu), torch.float32).cpu().numpy()
    a, b = gu[:, :688].astype(np.float64), gu[:, 688:].astype(np.float64)
    np.testing.assert_allclose(got, a / (1 + np.exp(-a)) * b, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("temperature", [0.0, 0.7])
def test_sampling_matches_oracle(temperature):
    rng = np.random.default_rng(2)
    B, V, v_limit = 6, 5003, 4999
    logits = rng.normal(size=(B, V)).astype(np.float32)
    logits[0, 4] = logits[0, 9] = 50.0            # exact tie: lowest id wins when greedy
    logits[1, v_limit + 1] = 99.0                 # beyond the shared vocabulary: never chosen
    row = np.array([0, 1, 2, 3, -1, 7], dtype=np.int32)
    pos = np.array([5, 5, 9, 1000, 3, 70000], dtype=np.int32)
    got = rb.k_sample(dev(logits), v_limit, temperature, 1234, 2, dev(row), dev(pos)).cpu().numpy()
    for b in range(B):
        if row[b] < 0:
            continue
        want, margin = oracle.sample(logits[b].astype(np.float64), v_limit, temperature, 1234, 2, row[b], pos[b] + 1)
        if margin > 1e-4 or temperature == 0.0:
            assert got[b] == want, (b, got[b], want, margin)
    if temperature == 0.0:
        assert got[0] == 4


def test_gate_compaction_all_masks_and_large():
    """Brute force (a serial loop over the rows) against the ballot / prefix path: EVERY accept mask of 12 rows, one
    call per mask as the step loop calls it, and every mask of 16 rows laid end to end in one call of 2^20 rows."""
    B = 12
    n_masks = 1 << B
    bits = (np.arange(n_masks)[:, None] >> np.arange(B)[None, :]) & 1               # [mask, row]
    r = np.where(bits == 1, np.float32(0.9), np.float32(0.1)).astype(np.float32)
    live = np.tile(np.array([1 if b % 5 else 0 for b in range(B)], dtype=np.uint8), (n_masks, 1))
    r_d, live_d = dev(r), dev(live)
    acc_d = torch.zeros(n_masks, B, dtype=torch.uint8, device="cuda")
    rej_d = torch.full((n_masks, B), -1, dtype=torch.int32, device="cuda")
    n_d = torch.zeros(n_masks, dtype=torch.int32, device="cuda")
    scratch = torch.zeros(64, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for m in range(n_masks):
        rc = rb.lib().rsd_k_gate_compact(r_d.data_ptr() + 4 * B * m, live_d.data_ptr() + B * m, 0.5, acc_d.data_ptr() + B * m,
                                         rej_d.data_ptr() + 4 * B * m, n_d.data_ptr() + 4 * m, B, scratch.data_ptr(), 64, stream)
        assert rc == 0
    acc, rej, n = acc_d.cpu().numpy(), rej_d.cpu().numpy(), n_d.cpu().numpy()
    for m in range(n_masks):
        want_rej = []
        for b in range(B):                                  # the serial definition
            if live[m, b] and not (r[m, b] >= np.float32(0.5)):
                want_rej.append(b)
        assert n[m] == len(want_rej), m
        assert rej[m, :len(want_rej)].tolist() == want_rej, m
        assert acc[m].tolist() == [int(live[m, b] and r[m, b] >= np.float32(0.5)) for b in range(B)], m
    # all 2^16 masks of 16 rows as consecutive segments of one call: the ascending global list, cut at the
    # segment boundaries, is every segment's own ascending list
    B = 16
    n_masks = 1 << B
    bits = (np.arange(n_masks)[:, None] >> np.arange(B)[None, :]) & 1
    r = np.where(bits == 1, np.float32(0.9), np.float32(0.1)).astype(np.float32).reshape(-1)
    live = np.tile(np.array([0 if b in (3, 11) else 1 for b in range(B)], dtype=np.uint8), n_masks)
    acc, rej, n = rb.k_gate_compact(dev(r), dev(live), 0.5)
    acc, rej, n = acc.cpu().numpy(), rej.cpu().numpy(), int(n.item())
    want = []
    for i in range(n_masks * B):
        if live[i] and not (r[i] >= np.float32(0.5)):
            want.append(i)
    assert n == len(want) and np.array_equal(rej[:n], np.array(want, dtype=np.int32))
    assert np.array_equal(acc, ((live == 1) & (r >= np.float32(0.5))).astype(np.uint8))
    seg = rej[:n] // B
    for m in (0, 1, 0x5A5A, 0xFFFF, 0x8001):
        want_rej = [b for b in range(B) if live[m * B + b] and not ((m >> b) & 1)]
        assert (rej[:n][seg == m] - m * B).tolist() == want_rej
    rng = np.random.default_rng(3)
    for B, p in [(1, 0.5), (1023, 0.3), (1024, 0.9), (1025, 0.1), (70001, 0.7), (1 << 20, 0.5)]:
        r = rng.random(B).astype(np.float32)
        live = (rng.random(B) < 0.95).astype(np.uint8)
        delta = np.float32(1 - p)
        acc, rej, n = rb.k_gate_compact(dev(r), dev(live), float(delta))
        want = np.nonzero((live == 1) & ~(r >= delta))[0]
        assert int(n.item()) == len(want)
        assert np.array_equal(rej.cpu().numpy()[:len(want)], want)
        assert np.array_equal(acc.cpu().numpy(), ((live == 1) & (r >= delta)).astype(np.uint8))
    # r == delta accepts; NaN rejects
    r = np.array([0.7, np.nan, np.nextafter(np.float32(0.7), np.float32(0))], dtype=np.float32)
    acc, rej, n = rb.k_gate_compact(dev(r), dev(np.ones(3, np.uint8)), 0.7)
    assert acc.cpu().numpy().tolist() == [1, 0, 0] and rej.cpu().numpy()[:2].tolist() == [1, 2]


def paged_kv(rng, B, KV, hd, ctx, dtype, max_pages, ext=False):
    """Random K/V per row scattered over randomly permuted pages; returns pool, table, dense K, V.
    ext: pages carry two more blocks with the low halves of keys and values (x = fp16 hi + fp16 lo)."""
    n_pages_row = [(c + 15) // 16 for c in ctx]
    total = sum(n_pages_row)
    perm = rng.permutation(total + 5)
    # page = keys [KV][16][hd] followed by values transposed [KV][hd][16]; unused slots hold NaN
    pool = np.full((total + 5, 4 if ext else 2, KV * 16 * hd), np.nan, dtype=np.float32)
    table = np.zeros((B, max_pages), dtype=np.int32)
    Ks, Vs = [], []
    nxt = 0
    for b in range(B):
        K = rng.normal(size=(ctx[b], KV, hd)).astype(np.float32)
        V = rng.normal(size=(ctx[b], KV, hd)).astype(np.float32)
        for i in range(n_pages_row[b]):
            pg = perm[nxt]; nxt += 1
            table[b, i] = pg
            n = min(16, ctx[b] - 16 * i)
            kk = pool[pg, 0].reshape(KV, 16, hd)
            vv = pool[pg, 1].reshape(KV, hd, 16)
            kblk = K[16 * i:16 * i + n].transpose(1, 0, 2)
            if ext:
                khi = kblk.astype(np.float16).astype(np.float32)
                kk[:, :n] = khi
                pool[pg, 2].reshape(KV, 16, hd)[:, :n] = kblk - khi
            else:
                kk[:, :n] = kblk
            vblk = V[16 * i:16 * i + n].transpose(1, 2, 0)
            if ext:
                vhi = vblk.astype(np.float16).astype(np.float32)
                vv[:, :, :n] = vhi
                pool[pg, 3].reshape(KV, hd, 16)[:, :, :n] = vblk - vhi
            else:
                vv[:, :, :n] = vblk
        Ks.append(K); Vs.append(V)
    pool_d = dev(pool, dtype)
    pool_back = pool_d.float().cpu().numpy()
    for b in range(B):       # the oracle sees the values as stored (bf16-rounded when 16-bit)
        for i in range(n_pages_row[b]):
            n = min(16, ctx[b] - 16 * i)
            Ks[b][16 * i:16 * i + n] = pool_back[table[b, i], 0].reshape(KV, 16, hd)[:, :n].transpose(1, 0, 2)
            Vs[b][16 * i:16 * i + n] = pool_back[table[b, i], 1].reshape(KV, hd, 16)[:, :, :n].transpose(2, 0, 1)
            if ext:
                Ks[b][16 * i:16 * i + n] += pool_back[table[b, i], 2].reshape(KV, 16, hd)[:, :n].transpose(1, 0, 2)
                Vs[b][16 * i:16 * i + n] += pool_back[table[b, i], 3].reshape(KV, hd, 16)[:, :, :n].transpose(2, 0, 1)
    return pool_d, dev(table), Ks, Vs


@pytest.mark.parametrize("dtype,hd,H,KV", [(torch.float32, 64, 4, 2), (torch.bfloat16, 128, 12, 2),
                                          (torch.bfloat16, 128, 28, 4), (torch.bfloat16, 128, 8, 1),
                                          (torch.bfloat16, 64, 6, 2), (torch.bfloat16, 128, 16, 1),
                                          (torch.bfloat16, 128, 64, 8), (torch.float16, 128, 12, 2),
                                          (torch.float16, 64, 4, 2), (torch.float16, 128, 28, 4)])
def test_decode_attention_against_definition(dtype, hd, H, KV):
    rng = np.random.default_rng(4)
    ctx = [1, 15, 16, 17, 33, 250, 1031, 2049]
    B = len(ctx)
    max_pages = 130
    # fp32 caches: fp32 arithmetic.  bf16 caches: the query and the softmax weights are rounded to
    # bf16 for the tensor-core products (relative 2^-9 each) on values of order one
    tol = {torch.float32: 2e-5, torch.bfloat16: 1.5e-2, torch.float16: 2e-3}[dtype]
    pool, table, Ks, Vs = paged_kv(rng, B, KV, hd, ctx, dtype, max_pages)
    q = rng.normal(size=(B, H, hd)).astype(np.float32)
    got = rb.k_attn_decode(dev(q), pool, table, dev(np.array(ctx, np.int32)), KV).cpu().numpy()
    for b in range(B):
        for h in range(H):
            g = h // (H // KV)
            s = Ks[b][:, g].astype(np.float64) @ q[b, h].astype(np.float64) / np.sqrt(hd)
            p = np.exp(s - s.max()); p /= p.sum()
            want = p @ Vs[b][:, g].astype(np.float64)
            np.testing.assert_allclose(got[b, h], want, rtol=0, atol=tol)


@pytest.mark.parametrize("dtype,hd,H,KV", [(torch.float16, 128, 12, 2), (torch.float16, 128, 28, 4), (torch.float16, 64, 4, 2),
                                          (torch.float32, 64, 4, 2), (torch.float16, 128, 64, 8), (torch.float16, 128, 8, 4),
                                          (torch.float16, 128, 3, 3), (torch.bfloat16, 128, 12, 2)])
def test_chunk_attention_against_definition(dtype, hd, H, KV):
    """Ragged chunks of several rows in one list: tiles that straddle rows, a chunk that starts in the
    middle of a page, long prefixes, one idle entry; every query against brute-force causal softmax."""
    rng = np.random.default_rng(8)
    ctx = [40, 1, 300, 17, 1031]                # cached positions per row after the chunk was written
    new = [40, 1, 37, 5, 70]                    # the last `new` positions of each row are the chunk
    B = len(ctx)
    max_pages = 70
    pool, table, Ks, Vs = paged_kv(rng, B, KV, hd, ctx, dtype, max_pages)
    rows, poss = [], []
    for b in range(B):
        for p in range(ctx[b] - new[b], ctx[b]):
            rows.append(b); poss.append(p)
    rows.insert(45, -1); poss.insert(45, 0)     # an idle entry in the middle of the list
    T = len(rows)
    q = rng.normal(size=(T, H, hd)).astype(np.float32)
    got = rb.k_attn_chunk(dev(q), pool, table, dev(np.array(rows, np.int32)), dev(np.array(poss, np.int32)), KV).cpu().numpy()
    tol = {torch.float32: 2e-5, torch.float16: 2e-3, torch.bfloat16: 1.5e-2}[dtype]
    for t in range(T):
        b, p = rows[t], poss[t]
        if b < 0:
            continue
        for h in range(0, H, max(1, H // 6)):
            g = h // (H // KV)
            s = Ks[b][:p + 1, g].astype(np.float64) @ q[t, h].astype(np.float64) / np.sqrt(hd)
            w = np.exp(s - s.max()); w /= w.sum()
            want = w @ Vs[b][:p + 1, g].astype(np.float64)
            np.testing.assert_allclose(got[t, h], want, rtol=0, atol=tol)


@pytest.mark.parametrize("H,KV", [(28, 4), (12, 2)])
def test_chunk_attention_long_prefix(H, KV):
    """Prefixes of more than a hundred pages (the page ids of a row are fetched in batches of 32, several batches a
    pass), a chunk that ends in the middle of a page, two rows in one tile; fp16 cache, head_dim 128."""
    rng = np.random.default_rng(21)
    hd = 128
    ctx = [2603, 531]
    new = [90, 70]
    B = len(ctx)
    max_pages = 170
    pool, table, Ks, Vs = paged_kv(rng, B, KV, hd, ctx, torch.float16, max_pages)
    rows, poss = [], []
    for b in range(B):
        for p in range(ctx[b] - new[b], ctx[b]):
            rows.append(b); poss.append(p)
    T = len(rows)
    q = rng.normal(size=(T, H, hd)).astype(np.float32)
    got = rb.k_attn_chunk(dev(q), pool, table, dev(np.array(rows, np.int32)), dev(np.array(poss, np.int32)), KV).cpu().numpy()
    assert np.isfinite(got).all()
    for t in range(0, T, 3):
        b, p = rows[t], poss[t]
        for h in range(0, H, max(1, H // 5)):
            g = h // (H // KV)
            s = Ks[b][:p + 1, g].astype(np.float64) @ q[t, h].astype(np.float64) / np.sqrt(hd)
            w = np.exp(s - s.max()); w /= w.sum()
            want = w @ Vs[b][:p + 1, g].astype(np.float64)
            np.testing.assert_allclose(got[t, h], want, rtol=0, atol=2e-3)


@pytest.mark.parametrize("hd,H,KV", [(128, 12, 2), (128, 64, 8), (64, 4, 2), (128, 16, 1)])
def test_extended_precision_attention(hd, H, KV):
    """fp16 cache with keys and values kept as hi + lo pairs, queries and softmax weights as hi + lo
    pairs: decode and chunk kernels alike agree with the fp64 definition to fp32 accuracy."""
    rng = np.random.default_rng(12)
    ctx = [1, 16, 33, 250, 1031]
    B = len(ctx)
    pool, table, Ks, Vs = paged_kv(rng, B, KV, hd, ctx, torch.float16, 70, ext=True)
    q = rng.normal(size=(B, H, hd)).astype(np.float32)
    got = rb.k_attn_decode(dev(q), pool, table, dev(np.array(ctx, np.int32)), KV, ext=True).cpu().numpy()
    rows = [b for b in range(B) for _ in range(min(ctx[b], 20))]
    poss = [p for b in range(B) for p in range(ctx[b] - min(ctx[b], 20), ctx[b])]
    qc = rng.normal(size=(len(rows), H, hd)).astype(np.float32)
    gotc = rb.k_attn_chunk(dev(qc), pool, table, dev(np.array(rows, np.int32)), dev(np.array(poss, np.int32)), KV, ext=True).cpu().numpy()

    def ref(b, p, qv, h):
        g = h // (H // KV)
        s = Ks[b][:p + 1, g].astype(np.float64) @ qv.astype(np.float64) / np.sqrt(hd)
        w = np.exp(s - s.max()); w /= w.sum()
        return w @ Vs[b][:p + 1, g].astype(np.float64)
    for b in range(B):
        for h in range(0, H, max(1, H // 4)):
            np.testing.assert_allclose(got[b, h], ref(b, ctx[b] - 1, q[b, h], h), rtol=0, atol=2e-5)
    for t in range(0, len(rows), 3):
        for h in range(0, H, max(1, H // 4)):
            np.testing.assert_allclose(gotc[t, h], ref(rows[t], poss[t], qc[t, h], h), rtol=0, atol=2e-5)


@pytest.mark.parametrize("M,N,K", [(129, 256, 64), (300, 1000, 520), (512, 1536, 1536), (2100, 640, 128), (4096, 2048, 1536)])
def test_dense_gemm_on_fp16_operands(M, N, K):
    """The dense form of the long passes (rsd_k_gemm impl 4): fp16 weights x one fp16 activation operand, more than
    128 rows, with and without adding into y; against the exact product of the fp16 values in fp64."""
    rng = np.random.default_rng(31)
    W = (rng.normal(size=(N, K)) * 0.05).astype(np.float16)
    x = rng.normal(size=(M, K)).astype(np.float16)
    want = x.astype(np.float64) @ W.astype(np.float64).T
    Wd, xd = torch.from_numpy(W).cuda(), torch.from_numpy(x).cuda()
    got = rb.k_gemm(Wd, xd, impl=4).cpu().numpy()
    tol = 2e-5 * np.sqrt(K) + 1e-6                      # fp32 accumulation of K products of order 0.05
    np.testing.assert_allclose(got, want, rtol=0, atol=tol)
    y0 = rng.normal(size=(M, N)).astype(np.float32)
    got2 = rb.k_gemm(Wd, xd, y=torch.from_numpy(y0.copy()).cuda(), accumulate=True, impl=4).cpu().numpy()
    np.testing.assert_allclose(got2, want + y0, rtol=0, atol=tol + 1e-6)
    with pytest.raises(rb.RsdError):
        rb.k_gemm(Wd, xd[:128].contiguous(), impl=4)    # the form is for more than 128 rows


@pytest.mark.parametrize("M,F,K", [(1, 64, 64), (5, 192, 512), (32, 1408, 512), (33, 128, 520), (70, 2048, 768),
                                   (129, 704, 1408), (300, 320, 256), (32, 8960, 1536), (200, 128, 520), (2100, 640, 128)])
def test_gate_up_gemm_with_swiglu_epilogue(M, F, K):
    """Gate/up projection with SwiGLU inside the GEMM epilogue (tile = 64 gate rows + the 64 matching up rows):
    against matmul + silu(g) * u written out in fp64.  Ragged M (all three tile heights and several x tiles), F of
    one to many tiles, K not a multiple of 64; the hi + lo output pair must carry the result to ~16 bits."""
    rng = np.random.default_rng(M * 13 + F)
    W = ri.cpu_tensor(3, 7, 2 * F, K, True) * 8.0          # pre-activations of order one, so silu is exercised
    W = dev(W, torch.bfloat16).float().cpu().numpy()
    x = rng.normal(size=(M, K)).astype(np.float32)
    xf = dev(x)
    hi = xf.to(torch.bfloat16)
    lo = (xf - hi.float()).to(torch.bfloat16)
    gu = oracle.matmul(W, (hi.float() + lo.float()).cpu().numpy()).astype(np.float64)
    g, u = gu[:, :F], gu[:, F:]
    want = g / (1.0 + np.exp(-g)) * u
    a_hi, a_lo = rb.k_gemm_gu(dev(W, torch.bfloat16), hi, lo)
    got = a_hi.float().cpu().numpy().astype(np.float64) + a_lo.float().cpu().numpy()
    scale = max(1.0, float(np.abs(want).max()))
    np.testing.assert_allclose(got, want, rtol=0, atol=(3e-5 * np.sqrt(K) + 2e-5) * scale)
    assert np.array_equal(a_hi.float().cpu().numpy(), torch.from_numpy(got.astype(np.float32)).to(torch.bfloat16).float().numpy()) or \
        np.abs(a_hi.float().cpu().numpy() - got).max() <= 2 ** -8 * scale
    again_hi, again_lo = rb.k_gemm_gu(dev(W, torch.bfloat16), hi, lo)
    assert torch.equal(again_hi, a_hi) and torch.equal(again_lo, a_lo)


def test_bounded_wait_runs_out_and_the_kernel_leaves_cleanly():
    """RSD_ERR_TIMEOUT without a fault: one CTA of the tensor-core GEMM whose copies are never issued.  Its wait
    (a few thousand polls in this mode) expires, the error flag is raised and reported, tensor memory is freed: the
    very next GEMMs on the same scratch are correct, many times over (a leaked allocation would stall them)."""
    rng = np.random.default_rng(5)
    W = dev(rng.normal(size=(128, 64)).astype(np.float32), torch.bfloat16)
    x = dev(rng.normal(size=(16, 64)).astype(np.float32), torch.bfloat16)
    y = torch.full((16, 128), 7.0, dtype=torch.float32, device="cuda")
    nbytes = rb.lib().rsd_k_gemm_scratch_bytes(16, 128, 64)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(3):
        rc = rb.lib().rsd_debug_gemm_wait_probe(W.data_ptr(), x.data_ptr(), y.data_ptr(), scratch.data_ptr(), nbytes, stream)
        assert rc == -5
        assert b"bounded wait" in rb.lib().rsd_last_error(None)
        assert int(scratch[4096:4100].view(torch.int32).item()) == 0           # cleared for the next use
        assert torch.all(y == 7.0)                                             # nothing was computed or written
    want = oracle.matmul(W.float().cpu().numpy(), x.float().cpu().numpy())
    for _ in range(40):                                  # 40 x 32 columns: more than the 512 a leak of 3 x 32 would leave
        got = torch.zeros(16, 128, dtype=torch.float32, device="cuda")
        assert rb.lib().rsd_k_gemm(W.data_ptr(), x.data_ptr(), None, got.data_ptr(), 16, 128, 64, 1, 0, 2, scratch.data_ptr(),
                                   nbytes, stream) == 0
        np.testing.assert_allclose(got.cpu().numpy(), want, rtol=0, atol=3e-4)
