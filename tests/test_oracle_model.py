"""Pins for the oracle's transformer, heads, random numbers, sampling and acceptance rule.

Each test checks the oracle against something that is not the oracle: a third-party Llama
implementation, library routines (attention, RMSNorm, SiLU, bfloat16), closed forms, invariants,
published known-answer vectors, or statistics with a known law.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import rsd_inputs as ri
from oracle import OracleModel

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def small_weights(shape, slot, seed, head_kind=ri.HEAD_LM, sigma_boost=5.0):
    w = ri.cpu_model_weights(shape, slot, seed, False, head_kind)
    # larger weights make attention and the MLP far from linear, so mistakes show
    for lw in w["layers"]:
        for k in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown"):
            lw[k] = lw[k] * sigma_boost
        lw["norm1"] = (1.0 + 0.1 * np.arange(shape.d_model) / shape.d_model).astype(np.float32)
        lw["norm2"] = (0.8 + 0.3 * np.arange(shape.d_model)[::-1] / shape.d_model).astype(np.float32)
    w["final_norm"] = (1.0 + 0.05 * np.sin(np.arange(shape.d_model))).astype(np.float32)
    w["tok_embed"] = w["tok_embed"] * 50.0
    return w


def hf_model(shape, w):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
                      num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
                      num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, max_position_embeddings=512, attn_implementation="eager")
    m = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": w["tok_embed"], "model.norm.weight": w["final_norm"],
          "lm_head.weight": w["head"]}
    names = dict(wq="self_attn.q_proj", wk="self_attn.k_proj", wv="self_attn.v_proj", wo="self_attn.o_proj",
                 wgate="mlp.gate_proj", wup="mlp.up_proj", wdown="mlp.down_proj",
                 norm1="input_layernorm", norm2="post_attention_layernorm")
    for l, lw in enumerate(w["layers"]):
        for k, n in names.items():
            sd[f"model.layers.{l}.{n}.weight"] = lw[k]
    missing = m.load_state_dict({k: torch.from_numpy(np.asarray(v, np.float64)) for k, v in sd.items()},
                                strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return m


@pytest.mark.parametrize("heads,kv", [(4, 2), (4, 4), (6, 1)])
def test_forward_matches_third_party_llama(heads, kv):
    """Whole forward (RMSNorm, RoPE pairing, GQA head mapping, causal softmax, SwiGLU, lm_head)."""
    shape = ri.ModelShape(2, heads * 16, heads, kv, 16, 172, 97)
    w = small_weights(shape, 0, 5)
    tokens = np.random.default_rng(0).integers(0, 97, size=23)
    om = OracleModel(w, 0)
    h = om.forward_full(tokens)
    got = np.stack([om.logits(h[t]) for t in range(len(tokens))])
    with torch.no_grad():
        want = hf_model(shape, w)(torch.from_numpy(tokens)[None]).logits[0].numpy()
    assert np.abs(want).max() > 0.5
    # the library builds its rotary cos/sin tables in fp32, which bounds the agreement near 1e-7
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)


def test_kv_cache_decode_equals_full_recompute(tiny_weights):
    d, _, _ = tiny_weights
    om = OracleModel(d, 0)
    tokens = np.random.default_rng(1).integers(0, 1024, size=40)
    full = om.forward_full(tokens)
    cache = om.new_cache(64)
    part = [om.forward(cache, tokens[:17], 0)]
    part.append(om.forward(cache, tokens[17:18], 17))
    part.append(om.forward(cache, tokens[18:33], 18))
    for p in range(33, 40):
        part.append(om.forward(cache, tokens[p:p + 1], p))
    got = np.concatenate(part)
    np.testing.assert_allclose(got, full, rtol=1e-10, atol=1e-12)
    # overwriting positions after a rollback leaves no trace of the dropped tokens
    other = tokens.copy()
    other[30:] = (other[30:] + 1) % 1024
    om.forward(cache, other[30:], 30)
    redo = om.forward(cache, tokens[30:], 30)
    np.testing.assert_allclose(redo, full[30:], rtol=1e-10, atol=1e-12)


def test_attention_against_library_softmax_attention():
    """One layer with wo = I and a zero MLP: x_out - x is the attention output, checked against
    torch's scaled_dot_product_attention on q, k, v rotated with explicit complex arithmetic."""
    H, KV, hd, T = 4, 2, 8, 11
    d = H * hd
    shape = ri.ModelShape(1, d, H, KV, hd, 16, 50)
    rng = np.random.default_rng(2)
    w = small_weights(shape, 0, 9)
    lw = w["layers"][0]
    lw["wo"] = np.eye(d, dtype=np.float32)
    lw["wdown"] = np.zeros_like(lw["wdown"])
    lw["norm1"] = np.ones(d, np.float32)
    om = OracleModel(w, 0)
    tokens = rng.integers(0, 50, size=T)
    x0 = om.embed(tokens)
    x1 = om.forward_full(tokens)
    att = x1 - x0

    xin = torch.from_numpy(x0)
    hn = torch.nn.functional.rms_norm(xin, (d,), eps=shape.rms_eps)
    q = (hn @ torch.from_numpy(lw["wq"]).double().T).view(T, H, hd)
    k = (hn @ torch.from_numpy(lw["wk"]).double().T).view(T, KV, hd)
    v = (hn @ torch.from_numpy(lw["wv"]).double().T).view(T, KV, hd)

    def rot(t):  # pair (i, i+hd/2) as the complex number a + ib, times exp(i * pos * theta^(-2i/hd))
        half = hd // 2
        z = torch.complex(t[..., :half], t[..., half:])
        freqs = shape.rope_theta ** (-2.0 * torch.arange(half, dtype=torch.float64) / hd)
        ang = torch.arange(T, dtype=torch.float64)[:, None] * freqs[None]
        z = z * torch.polar(torch.ones_like(ang), ang)[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    q, k = rot(q), rot(k)
    k = k.repeat_interleave(H // KV, dim=1)
    v = v.repeat_interleave(H // KV, dim=1)
    want = torch.nn.functional.scaled_dot_product_attention(
        q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None], is_causal=True)[0]
    want = want.transpose(0, 1).reshape(T, d).numpy()
    np.testing.assert_allclose(att, want, rtol=0, atol=1e-10)


def test_rope_depends_on_relative_position_only():
    rng = np.random.default_rng(3)
    q, k = rng.normal(size=64), rng.normal(size=64)
    ref = oracle.rope(q, 5, 1e4) @ oracle.rope(k, 2, 1e4)
    for m, n in [(3, 0), (103, 100), (4098, 4095)]:
        assert abs(oracle.rope(q, m, 1e4) @ oracle.rope(k, n, 1e4) - ref) < 1e-9
    assert np.allclose(oracle.rope(q, 0, 1e4), q)
    assert abs(np.linalg.norm(oracle.rope(q, 77, 1e4)) - np.linalg.norm(q)) < 1e-12
    # first pair turns by exactly `pos` radians, the last by pos * theta^(-(hd-2)/hd)
    e = np.zeros(64); e[0] = 1.0
    r = oracle.rope(e, 3, 1e4)
    assert abs(r[0] - math.cos(3.0)) < 1e-12 and abs(r[32] - math.sin(3.0)) < 1e-12
    e = np.zeros(64); e[31] = 1.0
    r = oracle.rope(e, 3, 1e4)
    ang = 3.0 * 1e4 ** (-62.0 / 64.0)
    assert abs(r[31] - math.cos(ang)) < 1e-12 and abs(r[63] - math.sin(ang)) < 1e-12


def test_rmsnorm_library_and_scale_invariance():
    rng = np.random.default_rng(4)
    x, g = rng.normal(size=(3, 96)), rng.normal(size=96).astype(np.float32)
    got = np.stack([oracle.rmsnorm(x[i], g, 1e-6) for i in range(3)])
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (96,), torch.from_numpy(g).double(), 1e-6).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=0)
    np.testing.assert_allclose(oracle.rmsnorm(1000.0 * x[0], g, 1e-12), oracle.rmsnorm(x[0], g, 1e-12), rtol=1e-9)


def test_matmul_orientation():
    rng = np.random.default_rng(5)
    W, X = rng.normal(size=(7, 13)).astype(np.float32), rng.normal(size=(4, 13))
    np.testing.assert_allclose(oracle.matmul(W, X), X @ W.astype(np.float64).T, rtol=1e-12)


def test_reward_range_and_zero_head(tiny_weights):
    _, p, _ = tiny_weights
    om = OracleModel(p, 1)
    tokens = np.random.default_rng(6).integers(0, 1024, size=20)
    h = om.forward_full(tokens)
    r = np.array([om.reward(h[t]) for t in range(20)])
    assert np.all(r >= 0.0) and np.all(r <= 1.0) and r.std() > 0
    # definition: sigmoid of the head's dot product with the final-normed hidden state
    hn = oracle.rmsnorm(h[7], p["final_norm"], p["shape"].rms_eps)
    assert abs(r[7] - 1.0 / (1.0 + math.exp(-float(p["head"][0].astype(np.float64) @ hn)))) < 1e-12
    zero = dict(p); zero["head"] = np.zeros_like(p["head"])
    assert OracleModel(zero, 1).reward(h[3]) == 0.5
    raw = dict(p); raw["head_kind"] = ri.HEAD_REWARD_RAW
    assert abs(OracleModel(raw, 1).reward(h[7]) - float(p["head"][0].astype(np.float64) @ hn)) < 1e-12


def test_philox_known_answers_and_uniform_range():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert list(oracle.philox4x32_10(w[0:4], w[4:6])) == w[6:10]
    # the oracle's and the input generator's implementations were written separately
    rng = np.random.default_rng(7)
    for _ in range(200):
        c, k = rng.integers(0, 2 ** 32, size=4, dtype=np.uint64), rng.integers(0, 2 ** 32, size=2, dtype=np.uint64)
        assert np.array_equal(oracle.philox4x32_10(c, k), ri.philox4x32_10(c, k))
    lib = oracle.lib()
    assert lib.orc_uniform_from_bits(0) == 0.5 / 2 ** 23
    assert lib.orc_uniform_from_bits(0xFFFFFFFF) == 1.0 - 0.5 / 2 ** 23
    # counter layout: word index%4 of block (index/4, position, row, stream), key = seed halves
    seed = (0xABCDEF01 << 32) | 0x12345678
    blk = oracle.philox4x32_10([9 // 4, 40, 3, 2], [0x12345678, 0xABCDEF01])
    assert oracle.uniform(seed, 2, 3, 40, 9) == lib.orc_uniform_from_bits(int(blk[1]))


def test_greedy_is_argmax_lowest_id_on_ties():
    logits = np.array([0.1, 2.0, -1.0, 2.0, 1.5])
    tok, margin = oracle.sample(logits, 5, 0.0, 0, 0, 0, 0)
    assert tok == 1 and margin == 0.0
    tok, margin = oracle.sample(logits, 3, 0.0, 0, 0, 0, 0)       # ids >= v_limit are not candidates
    assert tok == 1 and abs(margin - 1.9) < 1e-12


def test_gumbel_max_draws_from_softmax():
    logits = np.array([0.3, -0.7, 1.1, 0.0, 0.5, -1.5, 0.9, 0.2])
    T = 0.7
    p = np.exp(logits / T); p /= p.sum()
    n = 20000
    counts = np.zeros(8)
    for i in range(n):
        tok, _ = oracle.sample(logits, 8, T, 1234, 0, i % 64, i // 64)
        counts[tok] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 24.3       # chi-square, 7 degrees of freedom, p = 0.001
    # as T -> 0+ the draw is the argmax wherever the margin is clear
    for i in range(50):
        assert oracle.sample(logits, 8, 1e-3, 99, 0, i, 5)[0] == 2
    # noise is a function of (seed, model, row, position) only
    a = [oracle.sample(logits, 8, T, 5, 1, 2, pos)[0] for pos in range(40)]
    b = [oracle.sample(logits, 8, T, 5, 1, 2, pos)[0] for pos in range(40)]
    c = [oracle.sample(logits, 8, T, 5, 2, 2, pos)[0] for pos in range(40)]
    assert a == b and a != c


def test_weighting_functions_table():
    # Table 1: constant, binary step, clip, r/(1+r) floored at 0, logistic
    assert oracle.omega(0, 0.123, 0.4) == 0.4
    assert oracle.omega(1, 0.7, 0.7) == 1.0 and oracle.omega(1, 0.6999, 0.7) == 0.0
    assert oracle.omega(2, -0.5) == 0.0 and oracle.omega(2, 0.25) == 0.25 and oracle.omega(2, 1.5) == 1.0
    assert oracle.omega(3, 1.0) == 0.5 and oracle.omega(3, -0.5) == 0.0 and oracle.omega(3, 3.0) == 0.75
    assert oracle.omega(4, 0.7, 0.7, 10.0) == 0.5
    assert abs(oracle.omega(4, 0.9, 0.7, 10.0) - 1.0 / (1.0 + math.exp(-2.0))) < 1e-15
    for kind, a, b in [(1, 0.5, 0), (2, 0, 0), (3, 0, 0), (4, 0.5, 8.0)]:
        vals = [oracle.omega(kind, r, a, b) for r in np.linspace(0, 1, 101)]
        assert all(x <= y for x, y in zip(vals, vals[1:]))          # non-decreasing (Prop. 2.2 premise)
        assert all(0.0 <= v <= 1.0 for v in vals)


def test_acceptance_criterion():
    # Algorithm 2: omega in {0,1} decides alone; otherwise accept iff omega >= u
    assert oracle.accept(1, 0.8, 0.7, 0, u=0.999999) == 1
    assert oracle.accept(1, 0.6, 0.7, 0, u=1e-9) == 0
    assert oracle.accept(1, float("nan"), 0.7, 0, u=0.5) == 0
    assert oracle.accept(2, 0.3, 0, 0, u=0.29) == 1 and oracle.accept(2, 0.3, 0, 0, u=0.31) == 0
    assert oracle.accept(2, 1.0, 0, 0, u=0.9999) == 1 and oracle.accept(2, 0.0, 0, 0, u=1e-9) == 0
    n = 4000
    acc = sum(oracle.accept(0, 0.0, 0.35, 0, u=oracle.uniform(1, 3, i, 0, 0)) for i in range(n))
    assert abs(acc / n - 0.35) < 4 * math.sqrt(0.35 * 0.65 / n)
