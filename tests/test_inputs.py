"""The seeded input generators: Philox known answers, value recipe, bfloat16 rounding, prompts."""
import os

import numpy as np
import torch

import rsd_inputs as ri

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def kat_vectors():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out.append((w[0:4], w[4:6], w[6:10]))
    return out


def test_philox_known_answers():
    vecs = kat_vectors()
    assert len(vecs) == 3
    for ctr, key, want in vecs:
        assert list(ri.philox4x32_10(ctr, key)) == want


def test_weight_recipe_matches_definition():
    # value = (2 * sum of eight 16-bit fields - 8 * 65535) * scale, from the Philox block of the index
    seed, tid = 7, ri.tensor_id(2, 3, ri.KIND_WO)
    w = ri.cpu_tensor(seed, tid, 3, 5, bf16=False)
    for idx in range(15):
        o = ri.philox4x32_10([idx, 0, 0, 0x57454947], [seed, tid])
        s = sum(int(x) & 0xFFFF for x in o) + sum(int(x) >> 16 for x in o)
        want = np.float32(2 * s - 8 * 65535) * np.float32(ri.WEIGHT_SCALE)
        assert w.reshape(-1)[idx] == want


def test_weight_statistics_and_tensor_separation():
    a = ri.cpu_tensor(0, ri.tensor_id(0, 0, ri.KIND_WQ), 512, 512, False)
    b = ri.cpu_tensor(0, ri.tensor_id(1, 0, ri.KIND_WQ), 512, 512, False)
    assert abs(a.mean()) < 2e-4 and abs(a.std() - 0.02) < 2e-4
    assert abs(np.corrcoef(a.ravel(), b.ravel())[0, 1]) < 0.01      # draft and PRM trunks differ
    # the logical index does not depend on how rows are batched into calls
    part = ri.cpu_tensor(0, ri.tensor_id(0, 0, ri.KIND_WQ), 4, 512, False, first_row=100)
    assert np.array_equal(part, a[100:104])


def test_bf16_rounding_matches_library():
    a = ri.cpu_tensor(3, 11, 256, 256, False)
    r = ri.cpu_tensor(3, 11, 256, 256, True)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, want)


def test_norm_gains_are_seeded_distinct_and_away_from_one():
    """RMSNorm gains are 1 + 5 * (a weight-recipe draw): near 1 +- 0.1, a different vector for every norm of every
    layer and model, exactly representable in bfloat16 for 16-bit models."""
    sh = ri.SHAPES["tiny_draft"]
    for bf16 in (False, True):
        w = ri.cpu_model_weights(sh, ri.SLOT_DRAFT, 0, bf16, ri.HEAD_LM)
        p = ri.cpu_model_weights(sh, ri.SLOT_PRM, 0, bf16, ri.HEAD_REWARD_SIGMOID)
        gains = [w["final_norm"], p["final_norm"]] + [lw[k] for lw in w["layers"] + p["layers"] for k in ("norm1", "norm2")]
        for g in gains:
            assert g.shape == (sh.d_model,) and g.dtype == np.float32
            assert 0.5 < g.min() and g.max() < 1.5 and 0.05 < g.std() < 0.15
            if bf16:
                assert np.array_equal(g, torch.from_numpy(g).to(torch.bfloat16).float().numpy())
        for i in range(len(gains)):
            for j in range(i + 1, len(gains)):
                assert np.abs(gains[i] - gains[j]).max() > 0.1
    draw = ri.cpu_tensor(0, ri.tensor_id(0, 1, ri.KIND_NORM2), 1, sh.d_model, False)[0]
    want = np.float32(1.0) + np.float32(5.0) * draw
    assert np.array_equal(ri.cpu_model_weights(sh, 0, 0, False, ri.HEAD_LM)["layers"][1]["norm2"], want)


def test_prompts_shape_and_range():
    tok, off = ri.prompts(1, 32, 128, 512, 151936)
    lens = np.diff(off)
    assert off[0] == 0 and len(tok) == off[-1]
    assert lens.min() >= 128 and lens.max() <= 512
    assert tok.min() >= 0 and tok.max() < 151936
    tok2, off2 = ri.prompts(1, 32, 128, 512, 151936)
    assert np.array_equal(tok, tok2) and np.array_equal(off, off2)


def test_parameter_counts():
    # layer counts derived by hand from the shapes (d*Hhd*2 + 2*d*KVhd + 3*d*ffn + 2d)
    s = ri.SHAPES["1.5b"]
    assert s.n_params(ri.HEAD_LM) - 2 * s.vocab * s.d_model - s.d_model == 28 * 46_795_776
    s = ri.SHAPES["7b"]
    assert s.n_params(ri.HEAD_LM) - 2 * s.vocab * s.d_model - s.d_model == 28 * 233_053_184
    s = ri.SHAPES["72b"]
    assert s.n_params(ri.HEAD_LM) - 2 * s.vocab * s.d_model - s.d_model == 80 * 877_674_496
