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
