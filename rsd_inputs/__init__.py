"""Seeded synthetic inputs for the RSD step loop: model shapes, weights and prompts.

This module serves both the CPU oracle's callers and the GPU library's callers and holds none
of the decoding method's arithmetic.  Weights are random-init N(0, 0.02)-like values that are a
pure function of (seed, tensor id, logical element index) -- see ``weight_init.h`` -- so the CPU
(fp32 arrays) and GPU (fp32 or bfloat16 device arrays) copies are bit-identical.

Workload shapes stand in for the model families the paper serves (Section 3, "Models"): small
Llama-style test models plus the 1.5B / 7B / 72B decoder shapes used as draft, PRM and target.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass, asdict

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))

SIGMA = 0.02
# scale = sigma / (2 * std of the sum of eight 16-bit uniforms), rounded once to fp32
WEIGHT_SCALE = float(np.float32(SIGMA / (2.0 * math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0))))

KIND_EMBED, KIND_HEAD, KIND_WQ, KIND_WK, KIND_WV, KIND_WO, KIND_WGATE, KIND_WUP, KIND_WDOWN = range(9)
KIND_NORM1, KIND_NORM2, KIND_FINAL_NORM = 9, 10, 11
GAIN_SPREAD = 5.0   # RMSNorm gains = 1 + GAIN_SPREAD * (a weight-recipe draw of sigma 0.02): 1 +- 0.1
SLOT_DRAFT, SLOT_PRM, SLOT_TARGET = 0, 1, 2
HEAD_LM, HEAD_REWARD_SIGMOID, HEAD_REWARD_RAW = 0, 1, 2


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-6

    def n_params(self, head_kind: int = HEAD_LM) -> int:
        """All parameters: embedding, layers (with norm gains), final norm and head."""
        d, hd = self.d_model, self.head_dim
        per_layer = (d * self.n_heads * hd + 2 * d * self.n_kv_heads * hd + self.n_heads * hd * d
                     + 3 * d * self.d_ffn + 2 * d)
        head = self.vocab * d if head_kind == HEAD_LM else d
        return self.vocab * d + self.n_layers * per_layer + d + head

    def kv_bytes_per_token(self, elem_bytes: int) -> int:
        return self.n_layers * 2 * self.n_kv_heads * self.head_dim * elem_bytes


SHAPES = {
    "tiny_draft": ModelShape(2, 256, 4, 2, 64, 688, 1024),
    "tiny_target": ModelShape(4, 512, 8, 2, 64, 1376, 1024),
    # a second small family with head_dim 128, used to exercise the 16-bit kernels cheaply
    "mini_draft": ModelShape(2, 512, 4, 2, 128, 1408, 4096),
    "mini_target": ModelShape(3, 768, 6, 2, 128, 2048, 4096),
    "1.5b": ModelShape(28, 1536, 12, 2, 128, 8960, 151936),
    "7b": ModelShape(28, 3584, 28, 4, 128, 18944, 151936),
    "72b": ModelShape(80, 8192, 64, 8, 128, 29568, 152064),
}


def tensor_id(slot: int, layer: int, kind: int) -> int:
    return slot * 65536 + layer * 16 + kind


def _needs_build(target: str, sources: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build_cpu(force: bool = False) -> str:
    so = os.path.join(_HERE, "librsd_inputs_cpu.so")
    srcs = [os.path.join(_HERE, "gen_cpu.c"), os.path.join(_HERE, "weight_init.h")]
    if force or _needs_build(so, srcs):
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", so, srcs[0]])
    return so


def build_cuda(force: bool = False) -> str:
    so = os.path.join(_HERE, "librsd_inputs_cuda.so")
    srcs = [os.path.join(_HERE, "gen_cuda.cu"), os.path.join(_HERE, "weight_init.h")]
    if force or _needs_build(so, srcs):
        subprocess.check_call(["nvcc", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                               "-Xcompiler", "-fPIC", "-shared", "-o", so, srcs[0]])
    return so


_cpu_lib = None
_cuda_lib = None


def cpu_lib():
    global _cpu_lib
    if _cpu_lib is None:
        lib = ctypes.CDLL(build_cpu())
        lib.rsd_inputs_fill_f32.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64,
                                            ctypes.c_uint64, ctypes.c_float, ctypes.c_int]
        lib.rsd_inputs_fill_f32.restype = None
        lib.rsd_inputs_philox4x32_10.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.rsd_inputs_philox4x32_10.restype = None
        _cpu_lib = lib
    return _cpu_lib


def cuda_lib():
    global _cuda_lib
    if _cuda_lib is None:
        lib = ctypes.CDLL(build_cuda())
        lib.rsd_inputs_fill_device.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_uint32,
                                               ctypes.c_uint64, ctypes.c_uint64, ctypes.c_float, ctypes.c_void_p]
        lib.rsd_inputs_fill_device.restype = ctypes.c_int
        lib.rsd_inputs_fill_const_device.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64,
                                                     ctypes.c_float, ctypes.c_void_p]
        lib.rsd_inputs_fill_const_device.restype = ctypes.c_int
        _cuda_lib = lib
    return _cuda_lib


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    cpu_lib().rsd_inputs_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def cpu_tensor(seed: int, tid: int, rows: int, cols: int, bf16: bool, first_row: int = 0) -> np.ndarray:
    """fp32 host array [rows, cols] of tensor `tid`, starting at logical row `first_row`."""
    out = np.empty((rows, cols), dtype=np.float32)
    cpu_lib().rsd_inputs_fill_f32(out.ctypes.data, seed, tid, first_row * cols, rows * cols,
                                  WEIGHT_SCALE, 1 if bf16 else 0)
    return out


def _round_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array rounded to the nearest bfloat16 (ties to even), returned as fp32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return (((u + r) >> np.uint32(16)) << np.uint32(16)).view(np.float32)


def cpu_gain(seed: int, tid: int, d: int, bf16: bool) -> np.ndarray:
    """RMSNorm gain vector [d]: 1 + GAIN_SPREAD * draw (about 1 +- 0.1, never near zero: the draw is
    bounded by 4.9 sigma), a distinct tensor id per norm, so that a gain taken from the wrong layer, a
    skipped norm or a gain applied twice changes the result.  Computed on the host in fp32 (one multiply,
    one add, each rounded once) and, for 16-bit models, rounded to bfloat16; the GPU copy is an upload of
    these very values."""
    draw = cpu_tensor(seed, tid, 1, d, False)[0]
    g = (np.float32(1.0) + np.float32(GAIN_SPREAD) * draw).astype(np.float32)
    return _round_bf16(g) if bf16 else g


def layer_tensor_dims(shape: ModelShape) -> dict:
    d, hd = shape.d_model, shape.head_dim
    return {
        KIND_WQ: (shape.n_heads * hd, d), KIND_WK: (shape.n_kv_heads * hd, d), KIND_WV: (shape.n_kv_heads * hd, d),
        KIND_WO: (d, shape.n_heads * hd), KIND_WGATE: (shape.d_ffn, d), KIND_WUP: (shape.d_ffn, d),
        KIND_WDOWN: (d, shape.d_ffn),
    }


def cpu_layer_weights(shape: ModelShape, slot: int, layer: int, seed: int, bf16: bool) -> dict:
    """Un-fused weight matrices of one layer and its two RMSNorm gain vectors (fp32 host arrays)."""
    dims = layer_tensor_dims(shape)
    w = {k: cpu_tensor(seed, tensor_id(slot, layer, k), r, c, bf16) for k, (r, c) in dims.items()}
    return {
        "wq": w[KIND_WQ], "wk": w[KIND_WK], "wv": w[KIND_WV], "wo": w[KIND_WO],
        "wgate": w[KIND_WGATE], "wup": w[KIND_WUP], "wdown": w[KIND_WDOWN],
        "norm1": cpu_gain(seed, tensor_id(slot, layer, KIND_NORM1), shape.d_model, bf16),
        "norm2": cpu_gain(seed, tensor_id(slot, layer, KIND_NORM2), shape.d_model, bf16),
    }


def cpu_model_weights(shape: ModelShape, slot: int, seed: int, bf16: bool, head_kind: int,
                      with_layers: bool = True) -> dict:
    """All weights of one model as fp32 host arrays (bf16-rounded values when bf16=True)."""
    d = shape.d_model
    head_rows = shape.vocab if head_kind == HEAD_LM else 1
    out = {
        "shape": shape, "head_kind": head_kind,
        "tok_embed": cpu_tensor(seed, tensor_id(slot, 0, KIND_EMBED), shape.vocab, d, bf16),
        "final_norm": cpu_gain(seed, tensor_id(slot, 0, KIND_FINAL_NORM), d, bf16),
        "head": cpu_tensor(seed, tensor_id(slot, 0, KIND_HEAD), head_rows, d, bf16),
        "layers": [],
    }
    if with_layers:
        out["layers"] = [cpu_layer_weights(shape, slot, l, seed, bf16) for l in range(shape.n_layers)]
    return out


def gpu_model_tensors(shape: ModelShape, slot: int, seed: int, bf16: bool, head_kind: int) -> dict:
    """The same weights as cpu_model_weights, generated on the GPU into torch tensors in the fused
    storage the CUDA library reads: wqkv rows = Wq | Wk | Wv, wgu rows = Wgate | Wup."""
    import torch
    lib = cuda_lib()
    dt = torch.bfloat16 if bf16 else torch.float32
    code = 1 if bf16 else 0
    esz = 2 if bf16 else 4
    stream = torch.cuda.current_stream().cuda_stream

    def fill(t, row0, rows, cols, tid):
        rc = lib.rsd_inputs_fill_device(t.data_ptr() + row0 * cols * esz, code, seed, tid, 0, rows * cols,
                                        WEIGHT_SCALE, stream)
        assert rc == 0, f"fill kernel launch failed: {rc}"

    def gain(layer, kind):
        # the host's values, uploaded: bf16 values are exact in fp32, so the cast back is exact
        return torch.from_numpy(cpu_gain(seed, tensor_id(slot, layer, kind), shape.d_model, bf16)).to(dt).cuda()

    d, hd, H, KV, F = shape.d_model, shape.head_dim, shape.n_heads, shape.n_kv_heads, shape.d_ffn
    out = {"tok_embed": torch.empty(shape.vocab, d, dtype=dt, device="cuda"), "final_norm": gain(0, KIND_FINAL_NORM),
           "wqkv": [], "wo": [], "wgu": [], "wdown": [], "norm1": [], "norm2": []}
    fill(out["tok_embed"], 0, shape.vocab, d, tensor_id(slot, 0, KIND_EMBED))
    head_rows = shape.vocab if head_kind == HEAD_LM else 1
    out["head"] = torch.empty(head_rows, d, dtype=dt, device="cuda")
    fill(out["head"], 0, head_rows, d, tensor_id(slot, 0, KIND_HEAD))
    for l in range(shape.n_layers):
        wqkv = torch.empty((H + 2 * KV) * hd, d, dtype=dt, device="cuda")
        fill(wqkv, 0, H * hd, d, tensor_id(slot, l, KIND_WQ))
        fill(wqkv, H * hd, KV * hd, d, tensor_id(slot, l, KIND_WK))
        fill(wqkv, (H + KV) * hd, KV * hd, d, tensor_id(slot, l, KIND_WV))
        wo = torch.empty(d, H * hd, dtype=dt, device="cuda")
        fill(wo, 0, d, H * hd, tensor_id(slot, l, KIND_WO))
        wgu = torch.empty(2 * F, d, dtype=dt, device="cuda")
        fill(wgu, 0, F, d, tensor_id(slot, l, KIND_WGATE))
        fill(wgu, F, F, d, tensor_id(slot, l, KIND_WUP))
        wdown = torch.empty(d, F, dtype=dt, device="cuda")
        fill(wdown, 0, d, F, tensor_id(slot, l, KIND_WDOWN))
        out["wqkv"].append(wqkv); out["wo"].append(wo); out["wgu"].append(wgu); out["wdown"].append(wdown)
        out["norm1"].append(gain(l, KIND_NORM1)); out["norm2"].append(gain(l, KIND_NORM2))
    return out


def prompts(seed: int, batch: int, len_lo: int, len_hi: int, vocab: int):
    """Ragged uniform-random prompts: lengths uniform on [len_lo, len_hi], ids uniform on [0, vocab)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(len_lo, len_hi + 1, size=batch).astype(np.int32)
    offsets = np.zeros(batch + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(lens)
    tokens = rng.integers(0, vocab, size=int(offsets[-1])).astype(np.int32)
    return tokens, offsets


__all__ = [n for n in dir() if not n.startswith("_")]
