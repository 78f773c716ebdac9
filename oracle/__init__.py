"""TEST INFRASTRUCTURE -- CPU oracle of the RSD step loop (fp64 arithmetic on fp32-held weights).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA
library and its Python binding never do.  ``orc_model.c`` holds the transformer, heads, sampling
and acceptance rule; ``rsd_loop.py`` holds Algorithm 1 batched over rows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_lib = None


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "head_kind")] + \
               [("rope_theta", ctypes.c_double), ("rms_eps", ctypes.c_double)]


class _Layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm2")]


def build(force: bool = False) -> str:
    so = os.path.join(_HERE, "liborc.so")
    src = os.path.join(_HERE, "orc_model.c")
    if force or not os.path.exists(so) or os.path.getmtime(src) > os.path.getmtime(so):
        subprocess.check_call(["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", so, src, "-lm"])
    return so


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_double
        L.orc_rmsnorm.argtypes = [vp, vp, i32, f64, vp]
        L.orc_matmul.argtypes = [vp, i32, i32, vp, i32, vp]
        L.orc_rope.argtypes = [vp, i32, i32, f64]
        L.orc_embed.argtypes = [vp, vp, i32, i32, vp]
        L.orc_layer_forward.argtypes = [ctypes.POINTER(_Shape), ctypes.POINTER(_Layer), vp, i32, i32, vp, vp]
        L.orc_head_logits.argtypes = [ctypes.POINTER(_Shape), vp, vp, vp, vp]
        L.orc_head_reward.argtypes = [ctypes.POINTER(_Shape), vp, vp, vp]
        L.orc_head_reward.restype = f64
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
        L.orc_uniform.restype = f64
        L.orc_uniform_from_bits.argtypes = [ctypes.c_uint32]
        L.orc_uniform_from_bits.restype = f64
        L.orc_sample.argtypes = [vp, i32, f64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, vp]
        L.orc_sample.restype = i32
        L.orc_omega.argtypes = [i32, f64, f64, f64]
        L.orc_omega.restype = f64
        L.orc_accept.argtypes = [i32, f64, f64, f64, f64]
        L.orc_accept.restype = i32
        for f in (L.orc_rmsnorm, L.orc_matmul, L.orc_rope, L.orc_embed, L.orc_layer_forward,
                  L.orc_head_logits, L.orc_philox4x32_10):
            f.restype = None
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ----------------------------------------------------------------------------- thin wrappers

def rmsnorm(x, g, eps):
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = _f32(g)
    out = np.empty_like(x)
    lib().orc_rmsnorm(x.ctypes.data, g.ctypes.data, x.shape[-1], eps, out.ctypes.data)
    return out


def matmul(W, X):
    """Y[t, r] = sum_c W[r, c] X[t, c]."""
    W = _f32(W)
    X = np.ascontiguousarray(X, dtype=np.float64)
    T = X.shape[0]
    Y = np.empty((T, W.shape[0]), dtype=np.float64)
    lib().orc_matmul(W.ctypes.data, W.shape[0], W.shape[1], X.ctypes.data, T, Y.ctypes.data)
    return Y


def rope(v, pos, theta):
    v = np.array(v, dtype=np.float64)
    lib().orc_rope(v.ctypes.data, v.shape[-1], int(pos), float(theta))
    return v


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    o = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(c.ctypes.data, k.ctypes.data, o.ctypes.data)
    return o


def uniform(seed, stream, row, position, index):
    return lib().orc_uniform(seed, stream, row, position, index)


def sample(logits, v_limit, temperature, seed, model_id, row, position):
    """Returns (token, margin between the best and second-best compared score)."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    m = ctypes.c_double(0.0)
    t = lib().orc_sample(logits.ctypes.data, int(v_limit), float(temperature), int(seed), int(model_id),
                         int(row), int(position), ctypes.addressof(m))
    return int(t), float(m.value)


def omega(kind, r, a=0.0, b=0.0):
    return lib().orc_omega(kind, r, a, b)


def accept(kind, r, a=0.0, b=0.0, u=0.5):
    return lib().orc_accept(kind, r, a, b, u)


# ----------------------------------------------------------------------------- model objects

class KVCache:
    """Keys (after RoPE) and values of one sequence for every layer: [L, capacity, KV*hd] fp64."""

    def __init__(self, n_layers, capacity, kvd):
        self.k = np.zeros((n_layers, capacity, kvd), dtype=np.float64)
        self.v = np.zeros((n_layers, capacity, kvd), dtype=np.float64)
        self.capacity = capacity


class OracleModel:
    """One decoder-only transformer (draft m, target M or PRM r) held as un-fused fp32 matrices."""

    def __init__(self, weights: dict, model_id: int):
        sh = weights["shape"]
        self.shape = sh
        self.model_id = model_id
        self.head_kind = weights["head_kind"]
        self.w = weights
        self._cshape = _Shape(sh.n_layers, sh.d_model, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn,
                              sh.vocab, self.head_kind, sh.rope_theta, sh.rms_eps)
        self._clayers = [self._layer_struct(lw) for lw in weights["layers"]]
        self.n_params = sh.n_params(self.head_kind)

    @staticmethod
    def _layer_struct(lw):
        for k in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm2"):
            lw[k] = _f32(lw[k])
        return _Layer(*[lw[k].ctypes.data for k in
                        ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm2")])

    def new_cache(self, capacity: int) -> KVCache:
        return KVCache(self.shape.n_layers, capacity, self.shape.n_kv_heads * self.shape.head_dim)

    def embed(self, tokens) -> np.ndarray:
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        x = np.empty((len(tokens), self.shape.d_model), dtype=np.float64)
        e = self.w["tok_embed"]
        lib().orc_embed(e.ctypes.data, tokens.ctypes.data, len(tokens), self.shape.d_model, x.ctypes.data)
        return x

    def layer(self, l: int, x: np.ndarray, start_pos: int, cache: KVCache, layer_struct=None):
        ls = layer_struct if layer_struct is not None else self._clayers[l]
        lib().orc_layer_forward(ctypes.byref(self._cshape), ctypes.byref(ls), x.ctypes.data, x.shape[0],
                                int(start_pos), cache.k[l].ctypes.data, cache.v[l].ctypes.data)

    def forward(self, cache: KVCache, tokens, start_pos: int) -> np.ndarray:
        """Push tokens at positions start_pos.. through all layers; returns last-layer hidden [T, d]."""
        assert start_pos + len(tokens) <= cache.capacity
        x = self.embed(tokens)
        for l in range(self.shape.n_layers):
            self.layer(l, x, start_pos, cache)
        return x

    def forward_full(self, tokens) -> np.ndarray:
        """Full-sequence recompute from an empty cache."""
        return self.forward(self.new_cache(len(tokens)), tokens, 0)

    def logits(self, hidden_vec) -> np.ndarray:
        hv = np.ascontiguousarray(hidden_vec, dtype=np.float64)
        out = np.empty(self.shape.vocab, dtype=np.float64)
        lib().orc_head_logits(ctypes.byref(self._cshape), self.w["final_norm"].ctypes.data,
                              self.w["head"].ctypes.data, hv.ctypes.data, out.ctypes.data)
        return out

    def reward(self, hidden_vec) -> float:
        hv = np.ascontiguousarray(hidden_vec, dtype=np.float64)
        return lib().orc_head_reward(ctypes.byref(self._cshape), self.w["final_norm"].ctypes.data,
                                     self.w["head"].ctypes.data, hv.ctypes.data)
