"""ctypes binding of librsd.so: argument marshalling only.  Every step of the path runs in the
CUDA library; PyTorch provides device memory and the stream.  There is no CPU fallback: loading
fails loudly when the library is missing, and compute calls fail without a CUDA device."""
from __future__ import annotations

import ctypes
import os
from ctypes import c_float, c_int32, c_size_t, c_uint64, c_uint8, c_void_p, c_double, POINTER

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librsd.so")

RSD_F32, RSD_BF16 = 0, 1
RSD_DRAFT, RSD_PRM, RSD_TARGET = 0, 1, 2
RSD_HEAD_LM, RSD_HEAD_REWARD_SIGMOID, RSD_HEAD_REWARD_RAW = 0, 1, 2
RSD_DEBUG_KEEP_LOGITS = 1
RSD_DEBUG_NO_GRAPHS = 2
RSD_DEBUG_PERSISTENT_DECODE = 4
RSD_DEBUG_MEGA_PROFILE = 8
RSD_DEBUG_NO_F16_DENSE = 16
ERRORS = {0: "RSD_OK", -1: "RSD_ERR_ARG", -2: "RSD_ERR_STATE", -3: "RSD_ERR_OOM_PAGES", -4: "RSD_ERR_CUDA",
          -5: "RSD_ERR_TIMEOUT", -6: "RSD_ERR_UNSUPPORTED"}


class RsdError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERRORS.get(code, code)}: {msg}")
        self.code = code


class rsd_model(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn",
                                        "vocab", "dtype")] + \
               [("rope_theta", c_float), ("rms_eps", c_float), ("head_kind", c_int32),
                ("tok_embed", c_void_p), ("final_norm", c_void_p), ("head", c_void_p)] + \
               [(n, POINTER(c_void_p)) for n in ("wqkv", "wo", "wgu", "wdown", "norm1", "norm2")]


class rsd_config(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("max_batch", "max_seq_tokens", "max_step_tokens", "max_steps", "page_tokens",
                                        "step_end_id", "eos_id", "step_end_mod")] + \
               [("temperature", c_float), ("seed", c_uint64), ("omega_kind", c_int32), ("omega_alpha", c_float),
                ("max_chunk_tokens", c_int32), ("debug_flags", c_int32), ("kv_extended", c_int32), ("prm_shares_draft", c_int32),
                ("sd_tokens", c_int32), ("kv_pool", c_void_p * 3), ("kv_bytes", c_size_t * 3), ("workspace", c_void_p),
                ("workspace_bytes", c_size_t)]


class rsd_counters(ctypes.Structure):
    _fields_ = [("gen_tokens", c_uint64 * 3), ("ingest_tokens", c_uint64 * 3), ("score_tokens", c_uint64),
                ("steps", c_uint64), ("accepted_steps", c_uint64), ("rejected_steps", c_uint64),
                ("discarded_draft_tokens", c_uint64), ("flops_paper", c_double), ("flops_all_tokens", c_double),
                ("sd_rounds", c_uint64), ("sd_proposed", c_uint64), ("sd_matched", c_uint64), ("sd_verified", c_uint64)]


EXPORTS = ["rsd_query_sizes", "rsd_create", "rsd_load_models", "rsd_prefill", "rsd_step", "rsd_step_queued", "rsd_step_device", "rsd_get_target_step_rewards", "rsd_flops_counters",
           "rsd_reset", "rsd_destroy", "rsd_last_error", "rsd_debug_force", "rsd_debug_force_sd", "rsd_debug_get_logits",
           "rsd_debug_get_sampled", "rsd_debug_get_state", "rsd_debug_gemm_timing", "rsd_debug_gemm_timing_dense", "rsd_debug_launch_count", "rsd_debug_mega_profile", "rsd_debug_phase_ms", "rsd_k_gemm", "rsd_k_gemm_scratch_bytes", "rsd_debug_gemm_wait_probe",
           "rsd_k_attn_decode", "rsd_k_attn_decode_scratch_bytes", "rsd_k_attn_chunk", "rsd_k_gate_compact", "rsd_k_gate_compact_static", "rsd_k_gate_compact_static_error", "rsd_k_rmsnorm",
           "rsd_k_rope", "rsd_k_swiglu", "rsd_k_gemm_gu", "rsd_k_sample", "rsd_k_philox"]

_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2501_19324_b200.build` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp = c_void_p
        L.rsd_query_sizes.argtypes = [POINTER(rsd_model)] * 3 + [POINTER(rsd_config)]
        L.rsd_create.argtypes = [POINTER(rsd_config), POINTER(vp)]
        L.rsd_load_models.argtypes = [vp] + [POINTER(rsd_model)] * 3
        L.rsd_prefill.argtypes = [vp, vp, vp, c_int32, vp]
        L.rsd_step.argtypes = [vp, c_float, vp, vp, vp, vp, vp, vp]
        L.rsd_step_queued.argtypes = [vp, c_float, c_int32, vp, vp, vp, vp, vp, vp, vp]
        L.rsd_step_device.argtypes = [vp, c_float, c_int32, vp, vp, vp, vp, vp, vp, vp]
        L.rsd_get_target_step_rewards.argtypes = [vp, vp]
        L.rsd_flops_counters.argtypes = [vp, POINTER(rsd_counters)]
        L.rsd_reset.argtypes = [vp]
        L.rsd_destroy.argtypes = [vp]
        L.rsd_last_error.argtypes = [vp]
        L.rsd_last_error.restype = ctypes.c_char_p
        L.rsd_debug_force.argtypes = [vp, c_int32, vp, vp, vp]
        L.rsd_debug_force_sd.argtypes = [vp, vp, vp]
        L.rsd_debug_get_logits.argtypes = [vp, c_int32, vp]
        L.rsd_debug_get_sampled.argtypes = [vp, c_int32, vp]
        L.rsd_debug_get_state.argtypes = [vp] * 8
        L.rsd_debug_gemm_timing.argtypes = [vp, c_int32, vp, vp, vp]
        L.rsd_debug_gemm_timing_dense.argtypes = [vp, vp, vp, vp]
        L.rsd_debug_phase_ms.argtypes = [vp, c_int32, vp]
        L.rsd_debug_launch_count.argtypes = []
        L.rsd_debug_mega_profile.argtypes = [vp, c_int32, vp, c_int32, vp]
        L.rsd_debug_launch_count.restype = c_uint64
        L.rsd_k_gemm.argtypes = [vp, vp, vp, vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, vp, c_size_t, vp]
        L.rsd_debug_gemm_wait_probe.argtypes = [vp, vp, vp, vp, c_size_t, vp]
        L.rsd_k_gemm_scratch_bytes.argtypes = [c_int32, c_int32, c_int32]
        L.rsd_k_gemm_scratch_bytes.restype = c_size_t
        L.rsd_k_attn_decode.argtypes = [vp, vp, vp, vp, vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32,
                                        vp, c_size_t, vp]
        L.rsd_k_attn_chunk.argtypes = [vp, vp, vp, vp, vp, vp, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, vp]
        L.rsd_k_attn_decode_scratch_bytes.argtypes = [c_int32] * 4
        L.rsd_k_attn_decode_scratch_bytes.restype = c_size_t
        L.rsd_k_gate_compact.argtypes = [vp, vp, c_float, vp, vp, vp, c_int32, vp, c_size_t, vp]
        L.rsd_k_gate_compact_static.argtypes = [vp, vp, c_float, vp, vp, vp, c_int32, vp]
        L.rsd_k_gate_compact_static_error.argtypes = []
        L.rsd_k_gate_compact_static_error.restype = ctypes.c_char_p
        L.rsd_k_rmsnorm.argtypes = [vp, vp, vp, c_int32, c_int32, c_float, c_int32, vp]
        L.rsd_k_rope.argtypes = [vp, vp, c_int32, c_int32, c_int32, c_float, vp]
        L.rsd_k_swiglu.argtypes = [vp, vp, c_int32, c_int32, c_int32, vp]
        L.rsd_k_gemm_gu.argtypes = [vp, vp, vp, vp, vp, c_int32, c_int32, c_int32, vp, c_size_t, vp]
        L.rsd_k_sample.argtypes = [vp, c_int32, c_int32, c_int32, c_float, c_uint64, c_int32, vp, vp, vp, vp, c_size_t, vp]
        L.rsd_k_philox.argtypes = [vp, vp, vp, c_int32, vp]
        _lib = L
    return _lib


def _check(rc, ctx=None):
    if rc != 0:
        msg = lib().rsd_last_error(ctx)
        raise RsdError(rc, msg.decode() if msg else "")


def _stream():
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return c_void_p(t.data_ptr())


class Model:
    """A transformer's weights as torch CUDA tensors plus the rsd_model descriptor pointing at them.

    tensors: tok_embed [V, d], final_norm [d], head [V, d] or [d], and per-layer lists wqkv
    [(H+2KV)hd, d], wo [d, Hhd], wgu [2F, d], wdown [d, F], norm1 [d], norm2 [d].
    head_only: a PRM that is a head on the draft's trunk (prm_shares_draft) carries no layers."""

    def __init__(self, shape, tensors: dict, head_kind: int, head_only: bool = False):
        import torch
        self.shape, self.t, self.head_kind = shape, tensors, head_kind
        dt = tensors["tok_embed"].dtype
        assert dt in (torch.float32, torch.bfloat16)
        self.dtype = RSD_BF16 if dt == torch.bfloat16 else RSD_F32
        L = shape.n_layers
        self._arrays = {}
        for k in ("wqkv", "wo", "wgu", "wdown", "norm1", "norm2"):
            if head_only:
                self._arrays[k] = None
                continue
            assert len(tensors[k]) == L
            for w in tensors[k]:
                assert w.is_cuda and w.is_contiguous() and w.dtype == dt
            self._arrays[k] = (c_void_p * L)(*[w.data_ptr() for w in tensors[k]])
        self.desc = rsd_model(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                              shape.d_ffn, shape.vocab, self.dtype, shape.rope_theta, shape.rms_eps, head_kind,
                              tensors["tok_embed"].data_ptr(), tensors["final_norm"].data_ptr(),
                              tensors["head"].data_ptr(),
                              *[ctypes.cast(self._arrays[k], POINTER(c_void_p)) if self._arrays[k] is not None
                                else POINTER(c_void_p)() for k in ("wqkv", "wo", "wgu", "wdown", "norm1", "norm2")])


class Engine:
    """The RSD step loop on one GPU: rsd_load_models, rsd_prefill, rsd_step(delta), rsd_flops_counters."""

    def __init__(self, draft: Model, prm: Model, target: Model, *, max_batch, max_seq_tokens, max_step_tokens,
                 max_steps, step_end_id, eos_id=-1, step_end_mod=0, temperature=0.0, seed=0, omega_kind=1,
                 omega_alpha=0.0, max_chunk_tokens=0, debug_flags=0, kv_bytes=None, kv_extended=0,
                 prm_shares_draft=0, sd_tokens=0):
        import torch
        if not torch.cuda.is_available():
            raise RsdError(-4, "no CUDA device: this library has no CPU fallback")
        self.models = (draft, prm, target)
        self.B_max, self.S, self.C = max_batch, max_seq_tokens, max_step_tokens
        self.max_pages = (max_seq_tokens + 15) // 16
        self.sd_tokens = sd_tokens
        cfg = rsd_config(max_batch, max_seq_tokens, max_step_tokens, max_steps, 16, step_end_id, eos_id, step_end_mod,
                         temperature, seed, omega_kind, omega_alpha, max_chunk_tokens, debug_flags, kv_extended,
                         prm_shares_draft, sd_tokens)
        _check(lib().rsd_query_sizes(draft.desc, prm.desc, target.desc, cfg))
        if kv_bytes is not None:
            for i in range(3):
                cfg.kv_bytes[i] = kv_bytes[i]
        self._kv = [torch.empty(max(int(cfg.kv_bytes[i]), 256), dtype=torch.uint8, device="cuda") for i in range(3)]
        self._ws = torch.empty(int(cfg.workspace_bytes), dtype=torch.uint8, device="cuda")
        for i in range(3):
            cfg.kv_pool[i] = self._kv[i].data_ptr()
        cfg.workspace = self._ws.data_ptr()
        self.cfg = cfg
        self.ctx = c_void_p()
        _check(lib().rsd_create(cfg, ctypes.byref(self.ctx)))
        _check(lib().rsd_load_models(self.ctx, draft.desc, prm.desc, target.desc), self.ctx)
        self.B = 0

    def close(self):
        if getattr(self, "ctx", None):
            lib().rsd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        self.close()

    def prefill(self, tokens, offsets):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        offsets = np.ascontiguousarray(offsets, dtype=np.int32)
        self.B = len(offsets) - 1
        _check(lib().rsd_prefill(self.ctx, tokens.ctypes.data, offsets.ctypes.data, self.B, _stream()), self.ctx)

    def step(self, delta: float, min_target_rows: int = 1) -> dict:
        """rsd_step(delta); with min_target_rows > 1, rsd_step_queued: rejected rows wait (step_len 0,
        waiting 1) until that many wait, then the target writes all their steps in one pass."""
        B, C = self.B, self.C
        out = dict(step_tokens=np.zeros((B, C), np.int32), step_len=np.zeros(B, np.int32),
                   rewards=np.zeros(B, np.float32), accept=np.zeros(B, np.uint8), live=np.zeros(B, np.uint8),
                   waiting=np.zeros(B, np.uint8))
        ptrs = [out[k].ctypes.data for k in ("step_tokens", "step_len", "rewards", "accept", "live")]
        if min_target_rows == 1:
            _check(lib().rsd_step(self.ctx, delta, _stream(), *ptrs), self.ctx)
        else:
            _check(lib().rsd_step_queued(self.ctx, delta, min_target_rows, _stream(), *ptrs,
                                         out["waiting"].ctypes.data), self.ctx)
        return out

    def step_device(self, delta: float, min_target_rows: int = 1) -> dict:
        """rsd_step_device: the step's outputs as torch CUDA tensors, filled on the current stream."""
        import torch
        B, C = self.B, self.C
        out = dict(step_tokens=torch.zeros(B, C, dtype=torch.int32, device="cuda"),
                   step_len=torch.zeros(B, dtype=torch.int32, device="cuda"),
                   rewards=torch.zeros(B, dtype=torch.float32, device="cuda"),
                   accept=torch.zeros(B, dtype=torch.uint8, device="cuda"),
                   live=torch.zeros(B, dtype=torch.uint8, device="cuda"),
                   waiting=torch.zeros(B, dtype=torch.uint8, device="cuda"))
        _check(lib().rsd_step_device(self.ctx, delta, min_target_rows, _stream(),
                                     *[_ptr(out[k]) for k in ("step_tokens", "step_len", "rewards", "accept", "live", "waiting")]),
               self.ctx)
        return out

    def target_step_rewards(self) -> np.ndarray:
        """Reward of each row's latest target-written step (NaN where there is none yet)."""
        out = np.zeros(self.B, np.float32)
        _check(lib().rsd_get_target_step_rewards(self.ctx, out.ctypes.data), self.ctx)
        return out

    def counters(self) -> dict:
        c = rsd_counters()
        _check(lib().rsd_flops_counters(self.ctx, ctypes.byref(c)), self.ctx)
        return dict(gen_tokens=list(c.gen_tokens), ingest_tokens=list(c.ingest_tokens), score_tokens=c.score_tokens,
                    steps=c.steps, accepted_steps=c.accepted_steps, rejected_steps=c.rejected_steps,
                    discarded_draft_tokens=c.discarded_draft_tokens, flops_paper=c.flops_paper,
                    flops_all_tokens=c.flops_all_tokens, sd_rounds=c.sd_rounds, sd_proposed=c.sd_proposed,
                    sd_matched=c.sd_matched, sd_verified=c.sd_verified)

    def reset(self):
        _check(lib().rsd_reset(self.ctx), self.ctx)
        self.B = 0

    def gemm_timing(self, stride: int) -> dict:
        """Returns {ms, bytes, launches} gathered since the last call and installs a new stride."""
        ms, by, n = c_double(0), c_double(0), c_uint64(0)
        _check(lib().rsd_debug_gemm_timing(self.ctx, stride, ctypes.addressof(ms), ctypes.addressof(by),
                                           ctypes.addressof(n)), self.ctx)
        return dict(ms=ms.value, bytes=by.value, launches=n.value)

    def gemm_timing_dense(self) -> dict:
        """Dense GEMM launches (more than 128 rows) timed since the last call, by operand class:
        {"plain": {ms, flops, launches}, "split": {...}}."""
        ms, fl, n = (c_double * 2)(), (c_double * 2)(), (c_uint64 * 2)()
        _check(lib().rsd_debug_gemm_timing_dense(self.ctx, ms, fl, n), self.ctx)
        return {k: dict(ms=ms[i], flops=fl[i], launches=n[i]) for i, k in enumerate(("plain", "split"))}

    PHASES = ("draft_sync", "draft_decode", "prm_scoring", "gate_routing", "target_catchup", "target_decode", "commit")

    def phase_ms(self, enable: bool) -> dict:
        """Per-phase device time (ms) summed since the last call; switches the timing on or off."""
        out = (c_double * 7)()
        _check(lib().rsd_debug_phase_ms(self.ctx, int(enable), out), self.ctx)
        return dict(zip(self.PHASES, list(out)))

    # -- parity hooks ---------------------------------------------------------------------------
    def mega_profile(self, which: int) -> np.ndarray:
        """Global-timer stamps (ns) of the last persistent-decode launch of model `which` (RSD_DEBUG_MEGA_PROFILE)."""
        out = np.zeros(1024, dtype=np.uint64)
        n = ctypes.c_int32(0)
        _check(lib().rsd_debug_mega_profile(self.ctx, which, out.ctypes.data, 1024, ctypes.byref(n)), self.ctx)
        return out[:n.value]

    def force_tokens(self, which: int, steps: list):
        """steps[b]: list of token ids forced on row b in the next step (empty = free-running)."""
        tok = np.zeros((self.B, self.C), np.int32)
        ln = np.zeros(self.B, np.int32)
        for b, s in enumerate(steps):
            if s is not None and len(s):
                tok[b, :len(s)] = s
                ln[b] = len(s)
        _check(lib().rsd_debug_force(self.ctx, which, tok.ctypes.data, ln.ctypes.data, None), self.ctx)

    def force_sd_proposals(self, rounds: list):
        """rounds[b]: None, or the list of row b's rounds, each a list of proposed token ids (speculative decoding
        of rejected steps); imposed on the draft's proposals in the next step."""
        k = self.sd_tokens
        props = np.zeros((self.B, self.C, k), np.int32)
        on = np.zeros(self.B, np.uint8)
        for b, rs in enumerate(rounds):
            if rs is None:
                continue
            on[b] = 1
            for r, p in enumerate(rs):
                props[b, r, :len(p)] = p
        _check(lib().rsd_debug_force_sd(self.ctx, props.ctypes.data, on.ctypes.data), self.ctx)

    def force_accept(self, mask):
        m = np.array([255 if v is None else int(v) for v in mask], dtype=np.uint8)
        _check(lib().rsd_debug_force(self.ctx, RSD_PRM, None, None, m.ctypes.data), self.ctx)

    def logits(self, which: int) -> np.ndarray:
        V = self.models[which].shape.vocab
        out = np.zeros((self.B, self.C, V), np.float32)
        _check(lib().rsd_debug_get_logits(self.ctx, which, out.ctypes.data), self.ctx)
        return out

    def sampled(self, which: int) -> np.ndarray:
        out = np.zeros((self.B, self.C), np.int32)
        _check(lib().rsd_debug_get_sampled(self.ctx, which, out.ctypes.data), self.ctx)
        return out

    def state(self) -> dict:
        B, MP = self.B, self.max_pages
        z = np.zeros(B, np.int32); kv = np.zeros((3, B), np.int32); npg = np.zeros((3, B), np.int32)
        pt = np.zeros((3, B, MP), np.int32); nxt = np.zeros(3, np.int32); rej = np.zeros(B, np.int32)
        n_rej = c_int32(0)
        _check(lib().rsd_debug_get_state(self.ctx, z.ctypes.data, kv.ctypes.data, npg.ctypes.data, pt.ctypes.data,
                                         nxt.ctypes.data, rej.ctypes.data, ctypes.addressof(n_rej)), self.ctx)
        pages = [[pt[w, b, :npg[w, b]].tolist() for b in range(B)] for w in range(3)]
        return dict(z_len=z, kv_len=kv, n_pages=npg, pages=pages, next_page=nxt.tolist(),
                    rej_idx=rej[:n_rej.value].tolist())


# ---- single kernels ---------------------------------------------------------------------------

def k_gemm(W, x, y=None, accumulate=False, impl=0, x_lo=None):
    """y[M, N] (fp32) (+)= (x + x_lo)[M, K] @ W[N, K]^T on CUDA tensors."""
    import torch
    M, K = x.shape
    N = W.shape[0]
    if y is None:
        y = torch.zeros(M, N, dtype=torch.float32, device=x.device)
    nbytes = lib().rsd_k_gemm_scratch_bytes(M, N, K)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device=x.device)
    dt = RSD_BF16 if W.dtype in (torch.bfloat16, torch.float16) else RSD_F32     # fp16: impl 4 only (the element size)
    _check(lib().rsd_k_gemm(_ptr(W), _ptr(x), _ptr(x_lo) if x_lo is not None else None, _ptr(y), M, N, K, dt, int(accumulate), impl, _ptr(scratch), nbytes,
                            _stream()))
    if nbytes >= 4100 and int(scratch[4096:4100].view(torch.int32).item()) != 0:
        raise RsdError(-5, "a bounded wait inside the tensor-core GEMM expired")
    return y


def k_attn_decode(q, kv_pool, page_table, ctx_len, KV, ext=False):
    import torch
    B, H, hd = q.shape
    max_pages = page_table.shape[1]
    out = torch.empty_like(q)
    nbytes = lib().rsd_k_attn_decode_scratch_bytes(B, H, hd, max_pages * 16)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device=q.device)
    dt = {torch.bfloat16: RSD_BF16, torch.float16: 2, torch.float32: RSD_F32}[kv_pool.dtype]
    if ext:
        dt = 3
    _check(lib().rsd_k_attn_decode(_ptr(q), _ptr(kv_pool), _ptr(page_table), _ptr(ctx_len), _ptr(out), B, H, KV, hd,
                                   max_pages, dt, _ptr(scratch), nbytes, _stream()))
    return out


def k_attn_chunk(q, kv_pool, page_table, tok_row, tok_pos, KV, ext=False):
    import torch
    T, H, hd = q.shape
    out = torch.zeros_like(q)
    dt = {torch.bfloat16: RSD_BF16, torch.float16: 2, torch.float32: RSD_F32}[kv_pool.dtype]
    if ext:
        dt = 3
    _check(lib().rsd_k_attn_chunk(_ptr(q), _ptr(kv_pool), _ptr(page_table), _ptr(tok_row), _ptr(tok_pos), _ptr(out), T, H, KV,
                                  hd, page_table.shape[1], dt, _stream()))
    return out


def k_gate_compact(rewards, live, delta):
    import torch
    B = rewards.numel()
    accept = torch.empty(B, dtype=torch.uint8, device=rewards.device)
    rej = torch.empty(B, dtype=torch.int32, device=rewards.device)
    n_rej = torch.zeros(1, dtype=torch.int32, device=rewards.device)
    scratch = torch.zeros(4 * ((B + 1023) // 1024) + 16, dtype=torch.uint8, device=rewards.device)
    _check(lib().rsd_k_gate_compact(_ptr(rewards), _ptr(live), float(delta), _ptr(accept), _ptr(rej), _ptr(n_rej), B,
                                    _ptr(scratch), scratch.numel(), _stream()))
    return accept, rej, n_rej


def k_gate_compact_static(rewards, live, delta, accept, rej, n_rej):
    """Gate + compaction with the library's built-in scratch: the caller supplies every buffer and the
    call itself allocates nothing (for hosts that cannot call cudaMalloc).  Returns the status code."""
    return lib().rsd_k_gate_compact_static(_ptr(rewards), _ptr(live), float(delta), _ptr(accept), _ptr(rej),
                                           _ptr(n_rej), rewards.numel(), _stream())


def k_rmsnorm(x, gain, eps):
    import torch
    out = torch.empty(x.shape, dtype=gain.dtype, device=x.device)
    dt = RSD_BF16 if gain.dtype == torch.bfloat16 else RSD_F32
    _check(lib().rsd_k_rmsnorm(_ptr(x), _ptr(gain), _ptr(out), x.shape[0], x.shape[1], eps, dt, _stream()))
    return out


def k_rope(v, pos, theta):
    T, nh, hd = v.shape
    _check(lib().rsd_k_rope(_ptr(v), _ptr(pos), T, nh, hd, theta, _stream()))
    return v


def k_swiglu(gu, out_dtype):
    import torch
    T, F2 = gu.shape
    out = torch.empty(T, F2 // 2, dtype=out_dtype, device=gu.device)
    dt = RSD_BF16 if out_dtype == torch.bfloat16 else RSD_F32
    _check(lib().rsd_k_swiglu(_ptr(gu), _ptr(out), T, F2 // 2, dt, _stream()))
    return out


def k_gemm_gu(Wgu, x_hi, x_lo):
    """Gate/up projection + SwiGLU on the tensor-core path: returns (act_hi, act_lo), bf16 [M, F]."""
    import torch
    M, K = x_hi.shape
    F = Wgu.shape[0] // 2
    hi = torch.zeros(M, F, dtype=torch.bfloat16, device=x_hi.device)
    lo = torch.zeros(M, F, dtype=torch.bfloat16, device=x_hi.device)
    nbytes = lib().rsd_k_gemm_scratch_bytes(M, 2 * F, K)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device=x_hi.device)
    _check(lib().rsd_k_gemm_gu(_ptr(Wgu), _ptr(x_hi), _ptr(x_lo), _ptr(hi), _ptr(lo), M, F, K, _ptr(scratch), nbytes, _stream()))
    return hi, lo


def k_sample(logits, v_limit, temperature, seed, model_id, row, pos):
    import torch
    B, V = logits.shape
    tok = torch.zeros(B, dtype=torch.int32, device=logits.device)
    scratch = torch.zeros(B, dtype=torch.int64, device=logits.device)
    _check(lib().rsd_k_sample(_ptr(logits), B, V, v_limit, temperature, seed, model_id, _ptr(row), _ptr(pos), _ptr(tok),
                              _ptr(scratch), 8 * B, _stream()))
    return tok


def k_philox(ctr, key):
    import torch
    out = torch.empty_like(ctr)
    _check(lib().rsd_k_philox(_ptr(ctr), _ptr(key), _ptr(out), ctr.shape[0], _stream()))
    return out
