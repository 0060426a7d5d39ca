"""ctypes view of the CPU oracle (`adadecode_oracle.c`).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.  It never
imports the CUDA library or its binding, and holds no arithmetic of its own: every number comes
from the C file.  Inputs are NumPy arrays (fp32, or uint16 holding bf16 bit patterns).
"""

from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_SRC = os.path.join(_HERE, "adadecode_oracle.c")
_LIB = None


NU = 8   # random numbers per sequence position of a sampling decode call


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP across mat-vec output rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fopenmp-simd", "-march=native", "-std=c11", "-shared", "-fPIC",
               "-o", _SO, _SRC, "-lm"]
        subprocess.check_call(cmd)
    return _SO


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ff", C.c_int32),
                ("vocab", C.c_int32), ("wdtype", C.c_int32), ("kv_bf16", C.c_int32), ("rope_base", C.c_double),
                ("rms_eps", C.c_double)]


class LayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ("steps", "head_evals", "early_exits", "verify_steps", "accepted", "rejected",
                 "discarded", "row_layers", "truncated")] + [("exits_at_layer", C.c_int64 * 256)]

    def as_dict(self):
        d = {n: int(getattr(self, n)) for n, _ in self._fields_[:-1]}
        d["exits_at_layer"] = {i: int(v) for i, v in enumerate(self.exits_at_layer) if v}
        return d


def _lib():
    global _LIB
    if _LIB is None:
        build()
        L = C.CDLL(_SO)
        L.orc_model_create.restype = C.c_void_p
        L.orc_model_create.argtypes = [C.POINTER(Config), C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(LayerW)]
        L.orc_model_set_head.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_double]
        L.orc_model_destroy.argtypes = [C.c_void_p]
        L.orc_session_create.restype = C.c_void_p
        L.orc_session_create.argtypes = [C.c_void_p, C.c_int]
        L.orc_session_destroy.argtypes = [C.c_void_p]
        L.orc_session_record_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_session_record_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_session_record_heads.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        for f in ("orc_session_logits_recorded", "orc_session_trace_recorded", "orc_session_heads_recorded",
                  "orc_session_len"):
            getattr(L, f).argtypes = [C.c_void_p]
        L.orc_session_kv_len.argtypes = [C.c_void_p, C.c_int]
        L.orc_session_tokens.restype = C.POINTER(C.c_int32)
        L.orc_session_tokens.argtypes = [C.c_void_p]
        L.orc_session_kv.restype = C.POINTER(C.c_double)
        L.orc_session_kv.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_full_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_hidden_after.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_head_eval.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(C.c_double), C.c_void_p]
        L.orc_plain_decode.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(Stats)]
        L.orc_adaptive_decode.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_void_p, C.c_int, C.c_int,
                                          C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_int32),
                                          C.POINTER(Stats)]
        L.orc_sampling_decode.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_void_p, C.c_int, C.c_int,
                                          C.c_void_p, C.c_int, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(Stats),
                                          C.POINTER(C.c_double)]
        _LIB = L
    return _LIB


def to_numpy(t):
    """torch CPU tensor (fp32 or bf16) -> contiguous NumPy array (fp32, or uint16 bit patterns)."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


class Model:
    """Borrowed-weights oracle model.  `weights` uses the fused layout names
    (tok_embed, final_norm, [lm_head], layers.N.{attn_norm,wqkv,wo,ffn_norm,w_gate_up,w_down})."""

    def __init__(self, cfg, weights: Dict[str, np.ndarray], kv_bf16: Optional[bool] = None):
        lib = _lib()
        self.cfg = cfg
        self._keep = []
        bf16 = cfg.dtype == "bf16"
        want = np.uint16 if bf16 else np.float32

        def ptr(a):
            a = np.ascontiguousarray(a)
            assert a.dtype == want, (a.dtype, want)
            self._keep.append(a)
            return a.ctypes.data

        c = Config(cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff,
                   cfg.vocab, 1 if bf16 else 0, int(bf16 if kv_bf16 is None else kv_bf16), cfg.rope_base, cfg.rms_eps)
        nq, nkv = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
        layers = (LayerW * cfg.n_layers)()
        for l in range(cfg.n_layers):
            p = f"layers.{l}."
            qkv, gu = weights[p + "wqkv"], weights[p + "w_gate_up"]
            layers[l].attn_norm = ptr(weights[p + "attn_norm"])
            layers[l].wq = ptr(qkv[:nq])
            layers[l].wk = ptr(qkv[nq:nq + nkv])
            layers[l].wv = ptr(qkv[nq + nkv:])
            layers[l].wo = ptr(weights[p + "wo"])
            layers[l].ffn_norm = ptr(weights[p + "ffn_norm"])
            layers[l].w_gate = ptr(gu[:cfg.d_ff])
            layers[l].w_up = ptr(gu[cfg.d_ff:])
            layers[l].w_down = ptr(weights[p + "w_down"])
        lm = ptr(weights["lm_head"]) if "lm_head" in weights else None
        self.h = lib.orc_model_create(C.byref(c), ptr(weights["tok_embed"]), lm, ptr(weights["final_norm"]), layers)
        self._want = want

    def set_head(self, layer: int, T: Optional[np.ndarray], scale: float):
        p = None
        if T is not None:
            T = np.ascontiguousarray(T)
            assert T.dtype == self._want
            self._keep.append(T)
            p = T.ctypes.data
        rc = _lib().orc_model_set_head(self.h, layer, p, scale)
        if rc:
            raise ValueError(f"orc_model_set_head({layer}) -> {rc}")

    def full_logits(self, tokens: Sequence[int]) -> np.ndarray:
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        out = np.empty((len(tok), self.cfg.vocab), dtype=np.float64)
        rc = _lib().orc_full_logits(self.h, tok.ctypes.data, len(tok), out.ctypes.data)
        if rc:
            raise RuntimeError(f"orc_full_logits -> {rc}")
        return out

    def hidden_after(self, tokens: Sequence[int], upto_layer: int) -> np.ndarray:
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        out = np.empty(self.cfg.d_model, dtype=np.float64)
        rc = _lib().orc_hidden_after(self.h, tok.ctypes.data, len(tok), upto_layer, out.ctypes.data)
        if rc:
            raise RuntimeError(f"orc_hidden_after -> {rc}")
        return out

    def head_eval(self, layer: int, h: np.ndarray, want_probs: bool = False):
        h = np.ascontiguousarray(h, dtype=np.float64)
        p = C.c_double()
        probs = np.empty(self.cfg.vocab, dtype=np.float64) if want_probs else None
        tok = _lib().orc_head_eval(self.h, layer, h.ctypes.data, C.byref(p), probs.ctypes.data if want_probs else None)
        return (tok, p.value, probs) if want_probs else (tok, p.value)

    def __del__(self):
        try:
            _lib().orc_model_destroy(self.h)
        except Exception:
            pass


class Session:
    def __init__(self, model: Model, max_seq: int):
        self.model = model
        self.max_seq = max_seq
        self.h = _lib().orc_session_create(model.h, max_seq)
        if not self.h:
            raise MemoryError("orc_session_create")
        self._logits = self._trace = self._heads = None

    def record_logits(self, cap: int):
        self._logits = np.zeros((cap, self.model.cfg.vocab), dtype=np.float64)
        _lib().orc_session_record_logits(self.h, self._logits.ctypes.data, cap)

    def record_trace(self, cap: int = 1 << 16):
        self._trace = np.zeros((cap, 4), dtype=np.int32)
        _lib().orc_session_record_trace(self.h, self._trace.ctypes.data, cap)

    def record_heads(self, cap: int = 1 << 16):
        self._heads = np.zeros((cap, 4), dtype=np.float64)
        _lib().orc_session_record_heads(self.h, self._heads.ctypes.data, cap)

    @property
    def logits(self) -> np.ndarray:
        n = min(_lib().orc_session_logits_recorded(self.h), len(self._logits))
        return self._logits[:n]

    @property
    def trace(self) -> np.ndarray:
        """Rows (step, layer, first_pos, n_rows) for every processed layer."""
        n = min(_lib().orc_session_trace_recorded(self.h), len(self._trace))
        return self._trace[:n]

    @property
    def heads(self) -> np.ndarray:
        """Rows (step, layer, token, p) for every intermediate-head evaluation."""
        n = min(_lib().orc_session_heads_recorded(self.h), len(self._heads))
        return self._heads[:n]

    @property
    def len(self) -> int:
        return _lib().orc_session_len(self.h)

    def kv_len(self, layer0: int) -> int:
        return _lib().orc_session_kv_len(self.h, layer0)

    def tokens(self) -> np.ndarray:
        p = _lib().orc_session_tokens(self.h)
        return np.ctypeslib.as_array(p, shape=(self.len,)).copy()

    def kv(self, which: int, layer0: int, pos: int) -> np.ndarray:
        c = self.model.cfg
        p = _lib().orc_session_kv(self.h, which, layer0, pos)
        return np.ctypeslib.as_array(p, shape=(c.n_kv_heads * c.head_dim,)).copy()

    def prefill(self, prompt: Sequence[int]):
        tok = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
        rc = _lib().orc_prefill(self.h, tok.ctypes.data, len(tok))
        if rc:
            raise RuntimeError(f"orc_prefill -> {rc}")

    def plain_decode(self, n: int, stats: Optional[Stats] = None, eos_id: int = -1) -> np.ndarray:
        """Next n greedy tokens; with eos_id >= 0 generation stops at the first such token, `self.emitted`
        holds the number produced and the rest of the row is eos_id."""
        out = np.empty(n, dtype=np.int32)
        got = C.c_int32(0)
        rc = _lib().orc_plain_decode(self.h, n, eos_id, out.ctypes.data, C.byref(got),
                                     C.byref(stats) if stats is not None else None)
        if rc:
            raise RuntimeError(f"orc_plain_decode -> {rc}")
        self.emitted = got.value
        return out

    def adaptive_decode(self, n: int, gamma: float, exit_layers: Sequence[int], max_early: int = 5,
                        tape: Optional[Sequence[int]] = None, tape_tok: Optional[Sequence[int]] = None,
                        stats: Optional[Stats] = None, eos_id: int = -1) -> np.ndarray:
        out = np.empty(n, dtype=np.int32)
        got = C.c_int32(0)
        ex = np.ascontiguousarray(np.asarray(exit_layers, dtype=np.int32))
        n_tape = 0
        tp = tt = None
        if tape is not None:
            tp = np.ascontiguousarray(np.asarray(tape, dtype=np.uint8))
            n_tape = len(tp)
        if tape_tok is not None:
            tt = np.ascontiguousarray(np.asarray(tape_tok, dtype=np.int32))
            n_tape = max(n_tape, len(tt))
            if tp is None:
                tp = np.full(n_tape, 2, dtype=np.uint8)
            assert len(tp) == len(tt)
        rc = _lib().orc_adaptive_decode(self.h, n, gamma, ex.ctypes.data, len(ex), max_early,
                                        tp.ctypes.data if tp is not None else None,
                                        tt.ctypes.data if tt is not None else None, n_tape, eos_id,
                                        out.ctypes.data, C.byref(got), C.byref(stats) if stats is not None else None)
        if rc:
            raise RuntimeError(f"orc_adaptive_decode -> {rc}")
        self.emitted = got.value
        return out

    def sampling_decode(self, n: int, temperature: float, gamma: float, exit_layers: Sequence[int], max_early: int,
                        uniforms: np.ndarray, stats: Optional[Stats] = None, eos_id: int = -1) -> np.ndarray:
        """Algorithm 1 with sampled tokens (Eq. 1) and the acceptance test and resampling of Eq. 2.
        `uniforms[pos][k]`, float64 in [0, 1), k < NU: the random numbers of the token at sequence position pos
        ([0] draw at the last layer, [1] acceptance test, [2] resampling, [3 + e] draw at the e-th exit layer)."""
        out = np.empty(n, dtype=np.int32)
        got = C.c_int32(0)
        ex = np.ascontiguousarray(np.asarray(exit_layers, dtype=np.int32))
        u = np.ascontiguousarray(np.asarray(uniforms, dtype=np.float64))
        assert u.ndim == 2 and u.shape[1] == NU and u.shape[0] >= self.max_seq
        margin = C.c_double(1.0)
        rc = _lib().orc_sampling_decode(self.h, n, temperature, gamma, ex.ctypes.data, len(ex), max_early,
                                        u.ctypes.data, eos_id, out.ctypes.data, C.byref(got),
                                        C.byref(stats) if stats is not None else None, C.byref(margin))
        if rc:
            raise RuntimeError(f"orc_sampling_decode -> {rc}")
        self.emitted = got.value
        self.min_margin = margin.value   # smallest distance (in probability) of any random decision of the call from flipping
        return out

    def __del__(self):
        try:
            _lib().orc_session_destroy(self.h)
        except Exception:
            pass


def model_from_torch(cfg, weights, kv_bf16: Optional[bool] = None) -> Model:
    """Build an oracle model from the torch tensors of the input generator (moved to the CPU).
    kv_bf16 None: the cache holds bf16 exactly when the model is a bf16 model."""
    return Model(cfg, {k: to_numpy(v) for k, v in weights.items()}, kv_bf16=kv_bf16)
