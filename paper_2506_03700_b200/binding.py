"""ctypes binding of the C-ABI decode library (`include/adadecode.h`).

Argument marshalling only: every step of the decode path runs in the library's CUDA kernels.
PyTorch is used for device memory and the CUDA stream.  There is no CPU fallback: loading fails
loudly when the compiled library is missing.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadadecode.so")
_LIB = None

ADA_MAX_LAYERS = 256
ADA_MAX_BATCH = 16
ERRORS = {0: "ADA_OK", -1: "ADA_EINVAL", -2: "ADA_ESTATE", -3: "ADA_ECAPACITY", -4: "ADA_ECUDA",
          -5: "ADA_ETIMEOUT", -6: "ADA_EUNSUPPORTED"}

SAMPLE_NU = 8   # random numbers per sequence position of a sampling decode call

EXPORTS = [
    "ada_strerror", "ada_last_cuda_error", "ada_model_create", "ada_model_set_tensor", "ada_model_set_exit_head",
    "ada_model_finalize", "ada_model_destroy", "ada_session_scratch_bytes", "ada_kv_page_bytes",
    "ada_session_create", "ada_session_destroy", "ada_session_reset", "ada_prefill", "ada_plain_decode",
    "ada_adaptive_decode", "ada_debug_capture_logits", "ada_debug_logits_captured", "ada_debug_capture_heads",
    "ada_debug_set_exit_tape", "ada_debug_get_state", "ada_debug_read_kv", "ada_debug_set_path",
    "ada_debug_profile", "ada_debug_profile_read", "ada_debug_gemm", "ada_debug_gemm_plan", "ada_debug_gemm_work_bytes", "ada_debug_get_path", "ada_debug_set_launch_steps", "ada_debug_trace", "ada_gemm_noalloc",
    "ada_model_arena_bytes", "ada_model_set_arena", "ada_debug_set_wait_limit", "ada_debug_set_prefill",
    "ada_debug_dense_gemm", "ada_debug_dense_gemm_work_bytes", "ada_sampling_decode",
]


class AdaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = f"{where}: {ERRORS.get(code, code)}"
        try:
            lib = _LIB
            if lib is not None:
                msg += f" ({lib.ada_strerror(code).decode()})"
                if code in (-4, -5, -2) and lib.ada_last_cuda_error():
                    msg += f" [{lib.ada_last_cuda_error().decode()}]"
        except Exception:
            pass
        super().__init__(msg)


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32),
                ("dtype", C.c_int32), ("tied_lm_head", C.c_int32), ("rope_base", C.c_float), ("rms_eps", C.c_float)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in
                ("steps", "head_evals", "early_exits", "verify_steps", "accepted", "rejected", "discarded",
                 "row_layers", "truncated")] + \
               [("exits_at_layer", C.c_int64 * ADA_MAX_LAYERS), ("layer_passes", C.c_int64), ("host_syncs", C.c_int64),
                ("kernel_launches", C.c_int64), ("decode_ms", C.c_double), ("emitted", C.c_int64 * ADA_MAX_BATCH),
                ("finished", C.c_int64), ("path", C.c_int64)]

    def as_dict(self) -> dict:
        d = {n: getattr(self, n) for n, _ in self._fields_ if n not in ("exits_at_layer", "emitted")}
        d["exits_at_layer"] = {i: int(v) for i, v in enumerate(self.exits_at_layer) if v}
        d["emitted"] = [int(v) for v in self.emitted if v]
        return d


def load() -> C.CDLL:
    """Load the compiled library; raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_03700_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.ada_strerror.restype = C.c_char_p
        L.ada_strerror.argtypes = [C.c_int]
        L.ada_last_cuda_error.restype = C.c_char_p
        L.ada_model_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
        L.ada_model_set_tensor.argtypes = [vp, C.c_char_p, vp, sz]
        L.ada_model_set_exit_head.argtypes = [vp, i32, vp, C.c_float]
        L.ada_model_finalize.argtypes = [vp]
        L.ada_model_arena_bytes.restype = sz
        L.ada_model_arena_bytes.argtypes = [vp]
        L.ada_model_set_arena.argtypes = [vp, vp, sz]
        L.ada_debug_set_wait_limit.argtypes = [vp, C.c_uint64]
        L.ada_debug_set_prefill.argtypes = [vp, i32]
        L.ada_debug_dense_gemm_work_bytes.restype = sz
        L.ada_debug_dense_gemm_work_bytes.argtypes = [i32]
        L.ada_debug_dense_gemm.argtypes = [vp, i32, i32, vp, i32, vp, i32, i32, vp, sz, vp]
        L.ada_model_destroy.argtypes = [vp]
        L.ada_model_destroy.restype = None
        L.ada_session_scratch_bytes.restype = sz
        L.ada_session_scratch_bytes.argtypes = [vp, i32, i32, i32]
        L.ada_kv_page_bytes.restype = sz
        L.ada_kv_page_bytes.argtypes = [vp, i32]
        L.ada_session_create.argtypes = [vp, i32, i32, i32, i32, vp, sz, vp, sz, vp, C.POINTER(vp)]
        L.ada_session_destroy.argtypes = [vp]
        L.ada_session_destroy.restype = None
        L.ada_session_reset.argtypes = [vp, i32]
        L.ada_prefill.argtypes = [vp, i32, vp, i32]
        L.ada_plain_decode.argtypes = [vp, i32, i32, vp, C.POINTER(Stats)]
        L.ada_adaptive_decode.argtypes = [vp, i32, C.c_float, vp, i32, i32, i32, vp, C.POINTER(Stats)]
        L.ada_sampling_decode.argtypes = [vp, i32, C.c_float, C.c_float, vp, i32, i32, i32, vp, i32, i32, vp, C.POINTER(Stats)]
        L.ada_debug_capture_logits.argtypes = [vp, vp, i32]
        L.ada_debug_logits_captured.argtypes = [vp, C.POINTER(i32)]
        L.ada_debug_capture_heads.argtypes = [vp, vp, i32, C.POINTER(i32)]
        L.ada_debug_set_exit_tape.argtypes = [vp, vp, i32]
        L.ada_debug_get_state.argtypes = [vp, i32, C.POINTER(i32), vp]
        L.ada_debug_read_kv.argtypes = [vp, i32, i32, i32, i32, vp]
        L.ada_debug_set_path.argtypes = [vp, i32]
        L.ada_debug_get_path.argtypes = [vp, C.POINTER(i32)]
        L.ada_debug_set_launch_steps.argtypes = [vp, i32]
        L.ada_debug_trace.argtypes = [vp, vp, vp, C.c_uint32, i32, i32]
        L.ada_gemm_noalloc.argtypes = [vp, i32, i32, i32, vp, i32, vp, i32, vp]
        L.ada_debug_profile.argtypes = [vp, i32]
        L.ada_debug_profile_read.argtypes = [vp, vp, vp, vp]
        L.ada_debug_gemm_plan.argtypes = [i32, i32, i32, i32, i32, i32, C.POINTER(i32)]
        L.ada_debug_gemm_work_bytes.restype = sz
        L.ada_debug_gemm_work_bytes.argtypes = [i32]
        L.ada_debug_gemm.argtypes = [vp, i32, i32, i32, vp, i32, vp, sz, vp, i32, i32, vp, C.POINTER(C.c_float)]
        _LIB = L
    return _LIB


def _ck(rc: int, where: str):
    if rc != 0:
        raise AdaError(rc, where)


def debug_gemm_plan(N: int, K: int, mode: int, grid: int, cta: int, split: bool = True) -> dict:
    """ada_debug_gemm_plan: the share of CTA `cta` of `grid` in the streaming GEMM (host only, no GPU)."""
    out = (C.c_int32 * 9)()
    _ck(load().ada_debug_gemm_plan(N, K, mode, grid, cta, 1 if split else 0, out), "ada_debug_gemm_plan")
    keys = ("split", "t0", "t1", "n", "ta", "tb", "s0_own_k0", "s0_pub_k1", "sl_k1")
    return dict(zip(keys, list(out)))


def debug_gemm(W, X, mode: int = 0, repeat: int = 1):
    """The weight-streaming GEMM by itself: W bf16 [N, K] (cuda), X fp32 [cols, K] (cuda).
    Returns (Y fp32 [cols, N or N/2], device milliseconds of the kernel)."""
    import torch
    lib = load()
    N, K = W.shape
    cols = X.shape[0]
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.is_contiguous()
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.shape[1] == K
    n_out = N // 2 if mode == 1 else N
    wb = lib.ada_debug_gemm_work_bytes(K)
    work = torch.empty(wb + 256, dtype=torch.uint8, device="cuda")
    off = (-work.data_ptr()) % 256
    Y = torch.zeros(cols, n_out, dtype=torch.float32, device="cuda")
    ms = C.c_float(0.0)
    _ck(lib.ada_debug_gemm(W.data_ptr(), N, K, mode, X.data_ptr(), cols, work.data_ptr() + off, wb, Y.data_ptr(), n_out,
                           repeat, torch.cuda.current_stream().cuda_stream, C.byref(ms)), "ada_debug_gemm")
    return Y, ms.value


def debug_dense_gemm(W, X, Y=None):
    """The dense tcgen05 GEMM of the prompt pass by itself: W bf16 [N, K] (cuda), X fp32 [rows <= 128, K] (cuda).
    Returns Y fp32 [rows, N]; with Y given, the product is added to it in place."""
    import torch
    lib = load()
    N, K = W.shape
    rows = X.shape[0]
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.is_contiguous()
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.shape[1] == K
    acc = Y is not None
    if Y is None:
        Y = torch.full((rows, N), float("nan"), dtype=torch.float32, device="cuda")
    wb = lib.ada_debug_dense_gemm_work_bytes(K)
    work = torch.empty(wb + 256, dtype=torch.uint8, device="cuda")
    off = (-work.data_ptr()) % 256
    _ck(lib.ada_debug_dense_gemm(W.data_ptr(), N, K, X.data_ptr(), rows, Y.data_ptr(), Y.shape[1], 1 if acc else 0,
                                 work.data_ptr() + off, wb, torch.cuda.current_stream().cuda_stream), "ada_debug_dense_gemm")
    return Y


def gemm_noalloc(W, X, Y, mode: int = 0):
    """ada_gemm_noalloc: the streaming GEMM with the library's built-in scratch.  W bf16 [N, K], X
    fp32 [cols, K], Y fp32 [cols, N or N/2], all on the current CUDA device; Y is written in place.
    Nothing is allocated here or in the library."""
    import torch
    N, K = W.shape
    _ck(load().ada_gemm_noalloc(W.data_ptr(), N, K, mode, X.data_ptr(), X.shape[0], Y.data_ptr(), Y.shape[1],
                                torch.cuda.current_stream().cuda_stream), "ada_gemm_noalloc")
    return Y


class Model:
    """ada_model over borrowed torch CUDA tensors: the fused layout of `synth.make_weights` (wqkv,
    w_gate_up) or the separate matrices (wq, wk, wv, w_gate, w_up), as the caller holds them.  The
    arena the library repacks into is allocated here through torch and handed over."""

    def __init__(self, cfg, weights: Dict[str, "torch.Tensor"], tied: Optional[bool] = None):
        import torch
        lib = load()
        self.cfg = cfg
        tied = ("lm_head" not in weights) if tied is None else tied
        c = Config(cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff, cfg.vocab,
                   1 if cfg.dtype == "bf16" else 0, 1 if tied else 0, cfg.rope_base, cfg.rms_eps)
        h = C.c_void_p()
        _ck(lib.ada_model_create(C.byref(c), C.byref(h)), "ada_model_create")
        self.h = h
        self._keep = []
        for name, t in weights.items():
            assert t.is_cuda and t.is_contiguous() and t.dtype == cfg.torch_dtype, name
            self._keep.append(t)
            _ck(lib.ada_model_set_tensor(h, name.encode(), t.data_ptr(), t.numel() * t.element_size()),
                f"ada_model_set_tensor({name})")
        self._finalized = False
        self.arena = None

    def set_exit_head(self, layer: int, T=None, logit_scale: float = 1.0):
        ptr = None
        if T is not None:
            assert T.is_cuda and T.is_contiguous() and T.dtype == self.cfg.torch_dtype
            self._keep.append(T)
            ptr = T.data_ptr()
        _ck(load().ada_model_set_exit_head(self.h, layer, ptr, logit_scale), f"ada_model_set_exit_head({layer})")

    def finalize(self):
        if not self._finalized:
            import torch
            lib = load()
            need = lib.ada_model_arena_bytes(self.h)
            if need:
                self.arena = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
                off = (-self.arena.data_ptr()) % 256
                _ck(lib.ada_model_set_arena(self.h, self.arena.data_ptr() + off, need), "ada_model_set_arena")
            _ck(lib.ada_model_finalize(self.h), "ada_model_finalize")
            self._finalized = True

    def __del__(self):
        try:
            if self.h:
                load().ada_model_destroy(self.h)
                self.h = None
        except Exception:
            pass


class Session:
    """ada_session with its KV pool and scratch allocated through torch on the current device."""

    def __init__(self, model: Model, batch: int = 1, max_seq_len: int = 4096, page_tokens: int = 64,
                 max_early: int = 5, kv_pages: Optional[int] = None, stream=None):
        import torch
        lib = load()
        model.finalize()
        self.model = model
        self.batch = batch
        self.max_seq_len = max_seq_len
        self.vocab = model.cfg.vocab
        page_bytes = lib.ada_kv_page_bytes(model.h, page_tokens)
        if kv_pages is None:
            kv_pages = batch * ((max_seq_len + page_tokens - 1) // page_tokens)
        self.kv_pool = torch.empty(kv_pages * page_bytes, dtype=torch.uint8, device="cuda")
        sb = lib.ada_session_scratch_bytes(model.h, batch, max_seq_len, max_early)
        self.scratch = torch.empty(sb + 256, dtype=torch.uint8, device="cuda")
        off = (-self.scratch.data_ptr()) % 256
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        h = C.c_void_p()
        _ck(lib.ada_session_create(model.h, batch, max_seq_len, page_tokens, max_early, self.kv_pool.data_ptr(),
                                   self.kv_pool.numel(), self.scratch.data_ptr() + off, sb,
                                   self.stream.cuda_stream, C.byref(h)), "ada_session_create")
        self.h = h
        self._capture = None
        self._heads = None
        self._heads_n = C.c_int32(0)

    # ---- the calls of the boundary
    def reset(self, seq: int = -1):
        _ck(load().ada_session_reset(self.h, seq), "ada_session_reset")

    def prefill(self, prompt: Sequence[int], seq: int = 0):
        p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
        _ck(load().ada_prefill(self.h, seq, p.ctypes.data, len(p)), "ada_prefill")

    def plain_decode(self, n_tokens: int, stats: Optional[Stats] = None, out: Optional[np.ndarray] = None,
                     eos_id: int = -1) -> np.ndarray:
        out = np.empty((self.batch, n_tokens), dtype=np.int32) if out is None else out
        _ck(load().ada_plain_decode(self.h, n_tokens, eos_id, out.ctypes.data, C.byref(stats) if stats is not None else None),
            "ada_plain_decode")
        return out

    def adaptive_decode(self, n_tokens: int, threshold: float, exit_layers: Sequence[int], max_early: int = 5,
                        stats: Optional[Stats] = None, out: Optional[np.ndarray] = None, eos_id: int = -1) -> np.ndarray:
        out = np.empty((self.batch, n_tokens), dtype=np.int32) if out is None else out
        ex = np.ascontiguousarray(np.asarray(exit_layers, dtype=np.int32))
        _ck(load().ada_adaptive_decode(self.h, n_tokens, threshold, ex.ctypes.data if len(ex) else None, len(ex),
                                       max_early, eos_id, out.ctypes.data, C.byref(stats) if stats is not None else None),
            "ada_adaptive_decode")
        return out

    def sampling_decode(self, n_tokens: int, temperature: float, threshold: float, exit_layers: Sequence[int],
                        max_early: int, uniforms: np.ndarray, first_pos: int = 0, stats: Optional[Stats] = None,
                        out: Optional[np.ndarray] = None, eos_id: int = -1) -> np.ndarray:
        """`uniforms`: float32 [batch][n_pos][SAMPLE_NU], row j = the random numbers of sequence position first_pos + j."""
        out = np.empty((self.batch, n_tokens), dtype=np.int32) if out is None else out
        ex = np.ascontiguousarray(np.asarray(exit_layers, dtype=np.int32))
        u = np.ascontiguousarray(uniforms, dtype=np.float32)
        if u.ndim != 3 or u.shape[0] != self.batch or u.shape[2] != SAMPLE_NU:
            raise ValueError("uniforms must be [batch][n_pos][%d]" % SAMPLE_NU)
        _ck(load().ada_sampling_decode(self.h, n_tokens, temperature, threshold, ex.ctypes.data if len(ex) else None, len(ex),
                                       max_early, eos_id, u.ctypes.data, first_pos, u.shape[1], out.ctypes.data,
                                       C.byref(stats) if stats is not None else None), "ada_sampling_decode")
        return out

    # ---- test hooks
    def capture_logits(self, max_tokens: int):
        import torch
        self._capture = torch.zeros(max_tokens, self.vocab, dtype=torch.float32, device="cuda")
        _ck(load().ada_debug_capture_logits(self.h, self._capture.data_ptr(), max_tokens), "ada_debug_capture_logits")

    def captured_logits(self):
        n = C.c_int32(0)
        _ck(load().ada_debug_logits_captured(self.h, C.byref(n)), "ada_debug_logits_captured")
        return self._capture[:min(n.value, self._capture.shape[0])]

    def capture_heads(self, max_evals: int = 1 << 16):
        self._heads = np.zeros((max_evals, 4), dtype=np.float32)
        _ck(load().ada_debug_capture_heads(self.h, self._heads.ctypes.data, max_evals, C.byref(self._heads_n)),
            "ada_debug_capture_heads")

    def captured_heads(self) -> np.ndarray:
        """Rows (step, layer, token, p) of the last adaptive call."""
        return self._heads[:min(self._heads_n.value, len(self._heads))]

    def set_exit_tape(self, tape: Sequence[int]):
        t = np.ascontiguousarray(np.asarray(tape, dtype=np.uint8))
        _ck(load().ada_debug_set_exit_tape(self.h, t.ctypes.data if len(t) else None, len(t)), "ada_debug_set_exit_tape")

    def state(self, seq: int = 0):
        ln = C.c_int32(0)
        fill = np.zeros(self.model.cfg.n_layers, dtype=np.int32)
        _ck(load().ada_debug_get_state(self.h, seq, C.byref(ln), fill.ctypes.data), "ada_debug_get_state")
        return ln.value, fill

    def read_kv(self, which: int, layer0: int, pos: int, seq: int = 0) -> np.ndarray:
        c = self.model.cfg
        out = np.zeros(c.n_kv_heads * c.head_dim, dtype=np.float32)
        _ck(load().ada_debug_read_kv(self.h, seq, which, layer0, pos, out.ctypes.data), "ada_debug_read_kv")
        return out

    PROF_CLASSES = ("control", "rmsnorm", "qkv_gemm", "rope_kv", "attention", "o_gemm", "gate_up_gemm", "swiglu",
                    "down_gemm", "lm_head", "head_T", "other")

    def profile(self, on: bool):
        _ck(load().ada_debug_profile(self.h, 1 if on else 0), "ada_debug_profile")

    def profile_read(self) -> dict:
        """class -> dict(ms, launches, bytes) accumulated since profiling was switched on."""
        n = len(self.PROF_CLASSES)
        ms = np.zeros(n, dtype=np.float64)
        la = np.zeros(n, dtype=np.int64)
        by = np.zeros(n, dtype=np.float64)
        _ck(load().ada_debug_profile_read(self.h, ms.ctypes.data, la.ctypes.data, by.ctypes.data), "ada_debug_profile_read")
        return {c: dict(ms=float(ms[i]), launches=int(la[i]), bytes=float(by[i])) for i, c in enumerate(self.PROF_CLASSES)}

    def set_path(self, path: int):
        _ck(load().ada_debug_set_path(self.h, path), "ada_debug_set_path")

    def get_path(self) -> int:
        p = C.c_int32(-1)
        _ck(load().ada_debug_get_path(self.h, C.byref(p)), "ada_debug_get_path")
        return p.value

    def set_launch_steps(self, steps: int):
        _ck(load().ada_debug_set_launch_steps(self.h, steps), "ada_debug_set_launch_steps")

    def set_prefill(self, dense: bool):
        _ck(load().ada_debug_set_prefill(self.h, 1 if dense else 0), "ada_debug_set_prefill")

    def set_wait_limit(self, ns: int):
        _ck(load().ada_debug_set_wait_limit(self.h, ns), "ada_debug_set_wait_limit")

    def trace(self, cap_events: int, step0: int, step1: int):
        """Record the persistent kernel's events of steps [step0, step1) of every following launch
        (`cap_events` per CTA)."""
        import torch
        sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        self._trace = torch.zeros(sms, cap_events, 2, dtype=torch.int64, device="cuda")
        self._trace_n = torch.zeros(sms, dtype=torch.int32, device="cuda")
        _ck(load().ada_debug_trace(self.h, self._trace.data_ptr(), self._trace_n.data_ptr(), cap_events, step0, step1),
            "ada_debug_trace")

    def traced(self) -> np.ndarray:
        """Rows (ns, cta, arg, event) of the recorded events, in time order."""
        n = self._trace_n.cpu().numpy()
        t = self._trace.cpu().numpy()
        t = np.concatenate([t[i, :min(int(n[i]), t.shape[1])] for i in range(t.shape[0])], axis=0)
        code = t[:, 1]
        out = np.stack([t[:, 0], code >> 32, (code >> 8) & 0xffff, code & 0xff], axis=1)
        return out[np.argsort(out[:, 0], kind="stable")]

    def __del__(self):
        try:
            if self.h:
                load().ada_session_destroy(self.h)
                self.h = None
        except Exception:
            pass
