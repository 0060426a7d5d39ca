"""Seeded synthetic inputs: Llama-shaped weights and uniform-random prompts.

This module generates inputs only.  It holds none of the decoder's or the
decoding method's arithmetic, and it is the one module that both the CUDA
path's harness and the CPU oracle's harness use, so that both sides see the
same numbers.

Generator.  Element `i` of tensor stream `t` under seed `s` is

    bits = mix64(s, t, i)                      (integer-only, wrapping int64)
    w    = sigma * scale_t * Q(bits)

where `Q` maps the top 16 bits to a cell of a 65537-entry table of standard
normal quantiles (computed once on the CPU in float64) and interpolates
linearly inside the cell with the next 16 bits.  Hash, gather and the
interpolation use only integer ops and single IEEE float64 multiplies and adds,
so a tensor generated on `cuda` equals the one generated on `cpu` bit for bit.
bf16 tensors are rounded once (round-to-nearest-even) at generation.

The configurations follow the paper's model family (Llama-style decoders:
Section 3 names Llama-3.1-8B and CodeLlama-13B/34B); the datasets, checkpoints
and trained heads of the paper are replaced by these synthetic stand-ins.
"""

from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import torch

_MASK64 = (1 << 64) - 1


def _i64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_C1 = _i64(0xBF58476D1CE4E5B9)
_C2 = _i64(0x94D049BB133111EB)
_GOLD = _i64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def mix64(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """Counter-based 64-bit hash (splitmix64 finaliser over seed, stream, index)."""
    key = _i64((seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D))
    x = idx * _GOLD + key
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    x = x ^ _lsr(x, 31)
    return x


_TABLE: Optional[torch.Tensor] = None


def _quantile_table() -> torch.Tensor:
    global _TABLE
    if _TABLE is None:
        j = torch.arange(65537, dtype=torch.float64)
        _TABLE = torch.special.ndtri((j + 0.5) / 65537.0)
    return _TABLE


def standard_normal(seed: int, stream: int, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """`n` float64 standard-normal draws for counters start..start+n-1."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    bits = mix64(seed, stream, idx)
    cell = _lsr(bits, 48)
    frac = (_lsr(bits, 32) & 0xFFFF).to(torch.float64) * (1.0 / 65536.0)
    tab = _quantile_table().to(device)
    lo = tab[cell]
    hi = tab[cell + 1]
    d = hi - lo
    d = d * frac
    return lo + d


def normal_tensor(seed: int, stream: int, shape, sigma: float, dtype: torch.dtype, device="cpu",
                  out: Optional[torch.Tensor] = None, chunk: int = 1 << 24) -> torch.Tensor:
    """Tensor of N(0, sigma^2) draws in `dtype`, generated in chunks to bound temporaries."""
    n = 1
    for s in shape:
        n *= int(s)
    if out is None:
        out = torch.empty(n, dtype=dtype, device=device)
    flat = out.view(-1)
    assert flat.numel() == n
    for st in range(0, n, chunk):
        m = min(chunk, n - st)
        z = standard_normal(seed, stream, m, device=device, start=st)
        flat[st:st + m] = (z * sigma).to(dtype)
    return out.view(*shape)


def uniform_ids(seed: int, stream: int, n: int, vocab: int) -> torch.Tensor:
    """`n` token ids, uniform in [0, vocab), int32 on the CPU."""
    idx = torch.arange(n, dtype=torch.int64)
    bits = _lsr(mix64(seed, stream, idx), 11)
    return (bits % vocab).to(torch.int32)


@dataclasses.dataclass
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str            # "fp32" | "bf16"
    rope_base: float
    rms_eps: float = 1e-5
    resid_scale: float = 0.2   # multiplier on o_proj and down_proj
    sigma: float = 0.02
    exit_layers: tuple = ()
    logit_scale: float = 8.0   # intermediate-head logit scale s
    threshold: float = 0.8
    prompt_len: int = 16
    gen_len: int = 128
    batch: int = 1

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim


CONFIGS: Dict[str, ModelConfig] = {
    "tiny": ModelConfig("tiny", 4, 256, 4, 4, 64, 688, 2048, "fp32", 10000.0, resid_scale=0.1,
                        exit_layers=(2, 3), threshold=0.8, prompt_len=16, gen_len=128),
    "1b": ModelConfig("1b", 16, 2048, 32, 8, 64, 8192, 128256, "bf16", 500000.0,
                      exit_layers=(8, 12), threshold=0.8, prompt_len=512, gen_len=1024),
    "8b": ModelConfig("8b", 32, 4096, 32, 8, 128, 14336, 128256, "bf16", 500000.0,
                      exit_layers=(16, 20, 24, 28), threshold=0.8, prompt_len=1024, gen_len=2048),
    "8b-long": ModelConfig("8b-long", 32, 4096, 32, 8, 128, 14336, 128256, "bf16", 500000.0,
                           exit_layers=(16, 20, 24, 28), threshold=0.9, prompt_len=8192, gen_len=4096),
    "13b": ModelConfig("13b", 40, 5120, 40, 40, 128, 13824, 32000, "bf16", 10000.0,
                       exit_layers=(20, 25, 30, 35), threshold=0.8, prompt_len=2048, gen_len=1024, batch=4),
}


def small_config(name="small", **kw) -> ModelConfig:
    """A small odd-shaped config for unit tests (several tiles and ragged tails)."""
    base = dict(n_layers=3, d_model=192, n_q_heads=6, n_kv_heads=2, head_dim=32, d_ff=328, vocab=1000,
                dtype="fp32", rope_base=10000.0, resid_scale=0.1, exit_layers=(1, 2), prompt_len=7, gen_len=24)
    base.update(kw)
    return ModelConfig(name, **base)


# Stream ids: one per tensor, so tensors are independent of each other and of the layer count.
_S_EMBED, _S_LMHEAD, _S_PROMPT = 1, 2, 3
_PER_LAYER = {"wq": 0, "wk": 1, "wv": 2, "wo": 3, "w_gate": 4, "w_up": 5, "w_down": 6}


def _layer_stream(layer: int, which: str) -> int:
    return 1000 + 16 * layer + _PER_LAYER[which]


def make_weights(cfg: ModelConfig, seed: int = 1234, device="cpu", tied: bool = True,
                 norm_gain_jitter: float = 0.0) -> Dict[str, torch.Tensor]:
    """All tensors of a synthetic model, in the fused layout the CUDA library borrows.

    Returned names: tok_embed [V,d]; final_norm [d]; (lm_head [V,d] if not tied); per layer N:
    layers.N.attn_norm [d], layers.N.wqkv [(nq+2nkv)*hd, d] (q rows, then k, then v),
    layers.N.wo [d, nq*hd], layers.N.ffn_norm [d], layers.N.w_gate_up [2*d_ff, d] (gate rows,
    then up rows), layers.N.w_down [d, d_ff].  All row-major [out, in].
    `norm_gain_jitter` > 0 draws gains 1 + jitter*N(0,1) (tests use it so that a dropped gain
    shows); the benchmark configurations use gains of exactly 1.
    """
    dt = cfg.torch_dtype
    d, hd = cfg.d_model, cfg.head_dim
    nq, nkv = cfg.n_q_heads * hd, cfg.n_kv_heads * hd
    sg = cfg.sigma
    w: Dict[str, torch.Tensor] = {}
    w["tok_embed"] = normal_tensor(seed, _S_EMBED, (cfg.vocab, d), sg, dt, device)
    if not tied:
        w["lm_head"] = normal_tensor(seed, _S_LMHEAD, (cfg.vocab, d), sg, dt, device)

    def gain(stream):
        if norm_gain_jitter == 0.0:
            return torch.ones(d, dtype=dt, device=device)
        z = standard_normal(seed, stream, d, device=device)
        return (1.0 + norm_gain_jitter * z).to(dt)

    w["final_norm"] = gain(900)
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        w[p + "attn_norm"] = gain(_layer_stream(l, "wq") + 8)
        w[p + "ffn_norm"] = gain(_layer_stream(l, "wq") + 9)
        qkv = torch.empty(nq + 2 * nkv, d, dtype=dt, device=device)
        normal_tensor(seed, _layer_stream(l, "wq"), (nq, d), sg, dt, device, out=qkv[:nq])
        normal_tensor(seed, _layer_stream(l, "wk"), (nkv, d), sg, dt, device, out=qkv[nq:nq + nkv])
        normal_tensor(seed, _layer_stream(l, "wv"), (nkv, d), sg, dt, device, out=qkv[nq + nkv:])
        w[p + "wqkv"] = qkv
        w[p + "wo"] = normal_tensor(seed, _layer_stream(l, "wo"), (d, nq), sg * cfg.resid_scale, dt, device)
        gu = torch.empty(2 * cfg.d_ff, d, dtype=dt, device=device)
        normal_tensor(seed, _layer_stream(l, "w_gate"), (cfg.d_ff, d), sg, dt, device, out=gu[:cfg.d_ff])
        normal_tensor(seed, _layer_stream(l, "w_up"), (cfg.d_ff, d), sg, dt, device, out=gu[cfg.d_ff:])
        w[p + "w_gate_up"] = gu
        w[p + "w_down"] = normal_tensor(seed, _layer_stream(l, "w_down"), (d, cfg.d_ff),
                                        sg * cfg.resid_scale, dt, device)
    return w


def make_head_transform(cfg: ModelConfig, layer: int, seed: int = 1234, device="cpu",
                        noise: float = 0.0) -> torch.Tensor:
    """A dense d x d head transformation T = I + noise * N(0, 1/d) for exit layer `layer`."""
    d = cfg.d_model
    t = torch.eye(d, dtype=torch.float64, device=device)
    if noise != 0.0:
        z = standard_normal(seed, 5000 + layer, d * d, device=device).view(d, d)
        t = t + z * (noise / d ** 0.5)
    return t.to(cfg.torch_dtype)


def make_prompt(cfg: ModelConfig, seed: int = 5678, n: Optional[int] = None, seq: int = 0) -> torch.Tensor:
    """Uniform-random prompt ids (int32, CPU) for sequence `seq` of a batch."""
    n = cfg.prompt_len if n is None else n
    return uniform_ids(seed, _S_PROMPT + 7 * seq, n, cfg.vocab)


def batch_prompt_lengths(cfg: ModelConfig, seed: int = 5678, lo: int = 256, hi: int = 2048) -> List[int]:
    """Per-sequence prompt lengths, uniform in [lo, hi] (the ragged batch configuration)."""
    r = uniform_ids(seed, 77, cfg.batch, hi - lo + 1)
    return [lo + int(v) for v in r]
