"""Shared test helpers: an independent NumPy restatement of the decoder (used to pin the
oracle) and small conveniences.  Nothing here is imported by the oracle or the CUDA path."""

import numpy as np
import torch

from paper_2506_03700_b200 import synth


def widen(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16 through torch's own conversion (fp64 -> fp32 -> bf16)."""
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def np_decoder_logits(cfg, W, tokens, upto_layer=None, return_hidden=False, kv_bf16=False):
    """Final logits of every position, whole sequence at once, written with matrix ops, a
    causal mask and complex-number rotary embedding (a different formulation from the
    oracle's loops).  W: name -> float64 array in the fused layout."""
    tokens = np.asarray(tokens)
    n, hd = len(tokens), cfg.head_dim
    Hq, Hkv = cfg.n_q_heads, cfg.n_kv_heads
    nq, nkv, ff = Hq * hd, Hkv * hd, cfg.d_ff
    half = hd // 2
    inv = cfg.rope_base ** (-2.0 * np.arange(half) / hd)
    rot = np.exp(1j * np.arange(n)[:, None] * inv[None, :])

    def rms(x, g):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + cfg.rms_eps) * g

    def rope(t):
        z = (t[..., :half] + 1j * t[..., half:]) * rot[:, None, :]
        return np.concatenate([z.real, z.imag], -1)

    x = W["tok_embed"][tokens]
    L = cfg.n_layers if upto_layer is None else upto_layer
    for l in range(L):
        p = f"layers.{l}."
        a = rms(x, W[p + "attn_norm"])
        qkv = a @ W[p + "wqkv"].T
        q = rope(qkv[:, :nq].reshape(n, Hq, hd))
        k = rope(qkv[:, nq:nq + nkv].reshape(n, Hkv, hd))
        v = qkv[:, nq + nkv:].reshape(n, Hkv, hd)
        if kv_bf16:     # the cache holds bf16: K (rotated) and V are rounded when written
            k, v = bf16_round(k), bf16_round(v)
        k = np.repeat(k, Hq // Hkv, axis=1)
        v = np.repeat(v, Hq // Hkv, axis=1)
        s = np.einsum("qhd,khd->hqk", q, k) / np.sqrt(hd)
        s = s + np.triu(np.full((n, n), -np.inf), 1)[None]
        s = np.exp(s - s.max(-1, keepdims=True))
        pr = s / s.sum(-1, keepdims=True)
        o = np.einsum("hqk,khd->qhd", pr, v).reshape(n, nq)
        x = x + o @ W[p + "wo"].T
        b = rms(x, W[p + "ffn_norm"])
        gu = b @ W[p + "w_gate_up"].T
        g, u = gu[:, :ff], gu[:, ff:]
        x = x + ((g / (1.0 + np.exp(-g))) * u) @ W[p + "w_down"].T
    if return_hidden:
        return x
    E = W["lm_head"] if "lm_head" in W else W["tok_embed"]
    return rms(x, W["final_norm"]) @ E.T


def make_oracle(cfg, seed=1234, tied=True, jitter=0.05, heads=True, scale=None, kv_bf16=None, **kw):
    """(weights dict of torch tensors, oracle Model) with heads registered at cfg.exit_layers."""
    import oracle
    w = synth.make_weights(cfg, seed=seed, tied=tied, norm_gain_jitter=jitter)
    m = oracle.model_from_torch(cfg, w, kv_bf16=kv_bf16)
    if heads:
        for l in cfg.exit_layers:
            m.set_head(l, None, cfg.logit_scale if scale is None else scale)
    return w, m
