"""Shared test helpers: an independent NumPy restatement of the decoder (used to pin the
oracle) and small conveniences.  Nothing here is imported by the oracle or the CUDA path."""

import numpy as np
from scipy import stats as sps
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


# ---- sampled decoding: the closed-form law of a verified token, from the oracle's forward pass alone

def tempered(p, temperature):
    w = np.power(p, 1.0 / temperature)
    return w / w.sum()


def head_and_final_distributions(cfg, m, tokens, temperature):
    """q_i (one per exit layer) and p* for the successor of tokens[-1], from the oracle's forward pass only."""
    qs = []
    for l in cfg.exit_layers:
        h = m.hidden_after(tokens, l)
        _, _, probs = m.head_eval(l, h, want_probs=True)
        qs.append(tempered(np.asarray(probs), temperature))
    z = m.full_logits(tokens)[-1]
    p = np.exp((z - z.max()) / temperature)
    return qs, p / p.sum()


def law_of_a_verified_token(qs, pstar, gamma):
    """Law of the verified successor when every exit head is consulted in turn (derivation: a head's draw t is
    used iff q(t) > gamma, then accepted with probability min(1, p*(t)/q(t)) or replaced by a draw from the
    normalised positive part of p* - q; if no head emits, the token is drawn from p*)."""
    out = np.zeros_like(pstar)
    reach = 1.0
    for q in qs:
        emit = q > gamma
        acc = np.where(emit, np.minimum(q, pstar), 0.0)
        rej_mass = np.where(emit, q - np.minimum(q, pstar), 0.0).sum()
        res = np.maximum(0.0, pstar - q)
        res = res / res.sum() if res.sum() > 0 else pstar
        out += reach * (acc + rej_mass * res)
        reach *= 1.0 - q[emit].sum()
    return out + reach * pstar


def chi2_ok(counts, law, alpha=1e-4):
    n = counts.sum()
    exp = law * n
    big = exp >= 5
    obs = np.append(counts[big], counts[~big].sum())
    ex = np.append(exp[big], exp[~big].sum())
    if ex[-1] == 0:
        obs, ex = obs[:-1], ex[:-1]
    stat = ((obs - ex) ** 2 / ex).sum()
    return stat <= sps.chi2.ppf(1 - alpha, len(ex) - 1), stat
