"""Pins for the oracle's decoder: an independent NumPy restatement, closed forms, incremental
decoding against from-scratch recompute, and the intermediate head's definition."""

import numpy as np
import pytest
import torch

import oracle
from paper_2506_03700_b200 import synth
from helpers import make_oracle, np_decoder_logits, widen


@pytest.mark.parametrize("dtype,tied,kv,kv_bf16", [("fp32", True, 2, False), ("bf16", False, 6, False),
                                                    ("fp32", False, 1, False), ("bf16", True, 2, True)])
def test_logits_match_numpy_restatement(dtype, tied, kv, kv_bf16):
    """kv_bf16: the bf16 configurations keep K/V in a bf16 cache; the restatement rounds them with
    torch's conversion, the oracle with its own bit arithmetic."""
    cfg = synth.small_config(dtype=dtype, n_kv_heads=kv, resid_scale=1.0, sigma=0.1)
    w, m = make_oracle(cfg, tied=tied, heads=False, kv_bf16=kv_bf16)
    W = {k: widen(v) for k, v in w.items()}
    toks = synth.make_prompt(cfg, n=13).numpy()
    ref = np_decoder_logits(cfg, W, toks, kv_bf16=kv_bf16)
    if kv_bf16:   # the rounding is not a no-op on this model
        assert np.abs(ref - np_decoder_logits(cfg, W, toks)).max() > 1e-6
    got = m.full_logits(toks)
    assert np.abs(got - ref).max() < 1e-10 * max(1.0, np.abs(ref).max())
    # hidden state after an intermediate layer
    h = m.hidden_after(toks, 2)
    href = np_decoder_logits(cfg, W, toks, upto_layer=2, return_hidden=True, kv_bf16=kv_bf16)[-1]
    assert np.abs(h - href).max() < 1e-11


def test_zero_output_projections_leave_residual_stream():
    """W_o = W_down = 0  =>  logits = E* RMSNorm_f(embed(token)), whatever the context."""
    cfg = synth.small_config()
    w = synth.make_weights(cfg, norm_gain_jitter=0.1)
    for l in range(cfg.n_layers):
        w[f"layers.{l}.wo"].zero_()
        w[f"layers.{l}.w_down"].zero_()
    m = oracle.model_from_torch(cfg, w)
    toks = synth.make_prompt(cfg, n=5).numpy()
    got = m.full_logits(toks)
    E, g = widen(w["tok_embed"]), widen(w["final_norm"])
    x = E[toks]
    ref = (x / np.sqrt((x * x).mean(-1, keepdims=True) + cfg.rms_eps) * g) @ E.T
    assert np.abs(got - ref).max() < 1e-12


def test_single_position_attention_is_value_passthrough():
    """One token, one layer: softmax over one score is 1, so h = e + W_o W_v n1 + FFN(...);
    rotary angles are zero at position 0."""
    cfg = synth.small_config(n_layers=1, exit_layers=())
    w = synth.make_weights(cfg, norm_gain_jitter=0.1)
    m = oracle.model_from_torch(cfg, w)
    W = {k: widen(v) for k, v in w.items()}
    tok = 17
    e = W["tok_embed"][tok]
    rms = lambda x, g: x / np.sqrt((x * x).mean() + cfg.rms_eps) * g
    nq, nkv = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    v = W["layers.0.wqkv"][nq + nkv:] @ rms(e, W["layers.0.attn_norm"])
    att = np.repeat(v.reshape(cfg.n_kv_heads, cfg.head_dim), cfg.n_q_heads // cfg.n_kv_heads, axis=0).reshape(-1)
    h = e + W["layers.0.wo"] @ att
    gu = W["layers.0.w_gate_up"] @ rms(h, W["layers.0.ffn_norm"])
    g, u = gu[:cfg.d_ff], gu[cfg.d_ff:]
    h = h + W["layers.0.w_down"] @ (g / (1 + np.exp(-g)) * u)
    got = m.hidden_after([tok], 1)
    assert np.abs(got - h).max() < 1e-13


def test_zero_query_gives_uniform_attention():
    """W_q = 0 => all scores equal => attention output is the running mean of V."""
    cfg = synth.small_config(n_layers=1, exit_layers=())
    w = synth.make_weights(cfg)
    nq, nkv = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    w["layers.0.wqkv"][:nq].zero_()
    w["layers.0.w_down"].zero_()
    m = oracle.model_from_torch(cfg, w)
    W = {k: widen(v) for k, v in w.items()}
    toks = synth.make_prompt(cfg, n=6).numpy()
    x = W["tok_embed"][toks]
    a = x / np.sqrt((x * x).mean(-1, keepdims=True) + cfg.rms_eps) * W["layers.0.attn_norm"]
    v = a @ W["layers.0.wqkv"][nq + nkv:].T
    vmean = v.mean(0).reshape(cfg.n_kv_heads, cfg.head_dim)
    att = np.repeat(vmean, cfg.n_q_heads // cfg.n_kv_heads, axis=0).reshape(-1)
    h = x[-1] + W["layers.0.wo"] @ att
    got = m.hidden_after(toks, 1)
    assert np.abs(got - h).max() < 1e-13


def test_incremental_decode_equals_from_scratch():
    """KV-cache decoding: logits of each generated token equal the from-scratch logits of the
    whole prefix, and greedy tokens equal the from-scratch argmax."""
    cfg = synth.small_config(resid_scale=1.0)
    w, m = make_oracle(cfg, heads=False)
    prompt = synth.make_prompt(cfg, n=9).numpy()
    s = oracle.Session(m, 64)
    s.record_logits(32)
    s.prefill(prompt)
    out = s.plain_decode(12)
    seq = np.concatenate([prompt, out])
    full = m.full_logits(seq)
    for i in range(12):
        ref = full[len(prompt) - 1 + i]
        assert np.abs(s.logits[i] - ref).max() < 1e-11
        assert out[i] == int(np.argmax(ref))
    # chained calls continue the same sequence
    s2 = oracle.Session(m, 64)
    s2.prefill(prompt)
    a = s2.plain_decode(5)
    b = s2.plain_decode(7)
    assert np.array_equal(np.concatenate([a, b]), out)


def test_head_is_softmax_of_scaled_transformed_logits():
    """Section 2.1: p = softmax(h E^(i)T), E^(i) = E* T^(i).  Probabilities sum to one, the
    reported p is their maximum, and with T = I the head's token equals the argmax of the
    final-norm + LM-head logits of the same hidden state for any positive scale."""
    cfg = synth.small_config(dtype="fp32")
    w, m = make_oracle(cfg, heads=False)
    W = {k: widen(v) for k, v in w.items()}
    h = synth.standard_normal(7, 1, cfg.d_model).numpy()
    E, g = W["tok_embed"], W["final_norm"]
    xn = h / np.sqrt((h * h).mean() + cfg.rms_eps) * g
    z = E @ xn
    for scale in (1.0, 8.0):
        m.set_head(1, None, scale)
        tok, p, probs = m.head_eval(1, h, want_probs=True)
        assert abs(probs.sum() - 1.0) < 1e-12
        assert tok == int(np.argmax(z)) and abs(p - probs.max()) < 1e-15
        e = np.exp(scale * z - (scale * z).max())
        assert np.abs(probs - e / e.sum()).max() < 1e-14
    # dense T: logits = s * E (T xn); a scaled identity T equals the same logit scale (Lemma A.1's
    # decomposition with T = s I), and a random T matches the explicit product E T.
    T = synth.make_head_transform(cfg, 2, noise=0.5)
    m.set_head(2, oracle.to_numpy(T), 3.0)
    tok, p, probs = m.head_eval(2, h, want_probs=True)
    z2 = 3.0 * ((E @ widen(T)) @ xn)
    e = np.exp(z2 - z2.max())
    assert np.abs(probs - e / e.sum()).max() < 1e-13 and tok == int(np.argmax(z2))
    Ts = (torch.eye(cfg.d_model) * 4.0).to(cfg.torch_dtype)
    m.set_head(1, oracle.to_numpy(Ts), 2.0)
    tok_a, p_a = m.head_eval(1, h)
    m.set_head(1, None, 8.0)
    tok_b, p_b = m.head_eval(1, h)
    assert tok_a == tok_b and abs(p_a - p_b) < 1e-12
