"""The seeded input generators: determinism, distribution, layout."""

import numpy as np
import torch

from paper_2506_03700_b200 import synth


def test_normal_draws_are_deterministic_and_standard():
    a = synth.standard_normal(11, 3, 1 << 18)
    b = synth.standard_normal(11, 3, 1 << 18)
    assert torch.equal(a, b)
    # chunked generation gives the same stream
    c = torch.cat([synth.standard_normal(11, 3, 1000, start=0), synth.standard_normal(11, 3, 500, start=1000)])
    assert torch.equal(c, a[:1500])
    assert abs(a.mean().item()) < 0.01 and abs(a.std().item() - 1.0) < 0.01
    assert abs((a ** 4).mean().item() - 3.0) < 0.1
    assert not torch.equal(a, synth.standard_normal(12, 3, 1 << 18))
    assert not torch.equal(a, synth.standard_normal(11, 4, 1 << 18))


def test_weight_layout_and_scales():
    cfg = synth.CONFIGS["tiny"]
    w = synth.make_weights(cfg)
    d, hd = cfg.d_model, cfg.head_dim
    assert w["tok_embed"].shape == (cfg.vocab, d) and "lm_head" not in w
    assert w["layers.0.wqkv"].shape == ((cfg.n_q_heads + 2 * cfg.n_kv_heads) * hd, d)
    assert w["layers.3.w_gate_up"].shape == (2 * cfg.d_ff, d)
    assert w["layers.1.w_down"].shape == (d, cfg.d_ff)
    assert abs(w["layers.0.wqkv"].std().item() - 0.02) < 1e-3
    assert abs(w["layers.0.wo"].std().item() - 0.002) < 1e-4        # o_proj scaled by 0.1
    assert abs(w["layers.2.w_down"].std().item() - 0.002) < 1e-4    # down_proj scaled by 0.1
    assert torch.all(w["final_norm"] == 1) and torch.all(w["layers.0.attn_norm"] == 1)
    # chunk size does not change the values
    t1 = synth.normal_tensor(5, 9, (3, 1000), 0.02, torch.bfloat16, chunk=128)
    t2 = synth.normal_tensor(5, 9, (3, 1000), 0.02, torch.bfloat16)
    assert torch.equal(t1, t2)


def test_prompts_are_uniform_ids():
    cfg = synth.CONFIGS["1b"]
    p = synth.make_prompt(cfg)
    assert p.dtype == torch.int32 and len(p) == 512
    assert int(p.min()) >= 0 and int(p.max()) < cfg.vocab
    assert len(torch.unique(p)) > 500
    assert not torch.equal(p, synth.make_prompt(cfg, seq=1))
    lens = synth.batch_prompt_lengths(synth.CONFIGS["13b"])
    assert len(lens) == 4 and all(256 <= n <= 2048 for n in lens)
