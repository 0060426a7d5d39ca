"""Sampled decoding on the persistent path (Eq. 1 with a drawn token, Eq. 2 with the acceptance test and the
resampling) against the oracle.

Given the same random numbers the two sides take the same decisions unless a number falls within rounding of
a boundary of the CDF (the GPU's bf16-model probabilities differ from the oracle's by a few 1e-3).  The
exact comparison therefore uses peaked distributions (temperature 0.25: a handful of tokens with wide
intervals) and random numbers chosen, with the oracle alone, so that every decision of the oracle's run keeps
a distance of at least MARGIN from flipping; then tokens and counters must be identical.  Independently of
that, the law of a verified token at temperature 1.2 is compared by chi-square with its closed form."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2506_03700_b200 import binding, synth
from helpers import chi2_ok, head_and_final_distributions, law_of_a_verified_token
from test_gpu_parity import Pair
from test_gpu_persistent import gqa, hd128, mha

MARGIN = 0.012   # in probability; the head-probability error of these models stays below 1e-2
NU = binding.SAMPLE_NU
assert NU == oracle.NU


def _numbers_with_margin(pair, prompt, n, temperature, gamma, exits, max_early, max_seq, eos_id=-1, tries=400, seed0=0):
    """Random numbers (float32, used by both sides) for which every decision of the oracle's run is at least MARGIN
    away from flipping; returns them with the oracle's tokens, counters and session."""
    for seed in range(seed0, seed0 + tries):
        u = np.random.default_rng(seed).random((max_seq, NU), dtype=np.float32)
        s = pair.cpu(max_seq)
        s.prefill(prompt)
        st = oracle.Stats()
        out = s.sampling_decode(n, temperature, gamma, exits, max_early, u.astype(np.float64), stats=st, eos_id=eos_id)
        if s.min_margin >= MARGIN:
            s.seed = seed
            return u, out, st, s
    raise AssertionError("no seed keeps every decision away from the boundaries")


# o/down scale 0.1: the heads agree with the full model (acceptances); 0.25: they mostly do not (rejections, resampling)
CASES = [(gqa, 0.25, 0.05, 0.1), (hd128, 0.25, 0.2, 0.25), (hd128, 0.25, 0.2, 0.1), (mha, 0.25, 0.0, 0.1)]


@pytest.mark.parametrize("mk,temperature,gamma,resid_scale", CASES)
def test_same_numbers_same_decisions(mk, temperature, gamma, resid_scale):
    cfg = mk(logit_scale=2.0, resid_scale=resid_scale)
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=19).numpy()
    n, max_seq, max_early = 16, 64, 3
    u, want, ost, osess = _numbers_with_margin(pair, prompt, n, temperature, gamma, cfg.exit_layers, max_early, max_seq)
    S = binding.Session(pair.gm, 1, max_seq, 64, max_early)
    assert S.get_path() == 1
    S.prefill(prompt)
    st = binding.Stats()
    got = S.sampling_decode(n, temperature, gamma, cfg.exit_layers, max_early, u[None], 0, st)[0]
    assert np.array_equal(got, want), (got, want)
    for f in ("steps", "head_evals", "early_exits", "verify_steps", "accepted", "rejected", "discarded", "truncated", "row_layers"):
        assert getattr(st, f) == getattr(ost, f), f
    assert st.early_exits > 0 and (st.accepted > 0 if resid_scale < 0.2 else st.rejected > 3)
    ln, fill = S.state(0)
    assert ln == len(prompt) + n and (fill == len(prompt) + n - 1).all()
    # the cache behind a sampled run is the cache of its tokens: greedy continuation equals the oracle's
    more = S.plain_decode(6)[0]
    assert np.array_equal(more, osess.plain_decode(6))


def test_plain_sampling_chained_calls_and_end_of_sequence():
    cfg = hd128(logit_scale=2.0, resid_scale=0.25)
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=33).numpy()
    n, max_seq = 20, 96
    # no exit layers: every token is an inverse-CDF draw from the full model's distribution
    u, want, ost, _ = _numbers_with_margin(pair, prompt, n, 0.25, 0.5, (), 3, max_seq)
    assert len(set(want.tolist())) > 4
    S = binding.Session(pair.gm, 1, max_seq, 64, 3)
    S.prefill(prompt)
    st = binding.Stats()
    a = S.sampling_decode(8, 0.25, 0.5, (), 3, u[None], 0, st)[0]
    b = S.sampling_decode(n - 8, 0.25, 0.5, (), 3, u[None, len(prompt):], len(prompt), st)[0]   # rows from the prompt's end on suffice
    assert np.array_equal(np.concatenate([a, b]), want)
    assert st.head_evals == 0
    # an end-of-sequence token counts once it is verified: numbers whose run (with exits) keeps its margin both without
    # and with the end-of-sequence token, which is a token that run produces
    n, seed0 = 12, 0
    while True:
        u2, free_run, _, o1 = _numbers_with_margin(pair, prompt, n, 0.25, 0.2, cfg.exit_layers, 3, max_seq, seed0=seed0)
        seed0 = o1.seed + 1
        ks = [j for j in range(2, n - 1) if free_run[j] not in free_run[:j]]
        if not ks:
            continue
        k = ks[0]
        eos = int(free_run[k])
        o2 = pair.cpu(max_seq)
        o2.prefill(prompt)
        want2 = o2.sampling_decode(n, 0.25, 0.2, cfg.exit_layers, 3, u2.astype(np.float64), eos_id=eos)
        if o2.min_margin >= MARGIN:
            break
    assert o2.emitted == k + 1 and np.array_equal(want2[:k + 1], free_run[:k + 1])
    E = binding.Session(pair.gm, 1, max_seq, 64, 3)
    E.prefill(prompt)
    st = binding.Stats()
    got = E.sampling_decode(n, 0.25, 0.2, cfg.exit_layers, 3, u2[None], 0, st, eos_id=eos)[0]
    assert np.array_equal(got, want2) and st.emitted[0] == k + 1 and st.finished == 1


def test_rows_of_random_numbers_must_cover_the_call():
    cfg = gqa()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=9).numpy()
    S = binding.Session(pair.gm, 1, 64, 64, 3)
    S.prefill(prompt)
    u = np.zeros((1, 12, NU), dtype=np.float32)
    with pytest.raises(binding.AdaError) as e:
        S.sampling_decode(8, 1.0, 0.5, cfg.exit_layers, 3, u, 0)        # rows end before the call's last position
    assert e.value.code == -1
    with pytest.raises(binding.AdaError) as e:
        S.sampling_decode(2, 1.0, 0.5, cfg.exit_layers, 3, u, 11)       # rows start behind the pending token
    assert e.value.code == -1
    with pytest.raises(binding.AdaError) as e:
        S.sampling_decode(2, 0.0, 0.5, cfg.exit_layers, 3, u, 0)        # temperature must be positive
    assert e.value.code == -1
    Z = binding.Session(pair.gm, 1, 64, 64, 3)
    Z.set_path(0)
    Z.prefill(prompt)
    with pytest.raises(binding.AdaError) as e:
        Z.sampling_decode(2, 1.0, 0.5, cfg.exit_layers, 3, u, 0)        # only the persistent path draws tokens
    assert e.value.code == -6


@pytest.mark.parametrize("gamma", [0.0, 0.1])
def test_law_of_a_verified_token_on_the_gpu(gamma):
    """Frequencies of the first sampled token over 4 x 1500 runs (four sequences per call share the weight stream,
    each with its own random numbers) against the closed-form law computed from the oracle's distributions."""
    cfg = gqa(vocab=40, logit_scale=1.0, n_layers=4, exit_layers=(1, 2))
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=11).numpy()
    temperature, batch, calls = 1.2, 4, 1500
    o = pair.cpu(64)
    o.prefill(prompt)
    tokens = list(prompt) + [int(o.plain_decode(1)[0])]
    qs, pstar = head_and_final_distributions(cfg, pair.om, tokens, temperature)
    law = law_of_a_verified_token(qs, pstar, gamma)
    if gamma == 0.0:
        assert np.allclose(law, pstar, atol=1e-12)
    S = binding.Session(pair.gm, batch, 32, 64, 1)
    assert S.get_path() == 1
    rng = np.random.default_rng(77)
    counts = np.zeros(cfg.vocab, dtype=np.int64)
    st = binding.Stats()
    for _ in range(calls):
        for i in range(batch):
            S.reset(i)
            S.prefill(prompt, seq=i)
        u = rng.random((batch, 32, NU), dtype=np.float32)
        out = S.sampling_decode(2, temperature, gamma, cfg.exit_layers, 1, u, 0, st)
        assert (out[:, 0] == tokens[-1]).all()
        for i in range(batch):
            counts[out[i, 1]] += 1
    ok, stat = chi2_ok(counts, law)
    assert ok, (stat, counts / counts.sum(), law)
    assert st.early_exits > 0 and st.rejected > 0 and st.accepted > 0
    # the wrong rule a plausible mistake would implement (accept every early token) is told apart at this sample size
    assert not chi2_ok(counts, qs[0], alpha=1e-6)[0]


def test_same_numbers_same_decisions_for_every_sequence_of_a_batch():
    """Three sequences in one launch (one weight stream), each with its own prompt and its own random numbers: each
    equals the oracle's run of that sequence alone.  (The chi-square test cannot see a mix-up of the sequences' random
    numbers: any uniform number gives the right law.)"""
    cfg = hd128(logit_scale=2.0, resid_scale=0.1)
    pair = Pair(cfg)
    batch, n, max_seq, max_early = 3, 12, 64, 1
    prompts = [synth.make_prompt(cfg, n=m, seq=i).numpy() for i, m in enumerate((9, 21, 14))]
    us, wants, sts = [], [], []
    for i, p in enumerate(prompts):
        u, want, ost, _ = _numbers_with_margin(pair, p, n, 0.25, 0.2, cfg.exit_layers, max_early, max_seq, seed0=1000 * i)
        us.append(u); wants.append(want); sts.append(ost)
    S = binding.Session(pair.gm, batch, max_seq, 64, max_early)
    assert S.get_path() == 1
    for i, p in enumerate(prompts):
        S.prefill(p, seq=i)
    st = binding.Stats()
    got = S.sampling_decode(n, 0.25, 0.2, cfg.exit_layers, max_early, np.stack(us), 0, st)
    for i in range(batch):
        assert np.array_equal(got[i], wants[i]), (i, got[i], wants[i])
    for f in ("head_evals", "early_exits", "accepted", "rejected", "discarded"):
        assert getattr(st, f) == sum(getattr(o, f) for o in sts), f
    assert st.early_exits > 0 and st.accepted > 0
