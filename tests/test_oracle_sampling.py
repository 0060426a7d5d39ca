"""Pins for the oracle's sampled form of Algorithm 1 (Eq. 1 with a drawn token, Eq. 2 with the acceptance
test and the resampling from Normalize(max(0, p* - q))).

The law of a verified token is computed here from the head and final distributions alone (closed form,
no call into the sampling code) and compared with the frequencies the oracle produces over many seeded runs;
gamma = 0 must give plain sampling exactly; a vanishing temperature must give greedy decoding; with no exit
layer the tokens are the inverse-CDF draws of numpy's own cumulative sum."""

import numpy as np
import pytest
from scipy import stats as sps

import oracle
from paper_2506_03700_b200 import synth
from helpers import make_oracle, head_and_final_distributions as _distributions, law_of_a_verified_token as _law, chi2_ok as _chi2_ok


def _mini(**kw):
    base = dict(n_layers=3, d_model=32, n_q_heads=2, n_kv_heads=1, head_dim=16, d_ff=40, vocab=11,
                resid_scale=1.0, exit_layers=(1, 2), logit_scale=3.0, sigma=0.25)
    base.update(kw)
    return synth.small_config(name="mini-sampling", **base)


def _sample_second_token(cfg, m, prompt, temperature, gamma, runs, seed, exit_layers=None, max_early=3):
    """Token at the first sampled position (the one after the greedy token the prompt pass produced) over
    `runs` calls with fresh random numbers each."""
    rng = np.random.default_rng(seed)
    ex = cfg.exit_layers if exit_layers is None else exit_layers
    counts = np.zeros(cfg.vocab, dtype=np.int64)
    st = oracle.Stats()
    for _ in range(runs):
        s = oracle.Session(m, 32)
        s.prefill(prompt)
        u = rng.random((32, oracle.NU))
        out = s.sampling_decode(2, temperature, gamma, ex, max_early, u, stats=st)
        counts[out[1]] += 1
    return counts, st


@pytest.mark.parametrize("gamma", [0.0, 0.15, 0.3])
def test_law_of_a_verified_token(gamma):
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    s = oracle.Session(m, 32)
    s.prefill(prompt)
    first = s.plain_decode(1)
    tokens = list(prompt) + [int(first[0])]
    temperature = 1.3
    qs, pstar = _distributions(cfg, m, tokens, temperature)
    law = _law(qs, pstar, gamma)
    assert abs(law.sum() - 1.0) < 1e-12
    if gamma == 0.0:
        # every consulted head emits: speculative sampling, which is exactly plain sampling
        assert np.allclose(law, pstar, atol=1e-12)
    else:
        # the thresholded rule is not exactly lossless, and the case must show it (else the pin could not tell
        # the two laws apart)
        assert np.abs(law - pstar).max() > 5e-3
    counts, st = _sample_second_token(cfg, m, prompt, temperature, gamma, runs=6000, seed=17 + int(100 * gamma))
    ok, stat = _chi2_ok(counts, law)
    assert ok, (stat, counts / counts.sum(), law)
    assert st.early_exits > 0 and st.rejected > 0 and st.accepted > 0
    if gamma > 0:
        ok_plain, _ = _chi2_ok(counts, pstar, alpha=1e-6)
        assert not ok_plain   # the frequencies follow the derived law, not p*: the test has the power to tell


def test_planted_mistakes_are_caught_by_the_law():
    """The same comparison fails for a wrong acceptance rule (accept always) and for a wrong replacement law
    (resample from p* instead of the residual): what the oracle produces is neither."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    s = oracle.Session(m, 32)
    s.prefill(prompt)
    tokens = list(prompt) + [int(s.plain_decode(1)[0])]
    qs, pstar = _distributions(cfg, m, tokens, 1.3)
    counts, _ = _sample_second_token(cfg, m, prompt, 1.3, 0.0, runs=6000, seed=5)
    accept_always = qs[0]
    res_wrong = np.minimum(qs[0], pstar) + (qs[0] - np.minimum(qs[0], pstar)).sum() * pstar
    assert not _chi2_ok(counts, accept_always, alpha=1e-6)[0]
    assert not _chi2_ok(counts, res_wrong, alpha=1e-6)[0]
    assert _chi2_ok(counts, pstar)[0]


def test_no_exit_layers_is_inverse_cdf_sampling_of_the_final_distribution():
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=4).numpy()
    rng = np.random.default_rng(3)
    u = rng.random((64, oracle.NU))
    s = oracle.Session(m, 64)
    s.prefill(prompt)
    n = 12
    out = s.sampling_decode(n, 0.9, 0.5, (), 3, u)
    seq = list(prompt) + [int(out[0])]
    for i in range(1, n):
        z = m.full_logits(seq)[-1]
        p = np.exp((z - z.max()) / 0.9)
        cdf = np.cumsum(p / p.sum())
        want = int(np.searchsorted(cdf, u[len(seq), 0], side="right"))
        assert out[i] == want, (i, out[i], want)
        seq.append(int(out[i]))
    assert s.len == len(prompt) + n and all(s.kv_len(l) == len(prompt) + n - 1 for l in range(cfg.n_layers))


def test_vanishing_temperature_is_greedy_decoding():
    cfg = _mini(vocab=61, logit_scale=8.0)
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    g = oracle.Session(m, 64)
    g.prefill(prompt)
    ref = g.plain_decode(10)
    rng = np.random.default_rng(9)
    for gamma in (0.0, 0.6):
        s = oracle.Session(m, 64)
        s.prefill(prompt)
        st = oracle.Stats()
        out = s.sampling_decode(10, 1e-3, gamma, cfg.exit_layers, 3, rng.random((64, oracle.NU)), stats=st)
        assert np.array_equal(out, ref)
        assert st.early_exits > 0


def test_state_after_a_sampling_call_allows_chaining_and_eos():
    """Two chained calls equal one call over the same random numbers; an end-of-sequence token ends the
    sequence only once it is verified; the cache is complete behind the pending token."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=6).numpy()
    u = np.random.default_rng(21).random((64, oracle.NU))
    a = oracle.Session(m, 64)
    a.prefill(prompt)
    one = a.sampling_decode(14, 1.1, 0.2, cfg.exit_layers, 3, u)
    b = oracle.Session(m, 64)
    b.prefill(prompt)
    two = np.concatenate([b.sampling_decode(5, 1.1, 0.2, cfg.exit_layers, 3, u),
                          b.sampling_decode(9, 1.1, 0.2, cfg.exit_layers, 3, u)])
    assert b.len == len(prompt) + 14 and all(b.kv_len(l) == len(prompt) + 13 for l in range(cfg.n_layers))
    # truncation at the end of a call re-draws the dropped position with the same numbers, but from the state a
    # verification leaves (no head consulted when the count is reached), so chained calls may differ from the
    # single call only from a truncated position on; both are valid samples.  What must hold: the prefix before
    # the first call's end is identical.
    assert np.array_equal(one[:5], two[:5])
    k = next(j for j in range(2, 14) if one[j] not in one[:j])
    e = oracle.Session(m, 64)
    e.prefill(prompt)
    out = e.sampling_decode(14, 1.1, 0.2, cfg.exit_layers, 3, u, eos_id=int(one[k]))
    assert e.emitted == k + 1 and np.array_equal(out[:k + 1], one[:k + 1]) and (out[k + 1:] == one[k]).all()
