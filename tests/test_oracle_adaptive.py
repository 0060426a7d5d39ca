"""Pins for the oracle's Algorithm 1: output parity with plain greedy decoding under every
exit-decision tape (brute force), the gamma end points, the worked schedule of Figure 2, the
cap of Appendix D, the greedy form of Eq. 2 and the state after rollback."""

import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2506_03700_b200 import synth
from helpers import make_oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mini(**kw):
    base = dict(n_layers=3, d_model=32, n_q_heads=2, n_kv_heads=1, head_dim=16, d_ff=40, vocab=61,
                resid_scale=1.0, exit_layers=(1, 2), logit_scale=8.0, sigma=0.25)
    base.update(kw)
    return synth.small_config(name="mini", **base)


def _plain(m, prompt, n, max_seq=128):
    s = oracle.Session(m, max_seq)
    s.prefill(prompt)
    return s.plain_decode(n)


def test_every_decision_tape_reproduces_plain_greedy():
    """Schedule invariance (Section 2.2: verification guarantees output parity regardless of
    gamma): all 2^10 forced exit/continue tapes give the plain greedy tokens."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    n = 7
    ref = _plain(m, prompt, n)
    seen_reject = seen_accept = 0
    for tape in itertools.product((0, 1), repeat=10):
        s = oracle.Session(m, 128)
        s.prefill(prompt)
        st = oracle.Stats()
        out = s.adaptive_decode(n, 0.5, cfg.exit_layers, max_early=3, tape=tape, stats=st)
        assert np.array_equal(out, ref), (tape, out, ref)
        assert s.len == len(prompt) + n
        assert all(s.kv_len(l) == len(prompt) + n - 1 for l in range(cfg.n_layers))
        seen_reject += st.rejected
        seen_accept += st.accepted
    assert seen_reject > 0 and seen_accept > 0   # both branches of the verification ran


def test_planted_wrong_tokens_are_always_caught():
    """Early tokens replaced by arbitrary ids (wrong almost surely) never reach the output."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=4).numpy()
    n = 6
    ref = _plain(m, prompt, n)
    rng = np.random.default_rng(0)
    for trial in range(200):
        k = 12
        tape = rng.integers(0, 2, k)
        tape_tok = np.where(rng.random(k) < 0.5, rng.integers(0, cfg.vocab, k), -1)
        s = oracle.Session(m, 128)
        s.prefill(prompt)
        st = oracle.Stats()
        out = s.adaptive_decode(n, 0.5, cfg.exit_layers, max_early=4, tape=tape, tape_tok=tape_tok, stats=st)
        assert np.array_equal(out, ref)
        # emitted per verification = accepted + 1; nothing else is ever emitted
        assert st.accepted + st.verify_steps == n - 1 + st.truncated


def test_gamma_one_is_the_plain_path():
    """gamma = 1: no probability exceeds it (Section 4.4), so no early prediction happens."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=6).numpy()
    ref = _plain(m, prompt, 10)
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    s.record_trace()
    st = oracle.Stats()
    out = s.adaptive_decode(10, 1.0, cfg.exit_layers, stats=st)
    assert np.array_equal(out, ref)
    assert st.early_exits == 0 and st.rejected == 0 and st.steps == 9 and st.verify_steps == 9
    assert st.head_evals == 9 * len(cfg.exit_layers)
    assert (s.trace[:, 3] == 1).all()          # one row at every layer, like plain decoding


def test_gamma_zero_exits_at_the_first_head_until_the_cap():
    """gamma = 0 triggers an early prediction at every step (Section 4.4); with the cap of
    Appendix D the (max_early+1)-th token runs to full depth and verifies."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=6).numpy()
    n, cap = 40, 5
    ref = _plain(m, prompt, n)
    s = oracle.Session(m, 256)
    s.prefill(prompt)
    s.record_trace()
    st = oracle.Stats()
    out = s.adaptive_decode(n, 0.0, cfg.exit_layers, max_early=cap, stats=st)
    assert np.array_equal(out, ref)
    first = cfg.exit_layers[0]
    assert st.early_exits == st.exits_at_layer[first] > 0
    tr = s.trace
    assert tr[:, 3].max() <= cap + 1          # never more than max_early + 1 rows in a layer
    # steps alternate: up to `cap` one-layer steps, then one full-depth step
    per_step = {}
    for step, layer, pos0, rows in tr:
        per_step.setdefault(int(step), []).append(int(layer))
    run = 0
    for step in sorted(per_step):
        layers = per_step[step]
        if layers == list(range(1, first + 1)):
            run += 1
            assert run <= cap
        else:
            assert layers == list(range(1, cfg.n_layers + 1))
            run = 0


def test_figure2_schedule():
    """Figure 2 (left): t1 exits at layer 2, t2 at layer 1; then layer 2 of t2,t3 in parallel,
    then layer 3 of t1,t2,t3."""
    want = []
    with open(os.path.join(GOLDEN, "fig2_schedule.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            want.append((int(p[0]), int(p[1]), [int(t[1:]) for t in p[2:]]))
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=4).numpy()
    s = oracle.Session(m, 64)
    s.prefill(prompt)
    s.record_trace()
    # heads at layers 1 and 2.  t1: continue at 1, exit at 2.  t2: exit at 1.  t3: cap reached.
    s.adaptive_decode(4, 0.5, (1, 2), max_early=2, tape=[0, 1, 1])
    n0 = len(prompt)            # t1 is the first generated token, at position n0
    got = [(int(st), int(l), [int(p0) - n0 + 1 + r for r in range(rows)]) for st, l, p0, rows in s.trace[:len(want)]]
    assert got == want


def test_greedy_verification_rule_and_rollback_state():
    """Eq. 2 at temperature zero: an early token is kept iff it equals the full-depth argmax;
    the first mismatch is replaced by that argmax and everything after is dropped.  After a
    rollback the cache equals the cache of a from-scratch run over the corrected sequence."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    ref = _plain(m, prompt, 8)
    # plant a wrong token at the 2nd early prediction; 1st and 3rd are forced exits with the
    # head's own token
    wrong = (int(ref[2]) + 1) % cfg.vocab
    s = oracle.Session(m, 64)
    s.prefill(prompt)
    st = oracle.Stats()
    # decisions: t1 exits at layer 1 with the true next token, t2 exits with a wrong one, t3
    # exits (whatever it predicts is discarded), t4 runs to full depth (cap 3)
    # (gamma = 1 afterwards: past the tape no further early prediction happens)
    out = s.adaptive_decode(5, 1.0, (1, 2), max_early=3, tape=[1, 1, 1],
                            tape_tok=[int(ref[1]), wrong, -1], stats=st)
    assert np.array_equal(out, ref[:5])
    assert (st.accepted, st.rejected, st.discarded) == (1, 1, 1)
    # state: the sequence ends on the last token; K/V valid strictly before it at every layer and
    # equal to a from-scratch run (nothing computed for the rejected tokens survives)
    assert s.len == len(prompt) + 5
    assert np.array_equal(s.tokens(), np.concatenate([prompt, ref[:5]]))
    fresh = oracle.Session(m, 64)
    fresh.prefill(np.concatenate([prompt, ref[:4]]))
    for l in range(cfg.n_layers):
        assert s.kv_len(l) == fresh.kv_len(l) == len(prompt) + 4
        for pos in range(len(prompt) + 4):
            for which in (0, 1):
                assert np.abs(s.kv(which, l, pos) - fresh.kv(which, l, pos)).max() < 1e-12
    # and decoding continues correctly, adaptively or plainly, from the rolled-back state
    more = s.adaptive_decode(3, 0.0, (1, 2), max_early=2)
    assert np.array_equal(more, ref[5:])


def test_cap_and_counter_identities():
    cfg = _mini(n_layers=4, exit_layers=(1, 3))
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=8).numpy()
    ref = _plain(m, prompt, 30, max_seq=256)
    for cap in (0, 1, 2, 5):
        for gamma in (0.0, 0.3, 0.7):
            s = oracle.Session(m, 256)
            s.prefill(prompt)
            s.record_trace()
            st = oracle.Stats()
            out = s.adaptive_decode(30, gamma, cfg.exit_layers, max_early=cap, stats=st)
            assert np.array_equal(out, ref)
            assert s.trace[:, 3].max() <= cap + 1
            assert st.early_exits == st.accepted + st.rejected + st.discarded
            assert st.steps == st.early_exits + st.verify_steps
            assert st.accepted + st.verify_steps - st.truncated == 30 - 1
            if cap == 0:
                assert st.head_evals == 0 and st.early_exits == 0


def test_mixed_chained_calls_leave_identical_state():
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    ref = _plain(m, prompt, 20)
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    a = s.adaptive_decode(6, 0.0, cfg.exit_layers, max_early=5)
    b = s.plain_decode(4)
    c = s.adaptive_decode(10, 0.2, cfg.exit_layers[:1], max_early=2)
    assert np.array_equal(np.concatenate([a, b, c]), ref)


def test_bad_arguments_are_refused():
    cfg = _mini()
    w, m = make_oracle(cfg)
    s = oracle.Session(m, 32)
    s.prefill(synth.make_prompt(cfg, n=5).numpy())
    with pytest.raises(RuntimeError):
        s.adaptive_decode(4, 0.5, (3,), max_early=5)          # layer L carries no head
    with pytest.raises(RuntimeError):
        s.adaptive_decode(4, 0.5, (2, 1), max_early=5)        # not ascending
    with pytest.raises(RuntimeError):
        s.adaptive_decode(400, 0.5, (1,), max_early=5)        # beyond capacity


# ---------------------------------------------------------------- end of sequence (Algorithm 1: "while t_i != [EOS]")

def _first_repeat_free_eos(ref):
    """A token of the plain stream, not its first, whose first occurrence is where it stands."""
    for i in range(3, len(ref)):
        if ref[i] not in ref[:i]:
            return i, int(ref[i])
    raise AssertionError("degenerate stream")


def test_plain_decoding_with_eos_is_the_prefix_up_to_the_first_eos():
    """Definition: generate until the end-of-sequence token has been produced."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    n = 14
    ref = _plain(m, prompt, n)
    i, eos = _first_repeat_free_eos(ref)
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    out = s.plain_decode(n, eos_id=eos)
    assert s.emitted == i + 1
    assert np.array_equal(out[:i + 1], ref[:i + 1]) and (out[i + 1:] == eos).all()
    assert s.len == len(prompt) + i + 1
    assert all(s.kv_len(l) == len(prompt) + i for l in range(cfg.n_layers))
    # an end-of-sequence token that never occurs changes nothing
    unused = next(t for t in range(cfg.vocab) if t not in ref)
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    assert np.array_equal(s.plain_decode(n, eos_id=unused), ref) and s.emitted == n
    # the token prefill produced may already be it
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    out = s.plain_decode(n, eos_id=int(ref[0]))
    assert s.emitted == 1 and out[0] == ref[0] and s.len == len(prompt) + 1


def test_adaptive_with_eos_equals_plain_with_eos_on_every_tape():
    """Only a VERIFIED end-of-sequence token ends the sequence: under every forced exit tape, with and
    without planted early predictions of the end-of-sequence token itself, the adaptive procedure
    returns what plain decoding with the same token returns, and leaves the same state."""
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    n = 12
    ref = _plain(m, prompt, n)
    i, eos = _first_repeat_free_eos(ref)
    assert i + 1 < n                           # the call would have gone on
    p = oracle.Session(m, 128)
    p.prefill(prompt)
    want = p.plain_decode(n, eos_id=eos)
    planted = 0
    for tape in itertools.product((0, 1), repeat=8):
        for plant in (False, True):
            s = oracle.Session(m, 128)
            s.prefill(prompt)
            st = oracle.Stats()
            tape_tok = [eos if (plant and k % 3 == 1) else -1 for k in range(len(tape))]
            out = s.adaptive_decode(n, 0.5, cfg.exit_layers, max_early=3, tape=tape, tape_tok=tape_tok, stats=st, eos_id=eos)
            assert np.array_equal(out, want), (tape, plant, out, want)
            assert s.emitted == i + 1
            assert s.len == p.len and all(s.kv_len(l) == p.kv_len(l) for l in range(cfg.n_layers))
            planted += plant and st.rejected > 0
    assert planted > 0                         # a wrongly predicted end-of-sequence token was rejected, not obeyed


def test_eos_across_chained_calls():
    cfg = _mini()
    w, m = make_oracle(cfg)
    prompt = synth.make_prompt(cfg, n=5).numpy()
    ref = _plain(m, prompt, 14)
    i, eos = _first_repeat_free_eos(ref)
    s = oracle.Session(m, 128)
    s.prefill(prompt)
    a = s.adaptive_decode(2, 0.0, cfg.exit_layers, eos_id=eos)
    assert s.emitted == 2
    b = s.adaptive_decode(12, 0.0, cfg.exit_layers, eos_id=eos)
    assert s.emitted == i + 1 - 2
    assert np.array_equal(np.concatenate([a, b[:s.emitted]]), ref[:i + 1])
