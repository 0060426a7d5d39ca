"""The persistent decode kernel (path 1) against the CPU oracle and against itself, through the C ABI.

Tolerances: final logits within max|d| <= 2e-2 x logit std (bf16 models); token ids exact wherever
the oracle's top-2 gap exceeds that; adaptive decoding bit-exact (tokens and final-logit bits) with
the library's own plain decoding on the same path."""

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle
from paper_2506_03700_b200 import binding, synth
from test_gpu_parity import PTOL_BF16, Pair, check_against_oracle, schedule_parity, split_weights, tol


def gqa(**kw):      # 4 q heads per kv head, head_dim 64, ragged vocabulary tile, FFN depth with a short last k chunk
    base = dict(dtype="bf16", n_layers=6, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_ff=1408, vocab=5003,
                sigma=0.05, resid_scale=0.6, exit_layers=(2, 4), rope_base=500000.0)
    base.update(kw)
    return synth.small_config(name="pk-gqa", **base)


def hd128(**kw):    # head_dim 128, 2 q heads per kv head
    base = dict(dtype="bf16", n_layers=3, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=128, d_ff=704, vocab=3001,
                sigma=0.08, resid_scale=0.8, exit_layers=(1, 2), rope_base=10000.0)
    base.update(kw)
    return synth.small_config(name="pk-hd128", **base)


def mha(**kw):      # one q head per kv head
    base = dict(dtype="bf16", n_layers=4, d_model=256, n_q_heads=4, n_kv_heads=4, head_dim=64, d_ff=640, vocab=2048,
                sigma=0.08, resid_scale=0.8, exit_layers=(1, 3), rope_base=10000.0)
    base.update(kw)
    return synth.small_config(name="pk-mha", **base)


def session(pair, max_seq=256, max_early=5, **kw):
    S = binding.Session(pair.gm, 1, max_seq, 64, max_early, **kw)
    assert S.get_path() == 1, "the session did not qualify for the persistent kernel"
    return S


@pytest.mark.parametrize("mk,n_prompt,n_gen", [(gqa, 33, 24), (hd128, 70, 30), (mha, 9, 40)])
def test_plain_decode_matches_oracle(mk, n_prompt, n_gen):
    cfg = mk()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=n_prompt).numpy()
    S = session(pair)
    S.capture_logits(n_gen + 4)
    S.prefill(prompt)
    st = binding.Stats()
    out = S.plain_decode(n_gen, st)[0]
    lg = S.captured_logits().cpu().numpy()
    assert len(lg) >= n_gen
    check_against_oracle(pair, prompt, out, lg)
    assert st.kernel_launches <= 3 and st.layer_passes == (n_gen - 1) * cfg.n_layers
    assert len(set(out.tolist())) > 3


@pytest.mark.parametrize("mk", [gqa, hd128, mha])
def test_adaptive_is_bit_exact_with_plain(mk):
    cfg = mk()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=21).numpy()
    n = 48
    P = session(pair)
    P.capture_logits(n + 8)
    P.prefill(prompt)
    ref = P.plain_decode(n)[0]
    ref_lg = P.captured_logits()[:n].clone()
    seen = dict(exits=0, rejected=0, accepted=0)
    L = cfg.n_layers
    for gamma, exits, cap in [(0.0, cfg.exit_layers, 5), (0.3, cfg.exit_layers, 5), (0.6, cfg.exit_layers[:1], 2),
                              (0.9, cfg.exit_layers[1:], 1), (1.0, cfg.exit_layers, 5), (0.0, tuple(range(1, L)), 7),
                              (0.5, cfg.exit_layers, 0), (0.2, (), 5)]:
        for l in exits:
            pair.gm.set_exit_head(l, None, cfg.logit_scale)
        S = session(pair, max_early=7)
        S.capture_logits(n + 8)
        S.prefill(prompt)
        st = binding.Stats()
        out = S.adaptive_decode(n, gamma, exits, cap, st)[0]
        assert np.array_equal(out, ref), (gamma, exits, cap)
        assert torch.equal(S.captured_logits()[:n], ref_lg), (gamma, exits, cap)
        ln, fill = S.state()
        assert ln == len(prompt) + n and (fill == len(prompt) + n - 1).all()
        assert st.early_exits == st.accepted + st.rejected + st.discarded
        assert st.accepted + st.verify_steps - st.truncated == n - 1
        if gamma >= 1.0 or cap == 0 or not exits:
            assert st.early_exits == 0 and st.verify_steps == n - 1
        seen["exits"] += st.early_exits; seen["rejected"] += st.rejected; seen["accepted"] += st.accepted
    assert seen["exits"] > 0 and seen["rejected"] > 0 and seen["accepted"] > 0


@pytest.mark.parametrize("mk,T_noise", [(gqa, None), (hd128, None), (gqa, 0.3)])
def test_adaptive_schedule_and_heads_match_oracle(mk, T_noise):
    cfg = mk()
    pair = Pair(cfg, T_noise=T_noise)
    schedule_parity(pair, lambda: session(pair), 40, PTOL_BF16)


def test_forced_tapes_and_relaunches_never_change_the_output():
    cfg = gqa()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=9).numpy()
    n = 30
    P = session(pair)
    P.prefill(prompt)
    ref = P.plain_decode(n)[0]
    rng = np.random.default_rng(1)
    rej = 0
    for trial in range(10):
        S = session(pair, max_early=7)
        S.set_launch_steps(int(rng.integers(1, 9)))     # the kernel returns to the host every few steps
        S.prefill(prompt)
        S.set_exit_tape(rng.integers(0, 2, 64))
        st = binding.Stats()
        out = S.adaptive_decode(n, 0.5, cfg.exit_layers, int(rng.integers(1, 8)), st)[0]
        assert np.array_equal(out, ref)
        assert st.kernel_launches >= 3
        rej += st.rejected
    assert rej > 0


def test_rollback_leaves_the_cache_of_a_fresh_run():
    cfg = hd128()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=6).numpy()
    n = 20
    A = session(pair)
    A.prefill(prompt)
    A.set_exit_tape([1] * 64)
    st = binding.Stats()
    a = A.adaptive_decode(n, 0.5, cfg.exit_layers, 4, st)[0]
    assert st.rejected > 0
    B = session(pair)
    B.prefill(prompt)
    b = B.plain_decode(n)[0]
    assert np.array_equal(a, b)
    la, fa = A.state()
    lb, fb = B.state()
    assert la == lb and np.array_equal(fa, fb)
    O = pair.cpu()
    O.prefill(prompt)
    O.plain_decode(n)
    for l in range(cfg.n_layers):
        for pos in (0, 5, 6, 13, len(prompt) + n - 2):
            for which in (0, 1):
                ka, kb = A.read_kv(which, l, pos), B.read_kv(which, l, pos)
                assert np.array_equal(ka, kb)
                ref = O.kv(which, l, pos)
                assert np.abs(ka - ref).max() <= 2e-2 * max(1.0, np.abs(ref).max())


def test_chained_calls_and_both_paths_mixed():
    cfg = gqa()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=8).numpy()
    P = session(pair)
    P.capture_logits(40)
    P.prefill(prompt)
    ref = P.plain_decode(36)[0]
    ref_lg = P.captured_logits()[:36].clone()
    S = session(pair)
    S.capture_logits(40)
    S.prefill(prompt)
    st = binding.Stats()
    a = S.adaptive_decode(1, 0.0, cfg.exit_layers, 5, st)[0]
    b = S.adaptive_decode(9, 0.0, cfg.exit_layers, 5, st)[0]
    c = S.plain_decode(6, st)[0]
    d = S.adaptive_decode(20, 0.3, cfg.exit_layers[:1], 2, st)[0]
    assert np.array_equal(np.concatenate([a, b, c, d]), ref)
    assert st.path == 1 and st.emitted[0] == 36
    # one captured logits row per returned token, also across calls that ended by dropping a verified token
    lg = S.captured_logits()
    assert len(lg) == 36 and torch.equal(lg, ref_lg)
    S.prefill(prompt)
    assert np.array_equal(S.plain_decode(5)[0], ref[:5])
    # the one-kernel-per-operation path agrees within tolerance: same tokens on this model
    Q = session(pair)
    Q.set_path(0)
    Q.prefill(prompt)
    q = Q.plain_decode(36)[0]
    assert (q == ref).mean() > 0.9


def test_context_across_pages_and_attention_chunks():
    """Prompt + generation cross several 64-token KV pages and the 128-position attention split."""
    cfg = mha(n_layers=2, exit_layers=(1,))
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=250).numpy()
    n = 20
    S = session(pair, max_seq=300)
    S.capture_logits(n + 8)
    S.prefill(prompt)
    out = S.plain_decode(n)[0]
    check_against_oracle(pair, prompt, out, S.captured_logits().cpu().numpy())
    A = session(pair, max_seq=300)
    A.prefill(prompt)
    st = binding.Stats()
    assert np.array_equal(A.adaptive_decode(n, 0.2, cfg.exit_layers, 5, st)[0], out)
    assert st.early_exits > 0


def test_long_context_many_chunks():
    cfg = hd128(n_layers=2, exit_layers=(1,))
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=1100).numpy()
    n = 8
    S = session(pair, max_seq=1200)
    S.capture_logits(n + 4)
    S.prefill(prompt)
    out = S.plain_decode(n)[0]
    check_against_oracle(pair, prompt, out, S.captured_logits().cpu().numpy())
    A = session(pair, max_seq=1200)
    A.prefill(prompt)
    assert np.array_equal(A.adaptive_decode(n, 0.0, cfg.exit_layers, 5)[0], out)


def test_more_attention_work_items_than_ctas():
    """Sixteen kv heads at a context of 1600 positions: 13 chunks x 16 heads = 208 work items, more than
    any GPU has SMs, so CTAs take several items each and the chunk partials are merged by the
    designated CTAs (with fewer items than CTAs the last CTA to finish a head merges it)."""
    cfg = mha(n_layers=2, d_model=1024, n_q_heads=16, n_kv_heads=16, d_ff=704, exit_layers=(1,))
    assert 16 * (1600 // 128 + 1) > torch.cuda.get_device_properties(0).multi_processor_count
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=1600).numpy()
    n = 10
    S = session(pair, max_seq=1700)
    S.capture_logits(n + 4)
    S.prefill(prompt)
    out = S.plain_decode(n)[0]
    lg = S.captured_logits()[:n].clone()
    check_against_oracle(pair, prompt, out, lg.cpu().numpy())
    for gamma, tape in [(0.0, None), (0.5, [1] * 16)]:
        A = session(pair, max_seq=1700)
        A.capture_logits(n + 4)
        A.prefill(prompt)
        if tape:
            A.set_exit_tape(tape)
        assert np.array_equal(A.adaptive_decode(n, gamma, cfg.exit_layers, 5)[0], out)
        assert torch.equal(A.captured_logits()[:n], lg)


@pytest.mark.parametrize("mk", [gqa, hd128])
def test_end_of_sequence_token_stops_decoding(mk):
    """ "while t_i != [EOS]" inside the persistent kernel: the first verified end-of-sequence token ends
    the call, under every forced tape and across relaunches; an early-predicted one stops nothing."""
    cfg = mk()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=9).numpy()
    n = 30
    P = session(pair)
    P.prefill(prompt)
    ref = P.plain_decode(n)[0]
    i = next(k for k in range(4, n) if ref[k] not in ref[:k])
    eos = int(ref[i])
    Q = session(pair)
    Q.prefill(prompt)
    st = binding.Stats()
    want = Q.plain_decode(n, st, eos_id=eos)[0]
    assert st.emitted[0] == i + 1 and st.finished == 1 and st.path == 1
    assert np.array_equal(want[:i + 1], ref[:i + 1]) and (want[i + 1:] == eos).all()
    lq, fq = Q.state()
    assert lq == len(prompt) + i + 1 and (fq == len(prompt) + i).all()
    rng = np.random.default_rng(5)
    for trial in range(8):
        S = session(pair, max_early=7)
        S.set_launch_steps(int(rng.integers(1, 9)))
        S.prefill(prompt)
        S.set_exit_tape(rng.integers(0, 2, 64))
        st = binding.Stats()
        out = S.adaptive_decode(n, 0.5, cfg.exit_layers, int(rng.integers(1, 8)), st, eos_id=eos)[0]
        assert np.array_equal(out, want), trial
        assert st.emitted[0] == i + 1 and st.finished == 1
        ls, fs = S.state()
        assert ls == lq and np.array_equal(fs, fq)
    # the token prefill produced is itself the end-of-sequence token: one token, no step
    S = session(pair)
    S.prefill(prompt)
    st = binding.Stats()
    out = S.adaptive_decode(5, 0.0, cfg.exit_layers, 5, st, eos_id=int(ref[0]))[0]
    assert st.emitted[0] == 1 and st.steps == 0 and (out == ref[0]).all()
    # a prefill starts the sequence afresh
    S.prefill(prompt)
    assert np.array_equal(S.plain_decode(6)[0], ref[:6])


def test_separate_q_k_v_gate_up_tensors_give_the_same_bits():
    """Weights lent as wq, wk, wv, w_gate, w_up (separate allocations): the gate and up matrices are
    streamed through two tensor maps, q | k | v through the repacked copy in the arena."""
    cfg = gqa()
    pair = Pair(cfg)
    gm2 = binding.Model(cfg, split_weights(cfg, pair.w))
    for l in cfg.exit_layers:
        gm2.set_exit_head(l, None, cfg.logit_scale)
    prompt = synth.make_prompt(cfg, n=19).numpy()
    n = 24
    outs = []
    for gm in (pair.gm, gm2):
        S = binding.Session(gm, 1, 256, 64, 5)
        assert S.get_path() == 1
        S.capture_logits(n + 4)
        S.prefill(prompt)
        t = S.adaptive_decode(n, 0.3, cfg.exit_layers, 5)[0]
        outs.append((t, S.captured_logits()[:n].clone()))
    assert np.array_equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_a_wait_that_runs_out_ends_the_call_with_a_timeout_and_the_session_recovers():
    """Every device-side wait is bounded.  With the limit set far below what a grid-wide wait lasts, the
    first wait that is not satisfied at once gives up: the kernel raises its error word, every other
    wait falls through, the kernel ends and the call returns ADA_ETIMEOUT (no trap, no hang, the
    context stays usable).  After a reset and a prefill the same session decodes correctly."""
    cfg = gqa()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=12).numpy()
    n = 12
    P = session(pair)
    P.prefill(prompt)
    ref = P.plain_decode(n)[0]
    S = session(pair)
    S.prefill(prompt)
    S.set_wait_limit(20)                  # nanoseconds
    with pytest.raises(binding.AdaError) as e:
        S.plain_decode(n)
    assert e.value.code == -5
    torch.cuda.synchronize()              # the context is intact
    S.set_wait_limit(2_000_000_000)
    S.reset()
    S.prefill(prompt)
    assert np.array_equal(S.plain_decode(n)[0], ref)
    st = binding.Stats()
    S.prefill(prompt)
    assert np.array_equal(S.adaptive_decode(n, 0.3, cfg.exit_layers, 5, st)[0], ref) and st.early_exits > 0


@pytest.mark.parametrize("mk,n_prompt", [(gqa, 200), (hd128, 131), (mha, 77)])
def test_dense_prompt_pass_matches_the_pass_through_the_decode_path_and_the_oracle(mk, n_prompt):
    """KV cache <- LM(x): prompts of 32 tokens or more run in blocks of 128 positions through the tcgen05
    GEMMs.  The cache it leaves and the first token agree with the prompt pass through the decode kernel
    (eight positions at a time) within the cache's bf16 rounding, and decoding on from it matches the oracle."""
    cfg = mk()
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=n_prompt).numpy()
    n = 12
    D = session(pair, max_seq=n_prompt + 64)
    D.capture_logits(n + 4)
    D.prefill(prompt)                     # dense (the default)
    C = session(pair, max_seq=n_prompt + 64)
    C.set_prefill(False)
    C.prefill(prompt)
    ld, fd = D.state()
    lc, fc = C.state()
    assert ld == lc == n_prompt + 1 and np.array_equal(fd, fc)
    O = pair.cpu()
    O.prefill(prompt)
    for l in range(cfg.n_layers):
        for pos in (0, 1, 63, 64, 127, 128, n_prompt - 1):
            if pos >= n_prompt:
                continue
            for which in (0, 1):
                a, b, ref = D.read_kv(which, l, pos), C.read_kv(which, l, pos), O.kv(which, l, pos)
                scale = max(1.0, np.abs(ref).max())
                assert np.abs(a - ref).max() <= 2e-2 * scale and np.abs(a - b).max() <= 2e-2 * scale
    out = D.plain_decode(n)[0]
    check_against_oracle(pair, prompt, out, D.captured_logits().cpu().numpy())
    # adaptive decoding on top of a dense prompt pass equals plain decoding on top of one, bit for bit
    A = session(pair, max_seq=n_prompt + 64)
    A.prefill(prompt)
    st = binding.Stats()
    assert np.array_equal(A.adaptive_decode(n, 0.3, cfg.exit_layers, 5, st)[0], out) and st.early_exits > 0


def test_batch_of_ragged_sequences_on_the_persistent_path():
    """Independent sequences in one session (ragged prompt lengths, one of them long enough for the dense prompt
    pass): each equals its own single-sequence run bit for bit, plain and adaptive, with and without an
    end-of-sequence token."""
    cfg = gqa()
    pair = Pair(cfg)
    lens = [5, 19, 70]
    prompts = [synth.make_prompt(cfg, n=n, seq=i).numpy() for i, n in enumerate(lens)]
    n = 24
    singles = []
    for p in prompts:
        S = session(pair)
        S.prefill(p)
        singles.append(S.plain_decode(n)[0])
    B = binding.Session(pair.gm, 3, 256, 64, 5)
    assert B.get_path() == 1
    for i, p in enumerate(prompts):
        B.prefill(p, seq=i)
    st = binding.Stats()
    out = B.plain_decode(n, st)
    for i in range(3):
        assert np.array_equal(out[i], singles[i]), i
    assert st.path == 1 and list(st.emitted[:3]) == [n, n, n]
    A = binding.Session(pair.gm, 3, 256, 64, 5)
    for i, p in enumerate(prompts):
        A.prefill(p, seq=i)
    st = binding.Stats()
    a1 = A.adaptive_decode(10, 0.3, cfg.exit_layers, 5, st)
    a2 = A.adaptive_decode(n - 10, 0.0, cfg.exit_layers, 3, st)
    assert np.array_equal(np.concatenate([a1, a2], axis=1), out) and st.early_exits > 0
    for i in range(3):
        ln, fill = A.state(i)
        assert ln == lens[i] + n and (fill == lens[i] + n - 1).all()
    # an end-of-sequence token that only the second sequence meets: the others run on
    k = next(j for j in range(3, n) if singles[1][j] not in singles[1][:j] and singles[1][j] not in singles[0] and singles[1][j] not in singles[2])
    eos = int(singles[1][k])
    E = binding.Session(pair.gm, 3, 256, 64, 5)
    for i, p in enumerate(prompts):
        E.prefill(p, seq=i)
    st = binding.Stats()
    e = E.adaptive_decode(n, 0.3, cfg.exit_layers, 5, st, eos_id=eos)
    assert list(st.emitted[:3]) == [n, k + 1, n] and st.finished == 1
    assert np.array_equal(e[0], singles[0]) and np.array_equal(e[2], singles[2])
    assert np.array_equal(e[1][:k + 1], singles[1][:k + 1]) and (e[1][k + 1:] == eos).all()


@pytest.mark.parametrize("max_early,batch", [(1, 4), (3, 3), (0, 8)])
def test_sequences_sharing_one_weight_stream(max_early, batch):
    """Sessions whose sequences fit the kernel's eight token columns together (batch x (max_early + 1) <= 8, or
    groups of 8 / (max_early + 1)): every launch decodes the group in lock-step over one pass of the weights.  Each
    sequence still equals its own single-sequence run bit for bit: plain, adaptive (decisions differ per sequence),
    and with an end-of-sequence token that stops one sequence while the others run on."""
    cfg = gqa()
    pair = Pair(cfg)
    lens = [5, 19, 70, 33, 8, 41, 12, 27][:batch]
    prompts = [synth.make_prompt(cfg, n=n, seq=i).numpy() for i, n in enumerate(lens)]
    n = 24
    singles = []
    for p in prompts:
        S = session(pair)
        S.prefill(p)
        one = binding.Stats()
        singles.append(S.plain_decode(n, one)[0])

    def fresh():
        B = binding.Session(pair.gm, batch, 256, 64, max_early)
        assert B.get_path() == 1
        for i, p in enumerate(prompts):
            B.prefill(p, seq=i)
        return B

    st = binding.Stats()
    out = fresh().plain_decode(n, st)
    for i in range(batch):
        assert np.array_equal(out[i], singles[i]), i
    assert st.path == 1 and list(st.emitted[:batch]) == [n] * batch
    # one pass of the weights per step for the whole group, not one per sequence
    group = min(batch, 8 // (max_early + 1))
    launches_groups = -(-batch // group)
    assert st.layer_passes == launches_groups * one.layer_passes
    if max_early == 0:
        return
    A = fresh()
    st = binding.Stats()
    a1 = A.adaptive_decode(10, 0.3, cfg.exit_layers, max_early, st)
    a2 = A.adaptive_decode(n - 10, 0.0, cfg.exit_layers, max_early, st)
    assert np.array_equal(np.concatenate([a1, a2], axis=1), out) and st.early_exits > 0
    for i in range(batch):
        ln, fill = A.state(i)
        assert ln == lens[i] + n and (fill == lens[i] + n - 1).all()
    k = next(j for j in range(3, n) if singles[1][j] not in singles[1][:j]
             and all(singles[1][j] not in singles[o] for o in range(batch) if o != 1))
    eos = int(singles[1][k])
    E = fresh()
    st = binding.Stats()
    e = E.adaptive_decode(n, 0.3, cfg.exit_layers, max_early, st, eos_id=eos)
    want = [n] * batch
    want[1] = k + 1
    assert list(st.emitted[:batch]) == want and st.finished == 1
    for i in range(batch):
        if i != 1:
            assert np.array_equal(e[i], singles[i]), i
    assert np.array_equal(e[1][:k + 1], singles[1][:k + 1]) and (e[1][k + 1:] == eos).all()


def test_both_attention_arrangements_agree_with_more_items_than_ctas():
    """Four q heads per kv head at a context of 9700 positions: 2 x 76 work items, more than the GPU has SMs.  Plain
    decoding (one column: every query in the first tile, the two warp groups take different items) and adaptive decoding
    with forced exits (up to six columns: both query tiles in use, the groups share an item) must give the same tokens
    and the same final-logit bits: which warps compute an item does not change its arithmetic."""
    cfg = gqa(n_layers=2, exit_layers=(1,))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n_prompt = 128 * (sms // 2 + 2) - 28
    assert 2 * (n_prompt // 128 + 1) > sms
    pair = Pair(cfg)
    prompt = synth.make_prompt(cfg, n=n_prompt).numpy()
    n = 14
    P = session(pair, max_seq=n_prompt + 64)
    P.capture_logits(n + 4)
    P.prefill(prompt)
    out = P.plain_decode(n)[0]
    lg = P.captured_logits()[:n].clone()
    for tape in ([1] * 32, [1, 1, 0, 1, 1, 1, 1, 0] * 4):
        A = session(pair, max_seq=n_prompt + 64)
        A.capture_logits(n + 8)
        A.prefill(prompt)
        A.set_exit_tape(tape)
        st = binding.Stats()
        assert np.array_equal(A.adaptive_decode(n, 0.5, cfg.exit_layers, 5, st)[0], out)
        assert torch.equal(A.captured_logits()[:n], lg)
        assert st.early_exits >= 5
