#!/usr/bin/env python
"""Benchmark of the layer-parallel decode step (Algorithm 1) on a Llama-3.1-8B-shaped synthetic model.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8b|8b-long|13b|1b|tiny] [--impl ours|reference]

One "step" is one adaptive-decode call of about gen_len/K tokens on the benchmark sequence(s) (prompt
prefilled, untimed); K steps generate the configuration's full generation length (the last step
takes the remainder).  The same K steps are then timed with plain greedy decoding (the library's own
baseline).  Prints ONE JSON line; supplementary measurements (threshold and head-scale sweeps, the
pure-overhead checks, a dense head transformation, the adversarial weights of the long-context
configuration) ride along as extra keys of that line.  N > 1 runs N independent replicas (the path
does not shard), one per GPU under torchrun.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode_tokens_per_s_bs1"
UNIT = "tokens/s"
# dram__bytes_read+write of one launch of the persistent kernel over that launch's algorithmic bytes,
# from the ncu captures summarised in profiles/ (1B-shaped launches; traffic grows in proportion to the
# bytes streamed, so a ratio carries over to the larger shapes), keyed by decoding mode.  None = not
# captured for the kernel as it stands.
DRAM_TRAFFIC_RATIO = {"plain": 0.9961, "adaptive": 0.9976}   # profiles/k_decode_persistent_1b_dram_traffic_ncu.md
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of `values` over the ranks of the job (the slowest replica sets the time).
    The decode path does not shard: N GPUs run N independent replicas and exchange nothing else."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_max: float) -> float:
    """Throughput of the whole job: all replicas' tokens over the slowest replica's time."""
    return tokens_per_rank * world / (ms_max * 1e-3)


def byte_model(cfg, stats, ctx_sum: float, dense_T: bool = False) -> float:
    """Algorithmic HBM bytes of a decode call: every layer pass streams one layer's weights and
    reads that layer's K/V once for all rows (`ctx_sum` = cached positions summed over the
    sequences of the batch, averaged over the call); every head evaluation and every verification
    streams the LM head once (plus the d x d head transformation, if the heads carry a dense one)."""
    esz = 2 if cfg.dtype == "bf16" else 4
    d, hd = cfg.d_model, cfg.head_dim
    w_layer = ((cfg.n_q_heads + 2 * cfg.n_kv_heads) * hd * d + d * cfg.n_q_heads * hd + 3 * cfg.d_ff * d) * esz
    w_head = cfg.vocab * d * esz
    kv_layer = 2 * cfg.n_kv_heads * hd * esz * ctx_sum
    return (stats.layer_passes * (w_layer + kv_layer) + (stats.head_evals + stats.verify_steps) * w_head +
            (stats.head_evals * d * d * esz if dense_T else 0))


def step_sizes(gen_len: int, K: int):
    """K step sizes that add up to gen_len: gen_len // K each, the last one takes the remainder."""
    per = max(1, gen_len // K)
    sizes = [per] * K
    sizes[-1] = max(1, gen_len - per * (K - 1))
    return sizes


class Bench:
    """One model, one session, timed decode runs of it."""

    def __init__(self, cfg, torch, binding, synth, sizes, warm, dist=None, resid_scale=None, logit_scale=None,
                 dense_T=False, launch_steps=0, seed=1234, max_early=-1):
        import dataclasses
        self.torch, self.binding, self.dist = torch, binding, dist
        if resid_scale is not None:
            cfg = dataclasses.replace(cfg, resid_scale=resid_scale)
        self.cfg, self.sizes, self.dense_T = cfg, sizes, dense_T
        self.w = synth.make_weights(cfg, seed=seed, device="cuda")
        self.model = binding.Model(cfg, self.w)
        self.scale = cfg.logit_scale if logit_scale is None else logit_scale
        self.register_heads(self.scale, dense_T)
        self.batch = cfg.batch
        if self.batch > 1:
            lens = synth.batch_prompt_lengths(cfg, seed=5678)
            self.prompts = [synth.make_prompt(cfg, seed=5678, n=n, seq=i).numpy() for i, n in enumerate(lens)]
        else:
            self.prompts = [synth.make_prompt(cfg, seed=5678).numpy()]
        self.gen_len = sum(sizes)
        max_seq = max(len(p) for p in self.prompts) + max(self.gen_len, max(sizes) * max(warm, 1)) + 16
        # A sequence holds max_early + 1 of the persistent kernel's eight token columns.  One sequence: the paper's
        # setting of up to five early-predicted tokens.  A batch: as many as still let all its sequences share every
        # pass over the weights.
        self.max_early = max_early if max_early >= 0 else (5 if self.batch == 1 else max(0, 8 // self.batch - 1))
        self.sess = binding.Session(self.model, self.batch, max_seq, 64, self.max_early)
        if launch_steps > 0 and self.sess.get_path() == 1:
            self.sess.set_launch_steps(launch_steps)
        # launches a decode call needs for the batch (each streams the weights for its own sequences)
        self.groups = -(-self.batch // max(1, 8 // (self.max_early + 1))) if self.sess.get_path() == 1 else 1
        m = max(sizes)
        self.out = np.empty((self.batch, m), dtype=np.int32)
        try:
            self.out = torch.empty((self.batch, m), dtype=torch.int32).pin_memory().numpy()
        except Exception:
            pass
        self.prompt_bytes = sum(4 * len(p) for p in self.prompts)
        # cached positions one layer pass reads: those of the sequences that share the pass
        self.ctx_sum = (sum(len(p) for p in self.prompts) + self.batch * self.gen_len / 2) / self.groups

    def register_heads(self, scale, dense_T=False):
        torch = self.torch
        self.scale, self.dense_T = scale, dense_T
        for l in self.cfg.exit_layers:
            T = None
            if dense_T:   # the paper's head form E* T with a materialised d x d transformation (here the identity)
                T = torch.eye(self.cfg.d_model, dtype=self.cfg.torch_dtype, device="cuda").contiguous()
            self.model.set_exit_head(l, T, scale)

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def timed(self, mode, sizes=None, threshold=None, exit_layers=None, temperature=1.0):
        """Prefill (untimed), then one decode call per entry of `sizes`.  Returns device ms (CUDA events on
        the session stream around the calls), wall ms around the same calls, stats, tokens [batch][sum]."""
        torch, sess, cfg = self.torch, self.sess, self.cfg
        sizes = self.sizes if sizes is None else sizes
        threshold = cfg.threshold if threshold is None else threshold
        exit_layers = cfg.exit_layers if exit_layers is None else exit_layers
        for i, p in enumerate(self.prompts):
            sess.prefill(p, seq=i)
        st = self.binding.Stats()
        toks = []
        self.barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        ev0.record(sess.stream)
        for n in sizes:
            o = self.out[:, :n] if n == self.out.shape[1] else np.empty((self.batch, n), dtype=np.int32)
            if mode == "adaptive":
                sess.adaptive_decode(n, threshold, exit_layers, self.max_early, st, out=o)
            elif mode == "sampling":
                # every random number is an input of the call: rows for all positions, drawn on the host (seeded)
                sess.sampling_decode(n, temperature, threshold, exit_layers, self.max_early, self.uniforms(), 0, st, out=o)
            else:
                sess.plain_decode(n, st, out=o)
            toks.append(o.copy())
        ev1.record(sess.stream)
        self.barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3
        return ev0.elapsed_time(ev1), wall_ms, st, np.concatenate(toks, axis=1)

    def uniforms(self):
        if getattr(self, "_uniforms", None) is None:
            rng = np.random.default_rng(4321)
            self._uniforms = rng.random((self.batch, self.sess.max_seq_len, self.binding.SAMPLE_NU), dtype=np.float32)
        return self._uniforms

    def e2e(self, mode, sizes=None):
        """The same steps end to end through the C ABI with host buffers: every step's timed region holds the
        host-to-device copies of its inputs (the prompt, with its prefill, in the first step; the call's
        arguments in every step) and the device-to-host read of its tokens and counters."""
        sess = self.sess
        sizes = self.sizes if sizes is None else sizes
        for i in range(self.batch):
            sess.reset(i)
        self.barrier()
        st = self.binding.Stats()
        t0 = time.perf_counter()
        for i, p in enumerate(self.prompts):
            sess.prefill(p, seq=i)
        for n in sizes:
            o = self.out[:, :n] if n == self.out.shape[1] else np.empty((self.batch, n), dtype=np.int32)
            if mode == "adaptive":
                sess.adaptive_decode(n, self.cfg.threshold, self.cfg.exit_layers, self.max_early, st, out=o)
            else:
                sess.plain_decode(n, st, out=o)
        self.barrier()
        return (time.perf_counter() - t0) * 1e3

    def summary(self, ms, st, tokens_ref=None, tokens=None) -> dict:
        n_tok = self.batch * (tokens.shape[1] if tokens is not None else self.gen_len)
        d = {"tokens_per_s": n_tok / (ms * 1e-3), "early_exit_rate": st.early_exits / max(1, st.steps),
             "rejection_rate": st.rejected / max(1, st.accepted + st.rejected), "head_evals": int(st.head_evals),
             "steps": int(st.steps), "layer_passes": int(st.layer_passes),
             "step_gbs": byte_model(self.cfg, st, self.ctx_sum, self.dense_T) / (ms * 1e-3) / 1e9}
        if tokens_ref is not None and tokens is not None:
            d["equals_plain"] = bool(np.array_equal(tokens, tokens_ref[:, :tokens.shape[1]]))
        return d


def byte_model_speedup(cfg, st_adaptive, st_plain, ctx_sum, dense_T=False) -> float:
    """Speed-up the byte model predicts for these counters: plain bytes over adaptive bytes."""
    return byte_model(cfg, st_plain, ctx_sum) / byte_model(cfg, st_adaptive, ctx_sum, dense_T)


def run_ours(args):
    import torch
    from paper_2506_03700_b200 import binding, build, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        args.gpus = world
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    cfg = synth.CONFIGS[args.workload]
    K, Wm = args.steps, args.warmup
    gen_len = args.gen_len if args.gen_len > 0 else cfg.gen_len
    sizes = step_sizes(gen_len, K)
    warm = [sizes[0]] * max(Wm, 1)
    B = Bench(cfg, torch, binding, synth, sizes, max(Wm, 1), dist, launch_steps=args.launch_steps, max_early=args.max_early)
    path = B.sess.get_path()

    if args.plain_only or args.adaptive_only:
        # profiling aid: one mode only, so that every launch of the persistent kernel moves a known number of bytes
        mode = "plain" if args.plain_only else "adaptive"
        _, _, wst, _ = B.timed(mode, warm)
        ms, wall, st, tok = B.timed(mode)
        if rank == 0:
            # the warm-up's own counters too: a capture of every launch of the process is compared with the sum of both
            print(json.dumps({"mode": mode + "_only", "tokens_per_s": gen_len * cfg.batch / (ms * 1e-3), "decode_ms": st.decode_ms,
                              "launches": int(st.kernel_launches), "layer_passes": int(st.layer_passes),
                              "head_evals": int(st.head_evals), "verify_steps": int(st.verify_steps),
                              "algorithmic_bytes": byte_model(cfg, st, B.ctx_sum),
                              "warmup_launches": int(wst.kernel_launches),
                              "warmup_algorithmic_bytes": byte_model(cfg, wst, sum(len(q) for q in B.prompts) / B.groups + sum(warm) / 2)}))
        if dist is not None:
            dist.destroy_process_group()
        return

    # warm-up (W >= 3 steps of each mode), then the timed K steps from a fresh prefill
    B.timed("adaptive", warm)
    B.timed("plain", warm)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    a_ms, a_wall, a_st, a_tok = B.timed("adaptive")
    p_ms, p_wall, p_st, p_tok = B.timed("plain")
    clocks = sampler.stop() if rank == 0 else None
    e2e_ms = B.e2e("adaptive")
    parity = bool(np.array_equal(a_tok, p_tok))

    # instrumented pass: per-kernel-class device time of the same adaptive steps
    B.sess.profile(True)
    B.timed("adaptive")
    prof = B.sess.profile_read()
    B.sess.profile(False)

    a_ms, p_ms, a_wall, p_wall, e2e_ms = max_over_ranks([a_ms, p_ms, a_wall, p_wall, e2e_ms], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    n_tok = gen_len * cfg.batch
    a_bytes, p_bytes = byte_model(cfg, a_st, B.ctx_sum), byte_model(cfg, p_st, B.ctx_sum)
    a_gbs, p_gbs = a_bytes / (a_ms * 1e-3) / 1e9, p_bytes / (p_ms * 1e-3) / 1e9
    # The timed region launches one kernel of this library over and over: the persistent decode kernel (plus one
    # tiny set-up kernel per call) where the session runs on it, else one kernel per operation.  Achieved bandwidth
    # = algorithmic bytes of the calls (layer passes x layer bytes + head evaluations x LM-head bytes + KV reads)
    # over the device time of the calls (the library's CUDA events on the session stream around its launches).
    n_dec_launches = max(1, int(a_st.kernel_launches) - K) if path == 1 else int(a_st.kernel_launches)
    dom = "k_decode_persistent" if path == 1 else "k_gemv (one kernel per operation; the whole call is reported)"
    dom_gbs = a_bytes / (a_st.decode_ms * 1e-3) / 1e9
    ratio = DRAM_TRAFFIC_RATIO["adaptive"] if path == 1 else None
    prompt_desc = (f"{cfg.prompt_len}-token uniform-random prompt" if cfg.batch == 1 else
                   f"{cfg.batch} sequences, uniform-random prompts of {[len(p) for p in B.prompts]} tokens")
    line = {
        "metric": METRIC if cfg.batch == 1 else "decode_tokens_per_s_aggregate", "value": whole_job_tokens_per_s(n_tok, world, a_ms),
        "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": a_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"{cfg.name}-shaped decoder bs{cfg.batch}, {prompt_desc}, "
                               f"{gen_len} greedy tokens each, exits {list(cfg.exit_layers)}, gamma {cfg.threshold}, "
                               f"tied head logit scale {cfg.logit_scale}, max_early {B.max_early}, o/down scale {cfg.resid_scale}",
                   "tokens_per_step": sizes[0], "last_step_tokens": sizes[-1], "l2": "inputs_larger_than_l2 (weights stream >> 126 MB)",
                   "decode_path": ("persistent kernel" + ("" if cfg.batch == 1 else
                                                           ", all sequences share every pass over the weights" if B.groups == 1 else
                                                           f", sequences in {B.groups} groups, each group streams the weights for itself"))
                                  if path == 1 else "one kernel per operation",
                   "parallelism": "replicas" if world > 1 else "single"},
        "e2e": {"value": whole_job_tokens_per_s(n_tok, world, a_wall), "unit": UNIT,
                "h2d_bytes_per_step": int(64 + 4 * 16 + 4 * len(cfg.exit_layers)),
                "d2h_bytes_per_step": int(cfg.batch * sizes[0] * 4 + 8 * (9 + 256 + 4) + 8 * cfg.batch),
                "note": "host clock around the K decode calls of the C ABI (host buffers in and out: call arguments and exit "
                        "layers copied in, tokens and counters read back, every step); the prompt is already prefilled",
                "with_prompt_and_prefill": {"value": whole_job_tokens_per_s(n_tok, world, e2e_ms), "unit": UNIT,
                                            "h2d_bytes_first_step": int(B.prompt_bytes),
                                            "note": "the same plus the prompt's host-to-device copy and its prefill in the first step"}},
        "gpu_launches": int(a_st.kernel_launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": dom_gbs, "peak": peak, "unit": "GB/s", "frac": dom_gbs / peak,
                     "frac_of_nominal_8TBs": dom_gbs / NOMINAL_HBM_GBS,
                     "traffic": (ratio * a_bytes / n_dec_launches if ratio else None),
                     "kernel": dom, "peak_kind": peak_kind, "launches": n_dec_launches,
                     "avg_launch_ms": a_st.decode_ms / n_dec_launches,
                     "algorithmic_bytes_per_launch": a_bytes / n_dec_launches,
                     "plain_decode": {"achieved": p_bytes / (p_st.decode_ms * 1e-3) / 1e9,
                                      "frac": p_bytes / (p_st.decode_ms * 1e-3) / 1e9 / peak}},
        "cpu_baseline": None,
        "adaptive": {"tokens_per_s": n_tok / (a_ms * 1e-3), "step_gbs": a_gbs, "frac_of_nominal_8TBs": a_gbs / NOMINAL_HBM_GBS,
                     "frac_of_measured": a_gbs / peak, "stats": {k: v for k, v in a_st.as_dict().items()},
                     "early_exit_rate": a_st.early_exits / max(1, a_st.steps),
                     "rejection_rate": a_st.rejected / max(1, a_st.accepted + a_st.rejected)},
        "plain": {"tokens_per_s": n_tok / (p_ms * 1e-3), "step_gbs": p_gbs, "frac_of_nominal_8TBs": p_gbs / NOMINAL_HBM_GBS,
                  "frac_of_measured": p_gbs / peak, "gpu_launches": int(p_st.kernel_launches)},
        "speedup_vs_plain": p_ms / a_ms, "byte_model_speedup": byte_model_speedup(cfg, a_st, p_st, B.ctx_sum),
        "adaptive_equals_plain": parity,
        "kernel_classes": {c: {"ms": round(v["ms"], 3), "launches": v["launches"],
                               "us_per_launch": round(1e3 * v["ms"] / v["launches"], 2),
                               "gbs": (v["bytes"] / (v["ms"] * 1e-3) / 1e9 if v["ms"] > 0 and v["bytes"] > 0 else None)}
                           for c, v in prof.items() if v["launches"]},
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(cfg, B.w, args.cpu_tokens)
    if not args.no_extras and world == 1:
        line["extras"] = extras(args, B, p_tok, torch, binding, synth)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def extras(args, B, p_tok, torch, binding, synth) -> dict:
    """Supplementary measurements on the same model and session, each a shorter generation from a fresh
    prefill (`--extra-tokens` tokens), each with its own plain-decoding time over the same tokens."""
    cfg = B.cfg
    n = min(args.extra_tokens, B.gen_len)
    sz = step_sizes(n, max(1, min(args.steps, n)))
    out = {"tokens": n * cfg.batch}
    p_ms, _, p_st, _ = B.timed("plain", sz)
    out["plain_tokens_per_s"] = n * cfg.batch / (p_ms * 1e-3)

    def run(threshold=None, exit_layers=None):
        ms, _, st, tok = B.timed("adaptive", sz, threshold, exit_layers)
        d = B.summary(ms, st, p_tok, tok)
        d["speedup_vs_plain"] = p_ms / ms
        d["byte_model_speedup"] = byte_model_speedup(cfg, st, p_st, B.ctx_sum, B.dense_T)
        return d

    # thresholds of Eq. 1: the configuration's sweep, and gamma = 1 (no probability exceeds it: pure head overhead)
    sweep = {"1b": (0.6, 0.8, 0.95)}.get(cfg.name, (cfg.threshold,))
    out["threshold_sweep"] = {str(g): run(threshold=g) for g in sorted(set(sweep) | {1.0})}
    # no exit layers at all: the adaptive call must cost what plain decoding costs
    out["no_exit_layers"] = run(exit_layers=())
    if not args.no_scale_sweep:
        # logit scale s of the tied intermediate heads (the configurations leave it open): measured and modelled speed-up
        sc = {}
        for s_ in (1.0, 2.0, 4.0, 8.0):
            B.register_heads(s_)
            sc[str(s_)] = run()
        out["head_logit_scale_sweep"] = sc
        best = max(sc, key=lambda k: sc[k]["speedup_vs_plain"])
        out["head_logit_scale_best"] = {"scale": float(best), "why": "highest measured speed-up over plain decoding on these weights; "
                                        "with untrained heads a lower scale only lowers the confidence, so fewer wrong early exits are taken"}
        # the paper's head form with a materialised d x d transformation: its bytes are charged per evaluation
        B.register_heads(cfg.logit_scale, dense_T=True)
        out["dense_head_transformation"] = run()
        B.register_heads(cfg.logit_scale)
    if B.sess.get_path() == 1:
        # sampled decoding (Eq. 1 with a drawn token, Eq. 2 with acceptance test and resampling) at temperature 1:
        # plain sampling (no exit layers) and the adaptive form; the time over plain greedy decoding is what the draws cost
        sm = {}
        for name, ex in (("plain_sampling", ()), ("adaptive_sampling", cfg.exit_layers)):
            ms, _, st, tok = B.timed("sampling", sz, cfg.threshold, ex, temperature=1.0)
            sm[name] = {"tokens_per_s": n * cfg.batch / (ms * 1e-3), "early_exit_rate": st.early_exits / max(1, st.steps),
                        "rejection_rate": st.rejected / max(1, st.accepted + st.rejected), "time_vs_plain_greedy": ms / p_ms}
        out["sampled_decoding_temperature_1"] = sm
    if args.workload == "8b" and not args.no_regime:
        out["confident_head_regime"] = confident_regime(args, cfg, torch, binding, synth)
    if args.workload == "8b-long" and not args.no_regime:
        out["adversarial_o_down_scale_1"] = second_model_run(args, cfg, torch, binding, synth, 1.0, args.extra_tokens)
    return out


def second_model_run(args, cfg, torch, binding, synth, resid_scale, n_tok) -> dict:
    """The same shape with other o_proj / down_proj scaling, measured like the main run (adaptive and plain,
    K steps each from a fresh prefill)."""
    n = n_tok if n_tok > 0 else cfg.gen_len
    sz = step_sizes(n, max(1, min(args.steps, n)))
    B2 = Bench(cfg, torch, binding, synth, sz, 1, None, resid_scale=resid_scale)
    B2.timed("adaptive", sz[:1])
    B2.timed("plain", sz[:1])
    a_ms, _, a_st, a_tok = B2.timed("adaptive")
    p_ms, _, p_st, p_tok = B2.timed("plain")
    d = B2.summary(a_ms, a_st, p_tok, a_tok)
    d.update({"o_down_scale": resid_scale, "tokens": n, "plain_tokens_per_s": n * cfg.batch / (p_ms * 1e-3),
              "speedup_vs_plain": p_ms / a_ms, "byte_model_speedup": byte_model_speedup(cfg, a_st, p_st, B2.ctx_sum),
              "distinct_tokens": len(set(p_tok[0].tolist())), "exits_at_layer": a_st.as_dict()["exits_at_layer"]})
    if B2.sess.get_path() == 1:
        # the same with sampled tokens: plain sampling against the adaptive form with Eq. 2 in full, at a low and at a
        # moderate temperature (a shorter run each)
        n_s = min(n, 512)
        sz_s = step_sizes(n_s, max(1, min(args.steps, n_s)))
        sm = {}
        for T in (0.2, 0.7):
            r = {}
            for name, ex in (("plain_sampling", ()), ("adaptive_sampling", cfg.exit_layers)):
                ms, _, st, _ = B2.timed("sampling", sz_s, cfg.threshold, ex, temperature=T)
                r[name] = {"tokens_per_s": n_s * cfg.batch / (ms * 1e-3), "early_exit_rate": st.early_exits / max(1, st.steps),
                           "rejection_rate": st.rejected / max(1, st.accepted + st.rejected)}
            r["speedup_vs_plain_sampling"] = r["adaptive_sampling"]["tokens_per_s"] / r["plain_sampling"]["tokens_per_s"]
            sm[str(T)] = r
        d["sampled_decoding_by_temperature"] = sm
    del B2
    torch.cuda.empty_cache()
    return d


def confident_regime(args, cfg, torch, binding, synth) -> dict:
    """Supplementary measurement.  With the configured o_proj/down_proj scale (0.2) and d_model 4096 the
    random layers swamp the embedding, and an untrained head at layer 16 almost never agrees with the
    final argmax (the paper's "original LM head" ablation).  Scaling those projections by `--regime-scale`
    instead makes the intermediate heads predictive, as the paper's trained heads are (about 80 %
    early exits, a few % rejected): same shape, same kernels, same byte counts per layer, measured
    the same way (K steps from a fresh prefill, the configuration's full generation length)."""
    return second_model_run(args, cfg, torch, binding, synth, args.regime_scale, args.regime_tokens)


def cpu_baseline(cfg, w, n_tok: int, n_prompt: int = 16) -> dict:
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the same
    workload: a short prompt and a few plain greedy tokens of the same model."""
    import oracle
    from paper_2506_03700_b200 import synth
    om = oracle.model_from_torch(cfg, {k: v.cpu() for k, v in w.items()})
    S = oracle.Session(om, n_prompt + n_tok + 8)
    S.prefill(synth.make_prompt(cfg, n=n_prompt).numpy())
    t0 = time.perf_counter()
    S.plain_decode(n_tok + 1)
    dt = time.perf_counter() - t0
    return {"value": n_tok / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"plain greedy decoding of {n_tok} tokens after a {n_prompt}-token prompt on the same "
                      f"{cfg.name}-shaped weights (context {n_prompt}+ instead of {cfg.prompt_len}+), OpenMP on all host threads"}


def run_reference(args):
    """The reference arm is the CPU oracle (there is no reference implementation to install):
    each step is a bounded sample, `--ref-tokens` plain greedy tokens on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2506_03700_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = synth.make_weights(cfg, seed=1234, device=dev)
    om = oracle.model_from_torch(cfg, {k: v.cpu() for k, v in w.items()})
    del w
    n_prompt, per = 16, args.ref_tokens
    total = (args.steps + args.warmup) * per
    S = oracle.Session(om, n_prompt + total + 8)
    S.prefill(synth.make_prompt(cfg, n=n_prompt).numpy())
    S.plain_decode(1)
    for _ in range(args.warmup):
        S.plain_decode(per)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        S.plain_decode(per)
    dt = time.perf_counter() - t0
    val = args.steps * per / dt
    sample = (f"{per} plain greedy tokens per step after a {n_prompt}-token prompt on the {cfg.name}-shaped weights, "
              f"CPU oracle (double precision, OpenMP)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}-shaped decoder bs1 (bounded sample: {sample})"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--max-early", type=int, default=-1,
                    help="early-predicted tokens a sequence may hold (default: 5 for one sequence, 8 // batch - 1 for a batch)")
    ap.add_argument("--workload", default="8b", choices=["tiny", "1b", "8b", "8b-long", "13b"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-tokens", type=int, default=12)
    ap.add_argument("--ref-tokens", type=int, default=2)
    ap.add_argument("--no-regime", action="store_true", help="skip the supplementary run on a second set of weights")
    ap.add_argument("--regime-scale", type=float, default=0.02)
    ap.add_argument("--regime-tokens", type=int, default=0, help="tokens of the second-model run (0: the configuration's generation length)")
    ap.add_argument("--no-extras", action="store_true", help="skip every supplementary measurement")
    ap.add_argument("--no-scale-sweep", action="store_true", help="skip the head logit-scale sweep and the dense-T run")
    ap.add_argument("--extra-tokens", type=int, default=512, help="generation length of each supplementary run")
    ap.add_argument("--plain-only", action="store_true", help="time plain greedy decoding only (profiling runs)")
    ap.add_argument("--adaptive-only", action="store_true", help="time adaptive decoding only (profiling runs)")
    ap.add_argument("--gen-len", type=int, default=0, help="generate this many tokens instead of the workload's (profiling runs)")
    ap.add_argument("--launch-steps", type=int, default=0, help="decode steps per launch of the persistent kernel (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
