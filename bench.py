#!/usr/bin/env python
"""Benchmark of the layer-parallel decode step (Algorithm 1) on a Llama-3.1-8B-shaped synthetic model.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8b|1b|tiny] [--impl ours|reference]

One "step" is one adaptive-decode call of gen_len/K tokens on the benchmark sequence (prompt
prefilled, untimed); K steps generate the configuration's full generation length.  The same K
steps are then timed with plain greedy decoding (the library's own baseline).  Prints ONE JSON
line.  N > 1 runs N independent replicas (the path does not shard), one per GPU under torchrun.
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
# from the ncu capture summarised in profiles/ (1B-shaped plain decode; traffic grows in proportion
# to the bytes streamed, so the ratio carries over to the 8B shape).  None = not captured.
DRAM_TRAFFIC_RATIO = 0.996
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


def byte_model(cfg, stats, ctx_mean: float) -> float:
    """Algorithmic HBM bytes of a decode call: every layer pass streams one layer's weights and
    reads that layer's K/V once for all rows; every head evaluation and every verification streams
    the LM head once."""
    esz = 2 if cfg.dtype == "bf16" else 4
    d, hd = cfg.d_model, cfg.head_dim
    w_layer = ((cfg.n_q_heads + 2 * cfg.n_kv_heads) * hd * d + d * cfg.n_q_heads * hd + 3 * cfg.d_ff * d) * esz
    w_head = cfg.vocab * d * esz
    kv_layer = 2 * cfg.n_kv_heads * hd * esz * ctx_mean
    return stats.layer_passes * (w_layer + kv_layer) + (stats.head_evals + stats.verify_steps) * w_head


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
    per_step = max(1, gen_len // K)
    gen_len = per_step * K
    max_seq = cfg.prompt_len + per_step * max(K, Wm, 1) + 16

    w = synth.make_weights(cfg, seed=1234, device="cuda")
    model = binding.Model(cfg, w)
    for l in cfg.exit_layers:
        model.set_exit_head(l, None, cfg.logit_scale)
    prompt = synth.make_prompt(cfg, seed=5678).numpy()
    sess = binding.Session(model, 1, max_seq, 64, 5)
    if args.launch_steps > 0:
        sess.set_launch_steps(args.launch_steps)
    out = np.empty((1, per_step), dtype=np.int32)
    try:
        pinned = torch.empty((1, per_step), dtype=torch.int32).pin_memory()
        out = pinned.numpy()
    except Exception:
        pass

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(mode: str, steps: int):
        """Prefill (untimed), then `steps` decode calls.  Returns device ms (library's CUDA events on the
        session stream, summed), wall ms around the same calls, stats, tokens."""
        sess.prefill(prompt)
        st = binding.Stats()
        toks = []
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        ev0.record(sess.stream)
        for _ in range(steps):
            if mode == "adaptive":
                sess.adaptive_decode(per_step, cfg.threshold, cfg.exit_layers, 5, st, out=out)
            else:
                sess.plain_decode(per_step, st, out=out)
            toks.append(out.copy())
        ev1.record(sess.stream)
        barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3
        return ev0.elapsed_time(ev1), wall_ms, st, np.concatenate(toks, axis=1)

    if args.plain_only:
        # profiling aid: plain greedy decoding only, so that every launch of the persistent kernel
        # moves a known number of bytes (launch_steps x (L layers + LM head))
        timed("plain", max(Wm, 1))
        p_ms, p_wall, p_st, p_tok = timed("plain", K)
        if rank == 0:
            ctx_mean = cfg.prompt_len + gen_len / 2
            print(json.dumps({"mode": "plain_only", "tokens_per_s": gen_len / (p_ms * 1e-3), "decode_ms": p_st.decode_ms,
                              "launches": int(p_st.kernel_launches), "layer_passes": int(p_st.layer_passes),
                              "algorithmic_bytes": byte_model(cfg, p_st, ctx_mean)}))
        if dist is not None:
            dist.destroy_process_group()
        return

    # warm-up (W >= 3 steps of each mode), then the timed K steps from a fresh prefill
    timed("adaptive", max(Wm, 1))
    timed("plain", max(Wm, 1))
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    a_ms, a_wall, a_st, a_tok = timed("adaptive", K)
    p_ms, p_wall, p_st, p_tok = timed("plain", K)
    clocks = sampler.stop() if rank == 0 else None
    parity = bool(np.array_equal(a_tok, p_tok))

    # instrumented pass: per-kernel-class device time of the same adaptive steps
    sess.profile(True)
    timed("adaptive", K)
    prof = sess.profile_read()
    sess.profile(False)

    a_ms, p_ms, a_wall, p_wall = max_over_ranks([a_ms, p_ms, a_wall, p_wall], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    n_tok = gen_len * world
    ctx_mean = cfg.prompt_len + gen_len / 2
    a_bytes, p_bytes = byte_model(cfg, a_st, ctx_mean), byte_model(cfg, p_st, ctx_mean)
    a_gbs, p_gbs = a_bytes / (a_ms * 1e-3) / 1e9, p_bytes / (p_ms * 1e-3) / 1e9
    # The timed region launches one kernel of this library over and over: the persistent decode
    # kernel (plus one tiny set-up kernel per call).  Its achieved bandwidth = algorithmic bytes of
    # the calls (layer passes x layer bytes + head evaluations x LM-head bytes + KV reads) over the
    # device time of the calls (the library's CUDA events on the session stream around its launches).
    n_dec_launches = max(1, int(a_st.kernel_launches) - K)
    dom = "k_decode_persistent"
    dom_gbs = a_bytes / (a_st.decode_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": whole_job_tokens_per_s(gen_len, world, a_ms), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": a_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"{cfg.name}-shaped decoder bs1, {cfg.prompt_len}-token uniform-random prompt, "
                               f"{gen_len} greedy tokens, exits {list(cfg.exit_layers)}, gamma {cfg.threshold}, "
                               f"tied head logit scale {cfg.logit_scale}, max_early 5",
                   "tokens_per_step": per_step, "l2": "inputs_larger_than_l2 (weights stream >> 126 MB)",
                   "parallelism": "replicas" if world > 1 else "single"},
        "e2e": {"value": whole_job_tokens_per_s(gen_len, world, a_wall), "unit": UNIT, "h2d_bytes_per_step": 64 + 4 * 16,
                "d2h_bytes_per_step": int(per_step * 4 + 8 * (9 + 256 + 4))},
        "gpu_launches": int(a_st.kernel_launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": dom_gbs, "peak": peak, "unit": "GB/s", "frac": dom_gbs / peak,
                     "traffic": (DRAM_TRAFFIC_RATIO * a_bytes / n_dec_launches if DRAM_TRAFFIC_RATIO else None),
                     "kernel": dom, "peak_kind": peak_kind, "launches": n_dec_launches,
                     "avg_launch_ms": a_st.decode_ms / n_dec_launches,
                     "algorithmic_bytes_per_launch": a_bytes / n_dec_launches,
                     "plain_decode": {"achieved": p_bytes / (p_st.decode_ms * 1e-3) / 1e9,
                                      "frac": p_bytes / (p_st.decode_ms * 1e-3) / 1e9 / peak}},
        "cpu_baseline": None,
        "adaptive": {"tokens_per_s": gen_len / (a_ms * 1e-3), "step_gbs": a_gbs, "frac_of_nominal_8TBs": a_gbs / NOMINAL_HBM_GBS,
                     "frac_of_measured": a_gbs / peak, "stats": {k: v for k, v in a_st.as_dict().items()},
                     "early_exit_rate": a_st.early_exits / max(1, a_st.steps),
                     "rejection_rate": a_st.rejected / max(1, a_st.accepted + a_st.rejected)},
        "plain": {"tokens_per_s": gen_len / (p_ms * 1e-3), "step_gbs": p_gbs, "frac_of_nominal_8TBs": p_gbs / NOMINAL_HBM_GBS,
                  "frac_of_measured": p_gbs / peak, "gpu_launches": int(p_st.kernel_launches)},
        "speedup_vs_plain": p_ms / a_ms, "adaptive_equals_plain": parity,
        "kernel_classes": {c: {"ms": round(v["ms"], 3), "launches": v["launches"],
                               "gbs": (v["bytes"] / (v["ms"] * 1e-3) / 1e9 if v["ms"] > 0 and v["bytes"] > 0 else None)}
                           for c, v in prof.items() if v["launches"]},
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(cfg, w, args.cpu_tokens)
    if not args.no_regime and world == 1 and args.workload == "8b":
        del sess, model, w
        torch.cuda.empty_cache()
        line["confident_head_regime"] = confident_regime(cfg, args.regime_scale, args.regime_tokens)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def confident_regime(cfg, scale: float, n_tok: int) -> dict:
    """Supplementary measurement.  With the configured o_proj/down_proj scale (0.2) and d_model 4096 the
    random layers swamp the embedding, and an untrained head at layer 16 almost never agrees with the
    final argmax (the paper's "original LM head" ablation).  Scaling those projections by `scale`
    instead makes the intermediate heads predictive, as the paper's trained heads are (about 80 %
    early exits, a few % rejected): same shape, same kernels, same byte counts per layer, measured
    the same way on a shorter generation."""
    import dataclasses
    from paper_2506_03700_b200 import binding, synth
    c2 = dataclasses.replace(cfg, resid_scale=scale)
    w = synth.make_weights(c2, seed=1234, device="cuda")
    model = binding.Model(c2, w)
    for l in c2.exit_layers:
        model.set_exit_head(l, None, c2.logit_scale)
    prompt = synth.make_prompt(c2, seed=5678).numpy()
    sess = binding.Session(model, 1, c2.prompt_len + n_tok + 16, 64, 5)
    sess.prefill(prompt)
    sess.plain_decode(8)
    sess.prefill(prompt)
    ps = binding.Stats()
    pt = sess.plain_decode(n_tok, ps)[0]
    sess.prefill(prompt)
    st = binding.Stats()
    at = sess.adaptive_decode(n_tok, c2.threshold, c2.exit_layers, 5, st)[0]
    return {"o_down_scale": scale, "tokens": n_tok, "plain_tokens_per_s": n_tok / (ps.decode_ms * 1e-3),
            "adaptive_tokens_per_s": n_tok / (st.decode_ms * 1e-3), "speedup_vs_plain": ps.decode_ms / st.decode_ms,
            "adaptive_equals_plain": bool(np.array_equal(at, pt)), "distinct_tokens": len(set(pt.tolist())),
            "early_exit_rate": st.early_exits / max(1, st.steps),
            "rejection_rate": st.rejected / max(1, st.accepted + st.rejected),
            "exits_at_layer": st.as_dict()["exits_at_layer"]}


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
    ap.add_argument("--workload", default="8b", choices=["tiny", "1b", "8b"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-tokens", type=int, default=12)
    ap.add_argument("--ref-tokens", type=int, default=2)
    ap.add_argument("--no-regime", action="store_true", help="skip the supplementary confident-head measurement")
    ap.add_argument("--regime-scale", type=float, default=0.02)
    ap.add_argument("--regime-tokens", type=int, default=512)
    ap.add_argument("--plain-only", action="store_true", help="time plain greedy decoding only (profiling runs)")
    ap.add_argument("--gen-len", type=int, default=0, help="generate this many tokens instead of the workload's (profiling runs)")
    ap.add_argument("--launch-steps", type=int, default=0, help="decode steps per launch of the persistent kernel (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
