#!/usr/bin/env python
"""Benchmark of the Tandem + SPEED hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: the prompt pass (large model over
the prompt, FF_Tandem projection of every prompt position) followed by Tandem + SPEED greedy decoding of
`max_new` tokens per sequence (draft, block verify, projection, accept/rollback, repeated).  The default
workload is the "Small Tandem" configuration: bf16, batch 1, 512-token random prompt, gamma 3, 256 new
tokens, natural acceptance.  The metric is generated tokens per second of the decode phase over all ranks (the
step's prompt pass is timed in the same step and reported beside it); the default line also carries compact records
of the medium (batch 8) and large (batch 1) configurations.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload small|tiny|medium]
  python bench.py --workload micro [--micro-case B,T]     kernel micro-benchmark (decode attention, FF_Tandem projection)

With N > 1 (under torchrun) every rank runs an independent replica (sequences are independent units; there
is no collective on the path); the value is all ranks' tokens over the slowest rank's time.

`--impl reference` times the CPU checker (oracle/) on the host cores on a bounded sample of the same workload.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2402_08644_b200 import synth  # noqa: E402

METRIC = "tandem_speed_decode_tokens_per_s"
UNIT = "tokens/s"

WORKLOADS = {
    # name: (config name, batch, prompt length, gamma, new tokens, max_pos)
    "tiny": ("tiny", 1, 32, 4, 64, 128),
    "small": ("small", 1, 512, 3, 256, 1024),
    "medium": ("medium", 8, 2048, 3, 256, 2560),
    "large": ("large", 1, 8192, 3, 512, 8960),
    "large4": ("large", 4, 8192, 3, 512, 8960),
    "large_gqa": ("large", 1, 8192, 3, 512, 8960),   # the large pair with grouped-query attention: 8 key/value heads of 32 (16 -> 4 in the small model)
}
KV_HEADS = {"large_gqa": (8, 4)}
DEVICE_INIT = {"large", "large4", "large_gqa"}   # too big to draw on the host in reasonable time: N(0, 0.02^2) drawn on the device


def workload_desc(name):
    cfgname, B, P, gamma, new, _ = WORKLOADS[name]
    kv = f", key/value heads {KV_HEADS[name][0]} (large) / {KV_HEADS[name][1]} (small)" if name in KV_HEADS else ""
    return (f"{cfgname}: batch {B}, prompt {P} uniform-random ids, gamma {gamma}, {new} new tokens, "
            f"natural acceptance, random-init N(0,0.02) weights seed 0{kv}")


# DRAM bytes (read + write) of one decode iteration from one ncu capture of every kernel of an iteration, valid only
# while the kernel sources are the ones that were profiled (else the line reports null).
NCU_TRAFFIC = {"workload": "small", "bytes_per_iteration": 599.35e6, "sources_sha256_16": "2379be2240073bf1"}


def kernel_sources_hash():
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2402_08644_b200", "csrc")
    for fn in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, fn), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
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
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes_per_iteration(shape, B, gamma, T):
    """Weights of the large model once, of the small model gamma times, FF_Tandem and the small key/value maps
    once, plus both KV streams at context length T (bf16)."""
    esz = 2 if shape.dtype == synth.DTYPE_BF16 else 4
    def model(d):
        return d.n_layers * (2 * d.d_model ** 2 + 2 * d.d_model * d.d_kv + 2 * d.d_model * d.d_ff) + d.d_model * d.vocab
    L, S = shape.large, shape.small
    proj = S.n_layers * (S.d_model * L.d_model + 2 * S.d_model * S.d_kv) if shape.ff_tandem_kind == 0 else \
        S.n_layers * (shape.hidden * L.d_model + S.d_model * shape.hidden + 2 * S.d_model * S.d_kv)
    kv = B * T * (L.n_layers * 2 * L.d_kv + gamma * S.n_layers * 2 * S.d_kv)
    return esz * (model(L) + gamma * model(S) + proj + kv)


def run_reference(args):
    """The CPU checker as it stands, on the host cores, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import tandem_oracle as O
    cfgname, B, P, gamma, new, max_pos = WORKLOADS[args.workload]
    shape = synth.named_config(cfgname, max_pos)
    weights = synth.make_weights(shape, seed=0)
    prompt = [int(t) for t in synth.make_prompts(B, P, shape.large.vocab, seed=0)[0]]
    sample_new = min(new, 8)
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        o = O.TandemOracle(shape, weights)
        o.prefill(prompt)
        t1 = time.perf_counter()
        while len(o.tokens) - P < sample_new:
            o.step(gamma)
        t2 = time.perf_counter()
        if it >= args.warmup:
            # scale the sample to the full workload: one prompt pass plus `new` tokens at the sampled decode rate
            times.append((t1 - t0) + (t2 - t1) * new / (len(o.tokens) - P))
    sec = float(np.mean(times))
    value = B * new / sec
    cores = os.cpu_count()
    sample = (f"sequence 0 of the workload: full {P}-token prompt pass + {sample_new} new tokens per step, decode time "
              f"scaled to {new} tokens; numpy fp64")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_desc(args.workload)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def cpu_baseline(shape, weights, prompt, gamma, new):
    from oracle import tandem_oracle as O
    P = len(prompt)
    sample_new = min(new, 24)
    t0 = time.perf_counter()
    o = O.TandemOracle(shape, weights)
    o.prefill(prompt)
    t1 = time.perf_counter()
    while len(o.tokens) - P < sample_new:
        o.step(gamma)
    t2 = time.perf_counter()
    sec = (t1 - t0) + (t2 - t1) * new / (len(o.tokens) - P)
    return {"value": new / sec, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": (f"sequence 0: full {P}-token prompt pass ({t1 - t0:.1f} s) + {sample_new} new tokens "
                       f"({t2 - t1:.1f} s), decode time scaled to {new} tokens; numpy fp64 with its BLAS threads")}


def replicas_throughput(local_ms_per_step, units_per_rank, world, device=None):
    """Whole-job throughput of independent replicas: every rank processes `units_per_rank` units per step, the job
    takes as long as its slowest rank (MAX over ranks of the per-step time); returns (units / s, that time in ms)."""
    ms = float(local_ms_per_step)
    if world > 1:
        import torch
        import torch.distributed as dist
        tm = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        ms = float(tm.item())
    return world * units_per_rank / (ms * 1e-3), ms


def run_micro(args):
    """Kernel micro-benchmark: decode attention (16 heads x 64 as in the small models, and the large models' 128-wide
    heads; one query per (sequence, head)) over a large-derived context of T positions plus 4 own positions, and the FF_Tandem projection 4096 -> 1024 with
    the key/value maps, through the stand-alone C entry points.  L2 is flushed between timed calls."""
    import torch
    from paper_2402_08644_b200 import binding, build as _build
    _build.build()
    binding.load_library()
    peak, peak_kind = read_peaks()
    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev).manual_seed(0)

    def timed(fn):
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(5, args.steps)):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    To = 4
    cases = [(B, T, 16, 64) for B in (1, 8, 32) for T in (1024, 8192, 32768)]
    cases += [(1, 8192, 32, 128), (4, 8192, 32, 128), (8, 2048, 16, 128)]    # the large models' head shapes (128-wide heads)
    if args.micro_case:
        v = [int(x) for x in args.micro_case.split(",")]
        cases = [(v[0], v[1], v[2] if len(v) > 2 else 16, v[3] if len(v) > 3 else 64)]
    out = {"metric": "decode_attention_gbs", "unit": "GB/s", "peak": peak, "peak_kind": peak_kind, "dtype": "bf16",
           "data": "synthetic N(0,1) queries, keys and values", "attention": [], "ff_tandem_project": []}
    rn = lambda *s: torch.randn(*s, generator=g, device=dev).to(torch.bfloat16)
    for B, T, H, dh in cases:
        q, kd, vd, ko, vo = rn(B, H, dh), rn(B, H, T, dh), rn(B, H, T, dh), rn(B, H, To, dh), rn(B, H, To, dh)
        o = torch.empty_like(q)
        scratch = torch.empty(1 << 20, dtype=torch.uint8, device=dev)
        ms = timed(lambda: binding.tandem_decode_attention(q, kd, vd, ko, vo, o, scratch))
        byt = 2 * B * H * (T + To) * dh * 2 + 2 * B * H * dh * 2
        out["attention"].append({"batch": B, "heads": H, "d_head": dh, "derived_len": T, "own_len": To, "us": ms * 1e3, "algorithmic_bytes": byt,
                                 "gbs": byt / ms / 1e6, "frac": byt / ms / 1e6 / peak})
        del q, kd, vd, ko, vo
    if not args.micro_case:
        dL, dS = 4096, 1024
        for rows in (4, 32, 128):
            x = rn(rows, dL)
            wt, wk, wv = (rn(dS, k) * 0.02 for k in (dL, dS, dS))
            lg, lb = torch.ones(dS, device=dev), torch.zeros(dS, device=dev)
            ms = timed(lambda: binding.tandem_ff_tandem_project(x, wt, lg, lb, wk, wv))
            byt = (dS * dL + 2 * dS * dS) * 2 + rows * (dL + 2 * dS) * 2
            out["ff_tandem_project"].append({"rows": rows, "us": ms * 1e3, "algorithmic_bytes": byt, "gbs": byt / ms / 1e6,
                                             "frac": byt / ms / 1e6 / peak})
        # the streaming GEMM alone at the feed-forward shapes of the four configurations, 4 token rows
        out["block_linear"] = []
        for K, N in ((512, 2048), (1024, 4096), (2048, 8192), (4096, 11008), (11008, 4096), (4096, 32000)):
            x, w = rn(4, K), rn(N, K) * 0.02
            y = torch.empty(4, N, dtype=torch.bfloat16, device=dev)
            ms = timed(lambda: binding.tandem_block_linear(x, w, y))
            byt = 2 * N * K + 2 * 4 * (K + N)
            out["block_linear"].append({"rows": 4, "in": K, "out": N, "us": ms * 1e3, "algorithmic_bytes": byt,
                                        "gbs": byt / ms / 1e6, "frac": byt / ms / 1e6 / peak})
            del x, w, y
    print(json.dumps(out))


def measure_workload(name, steps, warmup, rank, local_rank, world, extras, keep_for_cpu=False):
    """Times `steps` steps of one workload on this rank's GPU.  Returns a dict of raw timings (ms, per step unless
    stated) plus, with `extras`, the accept-all and plain-greedy decode rates and the per-kernel pass."""
    import torch
    import torch.distributed as dist
    from paper_2402_08644_b200 import binding

    cfgname, B, P, gamma, new, max_pos = WORKLOADS[name]
    shape = synth.named_config(cfgname, max_pos)
    if name in KV_HEADS:
        from dataclasses import replace
        shape = replace(shape, large=replace(shape.large, n_kv_heads=KV_HEADS[name][0]),
                        small=replace(shape.small, n_kv_heads=KV_HEADS[name][1]))
    dev = torch.device("cuda", local_rank)
    if name in DEVICE_INIT:
        weights = synth.device_weights(shape, 0, dev)
    else:
        weights = synth.make_weights(shape, seed=0)
    prompts = [[int(t) for t in p] for p in synth.make_prompts(B, P, shape.large.vocab, seed=rank)]
    gmax = 2 * gamma if extras else gamma     # the adaptive block length of the extras drafts up to 2 gamma tokens
    t = binding.Tandem(shape, weights, max_batch=B, max_seq=P + new + gmax + 1, gamma_max=gmax, device=local_rank,
                       max_prefill_rows=B * P)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_decode(fn, reps):
        """Mean device time (ms) of fn() after a fresh prompt pass, events on the library's stream."""
        tot = 0.0
        for _ in range(reps):
            t.tandem_prefill(prompts)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream); fn(); e1.record(stream)
            torch.cuda.synchronize()
            tot += e0.elapsed_time(e1)
        return tot / reps

    for _ in range(warmup):
        t.tandem_prefill(prompts)
        t.tandem_speculative_generate(gamma, new, 0)

    # ---- device-timed region: K steps between events on the stream the library launches on ----
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    launches0 = t.tandem_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
    ev[0].record(stream)
    iters = 0
    for k in range(steps):
        t.tandem_prefill(prompts)
        ev[2 * k + 1].record(stream)
        out, lens, stats = t.tandem_speculative_generate(gamma, new, 0)
        ev[2 * k + 2].record(stream)
        iters += stats["iterations"]
    barrier()
    clocks = sampler.stop()
    r = {"name": name, "shape": shape, "B": B, "P": P, "gamma": gamma, "new": new, "clocks": clocks,
         "launches": t.tandem_launch_count() - launches0, "accept_hist": stats["accept_hist"],
         "step_ms": ev[0].elapsed_time(ev[-1]) / steps,
         "prefill_ms": sum(ev[2 * k].elapsed_time(ev[2 * k + 1]) for k in range(steps)) / steps,
         "decode_ms": sum(ev[2 * k + 1].elapsed_time(ev[2 * k + 2]) for k in range(steps)) / steps,
         "iters_per_step": iters / steps}

    # ---- end to end through the public calls with host buffers, wall clock, copies included ----
    barrier()
    t0 = time.perf_counter()
    for k in range(steps):
        t.tandem_prefill(prompts)
        out, lens, stats = t.tandem_speculative_generate(gamma, new, 0)
    torch.cuda.synchronize()
    r["e2e_step_ms"] = 1e3 * (time.perf_counter() - t0) / steps
    rows = B * (P - 1)
    group = 128 if shape.dtype == synth.DTYPE_BF16 else 16       # queries per attention group of the prompt pass
    r["h2d"] = 4 * (3 * rows + 2 * (rows // group + B) + 2 * B)  # row token/sequence/position, query groups, n, pending
    r["d2h"] = 4 * (B * new + B + 16) + stats["iterations"] * 20  # tokens, lengths, histogram; 5 counters per iteration

    if extras:
        # context: accept-all timing mode and plain greedy decoding of the large model alone (graphs warmed first)
        for fn in (lambda: t.tandem_speculative_generate(gamma, new, 1), lambda: t.tandem_large_greedy_generate(new)):
            t.tandem_prefill(prompts); fn(); t.tandem_prefill(prompts); fn()
        r["accept_all_decode_ms"] = timed_decode(lambda: t.tandem_speculative_generate(gamma, new, 1), 2)
        r["greedy_decode_ms"] = timed_decode(lambda: t.tandem_large_greedy_generate(new), 2)
        # stand-alone Tandem without the free token (the small model writes the response; Figure 3)
        rep_only = lambda: t.tandem_standalone_generate(gamma, binding.STANDALONE_REPRESENTATION_ONLY, new)
        t.tandem_prefill(prompts); rep_only(); t.tandem_prefill(prompts); rep_only()
        r["representation_only_decode_ms"] = timed_decode(rep_only, 2)
        # sampled SPEED at temperature 1 / 1 (two independent random models still overlap in distribution, so the
        # accept lengths are spread out, unlike the arg-max comparison)
        sampled = lambda: t.tandem_speculative_generate(gamma, new, binding.ACCEPT_SAMPLE, 1)
        t.tandem_prefill(prompts); sampled(); t.tandem_prefill(prompts); sampled()
        r["sampled_decode_ms"] = timed_decode(sampled, 2)
        t.tandem_prefill(prompts)
        r["sampled_accept_hist"] = sampled()[2]["accept_hist"]
        # adaptive block length with a random-init router (mechanism only: the paper's router is trained); gamma_max = 2 gamma
        if t.gamma_max >= 2 * gamma:
            t.tandem_set_router(synth.make_router(shape, 4, 64, seed=0), 0.5)
            adaptive = lambda: t.tandem_adaptive_generate(2 * gamma, new)
            t.tandem_prefill(prompts); adaptive(); t.tandem_prefill(prompts); adaptive()
            r["adaptive_decode_ms"] = timed_decode(adaptive, 2)
            t.tandem_prefill(prompts)
            st = adaptive()[2]
            r["adaptive_runs"] = {"large_runs": st["large_runs"], "small_runs": st["small_runs"], "gamma_max": 2 * gamma, "tau": 0.5}
        # per-kernel pass: the same step with every launch bracketed by events (serialises the stream: shares only)
        t.tandem_profile_enable(400000)
        t.tandem_prefill(prompts)
        t.tandem_speculative_generate(gamma, new, 0)
        r["prof"] = t.tandem_profile_read()
        t.tandem_profile_enable(0)
    t.close()
    if keep_for_cpu:
        r["weights"], r["prompt0"] = weights, prompts[0]
    del t, weights
    torch.cuda.empty_cache()
    return r


FLOP_CLASSES = ("gemm_tiled", "gemm_tc_tiled", "attn_prompt")     # prompt-pass kernels: work counted in flops


def iteration_roofline(r, peak):
    """Whole-iteration view of the decode phase: algorithmic bytes of one draft / verify iteration (weights of the
    large model once, of the small model gamma times, projection and key/value maps once, both KV streams at the
    mean context length) over the measured device time per iteration."""
    T_avg = r["P"] + r["new"] / 2
    it_bytes = algorithmic_bytes_per_iteration(r["shape"], r["B"], r["gamma"], T_avg)
    it_ms = r["decode_ms"] / r["iters_per_step"]
    gbs = it_bytes / 1e9 / (it_ms * 1e-3)
    return {"algorithmic_gb": it_bytes / 1e9, "us": 1e3 * it_ms, "achieved_gbs": gbs, "frac_of_peak": gbs / peak}


def sub_record(r, peak):
    """Compact record of one workload for the default line."""
    it = iteration_roofline(r, peak)
    toks = r["B"] * r["new"]
    rec = {"workload": workload_desc(r["name"]), "decode_tokens_per_s": toks / (r["decode_ms"] * 1e-3),
           "step_tokens_per_s": toks / (r["step_ms"] * 1e-3), "prefill_ms": r["prefill_ms"], "decode_ms": r["decode_ms"],
           "us_per_iteration": it["us"], "algorithmic_gb_per_iteration": it["algorithmic_gb"],
           "achieved_gbs": it["achieved_gbs"], "frac_of_peak": it["frac_of_peak"], "accept_hist": r["accept_hist"],
           "gpu_launches": int(r["launches"]), "clocks": r["clocks"]}
    if "accept_all_decode_ms" in r:
        rec["accept_all_decode_tokens_per_s"] = toks / (r["accept_all_decode_ms"] * 1e-3)
        rec["large_greedy_decode_tokens_per_s"] = toks / (r["greedy_decode_ms"] * 1e-3)
        rec["standalone_representation_only_decode_tokens_per_s"] = toks / (r["representation_only_decode_ms"] * 1e-3)
        rec["sampled_decode_tokens_per_s"] = toks / (r["sampled_decode_ms"] * 1e-3)
        rec["sampled_accept_hist"] = r["sampled_accept_hist"]
        if "adaptive_decode_ms" in r:
            rec["adaptive_decode_tokens_per_s"] = toks / (r["adaptive_decode_ms"] * 1e-3)
            rec["adaptive_runs"] = r["adaptive_runs"]
    return rec


def run_prefill_only(args, local_rank):
    """The prompt pass alone (large model over the prompt, FF_Tandem projection of every position): device time per
    pass and the tensor-core rate over its algorithmic flops (2 x parameters x rows for the linear maps, 2 d T^2 per
    layer and sequence for the causal attention)."""
    import torch
    from dataclasses import replace
    from paper_2402_08644_b200 import binding
    cfgname, B, P, gamma, new, max_pos = WORKLOADS[args.workload]
    shape = synth.named_config(cfgname, max_pos)
    if args.layers > 0:
        shape = synth.make_shape(replace(shape.large, n_layers=args.layers), replace(shape.small, n_layers=min(args.layers, shape.small.n_layers)),
                                 shape.ff_tandem_kind, shape.ff_tandem_hidden, None, shape.dtype)
    dev = torch.device("cuda", local_rank)
    weights = synth.device_weights(shape, 0, dev)
    prompts = [[int(t) for t in p] for p in synth.make_prompts(B, P, shape.large.vocab, seed=0)]
    t = binding.Tandem(shape, weights, max_batch=B, max_seq=P + 8, gamma_max=gamma, device=local_rank, max_prefill_rows=B * P)
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        t.tandem_prefill(prompts)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        t.tandem_prefill(prompts)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    L, S = shape.large, shape.small
    rows = B * (P - 1)
    lin = L.n_layers * (2 * L.d_model ** 2 + 2 * L.d_model * L.d_kv + 2 * L.d_model * L.d_ff) + \
        S.n_layers * (S.d_model * L.d_model + 2 * S.d_model * S.d_kv)
    flops = 2.0 * lin * rows + L.n_layers * 2.0 * L.d_model * B * float(P - 1) ** 2
    t.close()
    print(json.dumps({"metric": "prompt_pass_ms", "value": ms, "unit": "ms", "workload": workload_desc(args.workload),
                      "layers": [L.n_layers, S.n_layers], "rows": rows, "algorithmic_tflop": flops / 1e12,
                      "tflops": flops / 1e12 / (ms * 1e-3), "steps": args.steps, "warmup": args.warmup}))


def run_ours(args, rank, local_rank, world):
    import torch
    import torch.distributed as dist
    extras = rank == 0 and not args.no_extras
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and args.workload not in DEVICE_INIT
    r = measure_workload(args.workload, args.steps, args.warmup, rank, local_rank, world, extras, keep_for_cpu=want_cpu)
    B, new, shape = r["B"], r["new"], r["shape"]
    toks = B * new
    # value: generated tokens per second of the decode phase (all ranks' tokens over the slowest rank's time); the
    # prompt pass of the same step is timed separately (prefill_ms) and included in ms_per_step and step_tokens_per_s
    value, decode_ms = replicas_throughput(r["decode_ms"], toks, world, "cuda")
    step_value, ms_per_step = replicas_throughput(r["step_ms"], toks, world, "cuda")
    e2e_value, _ = replicas_throughput(r["e2e_step_ms"], toks, world, "cuda")
    peak, peak_kind = read_peaks()
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if shape.dtype == synth.DTYPE_BF16 else "f32", "data": "synthetic",
            "config": {"workload": workload_desc(args.workload), "parallelism": f"replicas x{world}",
                       "value_scope": "decode phase (draft, verify, project, accept) of each step; the step's prompt pass is "
                                      "in ms_per_step, prefill_ms and step_tokens_per_s",
                       "l2": "per-iteration working set (weights + KV) exceeds the 126 MB L2; no flush needed"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"],
                    "scope": "whole step through the C calls with host buffers (prompt pass + decode), wall clock"},
            "gpu_launches": int(r["launches"]), "clocks": r["clocks"], "prefill_ms": r["prefill_ms"], "decode_ms": decode_ms,
            "step_tokens_per_s": step_value, "iterations_per_step": r["iters_per_step"], "accept_hist": r["accept_hist"]}

    if extras:
        it = iteration_roofline(r, peak)
        prof = r["prof"]
        line["accept_all_decode_tokens_per_s"] = toks / (r["accept_all_decode_ms"] * 1e-3)
        line["large_greedy_decode_tokens_per_s"] = toks / (r["greedy_decode_ms"] * 1e-3)
        line["standalone_representation_only_decode_tokens_per_s"] = toks / (r["representation_only_decode_ms"] * 1e-3)
        line["sampled_decode_tokens_per_s"] = toks / (r["sampled_decode_ms"] * 1e-3)
        line["sampled_accept_hist"] = r["sampled_accept_hist"]
        if "adaptive_decode_ms" in r:
            line["adaptive_decode_tokens_per_s"] = toks / (r["adaptive_decode_ms"] * 1e-3)
            line["adaptive_runs"] = r["adaptive_runs"]
        tot = sum(v["ms"] for v in prof.values()) or 1.0
        # bracketed pass: work = algorithmic bytes (GB/s) for the streaming kernels, flops (TFLOP/s) for the prompt pass
        line["kernels_bracketed"] = {
            k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / tot, 4),
                "avg_us": round(1e3 * v["ms"] / max(1, v["launches"]), 3),
                "rate": round(v["work"] / (v["ms"] * 1e-3) / (1e12 if k in FLOP_CLASSES else 1e9), 1) if v["ms"] > 0 else 0.0}
            for k, v in prof.items() if v["launches"]}
        decode_classes = [k for k in prof if k not in FLOP_CLASSES]
        dec_tot = sum(prof[k]["ms"] for k in decode_classes) or 1.0
        dom = max(decode_classes, key=lambda k: prof[k]["ms"])
        g = prof[dom]
        # the dominant kernel inside the timed region: its share of the bracketed decode time applied to the
        # device-timed decode phase (graph replay, overlapped launches), so launches x time never exceeds the step
        piped_ms = r["decode_ms"] * g["ms"] / dec_tot
        traffic = None
        if args.workload == NCU_TRAFFIC["workload"] and kernel_sources_hash() == NCU_TRAFFIC["sources_sha256_16"]:
            traffic = NCU_TRAFFIC["bytes_per_iteration"]
        line["roofline"] = {
            "bound": "hbm", "scope": "one draft / verify iteration of the decode phase, all kernels",
            "achieved": it["achieved_gbs"], "peak": peak, "unit": "GB/s", "frac": it["frac_of_peak"], "traffic": traffic,
            "peak_kind": peak_kind, "algorithmic_bytes": it["algorithmic_gb"] * 1e9, "us": it["us"],
            "dominant_kernel": {"kernel": dom, "launches": g["launches"], "share_of_decode": g["ms"] / dec_tot,
                                "avg_launch_us": 1e3 * piped_ms / max(1, g["launches"]),
                                "algorithmic_bytes_per_launch": g["work"] / max(1, g["launches"]),
                                "achieved": g["work"] / 1e9 / (piped_ms * 1e-3),
                                "frac": g["work"] / 1e9 / (piped_ms * 1e-3) / peak}}
    if want_cpu:
        line["cpu_baseline"] = cpu_baseline(shape, r.pop("weights"), r.pop("prompt0"), r["gamma"], new)
    if extras and world == 1 and args.workload == "small" and not args.no_subrecords:
        # the other batch sizes of the metric: batch 8 (medium) and the bandwidth-bound batch 1 (large), few steps each
        line["workloads"] = {}
        for name in ("medium", "large", "large_gqa"):
            rr = measure_workload(name, 2, 3, rank, local_rank, world, extras=True)
            rr.pop("prof", None)
            line["workloads"][name] = sub_record(rr, peak)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="small", choices=sorted(WORKLOADS) + ["micro"])
    ap.add_argument("--micro-case", default="", help="with --workload micro: one attention case 'batch,context[,heads,d_head]'")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the accept-all / greedy / per-kernel passes")
    ap.add_argument("--no-subrecords", action="store_true", help="skip the medium / large sub-records of the default line")
    ap.add_argument("--prefill-only", action="store_true", help="time the prompt pass alone (steps = prompt passes); prints its own JSON line")
    ap.add_argument("--layers", type=int, default=0, help="with --prefill-only: cut both models to this many layers (small cases for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.workload == "micro":
        run_micro(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2402_08644_b200 import binding, build as _build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()

    if args.prefill_only:
        run_prefill_only(args, local_rank)
    else:
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
