#!/usr/bin/env python
"""Benchmark of the TPI-LLM decoder hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload C2]

One "step" is one pass of the whole per-token hot path (embedding, L x [norm,
column-sharded QKV + RoPE + KV append, attention over the cache, row-sharded O ->
N partials, rank-ordered sum + shortcut, norm, gate/up + SwiGLU, down -> partials,
sum + shortcut], final norm, task head, greedy argmax) on the workload C2:
a Llama-2-7B-shaped decoder, bf16 weights, fp32 accumulation, N = 4 shards
emulated on one GPU, prompt of 128 random tokens, all weights resident.

Prints ONE JSON line.  `value` is decode tokens/s with everything resident on the
device (token ids chained on the device, one host wait for the K steps, CUDA
events on the launching stream); `e2e` is the same metric through the public
per-token call with the token id copied host->device and the result device->host
every step.  TTFT (the prompt pass) and the whole-token roofline are extra keys.
With --gpus N > 1 (torchrun) every rank runs an independent replica: the method's
path on one GPU has no exchange step (all shards are emulated on-device).
"""
from __future__ import annotations

import argparse
import json
import os
import re
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import tpi_synth as S  # noqa: E402

METRIC = "decode_tokens_per_s_batch1"
UNIT = "tokens/s"


# ------------------------------------------------------------------ helpers
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak():
    """Measured dense bf16 throughput (TFLOP/s): (burst, sustained), kind."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


def ttft_roofline(shape, T, ttft_ms, weight_bytes, hbm_gbs):
    """The prompt pass against the slower of: every weight byte once over HBM, and its matrix products plus causal
    attention on the tensor cores at the measured bf16 rate (one product per activation: the split-bf16 scheme's second
    product is overhead).  The rate is the burst figure below ~10 ms of ideal time, the sustained one above."""
    a, b, d, h, s_, L, v = shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.hidden, shape.ffn, shape.n_layers, shape.vocab
    per_layer = (a + 2 * b) * d * h + a * d * h + 3 * h * s_
    flops = 2.0 * T * L * per_layer + 2.0 * v * h + 4.0 * (T * (T + 1) / 2) * a * d * L
    burst, sustained, kind = tensor_peak()
    t_hbm = weight_bytes / (hbm_gbs * 1e9) * 1e3
    t_tc = flops / (burst * 1e12) * 1e3
    if t_tc > 10.0:
        t_tc = flops / (sustained * 1e12) * 1e3
    ideal = max(t_hbm, t_tc)
    return {"bound": "hbm" if t_hbm >= t_tc else "tensor", "ideal_ms": ideal, "hbm_ms": t_hbm, "tensor_ms": t_tc,
            "flops": flops, "frac": ideal / ttft_ms, "peak_kind": kind}


def traffic_from_profile(workload: str):
    """DRAM bytes per launch of the dominant kernel, from the committed ncu summary (or None)."""
    p = os.path.join(ROOT, "profiles", f"wstream_gateup_{workload.lower()}.md")
    if os.path.exists(p):
        m = re.search(r"traffic_bytes_per_launch:\s*([0-9.eE+]+)", open(p).read())
        if m:
            return float(m.group(1))
    return None


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.rows, self.proc = index, [], None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                self.rows.append([c.strip() for c in line.split(",")])
        except Exception:
            pass

    def stop(self) -> dict:
        if self.proc:
            self.proc.terminate()
        self.join(timeout=2)
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = max(mx, float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except (ValueError, IndexError):
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


def tpi_config(shape: S.ModelShape, max_seq: int, max_prefill: int):
    import paper_2410_00531_b200 as P
    return P.make_config(n_layers=shape.n_layers, hidden=shape.hidden, n_heads=shape.n_heads,
                         n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn,
                         vocab=shape.vocab, max_seq=max_seq, max_prefill=max_prefill,
                         rms_eps=shape.rms_eps, rope_base=shape.rope_base, dtype=shape.dtype)


def make_oracle(shape: S.ModelShape):
    """The CPU fp64 oracle on the generator's weights (only the CPU-baseline legs come here)."""
    import functools
    from oracle.llama_oracle import LlamaOracle, OracleConfig

    @functools.lru_cache(maxsize=64)
    def w(layer: int, tid: int):
        return S.as_f64(S.gen_tensor(shape, layer, tid))
    cfg = OracleConfig(shape.n_layers, shape.hidden, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                       shape.vocab, shape.rms_eps, shape.rope_base, "bf16" if shape.dtype == "bf16" else "none")
    return LlamaOracle(cfg, w)


def oracle_sample(shape: S.ModelShape, n_tokens: int, l_red: int = 2, ctx: int = 16):
    """Time the CPU fp64 oracle, as it stands, on a bounded sample of the workload:
    `l_red` layers at full width + the task head, `n_tokens` decode steps after a `ctx`-token
    prompt; per-layer time is scaled linearly to the full depth.  Weight generation is excluded."""
    red = shape.with_(n_layers=l_red)
    orc = make_oracle(red)
    toks = S.prompt_tokens(red, ctx)
    orc.forward(toks)                       # also pulls every weight through the generator once
    t_steps = []
    tok = 1
    for _ in range(n_tokens):
        t0 = time.perf_counter()
        lg = orc.forward([tok])
        t_steps.append(time.perf_counter() - t0)
        tok = int(np.argmax(lg))
    # split one more step into layer part and head part
    t0 = time.perf_counter()
    x = orc.w(0, S.EMB)[[tok]]
    pos = np.array([orc.cache.length])
    for l in range(l_red):
        _, x, _, _ = orc.layer_unsharded(l, x, pos, orc.cache.K[l], orc.cache.V[l])
    t_layers = time.perf_counter() - t0
    t_step = float(np.median(t_steps))
    t_head = max(t_step - t_layers, 0.0)
    t_full = t_layers / l_red * shape.n_layers + t_head
    return 1.0 / t_full, t_steps, f"{l_red} of {shape.n_layers} layers at full width + head, {n_tokens} decode steps at context {ctx}, per-layer time scaled to {shape.n_layers} layers"


def run_reference(args, shape):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    # warm-up and timed steps are both bounded samples (2 layers + head per step)
    n = max(1, args.steps)
    t0 = time.perf_counter()
    value, steps, sample = oracle_sample(shape, args.warmup + n)
    steps = steps[args.warmup:]
    ms = float(np.mean(steps)) * 1e3
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": workload_name(shape, args),
                      "note": "ms_per_step is the timed step (a bounded sample: 2 layers + head); value is tokens/s "
                              "with the per-layer time scaled to the full depth",
                      "full_depth_ms_per_step_extrapolated": 1e3 / value},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0, "wall_s": time.perf_counter() - t0}
    print(json.dumps(out), flush=True)


def workload_name(shape, args):
    return (f"{args.workload}: {shape.name}, L{shape.n_layers} h{shape.hidden} a{shape.n_heads} b{shape.n_kv_heads} "
            f"s{shape.ffn} v{shape.vocab}, {shape.dtype} weights/KV, fp32 accumulate, N={shape.n_shards} shards "
            f"emulated on one GPU, prompt {shape.prompt_len}, all weights resident")


def max_over_ranks(x: float, device: str = "cpu") -> float:
    """Slowest rank's time: replicas run independently, the job is as slow as its slowest replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(steps: int, ms: float, world: int) -> float:
    """Tokens per second of the whole job: every one of `world` replicas decoded `steps` tokens in `ms`."""
    return world * steps / (ms * 1e-3)


# ------------------------------------------------------------------ GPU arm
def open_session(P, shape, local, max_seq, prefill_chunk, window=0, retain=0, longest_prompt=0):
    """Load a model (weights from the seeded generator) into fresh arenas; returns (session, seconds)."""
    import torch
    cfg = tpi_config(shape, max_seq, min(max(shape.prompt_len, longest_prompt), prefill_chunk))
    t0 = time.perf_counter()
    extra = 0
    if window > 0 and retain > 0:      # room for the kept FFN blocks beside the window (Prop. 6)
        extra = len(range(0, shape.n_layers, retain)) * P.block_bytes(cfg)[1]
    elif window > 0 and retain == -1:  # as many as fit in what the GPU has free (leave 8 GiB of headroom)
        free_b, _ = torch.cuda.mem_get_info(local)
        base = P.query_arena(cfg, shape.n_shards, window, True)[0]
        extra = max(0, min(shape.n_layers * P.block_bytes(cfg)[1], free_b - base - (8 << 30)))
    ses = P.Session(cfg, S.synth_fill(shape), shape.n_shards, window, device=local, extra_dev_bytes=extra)
    if extra:
        P.set_retention(ses.h, retain)           # -1: the library picks the smallest T that fits the arena
    return ses, time.perf_counter() - t0


def close_session(ses):
    import torch
    ses.close()
    del ses
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def kv_bytes_per_token(shape, ctx):
    B = 2 if shape.dtype == "bf16" else 4
    return 2 * shape.n_layers * shape.n_kv_heads * shape.head_dim * B * (ctx + 1)


def resident_decode(P, ses, shape, local, K, W, world=1, n_ttft=4):
    """TTFT (best of n_ttft - 1 prompt passes after a warm one) and K device-chained decode steps after W warm-up
    steps, timed with CUDA events on the launching stream between barriers, clocks sampled meanwhile."""
    import torch
    h, T = ses.h, shape.prompt_len
    toks = S.prompt_tokens(shape)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    ttft = []
    for _ in range(n_ttft):
        P.reset(h)
        t0 = time.perf_counter()
        first, _ = P.prefill(h, toks, 0)
        ttft.append((time.perf_counter() - t0) * 1e3)
    ttft_ms = min(ttft[1:]) if len(ttft) > 1 else ttft[0]
    tok = int(P.decode_run(h, first, W)[-1]) if W else first
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.5)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(ses.compute):
        e0.record()
        out = P.decode_run(h, tok, K)
        e1.record()
    barrier()
    dev_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    st = P.get_stats(h)
    dev_ms = max_over_ranks(dev_ms, f"cuda:{local}")
    token_bytes = st["weight_bytes_per_token"] + kv_bytes_per_token(shape, T + W + K / 2)
    return {"first": first, "out": out, "dev_ms": dev_ms, "clocks": clocks, "stats": st, "ttft_ms": ttft_ms,
            "token_bytes": token_bytes, "token_gbs": token_bytes / (dev_ms / K * 1e-3) / 1e9, "barrier": barrier}


def resident_leg(P, name, shape, local, K, W, prefill_chunk, long_ctx=0):
    """One more resident workload in compact form (tokens/s, whole-token HBM fraction, TTFT and its fraction).
    long_ctx > 0: on the same loaded model, also a prompt of that many tokens (TTFT, one pass) and 16 decoded tokens on
    top of it, reported under "long_context"."""
    T = shape.prompt_len
    peak, kind = measured_peaks()
    ses, load_s = open_session(P, shape, local, max(T + W + K, long_ctx + 24) + 8, prefill_chunk, longest_prompt=long_ctx)
    extra = None
    try:
        r = resident_decode(P, ses, shape, local, K, W, n_ttft=3)
        if long_ctx:
            sl = shape.with_(prompt_len=long_ctx)
            rl = resident_decode(P, ses, sl, local, 16, 3, n_ttft=1)
            trl = ttft_roofline(sl, long_ctx, rl["ttft_ms"], rl["stats"]["weight_bytes_per_token"], peak)
            extra = {"context": f"{long_ctx + 3}..{long_ctx + 19}", "steps": 16, "tokens_per_s": round(16 / (rl["dev_ms"] * 1e-3), 2),
                     "hbm_frac": round(rl["token_gbs"] / peak, 4), "ttft_ms": round(rl["ttft_ms"], 1), "ttft_prompt_tokens": long_ctx,
                     "ttft_bound": trl["bound"], "ttft_frac": round(trl["frac"], 4), "clocks": short_clocks(rl["clocks"])}
    finally:
        close_session(ses)
    tr = ttft_roofline(shape, T, r["ttft_ms"], r["stats"]["weight_bytes_per_token"], peak)
    out = _resident_leg_dict(name, shape, K, W, T, r, peak, tr)
    if extra:
        out["long_context"] = extra
    return out


def _resident_leg_dict(name, shape, K, W, T, r, peak, tr):
    return {"workload": f"{name} {shape.name} N={shape.n_shards} resident", "steps": K,
            "context": f"{T + W}..{T + W + K}", "tokens_per_s": round(K / (r["dev_ms"] * 1e-3), 2),
            "ms_per_step": round(r["dev_ms"] / K, 4), "hbm_gbs": round(r["token_gbs"], 1),
            "hbm_frac": round(r["token_gbs"] / peak, 4), "ttft_ms": round(r["ttft_ms"], 2), "ttft_prompt_tokens": T,
            "ttft_bound": tr["bound"], "ttft_frac": round(tr["frac"], 4), "clocks": short_clocks(r["clocks"])}


def short_clocks(c: dict) -> dict:
    return {"sm_mhz": c.get("sm_mhz"), "reasons": c.get("reasons"), "samples": c.get("samples")}


def host_link_peak(torch, local: int) -> float:
    """Pinned host -> device copy rate of this machine (GB/s), 2 GiB, best of 10 after two warm copies: the streamed runs'
    denominator (a plain cudaMemcpyAsync, so a well-fed ring can read a little above it)."""
    n = 2 << 30
    hbuf = torch.empty(n, dtype=torch.uint8, pin_memory=True)
    dbuf = torch.empty(n, dtype=torch.uint8, device=f"cuda:{local}")
    hbuf.zero_()
    best = 0.0
    for it in range(12):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dbuf.copy_(hbuf, non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        if it >= 2:
            best = max(best, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del hbuf, dbuf
    return best


def streamed_decode(P, ses, shape, local, K, W):
    """Window-streamed decode in its steady state: after the prompt pass and W warm-up tokens the device is drained
    (the window is then full and none of its bytes count), K tokens are enqueued in one call and the region ends when
    both streams are idle again, so every block copy issued inside the region also completed inside it.  Tokens/s and
    link GB/s are K tokens, resp. ALL bytes copied in the region, over the region's wall time."""
    import torch
    h = ses.h
    toks = S.prompt_tokens(shape)
    t0 = time.perf_counter()
    first, _ = P.prefill(h, toks, 0)
    ttft_ms = (time.perf_counter() - t0) * 1e3
    tok = int(P.decode_run(h, first, W)[-1]) if W else first
    sampler = ClockSampler(local)
    sampler.start()
    torch.cuda.synchronize()
    st0 = P.get_stats(h)
    t0 = time.perf_counter()
    out = P.decode_run(h, tok, K)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    clocks = sampler.stop()
    st = P.get_stats(h)
    region_bytes = st["link_bytes_total"] - st0["link_bytes_total"]
    return {"out": out, "wall_s": wall, "clocks": clocks, "stats": st, "ttft_ms": ttft_ms,
            "region_bytes": region_bytes, "link_gbs": region_bytes / wall / 1e9, "tokens_per_s": K / wall}


def streamed_leg(P, name, shape, local, K, W, window, link_peak, retain=0):
    # The first launch of a kernel in a process loads its code (tens of milliseconds per kernel): a one-layer resident
    # model of the same widths runs the prompt pass and two tokens first, so that the TTFT below times the streamed pass.
    warm = shape.with_(n_layers=1, vocab=1024)
    wses, _ = open_session(P, warm, local, warm.prompt_len + 8, 4096)
    try:
        t, _ = P.prefill(wses.h, S.prompt_tokens(warm), 0)
        P.decode_run(wses.h, t, 2)
    finally:
        close_session(wses)
    ses, load_s = open_session(P, shape, local, shape.prompt_len + W + K + 16, 4096, window, retain)
    try:
        r = streamed_decode(P, ses, shape, local, K, W)
        P.set_option(ses.h, P.OPT_PROFILE, 1)    # the paper's diagnostics on two more tokens, outside the timed region
        P.scheduler_reset(ses.h)
        P.decode_run(ses.h, int(r["out"][-1]), 2)
        import torch
        torch.cuda.synchronize()
        sched = P.scheduler_report(ses.h)
    finally:
        close_session(ses)
    st = r["stats"]
    return {"workload": f"{name} {shape.name} L{shape.n_layers} streamed, window {window}"
                        + (f", retain T={sched['retain_every_T']}" if retain else ""),
            "steps": K, "tokens_per_s": round(r["tokens_per_s"], 4), "ms_per_step": round(r["wall_s"] / K * 1e3, 2),
            "link_GB_per_token": round(r["region_bytes"] / K / 1e9, 3), "link_gbs": round(r["link_gbs"], 2),
            "link_peak_gbs": round(link_peak, 2), "link_frac": round(r["link_gbs"] / link_peak, 4),
            "ttft_ms": round(r["ttft_ms"], 1), "ttft_prompt_tokens": shape.prompt_len,
            "ttft_link_frac": round(r["region_bytes"] / K / (r["ttft_ms"] * 1e-3) / 1e9 / link_peak, 4),
            "tau_over_t": [round(sched["tau_attn_ms"] / max(sched["t_attn_ms"], 1e-9), 1),
                           round(sched["tau_ffn_ms"] / max(sched["t_ffn_ms"], 1e-9), 1)],
            "loose_holds": sched["loose_holds"], "clocks": short_clocks(r["clocks"])}


def tp_one_gpu_leg(P, shape, local, R, K, W):
    """The one-shard-per-rank form with all R ranks on THIS GPU (they take turns on it; every exchange is ordered by
    events): shows that the path runs at the workload's full size and what its launch sequence costs when nothing runs
    in parallel.  Not a multi-GPU measurement."""
    import torch
    import paper_2410_00531_b200.tp as TP
    T = shape.prompt_len
    cfg = tpi_config(shape, T + W + K + 8, T)
    t0 = time.perf_counter()
    g = TP.Group(cfg, S.synth_fill(shape), R, 0, device=local)
    load_s = time.perf_counter() - t0
    try:
        toks = S.prompt_tokens(shape)
        g.prefill(toks, 0)
        g.reset()
        t0 = time.perf_counter()
        first, _ = g.prefill(toks, 0)
        ttft_ms = (time.perf_counter() - t0) * 1e3
        tok = int(g.decode_run(first, W)[-1])
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.5)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        out = g.decode_run(tok, K)
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        clocks = sampler.stop()
        st = g.stats()
    finally:
        g.close()
        import gc
        gc.collect()
        torch.cuda.empty_cache()
    return {"workload": f"{shape.name}: {R} ranks, one shard each, ALL ON ONE GPU (time-shared; functional, not a multi-GPU number)",
            "steps": K, "tokens_per_s": round(K / wall, 2), "ms_per_step": round(wall / K * 1e3, 3), "ttft_ms": round(ttft_ms, 2),
            "ttft_prompt_tokens": T, "launches_per_token": st["kernel_launches_last"] // K,
            "exchange_bytes_per_token_per_rank": st["exchange_bytes_per_token"], "clocks": short_clocks(clocks)}


def extra_legs(P, args, local):
    """The other listed workloads, measured in the same process after the headline: the 8B shape at its 4096-token
    context and the 70B shape, both resident; then the window-streamed path on 70B-shaped blocks, bf16 and fp32, at a
    depth that keeps each run near half a minute (the bytes per block and the link rate are what is measured; depth
    only scales the time per token)."""
    import torch
    legs = {}

    def run(key, fn):
        t0 = time.perf_counter()
        try:
            legs[key] = fn()
            legs[key]["leg_s"] = round(time.perf_counter() - t0)
        except Exception as e:   # a leg that cannot run on this machine (memory) must not take the headline down
            legs[key] = {"error": f"{type(e).__name__}: {e}"[:300]}
            torch.cuda.empty_cache()

    want = set(args.legs.split(","))
    if "C3" in want:
        run("C3", lambda: resident_leg(P, "C3", S.CONFIGS["C3"], local, 256, 5, args.prefill_chunk))
    if "C5" in want:
        run("C5", lambda: resident_leg(P, "C5", S.CONFIGS["C5"], local, 32, 4, args.prefill_chunk, long_ctx=8192))
    if "TP" in want:
        run("C2_4_ranks_one_gpu", lambda: tp_one_gpu_leg(P, S.CONFIGS["C2"], local, 4, 32, 4))
    if "S5" in want or "S4" in want:
        link_peak = host_link_peak(torch, local)
        if "S5" in want:
            run("C5_streamed", lambda: streamed_leg(P, "C5-shaped", S.CONFIGS["C5"].with_(n_layers=10, prompt_len=512),
                                                    local, 16, 2, 8, link_peak))
        if "S4" in want:
            run("C4_streamed", lambda: streamed_leg(P, "C4-shaped", S.CONFIGS["C4"].with_(n_layers=5, prompt_len=512),
                                                    local, 16, 2, 8, link_peak))
    return legs


def run_gpu(args, shape):
    import torch
    import paper_2410_00531_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    K, W, T = args.steps, args.warmup, shape.prompt_len
    if args.window > 0:
        return run_streamed(args, shape, local, rank)
    if args.tp > 0:  # the one-shard-per-rank form with all ranks on this GPU, alone (short runs under a profiler)
        if rank == 0:
            print(json.dumps(tp_one_gpu_leg(P, shape, local, args.tp, K, W)), flush=True)
        return
    ses, t_load = open_session(P, shape, local, T + W + K + 8, args.prefill_chunk)
    h = ses.h
    toks = S.prompt_tokens(shape)
    r = resident_decode(P, ses, shape, local, K, W, world, n_ttft=1 if args.quick else 4)
    barrier, dev_ms, st, out = r["barrier"], r["dev_ms"], r["stats"], r["out"]
    launches = st["kernel_launches_last"]
    value = whole_job_value(K, dev_ms, world)

    if args.quick:   # profiling aid: device-resident decode only
        if rank == 0:
            print(json.dumps({"quick": True, "value": value, "ms_per_step": dev_ms / K, "gpu_launches": launches}), flush=True)
        ses.close()
        return
    # ---- end to end: the per-token public call, token id H2D and result D2H every step
    P.reset(h)
    first, _ = P.prefill(h, toks, 0)
    tok = first
    for _ in range(W):
        tok, _ = P.decode_step(h, tok, 0)
    barrier()
    t0 = time.perf_counter()
    for _ in range(K):
        tok, _ = P.decode_step(h, tok, 0)
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, f"cuda:{local}")
    e2e = whole_job_value(K, e2e_s * 1e3, world)

    # ---- roofline of the dominant kernel (gate/up GEMV): CUDA events around each launch.  Profile mode runs the step
    # as plain serialised stream launches (no graph, no programmatic dependent launch), so each launch is timed alone.
    P.set_option(h, P.OPT_PROFILE, 1)
    for _ in range(3):
        tok, _ = P.decode_step(h, tok, 0)
    sp = P.get_stats(h)
    P.set_option(h, P.OPT_PROFILE, 0)
    peak, peak_kind = measured_peaks()
    achieved = sp["dominant_kernel_bytes"] / (sp["dominant_kernel_ms"] * 1e-3) / 1e9 if sp["dominant_kernel_ms"] else None
    close_session(ses)
    if rank != 0:
        return
    # ---- CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        v, _, sample = oracle_sample(shape, 4)
        cpu = {"value": v, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle", "sample": sample}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": dev_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": shape.dtype, "data": "synthetic",
        "config": {"workload": workload_name(shape, args), "context": f"{T + W}..{T + W + K}",
                   "l2": "inputs larger than L2: every step streams %.2f GB of weights" % (st["weight_bytes_per_token"] / 1e9),
                   "parallelism": "replicas" if world > 1 else "single GPU, N shards emulated",
                   "graph": bool(st["graph_active"]), "load_s": round(t_load, 1)},
        "clocks": r["clocks"],
        "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": 4, "d2h_bytes_per_step": 8},
        "gpu_launches": launches,
        "ttft_ms": r["ttft_ms"], "ttft_prompt_tokens": T,
        "ttft_roofline": ttft_roofline(shape, T, r["ttft_ms"], st["weight_bytes_per_token"], peak),
        "token_roofline": {"bound": "hbm", "bytes_per_token": r["token_bytes"], "achieved": r["token_gbs"], "peak": peak,
                           "unit": "GB/s", "frac": r["token_gbs"] / peak, "peak_kind": peak_kind},
        "roofline": {"bound": "hbm", "kernel": "wstream_cols_kernel<bf16,EPI_SWIGLU> (gate/up + SwiGLU)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak if achieved else None, "traffic": traffic_from_profile(args.workload),
                     "bytes_per_launch": sp["dominant_kernel_bytes"], "ms_per_launch": sp["dominant_kernel_ms"],
                     "launches_timed": sp["dominant_kernel_samples"], "peak_kind": peak_kind},
        "cpu_baseline": cpu,
        "tokens_tail": [int(x) for x in out[-4:]],
    }
    if world == 1 and args.legs and args.workload == "C2" and not (args.layers or args.prompt or args.shards):
        line["legs"] = extra_legs(P, args, local)
    print(json.dumps(line), flush=True)


def run_streamed(args, shape, local, rank):
    """`--window W`: the streamed path as the headline of its own line (steady-state arithmetic as in the legs)."""
    import torch
    import paper_2410_00531_b200 as P
    K, W, T = args.steps, args.warmup, shape.prompt_len
    ses, t_load = open_session(P, shape, local, T + W + 2 * K + 24, args.prefill_chunk, args.window, args.retain)
    h = ses.h
    r = streamed_decode(P, ses, shape, local, K, W)
    st, out = r["stats"], r["out"]
    # e2e: the per-token public call (same link bytes per step, one host round trip per token)
    tok = int(out[-1])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(K):
        tok, _ = P.decode_step(h, tok, 0)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    attn_b, ffn_b = P.block_bytes(ses.cfg)
    # the paper's scheduler diagnostics on a few extra tokens (event-timed per block: outside every timed region)
    P.set_option(h, P.OPT_PROFILE, 1)
    P.scheduler_reset(h)
    P.decode_run(h, tok, min(K, 4))
    torch.cuda.synchronize()
    sched = P.scheduler_report(h)
    close_session(ses)
    peak = host_link_peak(torch, local)
    link_bytes = r["region_bytes"] / K
    line = {
        "metric": METRIC, "value": r["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
        "ms_per_step": r["wall_s"] / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": shape.dtype, "data": "synthetic",
        "config": {"workload": workload_name(shape, args).replace("all weights resident", f"layer blocks streamed from pinned host memory, window {args.window} blocks"),
                   "l2": "inputs larger than L2 (every block is copied from host memory each token)",
                   "timing": "wall time of K chained tokens between two device-wide synchronisations; every byte copied in the region counts",
                   "window_blocks": args.window, "window_device_bytes": st["window_peak_bytes"],
                   "retain_ffn_every": sched["retain_every_T"], "retained_blocks": st["retained_blocks"],
                   "retained_device_bytes": st["retained_bytes"],
                   "block_bytes": {"attention": attn_b, "ffn": ffn_b}, "load_s": round(t_load, 1)},
        "clocks": r["clocks"],
        "e2e": {"value": K / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(link_bytes) + 4, "d2h_bytes_per_step": 8},
        "gpu_launches": st["kernel_launches_last"],
        "ttft_ms": r["ttft_ms"], "ttft_prompt_tokens": T, "dev_ms_per_step": st["last_decode_dev_ms"] / K,
        "roofline": {"bound": "host_link", "kernel": "cudaMemcpyAsync of block images on the copy stream",
                     "achieved": r["link_gbs"], "peak": peak, "unit": "GB/s", "frac": r["link_gbs"] / peak,
                     "traffic": link_bytes, "bytes_in_timed_region": r["region_bytes"],
                     "peak_kind": "pinned H2D copy (2 GiB, best of 10) measured in this run"},
        "scheduler": sched,
        "cpu_baseline": None, "tokens_tail": [int(x) for x in out[-4:]],
    }
    if rank == 0:
        print(json.dumps(line), flush=True)


def run_timeline(args, shape):
    """One layer's schedule inside the graph-replayed decode step, from the kernels' own time stamps (a library built
    with TPI_TIMELINE=1; see paper_2410_00531_b200/build.py).  Prints, per kernel of the LAST layer, when its CTAs
    start, when their dependency wait returns, when their inputs are staged and when they end, in microseconds from
    the first CTA of the layer's QKV kernel, then one JSON line with the same numbers.  Not a benchmark line."""
    import ctypes
    import numpy as np
    import torch
    import paper_2410_00531_b200 as P
    from paper_2410_00531_b200 import binding
    lib = binding.lib()
    fn = lib.tpi_internal_timeline
    fn.argtypes, fn.restype = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int)], ctypes.c_int
    lay = (ctypes.c_int * 4)()
    if not fn(None, lay):
        raise SystemExit("this library carries no time stamps: TPI_TIMELINE=1 python -m paper_2410_00531_b200.build, "
                         "then TPI_TIMELINE=1 python bench.py --timeline ...")
    n_k, n_c, n_s, w0 = lay[0], lay[1], lay[2], lay[3]
    torch.cuda.set_device(0)
    buf = torch.zeros(n_k * n_c * n_s, dtype=torch.int64, device="cuda")
    fn(buf.data_ptr(), lay)
    ses, _ = open_session(P, shape, 0, shape.prompt_len + args.steps + args.warmup + 8, args.prefill_chunk)
    try:
        first, _ = P.prefill(ses.h, S.prompt_tokens(shape), 0)
        P.decode_run(ses.h, first, args.warmup + args.steps)
        torch.cuda.synchronize()
        t = buf.cpu().numpy().reshape(n_k, n_c, n_s)
    finally:
        fn(None, lay)
        close_session(ses)
    names = [(0, "qkv"), (6, "attention"), (4, "o_proj"), (1, "gate_up"), (5, "down_proj"), (3, "head")]
    t0, rows = None, {}
    for k, name in names:
        e = t[k][(t[k][:, 0] > 0) & (t[k][:, w0:].max(axis=1) > 0)]       # CTAs that did work (an idle split leaves no end stamp)
        if not len(e):
            continue
        t0 = e[:, 0].min() if t0 is None else t0
        us = lambda x: round(float(x - t0) / 1e3, 2)
        end = e[:, w0:].max(axis=1)
        rows[name] = {"ctas": int(len(e)), "entry": [us(e[:, 0].min()), us(e[:, 0].max())],
                      "wait_returned": [us(e[:, 1].min()), us(e[:, 1].max())],
                      "staged": [us(e[:, 2].min()), us(e[:, 2].max())] if e[:, 2].max() > 0 else None,
                      "cta_end": [us(end.min()), us(float(np.median(end))), us(end.max())]}
        r = rows[name]
        print(f"{name:10s} ctas {r['ctas']:3d}  entry {r['entry'][0]:7.2f}..{r['entry'][1]:7.2f}  wait returned "
              f"{r['wait_returned'][0]:7.2f}..{r['wait_returned'][1]:7.2f}  staged "
              + (f"{r['staged'][0]:7.2f}..{r['staged'][1]:7.2f}" if r["staged"] else "      -         ")
              + f"  CTA end min {r['cta_end'][0]:7.2f} median {r['cta_end'][1]:7.2f} max {r['cta_end'][2]:7.2f}", file=sys.stderr)
    print(json.dumps({"timeline_us": rows, "config": {"workload": f"{args.workload} {shape.name}", "layers": shape.n_layers,
                                                      "context": shape.prompt_len + args.warmup + args.steps}}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2", choices=sorted(S.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--legs", default="C3,C5,TP,S5,S4",
                    help="extra workloads measured after the default headline and reported under `legs` (C3, C5: resident; "
                         "TP: the 7B shape as 4 ranks with one shard each on this one GPU; S5, S4: 70B-shaped bf16 / fp32 "
                         "blocks window-streamed); empty string = none")
    ap.add_argument("--retain", type=int, default=0,
                    help="with --window: keep one FFN block in every T resident beside the window (0 = none, -1 = as many as fit)")
    ap.add_argument("--window", type=int, default=0,
                    help="stream the layer blocks through a window of this many blocks (0 = all resident)")
    ap.add_argument("--prompt", type=int, default=0, help="override the prompt length")
    ap.add_argument("--shards", type=int, default=0, help="override the number of emulated shards N")
    ap.add_argument("--prefill-chunk", type=int, default=4096, help="prompt positions processed per pass over the weights")
    ap.add_argument("--quick", action="store_true",
                    help="one prompt pass and the device-resident decode loop only (short runs under a profiler)")
    ap.add_argument("--tp", type=int, default=0,
                    help="run the workload as this many ranks with one shard each, all on this GPU, and print that leg alone")
    ap.add_argument("--layers", type=int, default=0, help="override the depth (small captures under a profiler)")
    ap.add_argument("--timeline", action="store_true",
                    help="print one layer's kernel schedule inside the replayed decode step instead of a benchmark line "
                         "(needs TPI_TIMELINE=1, which selects the library built with time stamps)")
    args = ap.parse_args()
    shape = S.CONFIGS[args.workload]
    if args.layers:
        shape = shape.with_(n_layers=args.layers)
    if args.prompt:
        shape = shape.with_(prompt_len=args.prompt)
    if args.shards:
        shape = shape.with_(n_shards=args.shards)
    if args.impl == "reference":
        run_reference(args, shape)
    elif args.timeline:
        run_timeline(args, shape)
    else:
        run_gpu(args, shape)


if __name__ == "__main__":
    main()
