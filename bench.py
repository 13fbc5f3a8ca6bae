#!/usr/bin/env python
"""Benchmark of the MixKVQ decode hot path on B200.

A step is one decode step of the whole path over all layers: for every layer `mixkvq_decode_step`, i.e. the
append of the new token (with the scoring + quantize + pack flush once per R steps) fused with decode attention.  The cache is pre-filled to the configured context with seeded synthetic
tensors; all timed inputs are resident in HBM.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config qwen7b|llama8b|tiny|...] [--impl reference]

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_19206_b200 import workloads as W  # noqa: E402
from paper_2512_19206_b200.replicas import dist_env, max_over_ranks, job_tokens_per_s  # noqa: E402

METRIC = "decode-attn us/step (all layers) over mixed-precision KV"
PREFILL_CHUNK = 4096


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, no MEASURED_PEAKS.json)"


# ---------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(w, n_streams=2, reps=3):
    """Times the oracle's attention on `n_streams` (layer, b, hk) streams at the full context.

    Returns (seconds per stream-step, description).  Inputs come from the same generator (CPU)."""
    from oracle import mixkvq_oracle as O
    import numpy as np
    secs = []
    for i in range(n_streams):
        layer, hk = i % w.n_layers, i % w.n_kv_heads
        one = W.small(w, batch=1)
        st = O.OracleStream(g=w.g, R=w.residual_len, G=w.group_size, score_bits=w.score_bits, tau_bf16=w.tau_bf16,
                            tau_u4=w.tau_u4)
        t = 0
        while t < w.tokens:
            n = min(PREFILL_CHUNK, w.tokens - t)
            k, v, q = W.tokens(one, layer, t, n)
            st.append_many(k[0, hk].float().numpy(), v[0, hk].float().numpy(),
                           q[0, hk * w.g:(hk + 1) * w.g].float().numpy())
            t += n
        qd = W.decode_query(one, layer, 0)[0, hk * w.g:(hk + 1) * w.g].float().numpy()
        st.attention(qd, W.softmax_scale())
        t0 = time.perf_counter()
        for _ in range(reps):
            st.attention(qd, W.softmax_scale())
        secs.append((time.perf_counter() - t0) / reps)
    return statistics.mean(secs), (f"oracle attention on {n_streams} of {w.n_layers * w.batch * w.n_kv_heads} "
                                   f"(layer, batch, kv-head) streams at T={w.tokens}, {reps} repetitions each, "
                                   "scaled linearly to all streams")


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return 1


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    steps = []
    for _ in range(args.warmup):
        oracle_sample(w, 1, 1)
    desc = ""
    for _ in range(max(1, args.steps)):
        s, desc = oracle_sample(w, 1, 1)
        steps.append(s)
    per_stream = statistics.mean(steps)
    n_streams = w.n_layers * w.batch * w.n_kv_heads
    us = per_stream * n_streams * 1e6
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args.importance_mode),
        "cpu_baseline": {"value": us, "unit": "us/step", "cores": oracle_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": us, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "tokens_per_s": w.batch / (us * 1e-6),
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------- GPU leg
def workload_config(w, importance_mode=0):
    return {"workload": w.name, "n_layers": w.n_layers, "batch": w.batch, "n_q_heads": w.n_q_heads,
            "n_kv_heads": w.n_kv_heads, "head_dim": 128, "context_tokens": w.tokens, "residual_len": w.residual_len,
            "group_size": w.group_size, "tau_bf16": w.tau_bf16, "tau_u4": w.tau_u4, "score_bits": w.score_bits,
            "importance_mode": importance_mode,
            "l2": "inputs larger than L2: every step streams all layers' packed cache once"}


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, reasons = [], [], set()
        for ln in out.strip().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [x for x in sm if x >= 0.5 * max(sm)]
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def prefill(cache, w, dev):
    """Fills every layer to the configured context; returns the device time (ms) spent inside the bulk
    mixkvq_quantize_append calls alone (input generation excluded)."""
    ms = 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for layer in range(w.n_layers):
        t = 0
        while t < w.tokens:
            n = min(PREFILL_CHUNK, w.tokens - t)
            k, v, q = W.tokens(w, layer, t, n, device=dev)
            e0.record()
            cache.quantize_append(layer, k, v, q)
            e1.record()
            e1.synchronize()
            ms += e0.elapsed_time(e1)
            t += n
    torch.cuda.synchronize()
    return ms


def tier_mix(cache, w):
    """Mean (n16, n4) per block over all layers/streams, from the block tables."""
    import numpy as np
    n16 = n4 = nb = 0
    for layer in range(w.n_layers):
        d = cache.describe(layer)
        for s in range(d.n_streams):
            start = d.table_off + d.table_stride * s
            t = cache.mem[start:start + d.n_blocks * 8].cpu().numpy().reshape(-1, 8)
            n16 += int(t[:, 4].sum()); n4 += int(t[:, 5].sum()); nb += t.shape[0]
    nb = max(nb, 1)
    return n16 / nb, n4 / nb


def measured_traffic(kernel, source_file, group_size, tokens_packed, streams):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture (profiles/dram_traffic.json),
    scaled by the packed tokens this launch streams; None when there is no capture for this kernel and group size
    or the kernel's source changed after the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    ent = json.load(open(path)).get(f"{kernel}:G{group_size}")
    src = os.path.join(ROOT, "paper_2512_19206_b200", "csrc", source_file)
    if not ent or hashlib.sha256(open(src, "rb").read()).hexdigest() != ent["source_sha256"]:
        return None
    return ent["dram_bytes_per_token_per_kv_head"] * tokens_packed * streams


def algorithmic_bytes_per_layer(w, n16, n4, r, tokens_packed, n_partials, v_bits=2):
    """Bytes the method must move for one decode-attention launch (one layer): packed keys and values with
    their scales/zeros, promoted channels, residual window, q, o and the split partials."""
    G, R, D, g = w.group_size, w.residual_len, 128, w.g
    n2 = D - n16 - n4
    k_tok = 2 * n16 + n4 / 2 + n2 / 4 + 4 * (n4 + n2) / G + 160 / R
    v_tok = D * v_bits / 8 + 4 * D / G
    streams = w.batch * w.n_kv_heads
    per_stream = tokens_packed * (k_tok + v_tok) + 2 * r * D * 2 + g * D * 2 + g * D * 4
    return streams * per_stream + 2 * n_partials * g * (D + 2) * 4


def run_gpu(args, w):
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2512_19206_b200 import build, binding
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.lib()

    K, Wm = args.steps, args.warmup
    n_steps = Wm + K + 4
    cfg = binding.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.tokens + n_steps + 2 * w.residual_len,
                              residual_len=w.residual_len, group_size=w.group_size, tau_bf16=w.tau_bf16,
                              tau_u4=w.tau_u4, score_bits=w.score_bits, block_layout=args.layout,
                              importance_mode=args.importance_mode, sink_len=args.sink_len, v_bits=args.v_bits,
                              budget_bf16=args.budget_bf16, budget_u4=args.budget_u4,
                              extras_budget_bytes=((w.tokens + n_steps) // w.residual_len + 3) * 8192 if w.score_bits == 4 else 0)
    cache = binding.Cache(cfg, device=dev)
    prefill_ms = prefill(cache, w, dev)
    assert cache.status() == 0
    scale = W.softmax_scale()

    # decode-step inputs, resident in HBM: [layer][step] -> (k, v, q) of one token
    steps_in = []
    for layer in range(w.n_layers):
        k, v, q = W.tokens(w, layer, w.tokens, n_steps, device=dev)
        steps_in.append([(k[:, :, i:i + 1].contiguous(), v[:, :, i:i + 1].contiguous(), q[:, :, i:i + 1].contiguous())
                         for i in range(n_steps)])
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)

    def step(i):
        for layer in range(w.n_layers):
            k, v, q = steps_in[layer][i]
            cache.decode_step(layer, k, v, q, scale, out=out[layer])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(Wm):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = cache.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.profiler.start()      # a profiler started with capture off sees only the timed region
    e0.record()
    for i in range(Wm, Wm + K):
        step(i)
    e1.record()
    barrier()
    torch.cuda.profiler.stop()
    ms = e0.elapsed_time(e1)
    launches = cache.launch_count() - launches0
    flushes = sum(1 for i in range(Wm, Wm + K) if (w.tokens + i) % w.residual_len == 0) * w.n_layers

    # ---- dominant kernel alone (split kernel, no combine), same state: average launch duration
    d0 = cache.describe(0)
    cache.set_attention_kernel(2)
    qs = [steps_in[layer][Wm + K][2].view(w.batch, w.n_q_heads, 128) for layer in range(w.n_layers)]
    reps = max(3, min(20, int(200 / max(1, w.n_layers))))
    for layer in range(w.n_layers):
        cache.decode_attention(layer, qs[layer], scale, out=out[layer])
    torch.cuda.synchronize()
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0.record()
    for _ in range(reps):
        for layer in range(w.n_layers):
            cache.decode_attention(layer, qs[layer], scale, out=out[layer])
    k1.record()
    torch.cuda.synchronize()
    kern_ms = k0.elapsed_time(k1) / (reps * w.n_layers)
    cache.set_attention_kernel(0)
    # ---- attention + combine for all layers from one CUDA graph (fixed state): launch gaps removed
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for layer in range(w.n_layers):
            cache.decode_attention(layer, qs[layer], scale, out=out[layer])
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=s):
            for layer in range(w.n_layers):
                cache.decode_attention(layer, qs[layer], scale, out=out[layer])
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(reps):
        g.replay()
    g1.record()
    torch.cuda.synchronize()
    graph_us = g0.elapsed_time(g1) / reps * 1e3
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end through the C ABI with host buffers: H2D of the step's inputs, D2H of its outputs
    n_e2e = min(K, 16)
    hk = torch.stack([torch.stack([steps_in[l][Wm + i][0] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
    hv = torch.stack([torch.stack([steps_in[l][Wm + i][1] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
    hq = torch.stack([torch.stack([steps_in[l][Wm + i][2] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
    hout = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    dk, dv, dq = [torch.empty(x.shape[1:], dtype=x.dtype, device=dev) for x in (hk, hv, hq)]
    barrier()
    t0 = time.perf_counter()
    for i in range(n_e2e):
        dk.copy_(hk[i], non_blocking=True); dv.copy_(hv[i], non_blocking=True); dq.copy_(hq[i], non_blocking=True)
        for layer in range(w.n_layers):
            cache.decode_step(layer, dk[layer], dv[layer], dq[layer], scale, out=out[layer])
        hout.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
    e2e_us = (time.perf_counter() - t0) / n_e2e * 1e6
    h2d = hk[0].numel() * 2 + hv[0].numel() * 2 + hq[0].numel() * 2
    d2h = out.numel() * 4
    status = cache.status()

    us = ms * 1e3 / K
    us, e2e_us, kern_ms, graph_us = max_over_ranks([us, e2e_us, kern_ms, graph_us], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    n16, n4 = tier_mix(cache, w)
    tokens_packed = d0.n_blocks * w.residual_len
    units = (tokens_packed // 32 + (d0.residual_tokens + 31) // 32) * w.batch * w.n_kv_heads
    # partials written per launch = CTAs of the split kernel: two per SM, a multiple of the stream count when there are
    # fewer streams than CTA slots (the library's grid rule), each CTA one partial per stream it touches
    streams = w.batch * w.n_kv_heads
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    n_part = min(2 * n_sms, units)
    n_part = n_part // streams * streams if n_part > streams else n_part + streams
    alg = algorithmic_bytes_per_layer(w, n16, n4, d0.residual_tokens, tokens_packed, n_part, args.v_bits)
    peak, peak_src = measured_peaks()
    achieved = alg / (kern_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "arithmetic": "2/4-bit codes and bf16 metadata expanded to fp16 tensor-core operands, fp32 accumulate and softmax",
        "config": workload_config(w, args.importance_mode),
        "tokens_per_s": job_tokens_per_s(w.batch, world, us),
        "attention_graph_us_per_step": graph_us,
        "prefill_quantize": {"ms": prefill_ms, "tokens_per_s": w.n_layers * w.batch * w.tokens / (prefill_ms * 1e-3),
                             "input_gb_per_s": w.n_layers * w.batch * w.tokens * 256 * (2 * w.n_kv_heads + w.n_q_heads)
                             / (prefill_ms * 1e-3) / 1e9},
        "flushes_in_timed_region": flushes,
        "tier_mix_mean": {"n16": n16, "n4": n4, "n2": 128 - n16 - n4},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     # the committed counters were taken on the two-tier mix (no UINT4 tier): other mixes have none
                     "traffic": None if (w.tau_u4 < w.tau_bf16 or args.v_bits != 2 or args.sink_len or args.budget_bf16 +
                                         args.budget_u4) else measured_traffic(
                         *(("attention_tc_kernel", "attention_tc.cu") if args.layout == 1 else
                           ("attention_ws_kernel", "attention_ws.cu")), w.group_size, tokens_packed,
                         w.batch * w.n_kv_heads),
                     "peak_source": peak_src,
                     "kernel": "attention_tc_kernel" if args.layout == 1 else "attention_ws_kernel", "kernel_us": kern_ms * 1e3, "algorithmic_bytes": alg},
        "e2e": {"value": e2e_us, "unit": "us/step", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": n_e2e},
        "gpu_launches": int(launches),
        "device_status": status,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        sec, desc = oracle_sample(w, n_streams=8, reps=5)
        n_streams = w.n_layers * w.batch * w.n_kv_heads
        line["cpu_baseline"] = {"value": sec * n_streams * 1e6, "unit": "us/step", "cores": oracle_threads(),
                                "kind": "oracle", "sample": desc}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="qwen7b", choices=sorted(W.CONFIGS))
    ap.add_argument("--group-size", type=int, default=None)
    ap.add_argument("--residual-len", type=int, default=None, help="R: residual window / block length (32 .. 256)")
    ap.add_argument("--importance-mode", type=int, default=0, choices=[0, 1, 2],
                    help="0: window importance (default), 1: cumulative, 2: error-only salience")
    ap.add_argument("--sink-len", type=int, default=0, help="sink tokens kept in bf16 (0, or a multiple of 32 up to 256)")
    ap.add_argument("--v-bits", type=int, default=2, choices=[2, 4], help="value bit-width (4: fragment layout only)")
    ap.add_argument("--budget-bf16", type=int, default=0, help="fixed-budget tiering: BF16 channels per window")
    ap.add_argument("--budget-u4", type=int, default=0, help="fixed-budget tiering: UINT4 channels per window")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--preset", default=None, choices=["P24", "P27", "P4BASE"],
                    help="threshold preset: two tiers (default), three tiers, or 4-bit base precision")
    ap.add_argument("--layout", type=int, default=0, choices=[0, 1],
                    help="0: fragment layout + mma.sync attention (default), 1: tile layout + tcgen05 attention")
    args = ap.parse_args()
    w = W.CONFIGS[args.config]
    over = {}
    if args.group_size:
        over["group_size"] = args.group_size
    if args.residual_len:
        over["residual_len"] = args.residual_len
    if args.tokens:
        over["tokens"] = args.tokens
    if args.layers:
        over["n_layers"] = args.layers
    if args.preset:
        over.update(getattr(W, args.preset))
    if over:
        w = W.small(w, **over)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
