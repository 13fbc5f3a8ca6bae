#!/usr/bin/env python
"""Benchmark of the MixKVQ decode hot path on B200.

A step is one decode step of the whole path over all layers: for every layer `mixkvq_decode_step`, i.e. the
append of the new token (with the scoring + quantize + pack flush once per R steps) fused with decode attention.
The cache is pre-filled to the configured context with seeded synthetic tensors; all timed inputs are resident
in HBM.  Prints one JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config qwen7b|llama8b|tiny|...] [--impl reference]

The line leads with the qwen2.5-7b shape (batch 8, 32768 cached tokens, 28 layers).  It also carries the separate
timings of the step's parts (attention, append, the step that flushes, the amortised step) and, under `configs`,
the decode-attention kernel on the other workload shapes (a few layers each).
`--gpus N` without launcher variables starts N ranks itself (one per GPU, independent replicas; only the measured
times are reduced, with MAX); under torchrun it takes rank and world size from the environment.
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
from paper_2512_19206_b200.replicas import dist_env, max_over_ranks, job_tokens_per_s, spawn_local_ranks  # noqa: E402

METRIC = "decode-attn us/step (all layers) over mixed-precision KV"
PREFILL_CHUNK = 4096
SPLIT_KERNEL = ("attention_ws_kernel", "attention_ws.cu")
TILE_KERNEL = ("attention_tc_kernel", "attention_tc.cu")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, no MEASURED_PEAKS.json)"


# ---------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_stream(w):
    from oracle import mixkvq_oracle as O
    return O.OracleStream(g=w.g, R=w.residual_len, G=w.group_size, score_bits=w.score_bits, tau_bf16=w.tau_bf16,
                          tau_u4=w.tau_u4)


def oracle_sample(w, n_streams=2, reps=3):
    """Times the oracle's attention on `n_streams` (layer, b, hk) streams at the full context.

    Returns (seconds per stream-step, description).  Inputs come from the same generator (CPU)."""
    secs = []
    for i in range(n_streams):
        layer, hk = i % w.n_layers, i % w.n_kv_heads
        one = W.small(w, batch=1)
        st = oracle_stream(w)
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


def oracle_flush_ms(w, n_blocks=6):
    """Mean time of one oracle flush (scoring, tiering, quantization of one R-token window of one stream)."""
    one = W.small(w, batch=1)
    st = oracle_stream(w)
    R = w.residual_len
    k, v, q = W.tokens(one, 0, 0, (n_blocks + 1) * R)
    kf, vf, qf = k[0, 0].float().numpy(), v[0, 0].float().numpy(), q[0, :w.g].float().numpy()
    st.append_many(kf[:R], vf[:R], qf[:, :R])                      # the window is full now
    secs = []
    for b in range(1, n_blocks + 1):
        t0 = time.perf_counter()
        st.append_many(kf[b * R:b * R + 1], vf[b * R:b * R + 1], qf[:, b * R:b * R + 1])   # flushes the full window first
        secs.append(time.perf_counter() - t0)
        st.append_many(kf[b * R + 1:(b + 1) * R], vf[b * R + 1:(b + 1) * R], qf[:, b * R + 1:(b + 1) * R])
    return statistics.mean(secs) * 1e3


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
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args.importance_mode),
        "cpu_baseline": {"value": us, "unit": "us/step", "cores": oracle_threads(), "kind": "oracle",
                         "impl": f"numpy, {oracle_threads()} BLAS threads", "sample": desc},
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
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
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


def make_cache(binding, w, args, dev, extra_tokens):
    cfg = binding.make_config(w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.tokens + extra_tokens,
                              residual_len=w.residual_len, group_size=w.group_size, tau_bf16=w.tau_bf16,
                              tau_u4=w.tau_u4, score_bits=w.score_bits, block_layout=args.layout,
                              importance_mode=args.importance_mode, sink_len=args.sink_len, v_bits=args.v_bits,
                              budget_bf16=args.budget_bf16, budget_u4=args.budget_u4,
                              extras_budget_bytes=((w.tokens + extra_tokens) // w.residual_len + 3) * 8192
                              if w.score_bits == 4 else 0)
    return binding.Cache(cfg, device=dev)


def prefill(cache, w, dev, t_from=0, t_to=None):
    """Appends tokens [t_from, t_to) to every layer in chunks; returns the device time (ms) spent inside the bulk
    mixkvq_quantize_append calls alone (input generation excluded)."""
    t_to = w.tokens if t_to is None else t_to
    ms = 0.0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for layer in range(w.n_layers):
        t = t_from
        while t < t_to:
            n = min(PREFILL_CHUNK, t_to - t)
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
    n16 = n4 = nb = 0
    for layer in range(w.n_layers):
        d = cache.describe(layer)
        for s in range(d.n_streams):
            start = d.table_off + d.table_stride * s
            blocks = cache.sequence_fill(layer, s // w.n_kv_heads)[0]
            t = cache.mem[start:start + blocks * 8].cpu().numpy().reshape(-1, 8)
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


def n_split_partials(w, d0, dev):
    """Partials written per launch = CTAs of the split kernel: two per SM, a multiple of the stream count when there
    are fewer streams than CTA slots (the library's grid rule), each CTA one partial per stream it touches."""
    streams = w.batch * w.n_kv_heads
    units = (d0.n_blocks * w.residual_len // 32 + (d0.residual_tokens + 31) // 32) * streams
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    n_part = min(2 * n_sms, units)
    return n_part // streams * streams if n_part > streams else n_part + streams


def time_loop(fn, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def attention_timings(cache, w, qs, out, scale):
    """(split kernel ms per launch, attention + combine us per layer) at the cache's current state."""
    def all_layers():
        for layer in range(w.n_layers):
            cache.decode_attention(layer, qs[layer], scale, out=out[layer])
    reps = max(3, min(20, int(200 / max(1, w.n_layers))))
    cache.set_attention_kernel(2)
    all_layers()
    kern_ms = time_loop(all_layers, reps) / w.n_layers
    cache.set_attention_kernel(0)
    all_layers()
    attn_us = time_loop(all_layers, reps) / w.n_layers * 1e3
    return kern_ms, attn_us


def roofline_entry(cache, w, dev, args, kern_ms):
    d0 = cache.describe(0)
    n16, n4 = tier_mix(cache, w)
    tokens_packed = d0.n_blocks * w.residual_len
    alg = algorithmic_bytes_per_layer(w, n16, n4, d0.residual_tokens, tokens_packed, n_split_partials(w, d0, dev), args.v_bits)
    peak, peak_src = measured_peaks()
    achieved = alg / (kern_ms * 1e-3) / 1e9
    return n16, n4, tokens_packed, alg, achieved, peak, peak_src


def other_config(binding, dev, args, name, w, label, contexts=None):
    """The decode-attention kernel on another workload shape, a few layers of it: one entry per context length."""
    entries = []
    contexts = contexts or [w.tokens]
    cache = make_cache(binding, W.small(w, tokens=max(contexts)), args, dev, 2 * w.residual_len + 8)
    scale = W.softmax_scale()
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    done = 0
    for T in contexts:
        prefill(cache, w, dev, done, T)
        done = T
        qs = [W.decode_query(w, layer, 0, device=dev) for layer in range(w.n_layers)]
        kern_ms, attn_us = attention_timings(cache, w, qs, out, scale)
        n16, n4, tokens_packed, alg, achieved, peak, _ = roofline_entry(cache, w, dev, args, kern_ms)
        entries.append({
            "workload": label, "shape": f"B={w.batch} Hq={w.n_q_heads} Hkv={w.n_kv_heads} T={T} G={w.group_size}",
            "layers_measured": w.n_layers, "layers_of_model": W.CONFIGS[name].n_layers,
            "kernel_us": kern_ms * 1e3, "algorithmic_bytes": alg, "achieved_gbs": achieved, "frac": achieved / peak,
            "attention_us_per_layer": attn_us,
            "attention_us_per_step_all_layers": attn_us * W.CONFIGS[name].n_layers,
            "tier_mix_mean": {"n16": n16, "n4": n4}, "device_status": cache.status()})
    cache.close()
    del cache
    torch.cuda.empty_cache()
    return entries


def ragged_config(binding, dev, args):
    """The decode-attention kernel on a batch of unequal lengths (the serving case): the headline model shape, four
    layers, eight sequences between 640 and 32768 tokens, appended with per-sequence counts."""
    w = W.small(W.CONFIGS["qwen7b"], n_layers=4)
    lengths = [32768, 29000, 23500, 17000, 12345, 9000, 4097, 640]
    cache = make_cache(binding, w, args, dev, 2 * w.residual_len + 8)
    for layer in range(w.n_layers):
        for t in range(0, max(lengths), PREFILL_CHUNK):
            n = min(PREFILL_CHUNK, max(lengths) - t)
            k, v, q = W.tokens(w, layer, t, n, device=dev)
            cache.quantize_append_ragged(layer, k, v, q, [min(max(L - t, 0), n) for L in lengths])
    torch.cuda.synchronize()
    scale = W.softmax_scale()
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    qs = [W.decode_query(w, layer, 0, device=dev) for layer in range(w.n_layers)]
    kern_ms, attn_us = attention_timings(cache, w, qs, out, scale)
    n16, n4 = tier_mix(cache, w)             # of sequence 0, the longest
    one = W.small(w, batch=1)
    alg, units = 0.0, 0
    for b in range(w.batch):
        nb, r, _ = cache.sequence_fill(0, b)
        alg += algorithmic_bytes_per_layer(one, n16, n4, r, nb * w.residual_len, 0, args.v_bits)
        units += (nb * w.residual_len // 32 + (r + 31) // 32) * w.n_kv_heads
    n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    alg += 2 * (min(2 * n_sms, units) + w.batch * w.n_kv_heads) * w.g * 130 * 4
    peak, _ = measured_peaks()
    entry = {"workload": "ragged batch: qwen2.5-7b shape, sequences of " + ", ".join(str(L) for L in lengths) + " tokens",
             "shape": f"B={w.batch} Hq={w.n_q_heads} Hkv={w.n_kv_heads} G={w.group_size}", "layers_measured": w.n_layers,
             "kernel_us": kern_ms * 1e3, "kernel_us_note": "the split kernel and the 2 us launch that writes the fill table",
             "algorithmic_bytes": alg, "achieved_gbs": alg / (kern_ms * 1e-3) / 1e9, "frac": alg / (kern_ms * 1e-3) / 1e9 / peak,
             "attention_us_per_layer": attn_us, "device_status": cache.status()}
    cache.close()
    del cache
    torch.cuda.empty_cache()
    return [entry]


def tensor_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json)"
    return 1590.0, 1400.0, "fallback (1.59 PFLOP/s burst, 1.4 sustained, no MEASURED_PEAKS.json)"


def prefill_attention_entries(binding, dev, args, contexts=(8192, 32768)):
    """The prefill call (causal full-precision attention of the prompt on the tensor cores, then the bulk quantizing
    append) on one layer of the headline model shape, one sequence: a tensor-bound path, reported against the
    measured bf16 GEMM peaks.  The flops are those of the causal definition: 4 D L (L + 1) / 2 per query head."""
    entries = []
    burst, sustained, src = tensor_peaks()
    for L in contexts:
        w = W.small(W.CONFIGS["qwen7b"], n_layers=1, batch=1, tokens=L)
        cache = make_cache(binding, w, args, dev, 0)
        k, v, q = W.tokens(w, 0, 0, L, device=dev)
        out = torch.empty(q.shape, dtype=torch.float32, device=dev)
        scratch = torch.empty(cache.prefill_scratch_bytes(L), dtype=torch.uint8, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn):
            ms = []
            for _ in range(6):
                cache.reset()
                e0.record()
                fn()
                e1.record()
                e1.synchronize()
                ms.append(e0.elapsed_time(e1))
            return ms

        call_ms = timed(lambda: cache.prefill(0, k, v, q, W.softmax_scale(), out=out, scratch=scratch))
        append_ms = timed(lambda: cache.quantize_append(0, k, v, q))
        call = sorted(call_ms[2:])[2]
        app = sorted(append_ms[2:])[2]
        flops = 4.0 * 128 * w.n_q_heads * L * (L + 1) / 2
        attn = call - app
        entries.append({
            "workload": "prefill: qwen2.5-7b shape, one layer, one sequence", "shape": f"B=1 Hq={w.n_q_heads} Hkv={w.n_kv_heads} L={L}",
            "call_ms": call, "append_ms": app, "attention_ms": attn, "flops": flops,
            "roofline": {"bound": "tensor", "kernel": "prefill_pack_kernel + prefill_attention_kernel",
                         "achieved": flops / (attn * 1e-3) / 1e12, "peak": sustained, "unit": "TFLOP/s",
                         "frac": flops / (attn * 1e-3) / 1e12 / sustained,
                         "frac_of_burst_peak": flops / (attn * 1e-3) / 1e12 / burst, "peak_source": src,
                         "note": "attention_ms = the call minus the bulk append timed alone; causal flops only "
                                 "(the masked half of the diagonal tiles is computed and not counted)"},
            "whole_call_tflops": flops / (call * 1e-3) / 1e12, "device_status": cache.status()})
        cache.close()
        del cache, k, v, q, out, scratch
        torch.cuda.empty_cache()
    return entries


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

    K, Wm, R = args.steps, args.warmup, w.residual_len
    n_steps = Wm + K + 4
    cache = make_cache(binding, w, args, dev, n_steps + 4 * R + 64)
    prefill_ms = prefill(cache, w, dev)
    assert cache.status() == 0
    scale = W.softmax_scale()

    # decode-step inputs, resident in HBM: [layer][step] -> (k, v, q) of one token
    n_in = n_steps + 2 * R + 40
    steps_in = []
    for layer in range(w.n_layers):
        k, v, q = W.tokens(w, layer, w.tokens, n_in, device=dev)
        steps_in.append([(k[:, :, i:i + 1].contiguous(), v[:, :, i:i + 1].contiguous(), q[:, :, i:i + 1].contiguous())
                         for i in range(n_in)])
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
    flushes = sum(1 for i in range(Wm, Wm + K) if (w.tokens + i) % R == 0) * w.n_layers

    # ---- dominant kernel alone (split kernel, no combine), and attention + combine, same state
    nxt = Wm + K                                    # next unused decode-step input
    qs = [steps_in[layer][nxt][2].view(w.batch, w.n_q_heads, 128) for layer in range(w.n_layers)]
    kern_ms, attn_us_layer = attention_timings(cache, w, qs, out, scale)
    reps = max(3, min(20, int(200 / max(1, w.n_layers))))
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
    graph_us = time_loop(g.replay, reps) * 1e3
    clocks = sampler.stop() if rank == 0 else None
    n16, n4, tokens_packed, alg, achieved, peak, peak_src = roofline_entry(cache, w, dev, args, kern_ms)

    # ---- the parts of the step on their own: the plain append of one token (no flush), and the step on which the
    # residual window is full, so that the append first scores, quantizes and packs it (once every R steps)
    def append_all(i):
        for layer in range(w.n_layers):
            k, v, q = steps_in[layer][i]
            cache.quantize_append(layer, k, v, q)

    def window_fill():
        return cache.describe(0).residual_tokens

    plain = []
    while window_fill() != R and len(plain) < 4:      # a few plain appends, timed one step at a time
        i = nxt
        plain.append(time_loop(lambda: append_all(i), 1) * 1e3)
        nxt += 1
    while window_fill() != R:                         # advance (untimed) until the window is full
        append_all(nxt)
        nxt += 1
    i = nxt
    flush_step_us = time_loop(lambda: append_all(i), 1) * 1e3      # flush + append on every layer
    nxt += 1
    while len(plain) < 4:
        i = nxt
        plain.append(time_loop(lambda: append_all(i), 1) * 1e3)
        nxt += 1
    append_us = statistics.median(plain)

    # ---- end to end through the C ABI with host buffers: H2D of the step's inputs, D2H of its outputs
    n_e2e = min(K, 16)
    hk = torch.stack([torch.stack([steps_in[l][nxt + i][0] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
    hv = torch.stack([torch.stack([steps_in[l][nxt + i][1] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
    hq = torch.stack([torch.stack([steps_in[l][nxt + i][2] for l in range(w.n_layers)]) for i in range(n_e2e)]).cpu().pin_memory()
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

    achieved = alg / (kern_ms * 1e-3) / 1e9
    attn_us = attn_us_layer * w.n_layers
    line = {
        "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "arithmetic": "2/4-bit codes and bf16 metadata expanded to fp16 tensor-core operands, fp32 accumulate and softmax",
        "config": workload_config(w, args.importance_mode),
        "tokens_per_s": job_tokens_per_s(w.batch, world, us),
        "step_parts": {
            "note": "all layers; `value` is the fused call (append inside the attention kernel) on steps without a flush",
            "attention_us": attn_us, "attention_graph_us": graph_us,
            "append_us": append_us, "flush_step_us": flush_step_us,
            "amortised_us_per_step": attn_us + append_us + (flush_step_us - append_us) / R,
            "fused_amortised_us_per_step": us + (flush_step_us - append_us) / R,
            "flush_every_steps": R},
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
                         *(TILE_KERNEL if args.layout == 1 else SPLIT_KERNEL), w.group_size, tokens_packed,
                         w.batch * w.n_kv_heads),
                     "peak_source": peak_src,
                     "kernel": (TILE_KERNEL if args.layout == 1 else SPLIT_KERNEL)[0], "kernel_us": kern_ms * 1e3,
                     "kernel_us_note": "mean over back-to-back launches of the split kernel alone (one per layer); each "
                                       "launch starts behind its predecessor with programmatic dependent launch, so set-up "
                                       "and the first requests of a launch overlap the tail of the one before",
                     "algorithmic_bytes": alg},
        "e2e": {"value": e2e_us, "unit": "us/step", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": n_e2e},
        "gpu_launches": int(launches),
        "device_status": status,
        "clocks": clocks,
    }
    cache.close()
    del cache, steps_in
    torch.cuda.empty_cache()
    if world == 1 and not args.no_configs and args.config == "qwen7b" and not args.tokens and not args.layers:
        cfgs = []
        cfgs += other_config(binding, dev, args, "tiny", W.CONFIGS["tiny"], "config 1: tiny (L2-resident)")
        l8 = W.small(W.CONFIGS["llama8b"], n_layers=4)
        cfgs += other_config(binding, dev, args, "llama8b", W.small(l8, **W.P24), "config 3: llama-3.1-8b, 2-bit base")
        cfgs += other_config(binding, dev, args, "llama8b", W.small(l8, **W.P4BASE), "config 3: llama-3.1-8b, 4-bit base")
        cfgs += other_config(binding, dev, args, "qwen32b", W.small(W.CONFIGS["qwen32b"], n_layers=3),
                             "config 4: qwen2.5-32b (3 distinct layers of 64)")
        cfgs += other_config(binding, dev, args, "longcot", W.small(W.CONFIGS["longcot"], n_layers=4),
                             "config 5: long-CoT stream", contexts=[8192, 32768, 65536, 131072])
        cfgs += other_config(binding, dev, args, "qwen7b", W.small(W.CONFIGS["qwen7b"], n_layers=4, **W.P27),
                             "config 2 with three tiers (the 2.7-bit mix), 4 layers")
        cfgs += ragged_config(binding, dev, args)
        line["configs"] = cfgs
        line["prefill_attention"] = prefill_attention_entries(binding, dev, args)
    if world == 1 and not args.no_cpu_baseline:
        sec, desc = oracle_sample(w, n_streams=8, reps=5)
        n_streams = w.n_layers * w.batch * w.n_kv_heads
        line["cpu_baseline"] = {"value": sec * n_streams * 1e6, "unit": "us/step", "cores": oracle_threads(),
                                "kind": "oracle", "impl": f"numpy, {oracle_threads()} BLAS threads", "sample": desc,
                                "flush_ms_per_block": oracle_flush_ms(w),
                                "flush_note": "one stream's window of R tokens: scoring, tiering, quantization (oracle); "
                                              "the GPU's flush_step_us covers all layers x streams"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
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
    ap.add_argument("--prefill-tokens", type=int, default=0,
                    help="run only the prefill call on a prompt of this many tokens (one layer, one sequence)")
    ap.add_argument("--no-configs", action="store_true", help="skip the other workload shapes")
    ap.add_argument("--preset", default=None, choices=["P24", "P27", "P4BASE"],
                    help="threshold preset: two tiers (default), three tiers, or 4-bit base precision")
    ap.add_argument("--layout", type=int, default=0, choices=[0, 1],
                    help="0: fragment layout + mma.sync attention (default), 1: tile layout + tcgen05 attention")
    args = ap.parse_args()
    launched = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if args.impl == "ours" and args.gpus > 1 and not launched:
        # no launcher: start the ranks here, one per GPU (independent replicas of the workload)
        sys.exit(spawn_local_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    if launched and args.impl == "ours" and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {os.environ['WORLD_SIZE']} ranks")
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
    elif args.prefill_tokens:
        # the prefill call alone on one GPU (for profiling it on a small case): one JSON line with its entries
        from paper_2512_19206_b200 import binding
        binding.lib()
        dev = torch.device("cuda", 0)
        torch.cuda.set_device(dev)
        print(json.dumps({"prefill_attention": prefill_attention_entries(binding, dev, args, (args.prefill_tokens,))}),
              flush=True)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
