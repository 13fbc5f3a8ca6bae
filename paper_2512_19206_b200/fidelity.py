"""Attention fidelity against effective key bit-width on synthetic streams: a sweep of the two salience thresholds.

The paper picks its thresholds by searching for the best benchmark accuracy at a given average key bit-width
(Appendix C) and reports accuracy against bits (Section 5).  Model weights and benchmark data are not part of this
library, so this tool scores a threshold pair by what the decode path itself can measure: the error of the quantized
decode attention (Eq. 1 over the mixed-precision cache) against the same attention over the unquantized bf16 keys and
values of the same seeded streams, next to the effective key bit-width B_eff the pair reaches (Appendix C).

    python -m paper_2512_19206_b200.fidelity --config qwen7b --tokens 8192

Every cache operation goes through the CUDA library; the unquantized reference is plain PyTorch on the GPU and is only
a yardstick (it is not part of any product path).
"""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import binding as B
from . import workloads as W


def effective_key_bits(n16: float, n4: float, head_dim: int = 128) -> float:
    """B_eff of Appendix C for keys: the tier counts weighted by 16, 4 and 2 bits, per channel."""
    n2 = head_dim - n16 - n4
    return (16.0 * n16 + 4.0 * n4 + 2.0 * n2) / head_dim


def tier_counts(cache: "B.Cache", layer: int):
    """Mean number of BF16 and UINT4 channels per packed block of a layer, read from the block tables."""
    d = cache.describe(layer)
    n16 = n4 = nb = 0
    for s in range(d.n_streams):
        start = d.table_off + d.table_stride * s
        t = cache.mem[start:start + d.n_blocks * 8].view(-1, 8)
        n16 += int(t[:, 4].sum())
        n4 += int(t[:, 5].sum())
        nb += t.shape[0]
    nb = max(nb, 1)
    return n16 / nb, n4 / nb


def reference_attention(k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, scale: float) -> torch.Tensor:
    """Unquantized decode attention in fp32: k, v [B, Hkv, T, D] bf16, q [B, Hq, D] bf16 -> [B, Hq, D] fp32.
    A yardstick for this tool's error columns only (plain PyTorch, no part of the decode path); the tests tie it and
    the tool's rows to the CPU oracle."""
    b, hkv, t, d = k.shape
    g = q.shape[1] // hkv
    qf = q.float().view(b, hkv, g, d)
    logits = torch.einsum("bhgd,bhtd->bhgt", qf, k.float()) * scale
    p = torch.softmax(logits, dim=-1)
    return torch.einsum("bhgt,bhtd->bhgd", p, v.float()).reshape(b, hkv * g, d)


def measure(w: "W.Workload", tau_bf16: float, tau_u4: float, score_bits: int = 2, importance_mode: int = 0,
            n_queries: int = 4, chunk: int = 4096, return_outputs: bool = False, budget_bf16: int = 0, budget_u4: int = 0,
            sink_len: int = 0):
    """Builds one layer of the workload with the given thresholds and returns (B_eff, n16, n4, max error, rms error)
    of decode attention against the unquantized reference, over n_queries decode queries (and, on request, the
    attention outputs themselves)."""
    # room in the promoted-channel arena for any tier mix (every channel promoted, dense UINT4 high plane)
    n_blocks = w.tokens // w.residual_len + 2
    budget = n_blocks * ((w.residual_len // 32) * (128 * 64 + 1024) + 512)
    cfg = B.make_config(1, w.batch, w.n_q_heads, w.n_kv_heads, w.tokens + 2 * w.residual_len,
                        residual_len=w.residual_len, group_size=w.group_size, tau_bf16=tau_bf16, tau_u4=tau_u4,
                        score_bits=score_bits, importance_mode=importance_mode, extras_budget_bytes=budget,
                        budget_bf16=budget_bf16, budget_u4=budget_u4, sink_len=sink_len)
    cache = B.Cache(cfg)
    ks, vs = [], []
    t = 0
    while t < w.tokens:
        n = min(chunk, w.tokens - t)
        k, v, q = W.tokens(w, 0, t, n, device="cuda")
        cache.quantize_append(0, k, v, q)
        ks.append(k)
        vs.append(v)
        t += n
    k_all, v_all = torch.cat(ks, dim=2), torch.cat(vs, dim=2)
    scale = W.softmax_scale()
    worst, sq, cnt = 0.0, 0.0, 0
    outs = []
    for i in range(n_queries):
        qd = W.decode_query(w, 0, i, device="cuda")
        out = cache.decode_attention(0, qd, scale)
        outs.append(out.clone())
        ref = reference_attention(k_all, v_all, qd, scale)
        err = (out - ref).abs()
        worst = max(worst, float(err.max()))
        sq += float((err.double() ** 2).sum())
        cnt += err.numel()
    if cache.status() != 0:
        raise RuntimeError(f"device status {cache.status()} (promoted-channel arena too small for these thresholds?)")
    n16, n4 = tier_counts(cache, 0)
    cache.close()
    res = (effective_key_bits(n16, n4), n16, n4, worst, math.sqrt(sq / max(cnt, 1)))
    return res + (outs,) if return_outputs else res


def sweep(w: "W.Workload", pairs, **kw):
    """One row per setting.  Besides the error against unquantized keys and values, `key_rms_err` is the error against
    the cache whose keys are all kept in bf16: the value codes do not depend on the thresholds, so this is the part of
    the error that the key tiers control."""
    *_, keys_bf16 = measure(w, -1.0, -1.0, return_outputs=True, **kw)
    rows = []
    for name, tau_bf16, tau_u4, score_bits, mode, *extra in pairs:
        more = extra[0] if extra else {}
        beff, n16, n4, worst, rms, outs = measure(w, tau_bf16, tau_u4, score_bits=score_bits, importance_mode=mode,
                                                  return_outputs=True, **more, **kw)
        sq = sum(float(((a - b).double() ** 2).sum()) for a, b in zip(outs, keys_bf16))
        key_rms = math.sqrt(sq / sum(a.numel() for a in outs))
        rows.append({"setting": name, "tau_bf16": tau_bf16, "tau_u4": tau_u4, "importance_mode": mode,
                     "key_bits": beff, "n16": n16, "n4": n4, "max_err": worst, "rms_err": rms, "key_rms_err": key_rms})
    return rows


def default_pairs():
    """(name, tau_bf16, tau_u4, score_bits, importance_mode[, further configuration fields]): uniform 2-bit, a sweep of the BF16 threshold, the two
    presets with a UINT4 tier, the error-only ablation at the first preset's threshold, and unquantized keys."""
    inf = 1e30
    pairs = [("uniform 2-bit keys", inf, inf, 2, 0)]
    pairs += [(f"two tiers, tau_bf16 = {t:g}", t, inf, 2, 0) for t in (13.0, 6.5, 3.25)]
    pairs += [(f"three tiers ({W.P27['tau_bf16']:g}, {W.P27['tau_u4']:g})", W.P27["tau_bf16"], W.P27["tau_u4"], 2, 0),
              ("three tiers (6.5, 2.0)", 6.5, 2.0, 2, 0)]
    pairs += [("error-only salience, tau_bf16 = 6.5", 6.5, inf, 2, 2)]
    pairs += [("fixed budget: 4 BF16", inf, inf, 2, 0, {"budget_bf16": 4}),
              ("fixed budget: 4 BF16 + 24 UINT4", inf, inf, 2, 0, {"budget_bf16": 4, "budget_u4": 24}),
              ("two tiers (6.5) + 32 sink tokens", 6.5, inf, 2, 0, {"sink_len": 32})]
    pairs += [(f"4-bit base ({W.P4BASE['tau_bf16']:g})", W.P4BASE["tau_bf16"], -1.0, 4, 0),
              ("all keys bf16 (values 2-bit)", -1.0, -1.0, 2, 0)]
    return pairs


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--config", default="qwen7b", choices=sorted(W.CONFIGS))
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--batch", type=int, default=2)
    ap.add_argument("--queries", type=int, default=4)
    ap.add_argument("--json", action="store_true", help="one JSON object per setting instead of the table")
    args = ap.parse_args()
    B.lib()
    w = W.small(W.CONFIGS[args.config], n_layers=1, batch=args.batch, tokens=args.tokens)
    rows = sweep(w, default_pairs(), n_queries=args.queries)
    if args.json:
        for r in rows:
            print(json.dumps(r))
        return
    print(f"{w.name}: batch {w.batch}, {w.n_kv_heads} KV heads x {w.g} query heads, {w.tokens} tokens, "
          f"R = {w.residual_len}, G = {w.group_size}; error of decode attention against unquantized bf16 K/V")
    print(f"{'setting':38s} {'key bits':>8s} {'n16':>6s} {'n4':>6s} {'max err':>10s} {'rms err':>10s} {'keys only':>10s}")
    for r in rows:
        print(f"{r['setting']:38s} {r['key_bits']:8.3f} {r['n16']:6.2f} {r['n4']:6.2f} {r['max_err']:10.2e} "
              f"{r['rms_err']:10.2e} {r['key_rms_err']:10.2e}")


if __name__ == "__main__":
    main()
