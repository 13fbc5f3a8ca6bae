"""CPU oracle for the MixKVQ decode hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy restatement of what the method computes, written from the
paper (arxiv 2512.19206) and from the written definition of the byte layouts (every position function below
states its formula).  It
shares no code with the CUDA path and must never be imported by the product package; only the
tests, the smoke check and the CPU-baseline leg of the benchmark may call it.

What each function follows:

* ``quantize_groups`` / ``dequantize``    Eq. 2 and Eq. 3 (B-bit asymmetric min/max quantizer),
                                          error bound of Appendix A.
* ``salience`` / ``assign_tiers``         importance, sensitivity and salience scores and the
                                          three-tier rule of Section 4.2 ("MixKVQ").
* ``OracleStream.append / flush``         the workflow of Section 4.2 and the lazy update of
                                          Appendix D.1; running |q| accumulator of Appendix D.2;
                                          GQA aggregation of Appendix D.
* ``OracleStream.attention``              Eq. 1 over the dequantized cache, fp64.
* ``pack_*``                              the storage layout (Appendix D "Storage Layout" gives
                                          the three stores; the bit positions are this repository's).
* ``effective_bits`` / ``fp16_cache_bytes``  B_eff of Appendix C; the footprint example of Section 1.
* ``causal_attention``                    Eq. 1 for the prompt (the prefill phase of Section 4.2): every position attends
                                          to itself and the positions before it, full precision, fp64.
* ``OracleStream.attention_partial`` /    Eq. 1 over a sequence whose tokens are spread over several caches (a context
  ``merge_partials``                      split over GPUs): each cache's output and log-denominator, merged by the
                                          log-sum-exp identity; equal to Eq. 1 over all tokens by construction.
* ``rope``                                the rotary embedding that Appendix D puts before the scores ("saliency
                                          evaluation is performed post-transformation"): keys and queries are
                                          rotated, then appended.

Precision: scores and attention in fp64.  The quantizer runs the fixed IEEE fp32 sequence
(subtract, divide by the stored bf16 scale, round half to even, clamp) because its integer result
must be reproduced bit for bit.

Parity pins: every function here is pinned by tests/test_oracle_*.py except the tier fractions
reached on real models (they need the models' weights): "parity unpinned" for those.

bf16 values are carried as float32 numbers whose low 16 bits are zero.
"""
from __future__ import annotations

import numpy as np

D = 128          # head dimension
TIER_U2, TIER_U4, TIER_BF16 = 0, 1, 2
TIER_BITS = {TIER_U2: 2, TIER_U4: 4, TIER_BF16: 16}


# --------------------------------------------------------------------------------------------
# bf16 helpers
# --------------------------------------------------------------------------------------------
def f32_bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def is_bf16(x) -> bool:
    return bool(np.all((f32_bits(x) & np.uint32(0xFFFF)) == 0))


def bf16_round_up(x):
    """Smallest bf16 value >= x, for finite x >= 0 (given as float32)."""
    b = f32_bits(x).astype(np.uint64)
    low = b & 0xFFFF
    b = np.where(low != 0, (b + 0x10000) & 0xFFFF0000, b)
    return b.astype(np.uint32).view(np.float32)


def bf16_rne(x):
    """Round float32 to bf16 (round to nearest even), returned as float32."""
    b = f32_bits(x).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(np.float32)


def bf16_to_u16(x):
    assert is_bf16(x)
    return (f32_bits(x) >> np.uint32(16)).astype(np.uint16)


def u16_to_bf16(u):
    return (np.asarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------------------------
# Eq. 2 / Eq. 3
# --------------------------------------------------------------------------------------------
def quantize_groups(x, bits):
    """B-bit asymmetric quantization of each row of ``x`` (float32 [..., n]) as one group.

    z = min, s = (max - min)/(2^B - 1) rounded up to bf16, c = round((x - z)/s) clamped.
    Returns (codes uint8 [..., n], s float32 [...], z float32 [...]).
    """
    x = np.asarray(x, dtype=np.float32)
    levels = np.float32((1 << bits) - 1)
    mx = x.max(axis=-1)
    mn = x.min(axis=-1)
    rng = (mx - mn).astype(np.float32)
    s = bf16_round_up((rng / levels).astype(np.float32))
    z = mn
    t = (x - z[..., None]).astype(np.float32)
    safe = np.where(s == 0, np.float32(1), s)
    y = (t / safe[..., None]).astype(np.float32)
    c = np.clip(np.rint(y), 0, float(levels))
    c = np.where((s == 0)[..., None], 0, c)
    return c.astype(np.uint8), s, z


def dequantize(codes, s, z):
    """Eq. 3 in fp64: x~ = c*s + z, with s, z broadcast over the last axis."""
    return codes.astype(np.float64) * np.asarray(s, np.float64)[..., None] + np.asarray(z, np.float64)[..., None]


# --------------------------------------------------------------------------------------------
# Section 4.2 scores
# --------------------------------------------------------------------------------------------
def salience(acc, cnt, k_window, score_bits):
    """I_d = acc_d / cnt, S_d = (max k_d - min k_d)/(2^B - 1) over the window, A_d = I_d * S_d."""
    k = np.asarray(k_window, dtype=np.float32)
    rng = k.max(axis=0).astype(np.float64) - k.min(axis=0).astype(np.float64)
    S = rng / float((1 << score_bits) - 1)
    I = np.asarray(acc, np.float64) / float(cnt)
    return I, S, I * S


def assign_tiers(A, tau_bf16, tau_u4):
    """BF16 if A > tau_bf16; else UINT4 if A > tau_u4; else UINT2.  Thresholds are float32 widened."""
    t16 = float(np.float32(tau_bf16))
    t4 = float(np.float32(tau_u4))
    A = np.asarray(A, np.float64)
    tiers = np.full(A.shape, TIER_U2, np.uint8)
    tiers[A > t4] = TIER_U4
    tiers[A > t16] = TIER_BF16
    return tiers


def assign_tiers_by_budget(A, budget_bf16, budget_u4):
    """Fixed-budget form of the tier rule of Section 4.2: the budget_bf16 channels of highest salience go to BF16, the next
    budget_u4 to UINT4, the rest to UINT2 (equal saliences: the lower channel index ranks first).  With no ties this is
    the threshold rule for any tau_bf16 between the budget_bf16-th and the next salience (and likewise tau_u4)."""
    A = np.asarray(A, np.float64)
    tiers = np.full(A.shape, TIER_U2, np.uint8)
    for d in range(A.shape[0]):
        rank = 0
        for e in range(A.shape[0]):
            if A[e] > A[d] or (A[e] == A[d] and e < d):
                rank += 1
        if rank < budget_bf16:
            tiers[d] = TIER_BF16
        elif rank < budget_bf16 + budget_u4:
            tiers[d] = TIER_U4
    return tiers


def importance_from_queries(q):
    """|q| summed in token-major, head-ascending order.  q float32 [g, n, D] -> (acc fp64 [D], cnt)."""
    q = np.asarray(q, np.float32)
    g, n, _ = q.shape
    mags = np.abs(q.astype(np.float64)).transpose(1, 0, 2).reshape(n * g, D)
    return sequential_sum(np.zeros(D), mags), n * g


def sequential_sum(start, rows):
    """start + rows[0] + rows[1] + ... added strictly in that order (fp64)."""
    if rows.shape[0] == 0:
        return np.array(start, np.float64)
    stacked = np.concatenate([np.asarray(start, np.float64)[None, :], rows], axis=0)
    return np.add.accumulate(stacked, axis=0)[-1]


def effective_bits(n16, n4, n2):
    """B_eff of Appendix C: mean of the per-channel bit-widths {16, 4, 2}."""
    return (16 * n16 + 4 * n4 + 2 * n2) / float(n16 + n4 + n2)


def fp16_cache_bytes(n_layers, n_kv_heads, head_dim, batch, tokens):
    """Bytes of an unquantized 16-bit KV cache (keys and values)."""
    return 2 * n_layers * n_kv_heads * head_dim * 2 * batch * tokens


# --------------------------------------------------------------------------------------------
# one (layer, batch element, KV head) stream
# --------------------------------------------------------------------------------------------
class Block:
    """One flushed R-token block, before packing."""
    __slots__ = ("tiers", "kcodes", "ks", "kz", "kraw", "vcodes", "vs", "vz", "A")


class OracleStream:
    def __init__(self, g, R=128, G=32, score_bits=2, tau_bf16=1e30, tau_u4=1e30, importance_mode=0, budget_bf16=0,
                 budget_u4=0, sink_len=0, v_bits=2):
        assert R % 32 == 0 and R % G == 0 and D % G == 0
        self.g, self.R, self.G = g, R, G
        self.score_bits, self.tau_bf16, self.tau_u4 = score_bits, tau_bf16, tau_u4
        self.importance_mode = importance_mode
        self.budget_bf16, self.budget_u4 = budget_bf16, budget_u4      # both 0: thresholds decide
        # sink tokens (the "sink length" of the paper's experimental settings, Appendix E): the first sink_len tokens of
        # the sequence stay in full precision for good; they never enter the residual window, the importance
        # accumulator or a quantized block
        self.sink_len = sink_len
        assert v_bits in (2, 4)
        self.v_bits = v_bits               # values: 2 bits per token-group code (Section 4.2), or 4
        self.sinkK = np.zeros((sink_len, D), np.float32)
        self.sinkV = np.zeros((sink_len, D), np.float32)
        self.n_sink = 0
        self.blocks: list[Block] = []
        self.resK = np.zeros((R, D), np.float32)
        self.resV = np.zeros((R, D), np.float32)
        self.r = 0
        self.acc = np.zeros(D, np.float64)
        self.cnt = 0
        self.n_flushes = 0

    # -- Appendix D.1: append into the residual buffer; flush lazily when it already holds R tokens
    def append(self, k, v, q):
        """k, v float32 [D]; q float32 [g, D] (all bf16-valued)."""
        if self.n_sink < self.sink_len:
            self.sinkK[self.n_sink] = k
            self.sinkV[self.n_sink] = v
            self.n_sink += 1
            return
        if self.r == self.R:
            self.flush()
        self.resK[self.r] = k
        self.resV[self.r] = v
        self.r += 1
        self.acc = sequential_sum(self.acc, np.abs(np.asarray(q, np.float32).astype(np.float64)))
        self.cnt += self.g

    def append_many(self, k, v, q):
        """k, v [n, D]; q [g, n, D].  Defined as n single appends in token order."""
        n = k.shape[0]
        t = 0
        while t < n and self.n_sink < self.sink_len:
            self.append(k[t], v[t], q[:, t])
            t += 1
        while t < n:
            if self.r == self.R:
                self.flush()
            m = min(n - t, self.R - self.r)
            self.resK[self.r:self.r + m] = k[t:t + m]
            self.resV[self.r:self.r + m] = v[t:t + m]
            mags = np.abs(np.asarray(q[:, t:t + m], np.float32).astype(np.float64))
            self.acc = sequential_sum(self.acc, mags.transpose(1, 0, 2).reshape(m * self.g, D))
            self.cnt += self.g * m
            self.r += m
            t += m

    def current_scores(self):
        I, S, A = salience(self.acc, self.cnt, self.resK[:self.r], self.score_bits)
        if self.importance_mode == 2:          # error-only ablation of the paper: the query term is dropped, A = S
            return np.ones_like(I), S, S.copy()
        return I, S, A

    def current_tiers(self):
        _, _, A = self.current_scores()
        if self.budget_bf16 + self.budget_u4 > 0:
            return assign_tiers_by_budget(A, self.budget_bf16, self.budget_u4), A
        return assign_tiers(A, self.tau_bf16, self.tau_u4), A

    def flush(self):
        assert self.r == self.R
        R, G = self.R, self.G
        tiers, A = self.current_tiers()
        blk = Block()
        blk.tiers, blk.A = tiers, A
        K = self.resK            # [R, D]
        NG = R // G
        blk.kcodes = np.zeros((R, D), np.uint8)
        blk.ks = np.zeros((NG, D), np.float32)
        blk.kz = np.zeros((NG, D), np.float32)
        blk.kraw = np.where((tiers == TIER_BF16)[None, :], K, np.float32(0)).astype(np.float32)
        grp = np.ascontiguousarray(K.T).reshape(D, NG, G)          # G consecutive tokens of channel d
        for tier in (TIER_U2, TIER_U4):
            c, s, z = quantize_groups(grp, TIER_BITS[tier])        # [D, NG, G], [D, NG], [D, NG]
            sel = tiers == tier
            blk.kcodes[:, sel] = c.reshape(D, R).T[:, sel]
            blk.ks[:, sel], blk.kz[:, sel] = s.T[:, sel], z.T[:, sel]
        V = self.resV.reshape(R, D // G, G)                    # G consecutive channels of a token
        c, s, z = quantize_groups(V, self.v_bits)
        blk.vcodes, blk.vs, blk.vz = c.reshape(R, D), s, z
        self.blocks.append(blk)
        self.r = 0
        self.n_flushes += 1
        if self.importance_mode != 1:
            self.acc = np.zeros(D, np.float64)
            self.cnt = 0

    # -- dequantized views (fp64)
    def keys(self):
        parts = [self.sinkK[:self.n_sink].astype(np.float64)]
        for b in self.blocks:
            NG = b.ks.shape[0]
            kq = (b.kcodes.reshape(NG, self.G, D).astype(np.float64) * b.ks.astype(np.float64)[:, None, :]
                  + b.kz.astype(np.float64)[:, None, :]).reshape(self.R, D)
            parts.append(np.where((b.tiers == TIER_BF16)[None, :], b.kraw.astype(np.float64), kq))
        parts.append(self.resK[:self.r].astype(np.float64))
        return np.concatenate(parts, axis=0)

    def values(self):
        parts = [self.sinkV[:self.n_sink].astype(np.float64)]
        for b in self.blocks:
            VG = D // self.G
            vq = (b.vcodes.reshape(self.R, VG, self.G).astype(np.float64) * b.vs.astype(np.float64)[..., None]
                  + b.vz.astype(np.float64)[..., None]).reshape(self.R, D)
            parts.append(vq)
        parts.append(self.resV[:self.r].astype(np.float64))
        return np.concatenate(parts, axis=0)

    @property
    def n_tokens(self):
        return self.n_sink + len(self.blocks) * self.R + self.r

    # -- Eq. 1
    def attention(self, q, scale, return_probs=False):
        """q float32 [g, D] -> o float32 [g, D]; softmax(q K~^T * scale) V~ in fp64."""
        Kt, Vt = self.keys(), self.values()
        logits = (np.asarray(q, np.float32).astype(np.float64) @ Kt.T) * float(scale)    # [g, T]
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        o = p @ Vt
        if return_probs:
            return o.astype(np.float32), p
        return o.astype(np.float32)

    def attention_partial(self, q, scale):
        """Eq. 1 restricted to the tokens this stream holds, in the form a sequence split needs: (o, lse) with
        o float64 [g, D] the softmax-weighted values over these tokens alone and lse float64 [g] the natural
        logarithm of the softmax denominator sum_j exp(scale q.k_j).  A stream without tokens gives o = 0, lse = -inf."""
        Kt, Vt = self.keys(), self.values()
        g = np.asarray(q).shape[0]
        if Kt.shape[0] == 0:
            return np.zeros((g, D), np.float64), np.full(g, -np.inf)
        logits = (np.asarray(q, np.float32).astype(np.float64) @ Kt.T) * float(scale)
        m = logits.max(axis=1, keepdims=True)
        p = np.exp(logits - m)
        den = p.sum(axis=1, keepdims=True)
        return (p @ Vt) / den, (m + np.log(den))[:, 0]


def merge_partials(os, lses):
    """Softmax attention over the union of disjoint token sets from the per-set results (the log-sum-exp identity):
    with w_r = exp(lse_r),  o = sum_r w_r o_r / sum_r w_r.  os [n, ..., D], lses [n, ...] (fp64); parts with
    lse = -inf (no tokens) carry weight 0; if every part is empty the result is 0."""
    os = np.asarray(os, np.float64)
    lses = np.asarray(lses, np.float64)
    top = lses.max(axis=0)
    safe = np.where(np.isfinite(top), top, 0.0)
    w = np.exp(lses - safe)                       # exp(-inf) = 0 for the empty parts
    den = w.sum(axis=0)
    num = (w[..., None] * os).sum(axis=0)
    return np.where(den[..., None] > 0, num / np.where(den > 0, den, 1.0)[..., None], 0.0)


def rope(x, cos, sin):
    """Rotary position embedding of bf16-valued rows x [..., n, D] at the n positions whose table rows are
    cos, sin [n, D/2] (float32, supplied by the caller: the oracle takes no trigonometric function).

    Pairing of the channels: (i, i + D/2), the "rotate-half" convention of the Llama and Qwen families.  With
    c = cos[p, i], s = sin[p, i]:   y[i] = x[i] c - x[i + D/2] s,   y[i + D/2] = x[i + D/2] c + x[i] s.
    Arithmetic: every product and the one sum are single IEEE fp32 operations (round to nearest, no fused
    multiply-add); the result is rounded to bf16 (nearest, ties to even).  Returned as float32 holding bf16 values.
    Appendix D fixes only that scores and keys are taken after this rotation; the order of the operations is this
    repository's, stated here so that the rotated bf16 bits are reproducible."""
    x = np.asarray(x, np.float32)
    cos = np.asarray(cos, np.float32)
    sin = np.asarray(sin, np.float32)
    h = x.shape[-1] // 2
    x1, x2 = x[..., :h], x[..., h:]
    a = (x1 * cos).astype(np.float32)
    b = (x2 * sin).astype(np.float32)
    c = (x2 * cos).astype(np.float32)
    d = (x1 * sin).astype(np.float32)
    y = np.concatenate([(a - b).astype(np.float32), (c + d).astype(np.float32)], axis=-1)
    return bf16_rne(y)


def unquantized_attention(q, K, V, scale):
    """Textbook Eq. 1 on raw tensors (fp64): q [g, D], K, V [T, D]."""
    logits = (np.asarray(q, np.float64) @ np.asarray(K, np.float64).T) * float(scale)
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    return p @ np.asarray(V, np.float64)


def causal_attention(q, K, V, scale):
    """Eq. 1 over a prompt, position by position: q [g, L, D], K, V [L, D] (bf16-valued) -> [g, L, D] float64.
    Position i sees keys and values 0..i: the plain definition, one softmax per row, nothing blocked or reused.
    The prompt's keys and values are attended in full precision (Section 4.2: quantization happens after the
    prefill computation; the cache the prompt leaves behind is that of append_many)."""
    q = np.asarray(q, np.float64)
    K = np.asarray(K, np.float64)
    V = np.asarray(V, np.float64)
    g, L, _ = q.shape
    out = np.zeros((g, L, V.shape[1]), np.float64)
    for i in range(L):
        logits = (q[:, i] @ K[:i + 1].T) * float(scale)
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        out[:, i] = p @ V[:i + 1]
    return out


# --------------------------------------------------------------------------------------------
# byte layout (one element at a time, from the stated position formulas)
# fragment layout (the default): blocks of any R
# --------------------------------------------------------------------------------------------
def unit_bytes_of(G, v_bits=2):
    """One 32-token unit: key low plane 1024, value low plane 1024, value scales and zero-points, and with 4-bit values the
    value high plane (codes >> 2, in the low plane's bit positions) 1024."""
    return 2048 + 128 * (D // G) + (1024 if v_bits == 4 else 0)


def base_bytes(R, G, v_bits=2):
    return (R // G) * 512 + (R // 32) * unit_bytes_of(G, v_bits)


def dense_high_plane(tau_u4):
    """4-bit base precision (tau_u4 < 0: no channel stays at 2 bits): the high plane of every block is a full
    1024-byte plane per unit in the low plane's bit order instead of 16 bytes per UINT4 channel pair."""
    return tau_u4 < 0


def extras_bytes(R, n16, n4, dense=False):
    n16p, n4p = (n16 + 1) // 2, 2 * ((n4 + 1) // 2)
    hi = 1024 if dense else 8 * n4p
    return 16 * ((2 * n16p + n4p + 15) // 16) + (R // 32) * (128 * n16p + hi)


def frag_meta_off(kg, G, unit_bytes):
    """Fragment layout: byte offset of key-meta group kg inside the base block (directly before the group's first unit)."""
    return kg * (G // 32) * unit_bytes + 512 * kg


def frag_unit_off(u, G, unit_bytes):
    """Fragment layout: byte offset of 32-token unit u inside the base block."""
    return u * unit_bytes + 512 * ((u * 32) // G + 1)


def _k_code_pos(jj, d):
    mt, row = divmod(jj, 16)
    rh, r = divmod(row, 8)
    kt, col = divmod(d, 16)
    ch, c8 = divmod(col, 8)
    t, e = divmod(c8, 2)
    lane, a = 4 * r + t, 2 * ch + rh
    return mt * 512 + lane * 16 + a * 4, 16 * e + 2 * kt


def _v_code_pos(jj, c):
    ct, row = divmod(c, 16)
    rh, r = divmod(row, 8)
    ks, col = divmod(jj, 16)
    ch, c8 = divmod(col, 8)
    t, e = divmod(c8, 2)
    lane = 4 * r + t
    return (ct // 4) * 512 + lane * 16 + (ct % 4) * 4, 16 * e + 2 * (4 * rh + 2 * ks + ch)


def _hi_plane_pos(jj, e):
    """UINT4 high plane: (byte offset inside the pair's 16 bytes, bit offset) of token jj, half e."""
    mt, row = divmod(jj, 16)
    rh, r = divmod(row, 8)
    return (r % 4) * 4, 16 * e + 8 * (r // 4) + 2 * (2 * mt + rh)


def _tables():
    """Position tables: the scalar layout functions evaluated for every (token, channel)."""
    if not hasattr(_tables, "cache"):
        kw = np.zeros((32, D), np.int64); kb = np.zeros((32, D), np.int64)
        vw = np.zeros((32, D), np.int64); vb = np.zeros((32, D), np.int64)
        for jj in range(32):
            for d in range(D):
                off, bit = _k_code_pos(jj, d)
                kw[jj, d], kb[jj, d] = off // 4, bit
                off, bit = _v_code_pos(jj, d)
                vw[jj, d], vb[jj, d] = off // 4, bit
        hw = np.zeros((32, 2), np.int64); hb = np.zeros((32, 2), np.int64)
        for jj in range(32):
            for e in range(2):
                off, bit = _hi_plane_pos(jj, e)
                hw[jj, e], hb[jj, e] = off // 4, bit
        # every (word, bit) target must be hit exactly once: the maps are bijections
        for w, b in ((kw, kb), (vw, vb)):
            assert len(set(zip(w.ravel().tolist(), b.ravel().tolist()))) == 32 * D
            assert w.max() == 255 and b.max() == 30
        _tables.cache = (kw, kb, vw, vb, hw, hb)
    return _tables.cache


def _scatter_codes(words, word_idx, bit_idx, codes):
    """OR 2-bit codes into 32-bit words; targets are disjoint so add == or."""
    np.add.at(words, word_idx.ravel(), (codes.astype(np.uint32) << bit_idx.astype(np.uint32)).ravel())


def pack_base(blk: Block, R, G, v_bits=2):
    NG, U, VG = R // G, R // 32, D // G
    kw, kb, vw, vb, _, _ = _tables()
    words = np.zeros(base_bytes(R, G, v_bits) // 4, np.uint32)
    quant = blk.tiers != TIER_BF16
    # K meta: entry (kg, d) at kg*512 + d*4 = {s, z}
    ks16 = np.where(quant[None, :], bf16_to_u16(blk.ks), 0).astype(np.uint32)
    kz16 = np.where(quant[None, :], bf16_to_u16(blk.kz), 0).astype(np.uint32)
    unit_bytes = unit_bytes_of(G, v_bits)
    meta = ks16 | (kz16 << 16)                                   # entry (kg, d) at frag_meta_off(kg) + d*4
    for kg in range(NG):
        mo = frag_meta_off(kg, G, unit_bytes) // 4
        words[mo:mo + 128] = meta[kg]
    vs16, vz16 = bf16_to_u16(blk.vs).astype(np.uint32), bf16_to_u16(blk.vz).astype(np.uint32)
    klow = np.where(quant[None, :], blk.kcodes & 3, 0)
    for u in range(U):
        ubase = frag_unit_off(u, G, unit_bytes) // 4
        sl = slice(32 * u, 32 * u + 32)
        _scatter_codes(words, ubase + kw, kb, klow[sl])
        _scatter_codes(words, ubase + 256 + vw, vb, blk.vcodes[sl] & 3)
        words[ubase + 512:ubase + 512 + 32 * VG] = (vs16[sl] | (vz16[sl] << 16)).reshape(32 * VG)
        if v_bits == 4:
            _scatter_codes(words, ubase + 512 + 32 * VG + vw, vb, blk.vcodes[sl] >> 2)
    return words.astype("<u4").tobytes()


def channel_lists(tiers):
    chan16 = [d for d in range(D) if tiers[d] == TIER_BF16]
    chan4 = [d for d in range(D) if tiers[d] == TIER_U4]
    return chan16, chan4


def pack_extras(blk: Block, R, dense=False):
    U = R // 32
    _, _, _, _, hw, hb = _tables()
    chan16, chan4 = channel_lists(blk.tiers)
    n16, n4 = len(chan16), len(chan4)
    n16p, n4p = (n16 + 1) // 2, 2 * ((n4 + 1) // 2)
    total = extras_bytes(R, n16, n4, dense)
    hdr = 16 * ((2 * n16p + n4p + 15) // 16)
    head = bytearray(hdr)
    l16 = chan16 + [0xFF] * (2 * n16p - n16)
    l4 = chan4 + [0xFF] * (n4p - n4)
    head[0:2 * n16p] = bytes(l16)
    head[2 * n16p:2 * n16p + n4p] = bytes(l4)
    words = np.zeros((total - hdr) // 4, np.uint32)
    unit_words = (128 * n16p + (1024 if dense else 8 * n4p)) // 4
    kw, kb = _tables()[0], _tables()[1]
    khigh = np.where((blk.tiers == TIER_U4)[None, :], blk.kcodes >> 2, 0)
    raw16 = bf16_to_u16(blk.kraw).astype(np.uint32)
    for u in range(U):
        ubase = u * unit_words
        sl = slice(32 * u, 32 * u + 32)
        for i in range(n16p):
            lo = raw16[sl, l16[2 * i]]
            hi = raw16[sl, l16[2 * i + 1]] if l16[2 * i + 1] != 0xFF else np.zeros(32, np.uint32)
            words[ubase + i * 32:ubase + i * 32 + 32] = lo | (hi << 16)       # word (i*32 + jj)
        hbase = ubase + 32 * n16p
        if dense:                                   # the low plane's positions, code >> 2 of UINT4 channels, 0 elsewhere
            _scatter_codes(words, hbase + kw, kb, khigh[sl])
            continue
        for i in range(n4p // 2):
            for e in range(2):
                ch = l4[2 * i + e]
                if ch == 0xFF:
                    continue
                _scatter_codes(words, hbase + i * 4 + hw[:, e], hb[:, e], blk.kcodes[sl, ch] >> 2)
    return bytes(head) + words.astype("<u4").tobytes(), n16, n4


def unpack_base(buf, R, G, v_bits=2):
    """Inverse of pack_base for the code planes and the metadata, element by element."""
    NG, U, VG = R // G, R // 32, D // G
    words = np.frombuffer(buf, dtype="<u4")
    halves = np.frombuffer(buf, dtype="<u2")
    ks = np.zeros((NG, D), np.float32)
    kz = np.zeros((NG, D), np.float32)
    unit_bytes = unit_bytes_of(G, v_bits)
    for kg in range(NG):
        for d in range(D):
            ks[kg, d] = u16_to_bf16(halves[(frag_meta_off(kg, G, unit_bytes) + d * 4) // 2])
            kz[kg, d] = u16_to_bf16(halves[(frag_meta_off(kg, G, unit_bytes) + d * 4) // 2 + 1])
    klow = np.zeros((R, D), np.uint8)
    vcodes = np.zeros((R, D), np.uint8)
    vs = np.zeros((R, VG), np.float32)
    vz = np.zeros((R, VG), np.float32)
    for u in range(U):
        ubase = frag_unit_off(u, G, unit_bytes)
        for jj in range(32):
            j = 32 * u + jj
            for d in range(D):
                off, bit = _k_code_pos(jj, d)
                klow[j, d] = (int(words[(ubase + off) // 4]) >> bit) & 3
                off, bit = _v_code_pos(jj, d)
                vcodes[j, d] = (int(words[(ubase + 1024 + off) // 4]) >> bit) & 3
                if v_bits == 4:
                    vcodes[j, d] |= ((int(words[(ubase + 2048 + 128 * VG + off) // 4]) >> bit) & 3) << 2
            for vg in range(VG):
                o = (ubase + 2048 + (jj * VG + vg) * 4) // 2
                vs[j, vg] = u16_to_bf16(halves[o])
                vz[j, vg] = u16_to_bf16(halves[o + 1])
    return klow, ks, kz, vcodes, vs, vz


# --------------------------------------------------------------------------------------------
# tile layout (optional, blocks of R = 128 tokens): one thread of the attention kernel owns one token's key codes
# and one channel's value codes, each a contiguous run of 2-bit fields
# --------------------------------------------------------------------------------------------
LAYOUT_FRAGMENT, LAYOUT_TILE = 0, 1


def tile_base_bytes(G):
    return (128 // G) * 512 + 4096 + 4096 + 128 * (D // G) * 4


def tile_extras_bytes(n16, n4):
    n16p, n4w = (n16 + 1) // 2, (n4 + 15) // 16
    return 16 * ((2 * n16p + 16 * n4w + 15) // 16) + 512 * (n16p + n4w)


def _tile_code_pos(row, i):
    """Code number i (0..127) of a 32-byte row: (byte offset of the 32-bit word inside the 4096-byte plane,
    bit offset).  Keys: row = token, i = channel.  Values: row = channel, i = token."""
    hh, rem = divmod(i, 64)
    w, rem = divmod(rem, 16)
    f, e = divmod(rem, 2)
    return hh * 2048 + row * 16 + w * 4, 16 * e + 2 * f


def _tile_tables():
    if not hasattr(_tile_tables, "cache"):
        wi = np.zeros((128, 128), np.int64); bi = np.zeros((128, 128), np.int64)
        for row in range(128):
            for i in range(128):
                off, bit = _tile_code_pos(row, i)
                wi[row, i], bi[row, i] = off // 4, bit
        assert len(set(zip(wi.ravel().tolist(), bi.ravel().tolist()))) == 128 * 128
        assert wi.max() == 1023 and bi.max() == 30
        _tile_tables.cache = (wi, bi)
    return _tile_tables.cache


def pack_base_tile(blk: Block, G):
    NG, VG = 128 // G, D // G
    wi, bi = _tile_tables()
    words = np.zeros(tile_base_bytes(G) // 4, np.uint32)
    quant = blk.tiers != TIER_BF16
    ks16 = np.where(quant[None, :], bf16_to_u16(blk.ks), 0).astype(np.uint32)
    kz16 = np.where(quant[None, :], bf16_to_u16(blk.kz), 0).astype(np.uint32)
    words[:NG * 128] = (ks16 | (kz16 << 16)).reshape(NG * 128)            # entry (kg, d) at kg*512 + d*4
    klow = np.where(quant[None, :], blk.kcodes & 3, 0)
    kbase = NG * 128
    _scatter_codes(words, kbase + wi, bi, klow)                            # row = token, i = channel
    _scatter_codes(words, kbase + 1024 + wi, bi, blk.vcodes.T)             # row = channel, i = token
    vs16, vz16 = bf16_to_u16(blk.vs).astype(np.uint32), bf16_to_u16(blk.vz).astype(np.uint32)
    words[kbase + 2048:kbase + 2048 + 128 * VG] = (vs16 | (vz16 << 16)).reshape(128 * VG)   # (j*VG + vg)*4
    return words.astype("<u4").tobytes()


def unpack_base_tile(buf, G):
    NG, VG = 128 // G, D // G
    words = np.frombuffer(buf, dtype="<u4")
    halves = np.frombuffer(buf, dtype="<u2")
    ks = np.zeros((NG, D), np.float32); kz = np.zeros((NG, D), np.float32)
    for kg in range(NG):
        for d in range(D):
            ks[kg, d] = u16_to_bf16(halves[(kg * 512 + d * 4) // 2])
            kz[kg, d] = u16_to_bf16(halves[(kg * 512 + d * 4) // 2 + 1])
    klow = np.zeros((128, D), np.uint8); vcodes = np.zeros((128, D), np.uint8)
    vs = np.zeros((128, VG), np.float32); vz = np.zeros((128, VG), np.float32)
    kb, vb, mb = NG * 512, NG * 512 + 4096, NG * 512 + 8192
    for j in range(128):
        for d in range(D):
            off, bit = _tile_code_pos(j, d)
            klow[j, d] = (int(words[(kb + off) // 4]) >> bit) & 3
            off, bit = _tile_code_pos(d, j)
            vcodes[j, d] = (int(words[(vb + off) // 4]) >> bit) & 3
        for vg in range(VG):
            o = (mb + (j * VG + vg) * 4) // 2
            vs[j, vg] = u16_to_bf16(halves[o]); vz[j, vg] = u16_to_bf16(halves[o + 1])
    return klow, ks, kz, vcodes, vs, vz


def pack_extras_tile(blk: Block):
    chan16, chan4 = channel_lists(blk.tiers)
    n16, n4 = len(chan16), len(chan4)
    n16p, n4w = (n16 + 1) // 2, (n4 + 15) // 16
    hdr = 16 * ((2 * n16p + 16 * n4w + 15) // 16)
    head = bytearray(hdr)
    l16 = chan16 + [0xFF] * (2 * n16p - n16)
    l4 = chan4 + [0xFF] * (16 * n4w - n4)
    head[0:2 * n16p] = bytes(l16)
    head[2 * n16p:2 * n16p + 16 * n4w] = bytes(l4)
    words = np.zeros(128 * (n16p + n4w), np.uint32)
    raw16 = bf16_to_u16(blk.kraw).astype(np.uint32)
    for i in range(n16p):                                                   # word (i*128 + j)
        lo = raw16[:, l16[2 * i]]
        hi = raw16[:, l16[2 * i + 1]] if l16[2 * i + 1] != 0xFF else np.zeros(128, np.uint32)
        words[i * 128:(i + 1) * 128] = lo | (hi << 16)
    for idx, ch in enumerate(chan4):                                        # word ((n16p + w)*128 + j)
        w, rem = divmod(idx, 16)
        f, e = divmod(rem, 2)
        words[(n16p + w) * 128:(n16p + w + 1) * 128] |= (blk.kcodes[:, ch] >> 2).astype(np.uint32) << np.uint32(16 * e + 2 * f)
    out = bytes(head) + words.astype("<u4").tobytes()
    assert len(out) == tile_extras_bytes(n16, n4)
    return out, n16, n4


def table_entry(extras_off16, n16, n4):
    return int(extras_off16).to_bytes(4, "little") + bytes([n16, n4, 0, 0])


def pack_stream(st: OracleStream, layout=LAYOUT_FRAGMENT):
    """All bytes the stream would hold in device memory, by region."""
    base, table, extras = [], [], []
    used16 = 0
    tile = layout == LAYOUT_TILE
    assert not tile or (st.R == 128 and st.v_bits == 2)
    for blk in st.blocks:
        if tile:
            base.append(pack_base_tile(blk, st.G))
            ex, n16, n4 = pack_extras_tile(blk)
        else:
            base.append(pack_base(blk, st.R, st.G, st.v_bits))
            ex, n16, n4 = pack_extras(blk, st.R, dense_high_plane(st.tau_u4) and st.budget_bf16 + st.budget_u4 == 0)
        table.append(table_entry(used16, n16, n4))
        extras.append(ex)
        used16 += len(ex) // 16
    state = bytearray(1152)
    state[0:1024] = st.acc.astype("<f8").tobytes()
    state[1024:1028] = int(st.cnt).to_bytes(4, "little")
    state[1028:1032] = int(used16).to_bytes(4, "little")
    return {
        "base": b"".join(base),
        "table": b"".join(table),
        "extras": b"".join(extras),
        "state": bytes(state),
        "resK": bf16_to_u16(st.resK[:st.r]).astype("<u2").tobytes(),
        "resV": bf16_to_u16(st.resV[:st.r]).astype("<u2").tobytes(),
        "sinkK": bf16_to_u16(st.sinkK[:st.n_sink]).astype("<u2").tobytes(),
        "sinkV": bf16_to_u16(st.sinkV[:st.n_sink]).astype("<u2").tobytes(),
    }
