"""Thin ctypes binding of libmixkvq.so: argument marshalling only.

Every step of the path (scoring, quantization, packing, attention) runs in the library's CUDA kernels.
PyTorch is used for device memory and the current stream.  If the shared library cannot be loaded this
module raises: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmixkvq.so")

EXPORTS = [
    "mixkvq_cache_bytes", "mixkvq_cache_init", "mixkvq_cache_destroy", "mixkvq_cache_reset",
    "mixkvq_select_channels", "mixkvq_select_channels_raw", "mixkvq_quantize_append",
    "mixkvq_decode_attention", "mixkvq_decode_attention_noalloc", "mixkvq_decode_step", "mixkvq_set_attention_kernel", "mixkvq_query_status",
    "mixkvq_cache_describe", "mixkvq_launch_count", "mixkvq_status_string",
    "mixkvq_cache_written_externally", "mixkvq_test_arm_copy_timeout", "mixkvq_rope_append", "mixkvq_rope_decode_step", "mixkvq_prefill", "mixkvq_prefill_scratch_bytes", "mixkvq_quantize_append_ragged", "mixkvq_sequence_fill", "mixkvq_decode_attention_partial", "mixkvq_merge_partials",
]

DEV_EXTRAS_FULL, DEV_COPY_TIMEOUT = 1, 2


class Config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("max_tokens", C.c_int32), ("residual_len", C.c_int32), ("group_size", C.c_int32),
        ("v_bits", C.c_int32), ("score_bits", C.c_int32), ("tau_bf16", C.c_float), ("tau_u4", C.c_float),
        ("importance_mode", C.c_int32), ("block_layout", C.c_int32), ("extras_budget_bytes", C.c_uint64),
        ("budget_bf16", C.c_int32), ("budget_u4", C.c_int32), ("sink_len", C.c_int32), ("reserved", C.c_int32),
    ]


class LayoutDesc(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "state_off", "state_stride", "table_off", "table_stride", "resk_off", "resk_stride",
        "resv_off", "resv_stride", "base_off", "base_stride", "extras_off", "extras_stride", "base_bytes")] + [
        (n, C.c_uint32) for n in ("max_blocks", "n_streams", "n_blocks", "residual_tokens")] + [
        ("sink_off", C.c_uint64), ("sink_stride", C.c_uint64), ("sink_tokens", C.c_uint32), ("sink_len", C.c_uint32)]


class MixKVQError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


_lib = None


def lib():
    """The loaded shared library; raises if it is missing (build it with `python -m paper_2512_19206_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA library first "
                               "(python -m paper_2512_19206_b200.build); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32, u64 = C.c_void_p, C.c_int, C.c_float, C.c_uint64
        L.mixkvq_cache_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        L.mixkvq_cache_init.argtypes = [C.POINTER(Config), vp, C.c_size_t, vp, C.POINTER(vp)]
        L.mixkvq_cache_destroy.argtypes = [vp]
        L.mixkvq_cache_reset.argtypes = [vp, i32, vp]
        L.mixkvq_select_channels.argtypes = [vp, i32, vp, vp, vp]
        L.mixkvq_select_channels_raw.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, f32, f32, vp, vp, vp]
        L.mixkvq_quantize_append.argtypes = [vp, i32, vp, vp, vp, i32, vp]
        L.mixkvq_decode_attention.argtypes = [vp, i32, vp, vp, f32, vp, C.c_size_t, vp]
        L.mixkvq_decode_attention_noalloc.argtypes = [vp, i32, vp, vp, f32, vp]
        L.mixkvq_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, f32, vp, C.c_size_t, vp]
        L.mixkvq_set_attention_kernel.argtypes = [vp, i32]
        L.mixkvq_quantize_append_ragged.argtypes = [vp, i32, vp, vp, vp, i32, C.POINTER(C.c_int32), vp]
        L.mixkvq_sequence_fill.argtypes = [vp, i32, i32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.mixkvq_decode_attention_partial.argtypes = [vp, i32, vp, vp, vp, f32, vp, C.c_size_t, vp]
        L.mixkvq_merge_partials.argtypes = [vp, vp, i32, i32, vp, vp]
        L.mixkvq_prefill.argtypes = [vp, i32, vp, vp, vp, i32, vp, f32, vp, C.c_size_t, vp]
        L.mixkvq_prefill_scratch_bytes.argtypes = [C.POINTER(Config), i32]
        L.mixkvq_prefill_scratch_bytes.restype = C.c_size_t
        L.mixkvq_rope_append.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32, i32, vp]
        L.mixkvq_rope_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32, vp, f32, vp, C.c_size_t, vp]
        L.mixkvq_cache_written_externally.argtypes = [vp]
        L.mixkvq_test_arm_copy_timeout.argtypes = [vp, C.c_uint32, C.c_uint32]
        L.mixkvq_query_status.argtypes = [vp, C.POINTER(i32), vp]
        L.mixkvq_cache_describe.argtypes = [vp, i32, C.POINTER(LayoutDesc)]
        L.mixkvq_launch_count.argtypes = [vp]
        L.mixkvq_launch_count.restype = u64
        L.mixkvq_status_string.argtypes = [i32]
        L.mixkvq_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("mixkvq_launch_count", "mixkvq_status_string"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().mixkvq_status_string(int(code)).decode()


def _check(code, what):
    if code != 0:
        raise MixKVQError(code, what)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: torch.Tensor | None):
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def make_config(n_layers, batch, n_q_heads, n_kv_heads, max_tokens, residual_len=128, group_size=32,
                tau_bf16=1e30, tau_u4=1e30, score_bits=2, importance_mode=0, extras_budget_bytes=0,
                block_layout=0, budget_bf16=0, budget_u4=0, sink_len=0, v_bits=2) -> Config:
    return Config(n_layers, batch, n_q_heads, n_kv_heads, 128, max_tokens, residual_len, group_size, v_bits, score_bits,
                  tau_bf16, tau_u4, importance_mode, block_layout, extras_budget_bytes, budget_bf16, budget_u4,
                  sink_len, 0)


def cache_bytes(cfg: Config):
    a, b = C.c_size_t(), C.c_size_t()
    _check(lib().mixkvq_cache_bytes(C.byref(cfg), C.byref(a), C.byref(b)), "mixkvq_cache_bytes")
    return a.value, b.value


def merge_partials(o_parts: torch.Tensor, lse_parts: torch.Tensor, out=None):
    """o_parts [n, ..., 128], lse_parts [n, ...] float32 (device) -> [..., 128]: attention over the union of the parts."""
    n = o_parts.shape[0]
    rows = lse_parts[0].numel()
    if out is None:
        out = torch.empty(o_parts.shape[1:], dtype=torch.float32, device=o_parts.device)
    if not (o_parts.is_cuda and o_parts.is_contiguous() and lse_parts.is_contiguous()):
        raise ValueError("merge_partials needs contiguous CUDA tensors")
    _check(lib().mixkvq_merge_partials(_ptr(o_parts), _ptr(lse_parts), n, rows, _ptr(out), _stream()),
           "mixkvq_merge_partials")
    return out


def select_channels_raw(q: torch.Tensor, k: torch.Tensor, score_bits, tau_bf16, tau_u4, want_salience=True):
    """q [B,Hq,Lq,128] bf16, k [B,Hkv,Lk,128] bf16 -> tiers uint8 [B,Hkv,128], salience float64 [B,Hkv,128]."""
    B, Hq, Lq, _ = q.shape
    _, Hkv, Lk, _ = k.shape
    tiers = torch.empty((B, Hkv, 128), dtype=torch.uint8, device=q.device)
    sal = torch.empty((B, Hkv, 128), dtype=torch.float64, device=q.device) if want_salience else None
    _check(lib().mixkvq_select_channels_raw(_ptr(q), _ptr(k), B, Hq, Hkv, Lq, Lk, score_bits, tau_bf16, tau_u4,
                                            _ptr(tiers), _ptr(sal), _stream()), "mixkvq_select_channels_raw")
    return tiers, sal


class Cache:
    """Owns the device memory (a torch uint8 tensor) and the library's host handle."""

    def __init__(self, cfg: Config, device="cuda"):
        self.cfg = cfg
        nbytes, ws_bytes = cache_bytes(cfg)
        self.mem = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        self.handle = C.c_void_p()
        with torch.cuda.device(self.mem.device):
            _check(lib().mixkvq_cache_init(C.byref(cfg), _ptr(self.mem), nbytes, _stream(), C.byref(self.handle)),
                   "mixkvq_cache_init")

    def close(self):
        if self.handle:
            lib().mixkvq_cache_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, layer=-1):
        _check(lib().mixkvq_cache_reset(self.handle, layer, _stream()), "mixkvq_cache_reset")

    def quantize_append(self, layer, k, v, q):
        """k, v [B,Hkv,n,128] bf16; q [B,Hq,n,128] bf16 (n may be 1: a decode step)."""
        n = k.shape[2]
        _check(lib().mixkvq_quantize_append(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), n, _stream()),
               "mixkvq_quantize_append")

    def decode_attention(self, layer, q, scale, out=None):
        """q [B,Hq,128] bf16 -> out [B,Hq,128] float32."""
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        _check(lib().mixkvq_decode_attention(self.handle, layer, _ptr(q), _ptr(out), float(scale),
                                             _ptr(self.workspace), self.workspace.numel(), _stream()),
               "mixkvq_decode_attention")
        return out

    def decode_step(self, layer, k, v, q, scale, out=None):
        """One decode step: k, v [B,Hkv,1,128], q [B,Hq,1,128] bf16 -> out [B,Hq,128] float32 (append + attention)."""
        if out is None:
            out = torch.empty((q.shape[0], q.shape[1], 128), dtype=torch.float32, device=q.device)
        _check(lib().mixkvq_decode_step(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), _ptr(out), float(scale),
                                        _ptr(self.workspace), self.workspace.numel(), _stream()), "mixkvq_decode_step")
        return out

    def decode_attention_partial(self, layer, q, scale, out=None, lse=None):
        """q [B,Hq,128] bf16 -> (out [B,Hq,128], lse [B,Hq]) float32: attention over this cache's tokens alone and the
        natural log of its softmax denominator (the inputs of merge_partials)."""
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        if lse is None:
            lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
        _check(lib().mixkvq_decode_attention_partial(self.handle, layer, _ptr(q), _ptr(out), _ptr(lse), float(scale),
                                                     _ptr(self.workspace), self.workspace.numel(), _stream()),
               "mixkvq_decode_attention_partial")
        return out, lse

    def quantize_append_ragged(self, layer, k, v, q, counts):
        """k, v [B,Hkv,n_max,128], q [B,Hq,n_max,128] bf16; counts: per-sequence token counts (host ints)."""
        arr = (C.c_int32 * len(counts))(*[int(c) for c in counts])
        _check(lib().mixkvq_quantize_append_ragged(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), k.shape[2], arr,
                                                   _stream()), "mixkvq_quantize_append_ragged")

    def sequence_fill(self, layer, b):
        """(n_blocks, residual_tokens, sink_tokens) of sequence b."""
        x = [C.c_uint32(0) for _ in range(3)]
        _check(lib().mixkvq_sequence_fill(self.handle, layer, b, C.byref(x[0]), C.byref(x[1]), C.byref(x[2])),
               "mixkvq_sequence_fill")
        return tuple(int(v.value) for v in x)

    def prefill(self, layer, k, v, q, scale, out=None, scratch=None):
        """Causal attention of the prompt over itself (k, v [B,Hkv,n,128], q [B,Hq,n,128] bf16 -> [B,Hq,n,128] float32),
        then the prompt goes into the (empty) layer as quantize_append would put it.  `scratch`: a uint8 device
        tensor of at least prefill_scratch_bytes(n) bytes (allocated here when absent)."""
        n = k.shape[2]
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        if scratch is None:
            scratch = torch.empty(self.prefill_scratch_bytes(n), dtype=torch.uint8, device=q.device)
        _check(lib().mixkvq_prefill(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), n, _ptr(out), float(scale),
                                    _ptr(scratch), scratch.numel(), _stream()), "mixkvq_prefill")
        return out

    def prefill_scratch_bytes(self, n_tokens):
        return int(lib().mixkvq_prefill_scratch_bytes(C.byref(self.cfg), int(n_tokens)))

    def rope_append(self, layer, k, v, q, cos, sin, pos0):
        """Rotates k [B,Hkv,n,128] and q [B,Hq,n,128] (bf16) IN PLACE with rows pos0.. of the float32 tables cos, sin
        [n_positions, 64], then appends them as quantize_append does."""
        assert cos.dtype == torch.float32 and sin.dtype == torch.float32
        _check(lib().mixkvq_rope_append(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), _ptr(cos), _ptr(sin), int(pos0),
                                        k.shape[2], _stream()), "mixkvq_rope_append")

    def rope_decode_step(self, layer, k, v, q, cos, sin, pos, scale, out=None):
        """One decode step with the rotation of k and q (in place) in front: see decode_step."""
        if out is None:
            out = torch.empty((q.shape[0], q.shape[1], 128), dtype=torch.float32, device=q.device)
        _check(lib().mixkvq_rope_decode_step(self.handle, layer, _ptr(k), _ptr(v), _ptr(q), _ptr(cos), _ptr(sin), int(pos),
                                             _ptr(out), float(scale), _ptr(self.workspace), self.workspace.numel(),
                                             _stream()), "mixkvq_rope_decode_step")
        return out

    def decode_attention_noalloc(self, layer, q, scale, out=None):
        """Same as decode_attention, but the library's built-in scratch array holds the split partials: for
        callers that cannot provide a workspace.  `out` should be passed by such callers (the default
        allocates it with torch for convenience).  Calls that overlap on the GPU race on the shared array."""
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        with torch.cuda.device(self.mem.device):
            _check(lib().mixkvq_decode_attention_noalloc(self.handle, layer, _ptr(q), _ptr(out), float(scale), _stream()),
                   "mixkvq_decode_attention_noalloc")
        return out

    def select_channels(self, layer, want_salience=True):
        B, Hkv = self.cfg.batch, self.cfg.n_kv_heads
        tiers = torch.empty((B, Hkv, 128), dtype=torch.uint8, device=self.mem.device)
        sal = torch.empty((B, Hkv, 128), dtype=torch.float64, device=self.mem.device) if want_salience else None
        _check(lib().mixkvq_select_channels(self.handle, layer, _ptr(tiers), _ptr(sal), _stream()),
               "mixkvq_select_channels")
        return tiers, sal

    def written_externally(self):
        _check(lib().mixkvq_cache_written_externally(self.handle), "mixkvq_cache_written_externally")

    def test_arm_copy_timeout(self, extra_bytes: int, max_polls: int):
        _check(lib().mixkvq_test_arm_copy_timeout(self.handle, extra_bytes, max_polls), "mixkvq_test_arm_copy_timeout")

    def set_attention_kernel(self, kind: int):
        _check(lib().mixkvq_set_attention_kernel(self.handle, kind), "mixkvq_set_attention_kernel")

    def status(self) -> int:
        s = C.c_int()
        _check(lib().mixkvq_query_status(self.handle, C.byref(s), _stream()), "mixkvq_query_status")
        return s.value

    def describe(self, layer) -> LayoutDesc:
        d = LayoutDesc()
        _check(lib().mixkvq_cache_describe(self.handle, layer, C.byref(d)), "mixkvq_cache_describe")
        return d

    def launch_count(self) -> int:
        return int(lib().mixkvq_launch_count(self.handle))

    # -- raw regions of one stream, for inspection and byte-level comparison
    def stream_regions(self, layer, stream):
        d = self.describe(layer)
        m = self.mem

        def cut(off, stride, n):
            start = off + stride * stream
            return m[start:start + n].cpu().numpy().tobytes()

        R = self.cfg.residual_len
        nb, r, n_sink = self.sequence_fill(layer, stream // self.cfg.n_kv_heads)
        state = cut(d.state_off, d.state_stride, 1152)
        used16 = int.from_bytes(state[1028:1032], "little")
        resk = cut(d.resk_off, d.resk_stride, R * 256)
        resv = cut(d.resv_off, d.resv_stride, R * 256)
        return {
            "base": cut(d.base_off, d.base_stride, nb * d.base_bytes),
            "table": cut(d.table_off, d.table_stride, nb * 8),
            "extras": cut(d.extras_off, d.extras_stride, used16 * 16),
            "state": state,
            "resK": resk[: r * 256],
            "resV": resv[: r * 256],
            "sinkK": cut(d.sink_off, d.sink_stride, n_sink * 256),
            "sinkV": cut(d.sink_off + d.sink_len * 256, d.sink_stride, n_sink * 256),
        }
