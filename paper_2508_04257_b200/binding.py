"""ctypes binding of libkvsink.so: the same entry points as include/kvsink.h, argument marshalling only.

Tensors are torch CUDA tensors used for device memory and the current stream; every step of the path runs in
the library's kernels.  The library must be present: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# KVSINK_LIB selects another build of the library (the debug build with index checks, for instance)
_LIB_PATH = os.environ.get("KVSINK_LIB") or os.path.join(_HERE, "libkvsink.so")

EXPORTS = ("kvsink_cache_sizes", "kvsink_predict_sinks", "kvsink_quantize_append", "kvsink_decode_attention",
           "kvsink_decode_attention_static", "kvsink_prefill_attention", "kvsink_calibrate", "kvsink_quantize_append_calibrated",
           "kvsink_decode_attention_calibrated", "kvsink_quantize_append_pertoken", "kvsink_decode_attention_pertoken",
           "kvsink_channel_absmax", "kvsink_quant_error", "kvsink_read_status",
           "kvsink_launch_count", "kvsink_strerror")
STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


class KvsinkError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "hidden", "bits", "group",
                                         "max_seq", "topk", "pfn_n", "n_channels")] + [("channels", C.c_int32 * 8)]


class _Cache(C.Structure):
    _fields_ = [("k_codes", C.c_void_p), ("v_codes", C.c_void_p), ("k_scale", C.c_void_p), ("k_zero", C.c_void_p),
                ("v_scale", C.c_void_p), ("v_zero", C.c_void_p), ("k_tail", C.c_void_p), ("sink_k", C.c_void_p),
                ("sink_v", C.c_void_p), ("sink_bitmask", C.c_void_p), ("sink_pos", C.c_void_p),
                ("sink_count", C.c_void_p), ("status", C.c_void_p), ("seq_len", C.c_int32)]


class _Sizes(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("k_codes_bytes", "v_codes_bytes", "k_param_floats", "v_param_floats",
                                         "k_tail_halfs", "sink_halfs", "bitmask_words", "sink_pos_ints",
                                         "predict_workspace_bytes", "decode_workspace_bytes", "calibrate_workspace_bytes")] + \
               [(n, C.c_int32) for n in ("sink_capacity", "v_group", "v_groups_per_row", "tile_bytes")]


_lib = None


def lib():
    """Loads libkvsink.so; raises if it has not been built (python -m paper_2508_04257_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2508_04257_b200.build`")
        _lib = C.CDLL(_LIB_PATH)
        _lib.kvsink_strerror.restype = C.c_char_p
        _lib.kvsink_launch_count.restype = C.c_ulonglong
        for name in EXPORTS:
            getattr(_lib, name)
    return _lib


def strerror(code: int) -> str:
    return lib().kvsink_strerror(C.c_int(code)).decode()


@dataclass
class Config:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden: int
    bits: int
    group: int
    max_seq: int
    topk: int
    pfn_n: int
    channels: Sequence[int] = field(default_factory=tuple)

    def c(self) -> _Cfg:
        ch = (C.c_int32 * 8)(*list(self.channels)[:8])
        return _Cfg(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.hidden, self.bits, self.group,
                    self.max_seq, self.topk, self.pfn_n, len(self.channels), ch)


def cache_sizes(cfg: Config) -> dict:
    s = _Sizes()
    rc = lib().kvsink_cache_sizes(C.byref(cfg.c()), C.byref(s))
    if rc:
        raise KvsinkError(rc, "kvsink_cache_sizes")
    return {n: getattr(s, n) for n, _ in _Sizes._fields_}


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> C.c_void_p:
    return C.c_void_p(0 if t is None else t.data_ptr())


class SinkSet:
    """Device buffers of one prompt's sink set (bitmask, ascending positions, counts); shareable by all layers."""

    def __init__(self, cfg: Config, device="cuda"):
        sz = cache_sizes(cfg)
        self.bitmask = torch.zeros(max(sz["bitmask_words"], 1), dtype=torch.int32, device=device)
        self.pos = torch.full((max(sz["sink_pos_ints"], 1),), -1, dtype=torch.int32, device=device)
        self.count = torch.zeros(cfg.batch, dtype=torch.int32, device=device)


class KVCache:
    """Device buffers of one layer's cache, zero-filled, in the layout kvsink.h documents.  With per_token_keys the key
    parameters take the value parameters' shape (for quantize_append_pertoken / decode_attention_pertoken)."""

    def __init__(self, cfg: Config, sinks: Optional[SinkSet] = None, device="cuda", per_token_keys: bool = False):
        sz = cache_sizes(cfg)
        self.cfg, self.sizes = cfg, sz
        z = lambda n, dt: torch.zeros(max(int(n), 1), dtype=dt, device=device)
        self.k_codes, self.v_codes = z(sz["k_codes_bytes"], torch.uint8), z(sz["v_codes_bytes"], torch.uint8)
        self.per_token_keys = per_token_keys
        nkp = sz["v_param_floats"] if per_token_keys else sz["k_param_floats"]
        self.k_scale, self.k_zero = z(nkp, torch.float32), z(nkp, torch.float32)
        self.v_scale, self.v_zero = z(sz["v_param_floats"], torch.float32), z(sz["v_param_floats"], torch.float32)
        self.k_tail = z(sz["k_tail_halfs"], torch.float16)
        self.sink_k, self.sink_v = z(sz["sink_halfs"], torch.float16), z(sz["sink_halfs"], torch.float16)
        self.sinks = sinks if sinks is not None else SinkSet(cfg, device)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        self.seq_len = 0

    def c(self) -> _Cache:
        s = self.sinks
        return _Cache(_ptr(self.k_codes), _ptr(self.v_codes), _ptr(self.k_scale), _ptr(self.k_zero), _ptr(self.v_scale),
                      _ptr(self.v_zero), _ptr(self.k_tail), _ptr(self.sink_k), _ptr(self.sink_v), _ptr(s.bitmask), _ptr(s.pos),
                      _ptr(s.count), _ptr(self.status), self.seq_len)


def predict_sinks(cfg: Config, hidden: torch.Tensor, sinks: SinkSet, workspace: Optional[torch.Tensor] = None) -> SinkSet:
    """kvsink_predict_sinks: hidden fp16 [B, S, d] on the device (last axis contiguous)."""
    assert hidden.is_cuda and hidden.dtype == torch.float16 and hidden.dim() == 3 and hidden.stride(2) == 1
    if workspace is None:
        workspace = torch.empty(cache_sizes(cfg)["predict_workspace_bytes"], dtype=torch.uint8, device=hidden.device)
    rc = lib().kvsink_predict_sinks(C.byref(cfg.c()), _ptr(hidden), C.c_int32(hidden.shape[1]), C.c_int64(hidden.stride(0)),
                                    C.c_int64(hidden.stride(1)), _ptr(sinks.bitmask), _ptr(sinks.pos), _ptr(sinks.count),
                                    _ptr(workspace), C.c_size_t(workspace.numel()), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_predict_sinks")
    return sinks


def quantize_append(cfg: Config, cache: KVCache, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
    """kvsink_quantize_append: k_new, v_new fp16 [B, Hkv, T, D] on the device with equal strides."""
    assert k_new.is_cuda and k_new.dtype == torch.float16 and k_new.dim() == 4 and k_new.stride(3) == 1
    assert v_new.shape == k_new.shape and v_new.stride() == k_new.stride() and v_new.dtype == torch.float16
    cc = cache.c()
    rc = lib().kvsink_quantize_append(C.byref(cfg.c()), C.byref(cc), _ptr(k_new), _ptr(v_new), C.c_int32(k_new.shape[2]),
                                      C.c_int64(k_new.stride(0)), C.c_int64(k_new.stride(1)), C.c_int64(k_new.stride(2)), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_quantize_append")
    cache.seq_len = cc.seq_len


def decode_attention(cfg: Config, cache: KVCache, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                     lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, want_lse: bool = True):
    """kvsink_decode_attention: q fp16 [B, Hq, D] contiguous. Returns (out fp32 [B,Hq,D], lse fp32 [B,Hq] or None)."""
    assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
    if out is None:
        out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(cache.sizes["decode_workspace_bytes"], dtype=torch.uint8, device=q.device)
    cc = cache.c()
    rc = lib().kvsink_decode_attention(C.byref(cfg.c()), C.byref(cc), _ptr(q), _ptr(out), _ptr(lse), _ptr(workspace),
                                       C.c_size_t(workspace.numel()), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_decode_attention")
    return out, lse


def prefill_attention(cfg: Config, cache: KVCache, q: torch.Tensor, q_pos0: int, out: Optional[torch.Tensor] = None,
                      lse: Optional[torch.Tensor] = None, want_lse: bool = True):
    """kvsink_prefill_attention: q fp16 [B, Hq, T, D] on the device (last axis contiguous); query t sits at position q_pos0 + t.
    Returns (out fp32 [B,Hq,T,D], lse fp32 [B,Hq,T] or None)."""
    assert q.is_cuda and q.dtype == torch.float16 and q.dim() == 4 and q.stride(3) == 1
    T = q.shape[2]
    if out is None:
        out = torch.empty((cfg.batch, cfg.n_q_heads, T, cfg.head_dim), dtype=torch.float32, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((cfg.batch, cfg.n_q_heads, T), dtype=torch.float32, device=q.device)
    cc = cache.c()
    rc = lib().kvsink_prefill_attention(C.byref(cfg.c()), C.byref(cc), _ptr(q), C.c_int32(T), C.c_int32(q_pos0), C.c_int64(q.stride(0)),
                                        C.c_int64(q.stride(1)), C.c_int64(q.stride(2)), _ptr(out), _ptr(lse), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_prefill_attention")
    return out, lse


def decode_attention_static(cfg: Config, cache: KVCache, q: torch.Tensor, out: torch.Tensor, lse: Optional[torch.Tensor] = None):
    """kvsink_decode_attention_static: decode attention for callers that may not allocate device memory.

    Same result as decode_attention, but the split partials go to a 4 MiB array built into the library instead of
    a workspace tensor, and this wrapper allocates nothing either: `out` (fp32 [B,Hq,D]) and, if wanted, `lse`
    (fp32 [B,Hq]) must be passed in.  Raises KvsinkError(-9) when the configuration needs more scratch than the
    built-in array holds.  Calls that may overlap on the GPU must not share a device (they share the array).
    """
    assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
    cc = cache.c()
    rc = lib().kvsink_decode_attention_static(C.byref(cfg.c()), C.byref(cc), _ptr(q), _ptr(out), _ptr(lse), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_decode_attention_static")
    return out, lse


class _Static(C.Structure):
    _fields_ = [("k_scale", C.c_void_p), ("k_zero", C.c_void_p), ("v_scale", C.c_void_p), ("v_zero", C.c_void_p)]


class StaticParams:
    """Device buffers of calibrated parameters: keys float32 [Hkv, D], values float32 [Hkv, D / v_group]."""

    def __init__(self, cfg: Config, device="cuda"):
        ngv = cfg.head_dim // min(cfg.group, cfg.head_dim)
        z = lambda *shape: torch.zeros(shape, dtype=torch.float32, device=device)
        self.k_scale, self.k_zero = z(cfg.n_kv_heads, cfg.head_dim), z(cfg.n_kv_heads, cfg.head_dim)
        self.v_scale, self.v_zero = z(cfg.n_kv_heads, ngv), z(cfg.n_kv_heads, ngv)

    def c(self) -> _Static:
        return _Static(_ptr(self.k_scale), _ptr(self.k_zero), _ptr(self.v_scale), _ptr(self.v_zero))


def calibrate(cfg: Config, k_cal: torch.Tensor, v_cal: torch.Tensor, sinks: SinkSet, params: Optional[StaticParams] = None) -> StaticParams:
    """kvsink_calibrate: k_cal, v_cal fp16 [B, Hkv, T, D] on the device; sinks = the batch's sink set."""
    assert k_cal.is_cuda and k_cal.dtype == torch.float16 and k_cal.dim() == 4 and k_cal.stride(3) == 1
    assert v_cal.shape == k_cal.shape and v_cal.stride() == k_cal.stride() and v_cal.dtype == torch.float16
    if params is None:
        params = StaticParams(cfg, k_cal.device)
    ws = torch.empty(cache_sizes(cfg)["calibrate_workspace_bytes"], dtype=torch.uint8, device=k_cal.device)
    cs = params.c()
    rc = lib().kvsink_calibrate(C.byref(cfg.c()), _ptr(k_cal), _ptr(v_cal), C.c_int32(k_cal.shape[2]), C.c_int64(k_cal.stride(0)),
                                C.c_int64(k_cal.stride(1)), C.c_int64(k_cal.stride(2)), _ptr(sinks.bitmask), C.byref(cs), _ptr(ws),
                                C.c_size_t(ws.numel()), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_calibrate")
    return params


def quantize_append_calibrated(cfg: Config, cache: KVCache, params: StaticParams, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
    """kvsink_quantize_append_calibrated: k_new, v_new fp16 [B, Hkv, T, D] on the device with equal strides."""
    assert k_new.is_cuda and k_new.dtype == torch.float16 and k_new.dim() == 4 and k_new.stride(3) == 1
    assert v_new.shape == k_new.shape and v_new.stride() == k_new.stride() and v_new.dtype == torch.float16
    cc, cs = cache.c(), params.c()
    rc = lib().kvsink_quantize_append_calibrated(C.byref(cfg.c()), C.byref(cc), C.byref(cs), _ptr(k_new), _ptr(v_new), C.c_int32(k_new.shape[2]),
                                                 C.c_int64(k_new.stride(0)), C.c_int64(k_new.stride(1)), C.c_int64(k_new.stride(2)), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_quantize_append_calibrated")
    cache.seq_len = cc.seq_len


def decode_attention_calibrated(cfg: Config, cache: KVCache, params: StaticParams, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                                lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, want_lse: bool = True):
    """kvsink_decode_attention_calibrated: q fp16 [B, Hq, D] contiguous. Returns (out fp32 [B,Hq,D], lse fp32 [B,Hq] or None)."""
    assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
    if out is None:
        out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(cache.sizes["decode_workspace_bytes"], dtype=torch.uint8, device=q.device)
    cc, cs = cache.c(), params.c()
    rc = lib().kvsink_decode_attention_calibrated(C.byref(cfg.c()), C.byref(cc), C.byref(cs), _ptr(q), _ptr(out), _ptr(lse), _ptr(workspace),
                                                  C.c_size_t(workspace.numel()), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_decode_attention_calibrated")
    return out, lse


def quantize_append_pertoken(cfg: Config, cache: KVCache, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
    """kvsink_quantize_append_pertoken: k_new, v_new fp16 [B, Hkv, T, D] on the device with equal strides."""
    assert cache.per_token_keys, "the cache was not sized for per-token key parameters"
    assert k_new.is_cuda and k_new.dtype == torch.float16 and k_new.dim() == 4 and k_new.stride(3) == 1
    assert v_new.shape == k_new.shape and v_new.stride() == k_new.stride() and v_new.dtype == torch.float16
    cc = cache.c()
    rc = lib().kvsink_quantize_append_pertoken(C.byref(cfg.c()), C.byref(cc), _ptr(k_new), _ptr(v_new), C.c_int32(k_new.shape[2]),
                                               C.c_int64(k_new.stride(0)), C.c_int64(k_new.stride(1)), C.c_int64(k_new.stride(2)), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_quantize_append_pertoken")
    cache.seq_len = cc.seq_len


def decode_attention_pertoken(cfg: Config, cache: KVCache, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                              lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, want_lse: bool = True):
    """kvsink_decode_attention_pertoken: q fp16 [B, Hq, D] contiguous. Returns (out fp32 [B,Hq,D], lse fp32 [B,Hq] or None)."""
    assert cache.per_token_keys, "the cache was not sized for per-token key parameters"
    assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
    if out is None:
        out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(cache.sizes["decode_workspace_bytes"], dtype=torch.uint8, device=q.device)
    cc = cache.c()
    rc = lib().kvsink_decode_attention_pertoken(C.byref(cfg.c()), C.byref(cc), _ptr(q), _ptr(out), _ptr(lse), _ptr(workspace),
                                                C.c_size_t(workspace.numel()), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_decode_attention_pertoken")
    return out, lse


def channel_absmax(hidden: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kvsink_channel_absmax: hidden fp16 [B, S, d] on the device (last axis contiguous) -> float32 [d]."""
    assert hidden.is_cuda and hidden.dtype == torch.float16 and hidden.dim() == 3 and hidden.stride(2) == 1
    if out is None:
        out = torch.empty(hidden.shape[2], dtype=torch.float32, device=hidden.device)
    rc = lib().kvsink_channel_absmax(_ptr(hidden), C.c_int32(hidden.shape[0]), C.c_int32(hidden.shape[1]), C.c_int32(hidden.shape[2]),
                                     C.c_int64(hidden.stride(0)), C.c_int64(hidden.stride(1)), _ptr(out), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_channel_absmax")
    return out


def quant_error(cfg: Config, x: torch.Tensor, sinks: SinkSet, per_channel: bool, exclude_sinks: bool,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """kvsink_quant_error: x fp16 [B, Hkv, T, D] on the device -> float64 [4] (sum sq err, count) without / with sink tokens."""
    assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 4 and x.stride(3) == 1
    if out is None:
        out = torch.empty(4, dtype=torch.float64, device=x.device)
    rc = lib().kvsink_quant_error(C.byref(cfg.c()), _ptr(x), C.c_int32(x.shape[2]), C.c_int64(x.stride(0)), C.c_int64(x.stride(1)),
                                  C.c_int64(x.stride(2)), C.c_int32(int(per_channel)), C.c_int32(int(exclude_sinks)), _ptr(sinks.bitmask),
                                  _ptr(out), _stream())
    if rc:
        raise KvsinkError(rc, "kvsink_quant_error")
    return out


def launch_count() -> int:
    """kvsink_launch_count: kernel launches the library has made in this process."""
    return int(lib().kvsink_launch_count())


def read_status(cache: KVCache) -> int:
    host = C.c_int32(0)
    cc = cache.c()
    rc = lib().kvsink_read_status(C.byref(cc), C.byref(host), _stream())
    if rc and not host.value:       # a raised status bit comes back as the word itself
        raise KvsinkError(rc, "kvsink_read_status")
    return int(host.value)
