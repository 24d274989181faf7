"""KVSink CPU oracle -- test infrastructure only.

A thin ctypes/numpy front end over ``kvsink_oracle.c`` (plain C, binary32 quantization per Eq. 8-11 of
arXiv 2508.04257, binary64 attention per Eq. 3 / Eq. 7, sink prediction per Algorithm 1 and Section 4.3).
Nothing here is imported by the CUDA library or its Python binding; only the tests, the smoke check and
the CPU-baseline leg of the benchmark may use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvsink_oracle.c")
_LIB = os.path.join(_HERE, "libkvsink_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (IEEE binary32, no FMA contraction, OpenMP over independent units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "hidden", "bits", "group",
                                         "max_seq", "topk", "pfn_n", "n_channels")] + [("channels", C.c_int32 * 8)]


class _Cache(C.Structure):
    _fields_ = [("k_codes", C.c_void_p), ("v_codes", C.c_void_p), ("k_scale", C.c_void_p), ("k_zero", C.c_void_p),
                ("v_scale", C.c_void_p), ("v_zero", C.c_void_p), ("k_tail", C.c_void_p), ("sink_k", C.c_void_p),
                ("sink_v", C.c_void_p), ("sink_bitmask", C.c_void_p), ("sink_pos", C.c_void_p),
                ("sink_count", C.c_void_p), ("seq_len", C.c_int32)]


class _Sizes(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("k_codes_bytes", "v_codes_bytes", "k_param_floats", "v_param_floats",
                                         "k_tail_halfs", "sink_halfs", "bitmask_words", "sink_pos_ints")] + \
               [(n, C.c_int32) for n in ("sink_capacity", "v_group", "v_groups_per_row", "tile_bytes")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.kvo_num_threads.restype = C.c_int
    return _lib


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


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with status {rc}")


def cache_sizes(cfg: Config) -> dict:
    s = _Sizes()
    _check(lib().kvo_cache_sizes(C.byref(cfg.c()), C.byref(s)), "cache_sizes")
    return {n: getattr(s, n) for n, _ in _Sizes._fields_}


def num_threads() -> int:
    return int(lib().kvo_num_threads())


def set_num_threads(n: int) -> None:
    lib().kvo_set_num_threads(C.c_int(n))


class Cache:
    """Host-side cache buffers (numpy, zero-initialised) in the library's layout."""

    def __init__(self, cfg: Config, bitmask: Optional[np.ndarray] = None, sink_pos: Optional[np.ndarray] = None,
                 sink_count: Optional[np.ndarray] = None, per_token_keys: bool = False):
        sz = cache_sizes(cfg)
        self.cfg, self.sizes = cfg, sz
        self.k_codes = np.zeros(sz["k_codes_bytes"], np.uint8)
        self.v_codes = np.zeros(sz["v_codes_bytes"], np.uint8)
        # per-token keys: the key parameters have the value parameters' shape [units][max_seq][D / v_group]
        self.k_scale = np.zeros(sz["v_param_floats" if per_token_keys else "k_param_floats"], np.float32)
        self.k_zero = np.zeros(sz["v_param_floats" if per_token_keys else "k_param_floats"], np.float32)
        self.v_scale = np.zeros(sz["v_param_floats"], np.float32)
        self.v_zero = np.zeros(sz["v_param_floats"], np.float32)
        self.k_tail = np.zeros(sz["k_tail_halfs"], np.uint16)
        self.sink_k = np.zeros(max(sz["sink_halfs"], 1), np.uint16)
        self.sink_v = np.zeros(max(sz["sink_halfs"], 1), np.uint16)
        words = (cfg.max_seq + 31) // 32
        self.sink_bitmask = np.zeros((cfg.batch, words), np.uint32) if bitmask is None else np.ascontiguousarray(bitmask, np.uint32)
        cap = max(sz["sink_capacity"], 1)
        self.sink_pos = np.full((cfg.batch, cap), -1, np.int32) if sink_pos is None else np.ascontiguousarray(sink_pos, np.int32)
        self.sink_count = np.zeros(cfg.batch, np.int32) if sink_count is None else np.ascontiguousarray(sink_count, np.int32)
        self.seq_len = 0

    def c(self) -> _Cache:
        p = lambda a: a.ctypes.data_as(C.c_void_p)
        return _Cache(p(self.k_codes), p(self.v_codes), p(self.k_scale), p(self.k_zero), p(self.v_scale), p(self.v_zero),
                      p(self.k_tail), p(self.sink_k), p(self.sink_v), p(self.sink_bitmask), p(self.sink_pos),
                      p(self.sink_count), self.seq_len)


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    assert a.dtype == np.uint16
    return a


def predict_sinks(cfg: Config, hidden: np.ndarray):
    """hidden: float16 [B, S, d] (last axis contiguous). Returns (bitmask [B, W] uint32, pos [B, cap] int32, count [B])."""
    h = _u16(hidden)
    assert h.ndim == 3 and h.strides[2] == 2
    B, S, _ = h.shape
    words = (cfg.max_seq + 31) // 32
    cap = max(cfg.topk + cfg.pfn_n, 1)
    bm = np.zeros((B, words), np.uint32)
    pos = np.full((B, cap), -1, np.int32)
    cnt = np.zeros(B, np.int32)
    rc = lib().kvo_predict_sinks(C.byref(cfg.c()), h.ctypes.data_as(C.c_void_p), C.c_int32(S), C.c_int64(h.strides[0] // 2),
                                 C.c_int64(h.strides[1] // 2), bm.ctypes.data_as(C.c_void_p), pos.ctypes.data_as(C.c_void_p),
                                 cnt.ctypes.data_as(C.c_void_p))
    _check(rc, "predict_sinks")
    return bm, pos, cnt


def quantize_append(cfg: Config, cache: Cache, k_new: np.ndarray, v_new: np.ndarray) -> None:
    """k_new, v_new: float16 [B, Hkv, T, D] (last axis contiguous, equal strides)."""
    k, v = _u16(k_new), _u16(v_new)
    assert k.shape == v.shape and k.strides == v.strides and k.strides[3] == 2
    T = k.shape[2]
    cc = cache.c()
    rc = lib().kvo_quantize_append(C.byref(cfg.c()), C.byref(cc), k.ctypes.data_as(C.c_void_p), v.ctypes.data_as(C.c_void_p),
                                   C.c_int32(T), C.c_int64(k.strides[0] // 2), C.c_int64(k.strides[1] // 2),
                                   C.c_int64(k.strides[2] // 2))
    _check(rc, "quantize_append")
    cache.seq_len = cc.seq_len


def decode_attention(cfg: Config, cache: Cache, q: np.ndarray):
    """q: float16 [B, Hq, D]. Returns (out float64 [B,Hq,D], lse float64 [B,Hq])."""
    qq = np.ascontiguousarray(_u16(q))
    out = np.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), np.float64)
    lse = np.zeros((cfg.batch, cfg.n_q_heads), np.float64)
    cc = cache.c()
    rc = lib().kvo_decode_attention(C.byref(cfg.c()), C.byref(cc), qq.ctypes.data_as(C.c_void_p),
                                    out.ctypes.data_as(C.c_void_p), lse.ctypes.data_as(C.c_void_p))
    _check(rc, "decode_attention")
    return out, lse


def dequant_dense(cfg: Config, cache: Cache):
    """Dense K', V' float64 [B,Hkv,seq_len,D] exactly as attention consumes them (sink rows exact)."""
    n = cache.seq_len
    kd = np.zeros((cfg.batch, cfg.n_kv_heads, n, cfg.head_dim), np.float64)
    vd = np.zeros_like(kd)
    cc = cache.c()
    _check(lib().kvo_dequant_dense(C.byref(cfg.c()), C.byref(cc), kd.ctypes.data_as(C.c_void_p),
                                   vd.ctypes.data_as(C.c_void_p)), "dequant_dense")
    return kd, vd


def unpack_codes(cfg: Config, codes: np.ndarray, kind: str, seq: int) -> np.ndarray:
    """Logical codes int8 [B,Hkv,seq,D] from a packed array; kind is 'k' or 'v'."""
    codes = np.ascontiguousarray(codes, np.uint8)
    out = np.zeros((cfg.batch, cfg.n_kv_heads, seq, cfg.head_dim), np.int8)
    _check(lib().kvo_unpack_codes(C.byref(cfg.c()), codes.ctypes.data_as(C.c_void_p), C.c_int(0 if kind == "k" else 1),
                                  C.c_int(seq), out.ctypes.data_as(C.c_void_p)), "unpack_codes")
    return out


def quantize_group(x: np.ndarray, member: np.ndarray, bits: int):
    """Eq. 8-11 on one group. Returns (scale float32, zero float32, codes int32[n])."""
    x = np.ascontiguousarray(x, np.float32)
    m = np.ascontiguousarray(member, np.uint8)
    codes = np.zeros(x.shape[0], np.int32)
    sc, ze = C.c_float(0), C.c_float(0)
    lib().kvo_quantize_group(x.ctypes.data_as(C.c_void_p), m.ctypes.data_as(C.c_void_p), C.c_int(x.shape[0]),
                             C.c_int(bits), C.byref(sc), C.byref(ze), codes.ctypes.data_as(C.c_void_p))
    return np.float32(sc.value), np.float32(ze.value), codes


# ---- analysis routines (Section 3.1 / Appendix D; Section 4.1, Table 1) ----
def channel_absmax(hidden: np.ndarray) -> np.ndarray:
    """hidden: float16 [B, S, d] (last axis contiguous). Returns float32 [d]: the largest |H| of every channel."""
    h = _u16(hidden)
    assert h.ndim == 3 and h.strides[2] == 2
    B, S, d = h.shape
    out = np.zeros(d, np.float32)
    _check(lib().kvo_channel_absmax(h.ctypes.data_as(C.c_void_p), C.c_int32(B), C.c_int32(S), C.c_int32(d), C.c_int64(h.strides[0] // 2),
                                    C.c_int64(h.strides[1] // 2), out.ctypes.data_as(C.c_void_p)), "channel_absmax")
    return out


def quant_error(cfg: Config, x: np.ndarray, bitmask: np.ndarray, per_channel: bool, exclude_sinks: bool) -> np.ndarray:
    """x: float16 [B, Hkv, T, D]. Returns float64 [4]: (sum sq err, elements) over groups without / with a sink token."""
    a = _u16(x)
    assert a.ndim == 4 and a.strides[3] == 2
    bm = np.ascontiguousarray(bitmask, np.uint32)
    out = np.zeros(4, np.float64)
    _check(lib().kvo_quant_error(C.byref(cfg.c()), a.ctypes.data_as(C.c_void_p), C.c_int32(a.shape[2]), C.c_int64(a.strides[0] // 2),
                                 C.c_int64(a.strides[1] // 2), C.c_int64(a.strides[2] // 2), C.c_int(int(per_channel)),
                                 C.c_int(int(exclude_sinks)), bm.ctypes.data_as(C.c_void_p), out.ctypes.data_as(C.c_void_p)), "quant_error")
    return out


# ---- static (calibrated) parameters (Section 5.1 scheme; Appendix C; Algorithm 1's remark on calibration) ----
class _Static(C.Structure):
    _fields_ = [("k_scale", C.c_void_p), ("k_zero", C.c_void_p), ("v_scale", C.c_void_p), ("v_zero", C.c_void_p)]


class StaticParams:
    """Calibrated (scale, zero): keys float32 [Hkv, D] per channel, values float32 [Hkv, D / v_group] per channel group."""

    def __init__(self, cfg: Config):
        ngv = cfg.head_dim // min(cfg.group, cfg.head_dim)
        self.k_scale = np.zeros((cfg.n_kv_heads, cfg.head_dim), np.float32)
        self.k_zero = np.zeros_like(self.k_scale)
        self.v_scale = np.zeros((cfg.n_kv_heads, ngv), np.float32)
        self.v_zero = np.zeros_like(self.v_scale)

    def c(self) -> _Static:
        p = lambda a: a.ctypes.data_as(C.c_void_p)
        return _Static(p(self.k_scale), p(self.k_zero), p(self.v_scale), p(self.v_zero))


def calibrate(cfg: Config, k_cal: np.ndarray, v_cal: np.ndarray, bitmask: np.ndarray) -> StaticParams:
    """Global min-max calibration over k_cal, v_cal float16 [B, Hkv, T, D] with the masked (sink) tokens left out."""
    k, v = _u16(k_cal), _u16(v_cal)
    assert k.shape == v.shape and k.strides == v.strides and k.strides[3] == 2
    bm = np.ascontiguousarray(bitmask, np.uint32)
    sp = StaticParams(cfg)
    cs = sp.c()
    _check(lib().kvo_calibrate(C.byref(cfg.c()), k.ctypes.data_as(C.c_void_p), v.ctypes.data_as(C.c_void_p), C.c_int32(k.shape[2]),
                               C.c_int64(k.strides[0] // 2), C.c_int64(k.strides[1] // 2), C.c_int64(k.strides[2] // 2),
                               bm.ctypes.data_as(C.c_void_p), C.byref(cs)), "calibrate")
    return sp


def quantize_append_calibrated(cfg: Config, cache: Cache, sp: StaticParams, k_new: np.ndarray, v_new: np.ndarray) -> None:
    k, v = _u16(k_new), _u16(v_new)
    assert k.shape == v.shape and k.strides == v.strides and k.strides[3] == 2
    cc, cs = cache.c(), sp.c()
    rc = lib().kvo_quantize_append_calibrated(C.byref(cfg.c()), C.byref(cc), C.byref(cs), k.ctypes.data_as(C.c_void_p),
                                              v.ctypes.data_as(C.c_void_p), C.c_int32(k.shape[2]), C.c_int64(k.strides[0] // 2),
                                              C.c_int64(k.strides[1] // 2), C.c_int64(k.strides[2] // 2))
    _check(rc, "quantize_append_calibrated")
    cache.seq_len = cc.seq_len


def decode_attention_calibrated(cfg: Config, cache: Cache, sp: StaticParams, q: np.ndarray):
    qq = np.ascontiguousarray(_u16(q))
    out = np.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), np.float64)
    lse = np.zeros((cfg.batch, cfg.n_q_heads), np.float64)
    cc, cs = cache.c(), sp.c()
    _check(lib().kvo_decode_attention_calibrated(C.byref(cfg.c()), C.byref(cc), C.byref(cs), qq.ctypes.data_as(C.c_void_p),
                                                 out.ctypes.data_as(C.c_void_p), lse.ctypes.data_as(C.c_void_p)), "decode_attention_calibrated")
    return out, lse


def prefill_attention(cfg: Config, cache: Cache, q: np.ndarray, q_pos0: int):
    """q: float16 [B, Hq, T, D]; query t sits at position q_pos0 + t. Returns (out float64 [B,Hq,T,D], lse [B,Hq,T])."""
    qq = _u16(q)
    assert qq.ndim == 4 and qq.strides[3] == 2
    T = qq.shape[2]
    out = np.zeros((cfg.batch, cfg.n_q_heads, T, cfg.head_dim), np.float64)
    lse = np.zeros((cfg.batch, cfg.n_q_heads, T), np.float64)
    cc = cache.c()
    _check(lib().kvo_prefill_attention(C.byref(cfg.c()), C.byref(cc), qq.ctypes.data_as(C.c_void_p), C.c_int32(T), C.c_int32(q_pos0),
                                       C.c_int64(qq.strides[0] // 2), C.c_int64(qq.strides[1] // 2), C.c_int64(qq.strides[2] // 2),
                                       out.ctypes.data_as(C.c_void_p), lse.ctypes.data_as(C.c_void_p)), "prefill_attention")
    return out, lse


# ---- per-token keys (Section 4.1 "Per-token quantization"; Section 5.1's per-token Key and Value dynamic scheme) ----
def quantize_append_pertoken(cfg: Config, cache: Cache, k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Keys and values per token, dynamic; `cache` must have been made with per_token_keys=True."""
    k, v = _u16(k_new), _u16(v_new)
    assert k.shape == v.shape and k.strides == v.strides and k.strides[3] == 2
    assert cache.k_scale.size == cache.sizes["v_param_floats"]
    cc = cache.c()
    rc = lib().kvo_quantize_append_pertoken(C.byref(cfg.c()), C.byref(cc), k.ctypes.data_as(C.c_void_p), v.ctypes.data_as(C.c_void_p),
                                            C.c_int32(k.shape[2]), C.c_int64(k.strides[0] // 2), C.c_int64(k.strides[1] // 2),
                                            C.c_int64(k.strides[2] // 2))
    _check(rc, "quantize_append_pertoken")
    cache.seq_len = cc.seq_len


def decode_attention_pertoken(cfg: Config, cache: Cache, q: np.ndarray):
    qq = np.ascontiguousarray(_u16(q))
    out = np.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), np.float64)
    lse = np.zeros((cfg.batch, cfg.n_q_heads), np.float64)
    cc = cache.c()
    _check(lib().kvo_decode_attention_pertoken(C.byref(cfg.c()), C.byref(cc), qq.ctypes.data_as(C.c_void_p),
                                               out.ctypes.data_as(C.c_void_p), lse.ctypes.data_as(C.c_void_p)), "decode_attention_pertoken")
    return out, lse
