"""Helpers for the GPU-vs-oracle parity tests: run both sides on the same seeded bits and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

ATOL, RTOL = 2e-3, 1e-2      # attention tolerance: |gpu - oracle| <= ATOL + RTOL * |oracle|


def configs(wl: synth.Workload, max_seq=None):
    ms = wl.max_seq if max_seq is None else max_seq
    args = (wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, ms, wl.topk, wl.pfn_n, wl.channels)
    return oracle.Config(*args), kv.Config(*args)


def np16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy()


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.shape == b.shape and a.tobytes() == b.tobytes()


def assert_close(gpu: np.ndarray, ref: np.ndarray, what: str, atol=ATOL, rtol=RTOL):
    err = np.abs(gpu.astype(np.float64) - ref)
    bound = atol + rtol * np.abs(ref)
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, worst err {err.max():.3e} (ref {ref.flat[np.argmax(err)]:.4e})"
    return float(err.max())


def compare_sinks(gs: kv.SinkSet, bm, pos, cnt, cap):
    B = cnt.shape[0]
    assert bits_equal(gs.bitmask.cpu().numpy().view(np.uint32)[:bm.size].reshape(bm.shape), bm), "sink bitmask"
    assert bits_equal(gs.count.cpu().numpy(), cnt), "sink count"
    if cap > 0:
        assert bits_equal(gs.pos.cpu().numpy()[:B * cap].reshape(B, cap), pos[:, :cap]), "sink positions"


def compare_cache(gc: kv.KVCache, oc: oracle.Cache, wl, what=""):
    """Bit-exact comparison of every cache array over the region the two sides define."""
    assert gc.seq_len == oc.seq_len
    n, G, D = oc.seq_len, wl.group, wl.head_dim
    units = wl.batch * wl.n_kv_heads
    for name in ("k_codes", "v_codes", "v_scale", "v_zero", "k_scale", "k_zero"):
        g = getattr(gc, name).cpu().numpy()
        o = getattr(oc, name)
        assert bits_equal(g[:o.size].view(o.dtype) if g.dtype != o.dtype else g[:o.size], o), f"{what}{name} differs"
    if oc.sizes["sink_halfs"] > 0:
        for name in ("sink_k", "sink_v"):
            g = getattr(gc, name).cpu().numpy().view(np.uint16)
            o = getattr(oc, name)
            assert bits_equal(g[:o.size], o), f"{what}{name} differs"
    r = n % G
    if r:
        gt = gc.k_tail.cpu().numpy().view(np.uint16).reshape(units, G, D)[:, :r]
        ot = oc.k_tail.reshape(units, G, D)[:, :r]
        assert bits_equal(gt, ot), f"{what}k_tail differs"


CANARY, PAD = 0xA5, 256


def guard(obj, names, device="cuda"):
    """Moves the named tensors of a cache / sink set into buffers with PAD canary bytes before and after them."""
    obj._guards = []
    for name in names:
        t = getattr(obj, name)
        nbytes = t.numel() * t.element_size()
        buf = torch.full((nbytes + 2 * PAD,), CANARY, dtype=torch.uint8, device=device)
        mid = buf[PAD:PAD + nbytes].view(t.dtype)
        mid.copy_(t.reshape(-1))
        setattr(obj, name, mid.view(t.shape))
        obj._guards.append((name, buf, nbytes))
    return obj


def check_guards(obj):
    """No kernel wrote past the ends of a guarded buffer."""
    for name, buf, nbytes in obj._guards:
        host = buf.cpu().numpy()
        assert (host[:PAD] == CANARY).all() and (host[PAD + nbytes:] == CANARY).all(), f"write outside {name}"


CACHE_BUFFERS = ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero", "k_tail", "sink_k", "sink_v", "status")
SINK_BUFFERS = ("bitmask", "pos", "count")


def run_both(wl: synth.Workload, appends: int = 0, device="cuda", check=True, H=None, K=None, V=None, max_seq=None):
    """Full path on both sides: predict -> prefill quantize -> `appends` single-token appends -> decode attention."""
    ocfg, gcfg = configs(wl, max_seq)
    H = synth.make_hidden(wl, device) if H is None else H
    if K is None:
        K, V = synth.make_kv(wl, 0, device)
    # GPU
    gs = guard(kv.SinkSet(gcfg, device), SINK_BUFFERS, device)
    kv.predict_sinks(gcfg, H, gs)
    gc = guard(kv.KVCache(gcfg, gs, device), CACHE_BUFFERS, device)
    kv.quantize_append(gcfg, gc, K, V)
    # oracle
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    oc = oracle.Cache(ocfg, bm, pos, cnt)
    oracle.quantize_append(ocfg, oc, np16(K), np16(V))
    cap = wl.topk + wl.pfn_n
    if check:
        compare_sinks(gs, bm, pos, cnt, cap)
        compare_cache(gc, oc, wl, "prefill: ")
    for step in range(appends):
        k1, v1 = synth.make_new_token(wl, 0, step, device)
        kv.quantize_append(gcfg, gc, k1, v1)
        oracle.quantize_append(ocfg, oc, np16(k1), np16(v1))
        if check:
            compare_cache(gc, oc, wl, f"append {step}: ")
    q = synth.make_query(wl, K)
    out, lse = kv.decode_attention(gcfg, gc, q)
    ref, ref_lse = oracle.decode_attention(ocfg, oc, np16(q))
    torch.cuda.synchronize()
    assert kv.read_status(gc) == 0
    check_guards(gs)
    check_guards(gc)
    err = None
    if check:
        err = assert_close(out.cpu().numpy(), ref, "attention output")
        if oc.seq_len > 0:
            assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-3 + 1e-3 * np.abs(ref_lse).max(), "lse"
    return dict(gpu_cache=gc, oracle_cache=oc, out=out, ref=ref, lse=lse, ref_lse=ref_lse, err=err, q=q, K=K, V=V, H=H)
