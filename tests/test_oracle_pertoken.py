"""Pins for the oracle's per-token key path (Section 4.1 "Per-token quantization"): the key quantizer is the value
quantizer (pinned by its own tests) -- the same tensor passed as K and as V gives the same logical codes and the same
parameters; sink rows are exact; chunked = bulk; attention is textbook softmax attention in numpy over tensors
dequantised in numpy; a single sink-free token group reproduces the dynamic per-channel result only by accident, so the
two schemes are told apart on a tensor with a per-channel offset (the paper's reason for per-channel keys)."""
import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth

TINY = synth.WORKLOADS["tiny"]


def _setup(bits, rep=2, seq=75, group=32, d=64, seed=0):
    wl = TINY.scaled(bits=bits, batch=2, seq=seq, group=group, head_dim=d, n_q_heads=2 * rep, n_kv_heads=2, topk=4, pfn_n=1, seed=500 + bits + seed)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    H = synth.make_hidden(wl).numpy()
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    return wl, cfg, K, V, bm, pos, cnt


@pytest.mark.parametrize("bits,group,d", [(2, 32, 64), (3, 64, 128), (4, 128, 128), (4, 16, 64), (2, 256, 128)])
def test_keys_take_the_value_path(bits, group, d):
    wl, cfg, K, V, bm, pos, cnt = _setup(bits, group=group, d=d)
    cache = oracle.Cache(cfg, bm, pos, cnt, per_token_keys=True)
    oracle.quantize_append_pertoken(cfg, cache, K, K)                 # the same tensor as keys and as values
    kc = oracle.unpack_codes(cfg, cache.k_codes, "k", wl.seq)
    vc = oracle.unpack_codes(cfg, cache.v_codes, "v", wl.seq)
    assert np.array_equal(kc, vc)
    assert np.array_equal(cache.k_scale, cache.v_scale) and np.array_equal(cache.k_zero, cache.v_zero)
    # and that value path is the one the per-channel scheme uses for its values
    ref = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, ref, V, K)
    assert ref.v_codes.tobytes() == cache.v_codes.tobytes() and np.array_equal(ref.v_scale, cache.v_scale)
    assert np.array_equal(cache.sink_k, cache.sink_v) and np.array_equal(cache.sink_k, ref.sink_v)
    # chunks give the same bytes
    c2 = oracle.Cache(cfg, bm, pos, cnt, per_token_keys=True)
    at = 0
    for n in (1, 20, 17, wl.seq - 38):
        oracle.quantize_append_pertoken(cfg, c2, K[:, :, at:at + n], K[:, :, at:at + n])
        at += n
    assert c2.k_codes.tobytes() == cache.k_codes.tobytes() and np.array_equal(c2.k_scale, cache.k_scale)


@pytest.mark.parametrize("bits,rep", [(2, 1), (4, 2), (3, 4)])
def test_attention_is_textbook_attention_on_the_dequantised_tensors(bits, rep):
    wl, cfg, K, V, bm, pos, cnt = _setup(bits, rep=rep, seed=3)
    cache = oracle.Cache(cfg, bm, pos, cnt, per_token_keys=True)
    oracle.quantize_append_pertoken(cfg, cache, K, V)
    q = synth.make_query(wl, synth.make_kv(wl)[0]).numpy()
    out, lse = oracle.decode_attention_pertoken(cfg, cache, q)
    gv = min(wl.group, wl.head_dim)
    ngv = wl.head_dim // gv
    units = wl.batch * wl.n_kv_heads

    def dense(codes, scale, zero, orig):
        c = oracle.unpack_codes(cfg, codes, "k" if orig is K else "v", wl.seq).astype(np.float32)
        s = np.repeat(scale.reshape(units, -1, ngv)[:, :wl.seq], gv, axis=2).reshape(c.shape)
        z = np.repeat(zero.reshape(units, -1, ngv)[:, :wl.seq], gv, axis=2).reshape(c.shape)
        d = (s * (c - z)).astype(np.float64)
        for b in range(wl.batch):
            for j in range(cnt[b]):
                d[b, :, pos[b, j]] = orig[b, :, pos[b, j]].astype(np.float64)
        return d

    kd = dense(cache.k_codes, cache.k_scale, cache.k_zero, K)
    vd = dense(cache.v_codes, cache.v_scale, cache.v_zero, V)
    for b in range(wl.batch):
        for hq in range(wl.n_q_heads):
            h = hq // rep
            s = kd[b, h] @ q[b, hq].astype(np.float64) / np.sqrt(wl.head_dim)
            w = np.exp(s - s.max())
            assert np.allclose(out[b, hq], (w[:, None] * vd[b, h]).sum(0) / w.sum(), rtol=1e-12, atol=1e-14)
            assert np.isclose(lse[b, hq], s.max() + np.log(w.sum()), rtol=1e-13)


def test_per_channel_keys_beat_per_token_keys_on_channel_offsets():
    # Section 4.1: keys have outliers along channels, which per-channel groups absorb and per-token groups do not
    wl = synth.WORKLOADS["llama3_8b_gqa"].scaled(batch=1, seq=512, n_q_heads=4, n_kv_heads=2, topk=3, group=64, bits=4)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, synth.make_hidden(wl).numpy())
    per_channel = oracle.quant_error(cfg, K, bm, True, True)
    per_token = oracle.quant_error(cfg, K, bm, False, True)
    assert per_token[0] / per_token[1] > 3 * per_channel[0] / per_channel[1]
