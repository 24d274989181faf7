"""Pins for the oracle's decode attention (Eq. 3, Eq. 7): textbook fp64 softmax attention written with numpy
on materialised tensors, the all-sinks special case (exact fp16 attention on the original inputs), GQA head
mapping, and Eq. 7's split of one softmax into a sink part and a non-sink part."""
import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth


def _setup(bits=4, group=32, d=64, hq=4, hkv=2, batch=2, seq=117, topk=3, pfn=1, seed=21):
    wl = synth.WORKLOADS["tiny"].scaled(bits=bits, group=group, head_dim=d, n_q_heads=hq, n_kv_heads=hkv, batch=batch,
                                         seq=seq, topk=topk, pfn_n=pfn, seed=seed)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq,
                        wl.topk, wl.pfn_n, wl.channels)
    H = synth.make_hidden(wl)
    K, V = synth.make_kv(wl)
    q = synth.make_query(wl, K)
    return wl, cfg, H.numpy(), K.numpy(), V.numpy(), q.numpy()


def _textbook(q, Kd, Vd, rep):
    """softmax(q K^T / sqrt(D)) V in float64, query head hq reading KV head hq // rep."""
    B, Hq, D = q.shape
    out = np.zeros((B, Hq, D))
    lse = np.zeros((B, Hq))
    for b in range(B):
        for h in range(Hq):
            s = Kd[b, h // rep] @ q[b, h].astype(np.float64) / np.sqrt(D)
            m = s.max()
            w = np.exp(s - m)
            out[b, h] = (w[:, None] * Vd[b, h // rep]).sum(0) / w.sum()
            lse[b, h] = m + np.log(w.sum())
    return out, lse


@pytest.mark.parametrize("bits,group,d,hq,hkv", [(4, 32, 64, 4, 2), (2, 64, 128, 8, 2), (3, 64, 128, 3, 3)])
def test_matches_textbook_attention_on_the_dequantised_cache(bits, group, d, hq, hkv):
    wl, cfg, H, K, V, q = _setup(bits=bits, group=group, d=d, hq=hq, hkv=hkv)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    out, lse = oracle.decode_attention(cfg, cache, q)
    kd, vd = oracle.dequant_dense(cfg, cache)
    ref, ref_lse = _textbook(q, kd, vd, hq // hkv)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(lse, ref_lse, rtol=1e-12, atol=1e-12)


def test_every_token_a_sink_is_exact_fp16_attention():
    wl, cfg, H, K, V, q = _setup(seq=64, topk=64, pfn=0)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    assert np.all(cnt == 64)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    out, lse = oracle.decode_attention(cfg, cache, q)
    ref, ref_lse = _textbook(q, K.astype(np.float64), V.astype(np.float64), wl.n_q_heads // wl.n_kv_heads)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(lse, ref_lse, rtol=1e-12, atol=1e-12)


def test_quantisation_error_shrinks_with_bits_and_tail_is_exact():
    errs = []
    for bits in (2, 3, 4):
        wl, cfg, H, K, V, q = _setup(bits=bits, group=64, d=128, hq=2, hkv=2, seq=190)
        cache = oracle.Cache(cfg)                       # no sinks
        oracle.quantize_append(cfg, cache, K, V)
        out, _ = oracle.decode_attention(cfg, cache, q)
        ref, _ = _textbook(q, K.astype(np.float64), V.astype(np.float64), 1)
        errs.append(np.abs(out - ref).max())
        kd, _ = oracle.dequant_dense(cfg, cache)
        assert np.array_equal(kd[:, :, 128:], K[:, :, 128:].astype(np.float64))   # keys of the open group: fp16 tail
    assert errs[0] > errs[1] > errs[2]


def test_eq7_split_merges_to_the_single_softmax():
    wl, cfg, H, K, V, q = _setup(bits=4, seq=96, topk=5)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    out, lse = oracle.decode_attention(cfg, cache, q)
    kd, vd = oracle.dequant_dense(cfg, cache)
    rep = wl.n_q_heads // wl.n_kv_heads
    for b in range(wl.batch):
        sink = np.zeros(wl.seq, bool)
        sink[pos[b, :cnt[b]]] = True
        parts = []
        for sel in (sink, ~sink):
            o, l = _textbook(q[b:b + 1], kd[b:b + 1][:, :, sel], vd[b:b + 1][:, :, sel], rep)
            parts.append((o[0], l[0]))
        (o1, l1), (o2, l2) = parts
        m = np.maximum(l1, l2)
        w1, w2 = np.exp(l1 - m), np.exp(l2 - m)
        merged = (o1 * w1[:, None] + o2 * w2[:, None]) / (w1 + w2)[:, None]
        assert np.allclose(merged, out[b], rtol=1e-11, atol=1e-13)
        assert np.allclose(m + np.log(w1 + w2), lse[b], rtol=1e-12)


def test_append_then_attend_sees_the_new_token():
    wl, cfg, H, K, V, q = _setup(bits=2, group=32, d=64, seq=95)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    k1, v1 = [t.numpy() for t in synth.make_new_token(wl)]
    oracle.quantize_append(cfg, cache, k1, v1)          # completes the third group of 32
    assert cache.seq_len == 96
    kd, vd = oracle.dequant_dense(cfg, cache)
    assert kd.shape[2] == 96
    assert not np.array_equal(kd[:, :, 95], k1[:, :, 0].astype(np.float64))      # now quantized with its group
    assert np.abs(kd[:, :, 95] - k1[:, :, 0]).max() < 1.5
    out, _ = oracle.decode_attention(cfg, cache, q)
    ref, _ = _textbook(q, kd, vd, wl.n_q_heads // wl.n_kv_heads)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-13)
