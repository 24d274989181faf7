"""Pins for the oracle's prompt attention over the quantized cache (Algorithm 1's attention statement): a single query
at the last position is decode attention (pinned by its own tests); every query is textbook causal softmax attention in
numpy over the dense tensors attention reads; a prompt of sink tokens only is exact fp16 causal attention."""
import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth

TINY = synth.WORKLOADS["tiny"]


def _setup(bits, rep, seq, group=32, topk=3, pfn=1, seed=0):
    wl = TINY.scaled(bits=bits, batch=2, seq=seq, group=group, head_dim=64, n_q_heads=2 * rep, n_kv_heads=2, topk=topk, pfn_n=pfn, seed=400 + seed)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    H = synth.make_hidden(wl).numpy()
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    rng = np.random.default_rng(seed)
    return wl, cfg, cache, K, V, rng


def test_one_query_at_the_end_is_decode_attention():
    wl, cfg, cache, K, V, rng = _setup(4, 2, 75)
    q = rng.standard_normal((wl.batch, wl.n_q_heads, 1, wl.head_dim)).astype(np.float16)
    out, lse = oracle.prefill_attention(cfg, cache, q, wl.seq - 1)
    ref, ref_lse = oracle.decode_attention(cfg, cache, q[:, :, 0])
    assert np.allclose(out[:, :, 0], ref, rtol=1e-13, atol=0) and np.allclose(lse[:, :, 0], ref_lse, rtol=1e-13)


@pytest.mark.parametrize("bits,rep,seq,T,pos0", [(2, 1, 70, 70, 0), (3, 4, 70, 20, 50), (4, 2, 33, 5, 10)])
def test_textbook_causal_attention_on_the_dequantised_tensors(bits, rep, seq, T, pos0):
    wl, cfg, cache, K, V, rng = _setup(bits, rep, seq, seed=bits)
    q = rng.standard_normal((wl.batch, wl.n_q_heads, T, wl.head_dim)).astype(np.float16)
    out, lse = oracle.prefill_attention(cfg, cache, q, pos0)
    kd, vd = oracle.dequant_dense(cfg, cache)
    for b in range(wl.batch):
        for hq in range(wl.n_q_heads):
            h = hq // rep
            s = q[b, hq].astype(np.float64) @ kd[b, h].T / np.sqrt(wl.head_dim)           # [T, seq]
            visible = np.arange(seq)[None, :] <= (pos0 + np.arange(T))[:, None]
            s = np.where(visible, s, -np.inf)
            w = np.exp(s - s.max(axis=1, keepdims=True))
            assert np.allclose(out[b, hq], (w @ vd[b, h]) / w.sum(axis=1, keepdims=True), rtol=1e-12, atol=1e-14)
            assert np.allclose(lse[b, hq], s.max(axis=1) + np.log(w.sum(axis=1)), rtol=1e-13)
    # strided queries ([B, T, Hq, D] storage) give the same
    qt = np.ascontiguousarray(q.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    out2, _ = oracle.prefill_attention(cfg, cache, qt, pos0)
    assert np.array_equal(out, out2)


def test_a_prompt_of_sink_tokens_is_exact_causal_attention():
    wl, cfg, cache, K, V, rng = _setup(2, 1, 24, topk=0, pfn=24, seed=9)
    q = rng.standard_normal((wl.batch, wl.n_q_heads, wl.seq, wl.head_dim)).astype(np.float16)
    out, _ = oracle.prefill_attention(cfg, cache, q, 0)
    for hq in range(wl.n_q_heads):
        s = q[0, hq].astype(np.float64) @ K[0, hq].astype(np.float64).T / np.sqrt(wl.head_dim)
        s = np.where(np.tril(np.ones((wl.seq, wl.seq), bool)), s, -np.inf)
        w = np.exp(s - s.max(axis=1, keepdims=True))
        assert np.allclose(out[0, hq], (w @ V[0, hq].astype(np.float64)) / w.sum(axis=1, keepdims=True), rtol=1e-12)


def test_queries_beyond_the_cache_are_refused():
    wl, cfg, cache, K, V, rng = _setup(2, 1, 20)
    q = np.zeros((wl.batch, wl.n_q_heads, 4, wl.head_dim), np.float16)
    with pytest.raises(RuntimeError):
        oracle.prefill_attention(cfg, cache, q, 18)
