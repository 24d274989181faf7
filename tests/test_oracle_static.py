"""Pins for the oracle's static (calibrated) path: global min-max calibration without the sink tokens, quantization
with fixed parameters (clamping outside the calibrated range), and attention over such a cache.

Calibration is pinned to numpy's min / max plus the already pinned group routine; codes to exact rationals and to the
clamp; the paper's observation that calibrating with sink tokens widens every range (Section 4.1, static rows of
Table 1) by direction; attention to textbook softmax attention in numpy over tensors dequantised in numpy.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth

TINY = synth.WORKLOADS["tiny"]


def _setup(bits, seed=0, rep=2, seq=90):
    wl = TINY.scaled(bits=bits, batch=2, seq=seq, group=32, head_dim=64, n_q_heads=2 * rep, n_kv_heads=2, topk=4, pfn_n=1, seed=300 + bits + seed)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    H = synth.make_hidden(wl).numpy()
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    return wl, cfg, K, V, bm, pos, cnt


def _keep(wl, pos, cnt):
    keep = np.ones((wl.batch, wl.seq), bool)
    for b in range(wl.batch):
        keep[b, pos[b, :cnt[b]]] = False
    return keep


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_calibration_is_the_group_routine_on_numpys_extremes(bits):
    wl, cfg, K, V, bm, pos, cnt = _setup(bits)
    sp = oracle.calibrate(cfg, K, V, bm)
    keep = _keep(wl, pos, cnt)
    gv = min(wl.group, wl.head_dim)
    for h in range(wl.n_kv_heads):
        kh = K[:, h][keep]                       # [tokens kept, D]
        vh = V[:, h][keep]
        for ch in range(0, wl.head_dim, 7):
            col = kh[:, ch].astype(np.float32)
            s, z, _ = oracle.quantize_group(np.array([col.min(), col.max()], np.float32), np.ones(2, np.uint8), bits)
            assert sp.k_scale[h, ch] == s and sp.k_zero[h, ch] == z
        for j in range(wl.head_dim // gv):
            blk = vh[:, j * gv:(j + 1) * gv].astype(np.float32)
            s, z, _ = oracle.quantize_group(np.array([blk.min(), blk.max()], np.float32), np.ones(2, np.uint8), bits)
            assert sp.v_scale[h, j] == s and sp.v_zero[h, j] == z


def test_calibrating_with_the_sink_tokens_widens_the_ranges():
    # sink rows are small, the other rows carry per-channel offsets: without exclusion every channel's range must reach
    # down to the sinks' near-zero values (Section 4.1: the sinks' influence spreads to all groups under static quantization)
    wl = synth.WORKLOADS["llama3_8b_gqa"].scaled(batch=2, seq=512, n_q_heads=4, n_kv_heads=2, topk=5, group=64, bits=2, k_outlier_channels=0)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    K, V = (t.numpy() for t in synth.make_kv(wl))
    K = (K.astype(np.float32) * 0.1 + 6.0).astype(np.float16)          # every channel sits well away from zero ...
    for b, p in enumerate(synth.sink_positions(wl)):
        K[b, :, p, :] = (K[b, :, p, :].astype(np.float32) * 0.01).astype(np.float16)   # ... except at the sink tokens
    bm, pos, cnt = oracle.predict_sinks(cfg, synth.make_hidden(wl).numpy())
    without = oracle.calibrate(cfg, K, V, bm)
    with_sinks = oracle.calibrate(cfg, K, V, np.zeros_like(bm))
    assert np.all(with_sinks.k_scale >= without.k_scale) and np.all(with_sinks.k_scale > 3 * without.k_scale)
    # and the error of the non-sink tokens under the wider parameters is larger
    keep = _keep(wl, pos, cnt)
    errs = []
    for sp in (without, with_sinks):
        cache = oracle.Cache(cfg, bm, pos, cnt)
        oracle.quantize_append_calibrated(cfg, cache, sp, K, V)
        codes = oracle.unpack_codes(cfg, cache.k_codes, "k", wl.seq).astype(np.float32)
        deq = sp.k_scale[None, :, None, :] * (codes - sp.k_zero[None, :, None, :])
        errs.append((((K.astype(np.float32) - deq) ** 2)[np.broadcast_to(keep[:, None, :, None], K.shape)]).mean())
    assert errs[1] > 4 * errs[0]


def _round_half_even(fr: Fraction) -> int:
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem != Fraction(1, 2):
        return fl + (1 if rem > Fraction(1, 2) else 0)
    return fl if fl % 2 == 0 else fl + 1


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_static_codes_against_exact_rationals_clamp_sinks_and_chunking(bits):
    wl, cfg, K, V, bm, pos, cnt = _setup(bits, seed=5)
    sp = oracle.calibrate(cfg, K[:, :, :40], V[:, :, :40], bm)          # calibrated on a prefix: later tokens fall outside
    sp.k_scale[0, 3] = 0.0                                               # a channel that saw no data
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append_calibrated(cfg, cache, sp, K, V)
    kc = oracle.unpack_codes(cfg, cache.k_codes, "k", wl.seq)
    vc = oracle.unpack_codes(cfg, cache.v_codes, "v", wl.seq)
    qmax = (1 << bits) - 1
    keep = _keep(wl, pos, cnt)
    gv = min(wl.group, wl.head_dim)
    rng = np.random.default_rng(bits)
    checked = clamped = 0
    for _ in range(1500):
        b, h, t, ch = (int(rng.integers(n)) for n in (wl.batch, wl.n_kv_heads, wl.seq, wl.head_dim))
        for x, s, z, got in ((K[b, h, t, ch], sp.k_scale[h, ch], sp.k_zero[h, ch], kc[b, h, t, ch]),
                             (V[b, h, t, ch], sp.v_scale[h, ch // gv], sp.v_zero[h, ch // gv], vc[b, h, t, ch])):
            if not keep[b, t] or s == 0.0:
                assert got == 0
                continue
            quo = Fraction(float(x)) / Fraction(float(s))
            if abs((quo % 1) - Fraction(1, 2)) < Fraction(1, 1000) or abs(quo) > 2 ** 20:
                continue                                                   # within rounding distance of a tie
            want = _round_half_even(quo) + int(z)
            clamped += want < 0 or want > qmax
            assert got == min(max(want, 0), qmax)
            checked += 1
    assert checked > 1000 and clamped > 0
    assert np.all(kc[:, 0, :, 3] == 0)
    # sink rows are exact, in rank order
    for b in range(wl.batch):
        for j in range(cnt[b]):
            for h in range(wl.n_kv_heads):
                u = b * wl.n_kv_heads + h
                row = cache.sink_k.reshape(-1, wl.topk + wl.pfn_n, wl.head_dim)[u, j]
                assert np.array_equal(row, K[b, h, pos[b, j]].view(np.uint16))
    # appending in chunks gives the same bytes
    c2 = oracle.Cache(cfg, bm, pos, cnt)
    at = 0
    for n in (1, 30, 17, wl.seq - 48):
        oracle.quantize_append_calibrated(cfg, c2, sp, K[:, :, at:at + n], V[:, :, at:at + n])
        at += n
    assert c2.seq_len == cache.seq_len == wl.seq
    assert c2.k_codes.tobytes() == cache.k_codes.tobytes() and c2.v_codes.tobytes() == cache.v_codes.tobytes()
    assert c2.sink_v.tobytes() == cache.sink_v.tobytes()


@pytest.mark.parametrize("bits,rep", [(2, 1), (4, 2), (3, 4)])
def test_calibrated_attention_is_textbook_attention_on_the_dequantised_tensors(bits, rep):
    wl, cfg, K, V, bm, pos, cnt = _setup(bits, seed=9, rep=rep, seq=77)
    sp = oracle.calibrate(cfg, K, V, bm)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append_calibrated(cfg, cache, sp, K, V)
    q = synth.make_query(wl, synth.make_kv(wl)[0]).numpy()
    out, lse = oracle.decode_attention_calibrated(cfg, cache, sp, q)
    gv = min(wl.group, wl.head_dim)
    kc = oracle.unpack_codes(cfg, cache.k_codes, "k", wl.seq).astype(np.float32)
    vc = oracle.unpack_codes(cfg, cache.v_codes, "v", wl.seq).astype(np.float32)
    kd = (sp.k_scale[None, :, None, :] * (kc - sp.k_zero[None, :, None, :])).astype(np.float64)
    vs, vz = np.repeat(sp.v_scale, gv, axis=1), np.repeat(sp.v_zero, gv, axis=1)
    vd = (vs[None, :, None, :] * (vc - vz[None, :, None, :])).astype(np.float64)
    for b in range(wl.batch):                    # sink tokens: the exact rows
        for j in range(cnt[b]):
            kd[b, :, pos[b, j]] = K[b, :, pos[b, j]].astype(np.float64)
            vd[b, :, pos[b, j]] = V[b, :, pos[b, j]].astype(np.float64)
    for b in range(wl.batch):
        for hq in range(wl.n_q_heads):
            h = hq // rep
            s = kd[b, h] @ q[b, hq].astype(np.float64) / np.sqrt(wl.head_dim)
            w = np.exp(s - s.max())
            assert np.allclose(out[b, hq], (w[:, None] * vd[b, h]).sum(0) / w.sum(), rtol=1e-12, atol=1e-14)
            assert np.isclose(lse[b, hq], s.max() + np.log(w.sum()), rtol=1e-13)


def test_every_token_a_sink_is_exact_attention():
    wl = TINY.scaled(batch=1, seq=20, group=32, head_dim=64, n_q_heads=2, n_kv_heads=2, topk=0, pfn_n=20, seed=3)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                        wl.channels)
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, synth.make_hidden(wl).numpy())
    sp = oracle.calibrate(cfg, K, V, bm)
    assert not sp.k_scale.any() and not sp.v_scale.any()                # nothing left to calibrate on
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append_calibrated(cfg, cache, sp, K, V)
    q = synth.make_query(wl, synth.make_kv(wl)[0]).numpy()
    out, _ = oracle.decode_attention_calibrated(cfg, cache, sp, q)
    for hq in range(wl.n_q_heads):
        s = K[0, hq].astype(np.float64) @ q[0, hq].astype(np.float64) / np.sqrt(wl.head_dim)
        w = np.exp(s - s.max())
        assert np.allclose(out[0, hq], (w[:, None] * V[0, hq].astype(np.float64)).sum(0) / w.sum(), rtol=1e-12)
