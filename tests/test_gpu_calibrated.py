"""GPU parity of the static (calibrated) path against the CPU oracle: calibrated parameters, packed codes and side buffer
bit for bit; attention within |gpu - oracle| <= 2e-3 + 1e-2 |oracle|."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, bits_equal, configs, np16

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


def _both(wl, chunks=None, cal_tokens=None):
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    nc = wl.seq if cal_tokens is None else cal_tokens
    gp = kv.calibrate(gcfg, K[:, :, :nc], V[:, :, :nc], gs)
    op = oracle.calibrate(ocfg, np16(K[:, :, :nc]), np16(V[:, :, :nc]), bm)
    for name in ("k_scale", "k_zero", "v_scale", "v_zero"):
        assert bits_equal(getattr(gp, name).cpu().numpy(), getattr(op, name)), name
    gc, oc = kv.KVCache(gcfg, gs), oracle.Cache(ocfg, bm, pos, cnt)
    at = 0
    for n in (chunks or (wl.seq,)):
        kv.quantize_append_calibrated(gcfg, gc, gp, K[:, :, at:at + n], V[:, :, at:at + n])
        oracle.quantize_append_calibrated(ocfg, oc, op, np16(K[:, :, at:at + n]), np16(V[:, :, at:at + n]))
        at += n
        assert gc.seq_len == oc.seq_len
        # the region both sides define: the tiles that hold tokens
        nb = (at + 15) // 16 * 16 * wl.head_dim * wl.bits // 8
        per = wl.max_seq * wl.head_dim * wl.bits // 8
        for name in ("k_codes", "v_codes"):
            g = getattr(gc, name).cpu().numpy().reshape(-1, per)[:, :nb]
            o = getattr(oc, name).reshape(-1, per)[:, :nb]
            assert bits_equal(g, o), f"{name} after {at} tokens"
    if oc.sizes["sink_halfs"] > 0:
        for name in ("sink_k", "sink_v"):
            assert bits_equal(getattr(gc, name).cpu().numpy().view(np.uint16)[:getattr(oc, name).size], getattr(oc, name)), name
    q = synth.make_query(wl, K)
    out, lse = kv.decode_attention_calibrated(gcfg, gc, gp, q)
    ref, ref_lse = oracle.decode_attention_calibrated(ocfg, oc, op, np16(q))
    torch.cuda.synchronize()
    assert kv.read_status(gc) == 0
    err = assert_close(out.cpu().numpy(), ref, "attention output")
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-3 + 1e-3 * np.abs(ref_lse).max()
    return err


@pytest.mark.parametrize("bits,group", [(2, 128), (2, 64), (3, 64), (4, 64), (4, 128), (3, 128)])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (6, 2), (16, 2)])
def test_grid_of_shapes(bits, group, hq, hkv):
    seq = 3 * group + 37
    wl = TINY.scaled(bits=bits, head_dim=128, group=group, n_q_heads=hq, n_kv_heads=hkv, batch=2, seq=seq, topk=5, pfn_n=2,
                     seed=9000 + bits * 100 + group + hq)
    _both(wl)


@pytest.mark.parametrize("seq", [1, 15, 16, 17, 63, 64, 65, 200])
def test_short_and_ragged_lengths(seq):
    wl = TINY.scaled(seq=seq, topk=min(2, seq), batch=2, group=64, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=2, seed=177 + seq)
    _both(wl)


def test_chunked_appends_and_values_outside_the_calibrated_range():
    # calibrated on the first 50 tokens only: later tokens clamp; chunks start and end inside tiles
    wl = TINY.scaled(seq=333, group=64, bits=3, head_dim=128, n_q_heads=4, n_kv_heads=2, batch=2, topk=6, pfn_n=1, seed=55)
    _both(wl, chunks=(1, 14, 1, 33, 100, 1, 183), cal_tokens=50)


@pytest.mark.parametrize("bits,group", [(2, 64), (2, 128), (3, 64), (4, 64), (4, 128)])
@pytest.mark.parametrize("cal_tokens", [40, 3])
def test_chunks_through_the_bulk_quantizer_with_values_outside_the_calibrated_range(bits, group, cal_tokens):
    # chunks that start on a multiple of the group size send their whole spans to the bulk kernel, the rest to the tile kernels;
    # calibrated on a few tokens only, so later tokens clamp at both ends (three tokens: most of them do)
    G = group
    wl = TINY.scaled(seq=5 * G + 19, group=G, bits=bits, head_dim=128, n_q_heads=4, n_kv_heads=2, batch=2, topk=7, pfn_n=2, seed=81 + G + bits)
    _both(wl, chunks=(G, G + 6, G - 6, 2 * G, 19), cal_tokens=cal_tokens)


def test_static_pairs_that_force_the_literal_formula():
    # hand-made pairs: a tiny scale with a huge zero-point (the fast coder declines), scale 0, and a scale so large that every
    # value codes to the zero-point; the codes must still be the oracle's bit for bit
    wl = TINY.scaled(seq=256, group=64, bits=4, head_dim=128, n_q_heads=2, n_kv_heads=2, batch=1, topk=3, pfn_n=1, seed=5)
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    gp, op = kv.StaticParams(gcfg), oracle.StaticParams(ocfg)
    rng = np.random.default_rng(11)
    ks = rng.uniform(0.05, 0.5, size=(2, 128)).astype(np.float32)
    kz = np.rint(rng.uniform(0, 15, size=(2, 128))).astype(np.float32)
    ks[:, 0] = 1e-6; kz[:, 0] = 5e6          # |zero| far beyond the fast coder's range
    ks[:, 1] = 0.0; kz[:, 1] = 0.0           # never calibrated
    ks[:, 2] = 1e4; kz[:, 2] = 7.0           # every value rounds to 0: code 7
    ks[:, 3] = 3e-4; kz[:, 3] = 40000.0      # integer part beyond 16 bits: literal formula
    ks[:, 4] = 2e-3; kz[:, 4] = -29990.0     # just inside the fast coder's range
    vs = np.array([[0.3, 1e-5]] * 2, np.float32)
    vz = np.array([[8.0, -70000.0]] * 2, np.float32)
    for name, arr in (("k_scale", ks), ("k_zero", kz), ("v_scale", vs), ("v_zero", vz)):
        getattr(gp, name).copy_(torch.from_numpy(arr))
        getattr(op, name)[...] = arr.reshape(getattr(op, name).shape)
    gc, oc = kv.KVCache(gcfg, gs), oracle.Cache(ocfg, bm, pos, cnt)
    kv.quantize_append_calibrated(gcfg, gc, gp, K, V)
    oracle.quantize_append_calibrated(ocfg, oc, op, np16(K), np16(V))
    torch.cuda.synchronize()
    per, nb = wl.max_seq * wl.head_dim * wl.bits // 8, wl.seq * wl.head_dim * wl.bits // 8
    for name in ("k_codes", "v_codes"):
        assert bits_equal(getattr(gc, name).cpu().numpy().reshape(-1, per)[:, :nb], getattr(oc, name).reshape(-1, per)[:, :nb]), name
    assert kv.read_status(gc) == 0


def test_many_splits_and_clusters():
    # few units and a long sequence (merge kernel), then many units (cluster merge)
    _both(TINY.scaled(seq=64 * 40 + 5, group=64, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=1, batch=1, topk=20, seed=12))
    _both(TINY.scaled(seq=64 * 24 + 11, group=64, bits=4, head_dim=128, n_q_heads=16, n_kv_heads=16, batch=8, topk=6, pfn_n=1, seed=13))


def test_unsupported_shapes_are_refused_on_the_host():
    wl = TINY.scaled(seq=64, group=32, bits=2, head_dim=128, n_q_heads=2, n_kv_heads=2, batch=1)      # four value groups per row
    _, gcfg = configs(wl)
    gs = kv.SinkSet(gcfg)
    gc, gp = kv.KVCache(gcfg, gs), kv.StaticParams(gcfg)
    q = torch.zeros((1, 2, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(kv.KvsinkError) as e:
        kv.decode_attention_calibrated(gcfg, gc, gp, q)
    assert e.value.code == -3
