"""GPU parity of the per-token key path (Section 4.1 "Per-token quantization"; Section 5.1's per-token Key and Value scheme)
against the CPU oracle: packed codes, per-token parameters and side buffer bit for bit; attention within
|gpu - oracle| <= 2e-3 + 1e-2 |oracle|."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, bits_equal, configs, np16

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


def _both(wl, chunks=None, poison=False):
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    gc, oc = kv.KVCache(gcfg, gs, per_token_keys=True), oracle.Cache(ocfg, bm, pos, cnt, per_token_keys=True)
    if poison:   # what lies beyond the sequence must never reach a result
        for name in ("k_scale", "k_zero", "v_scale", "v_zero"):
            getattr(gc, name).fill_(float("nan"))
        gc.k_codes.fill_(0xFF)
        gc.v_codes.fill_(0xFF)
    ngv = wl.head_dim // min(wl.group, wl.head_dim)
    units = wl.batch * wl.n_kv_heads
    per = wl.max_seq * wl.head_dim * wl.bits // 8
    at = 0
    for n in (chunks or (wl.seq,)):
        kv.quantize_append_pertoken(gcfg, gc, K[:, :, at:at + n], V[:, :, at:at + n])
        oracle.quantize_append_pertoken(ocfg, oc, np16(K[:, :, at:at + n]), np16(V[:, :, at:at + n]))
        at += n
        assert gc.seq_len == oc.seq_len == at
        if not poison:   # codes: the tiles that hold tokens (fields of tokens not yet appended are zero on both sides)
            nb = (at + 15) // 16 * 16 * wl.head_dim * wl.bits // 8
            for name in ("k_codes", "v_codes"):
                g = getattr(gc, name).cpu().numpy().reshape(-1, per)[:, :nb]
                o = getattr(oc, name).reshape(-1, per)[:, :nb]
                assert bits_equal(g, o), f"{name} after {at} tokens"
        for name in ("k_scale", "k_zero", "v_scale", "v_zero"):
            g = getattr(gc, name).cpu().numpy().reshape(units, wl.max_seq, ngv)[:, :at]
            o = getattr(oc, name).reshape(units, wl.max_seq, ngv)[:, :at]
            assert bits_equal(g, o), f"{name} after {at} tokens"
    if oc.sizes["sink_halfs"] > 0:
        for name in ("sink_k", "sink_v"):
            assert bits_equal(getattr(gc, name).cpu().numpy().view(np.uint16)[:getattr(oc, name).size], getattr(oc, name)), name
    q = synth.make_query(wl, K)
    out, lse = kv.decode_attention_pertoken(gcfg, gc, q)
    ref, ref_lse = oracle.decode_attention_pertoken(ocfg, oc, np16(q))
    torch.cuda.synchronize()
    assert kv.read_status(gc) == 0
    err = assert_close(out.cpu().numpy(), ref, "attention output")
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-3 + 1e-3 * np.abs(ref_lse).max()
    return err


@pytest.mark.parametrize("bits,group", [(2, 128), (2, 64), (4, 64), (4, 128), (2, 256)])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (8, 2), (6, 2)])
def test_grid_of_shapes(bits, group, hq, hkv):
    seq = 3 * group + 37
    wl = TINY.scaled(bits=bits, head_dim=128, group=group, n_q_heads=hq, n_kv_heads=hkv, batch=2, seq=seq, topk=5, pfn_n=2,
                     seed=9100 + bits * 100 + group + hq)
    _both(wl)


@pytest.mark.parametrize("group", [128, 256])
def test_three_bit_one_group_one_head(group):
    wl = TINY.scaled(bits=3, head_dim=128, group=group, n_q_heads=4, n_kv_heads=4, batch=2, seq=2 * group + 21, topk=5, pfn_n=2, seed=931 + group)
    _both(wl)


@pytest.mark.parametrize("seq", [1, 15, 16, 17, 63, 64, 65, 200])
def test_short_and_ragged_lengths(seq):
    wl = TINY.scaled(seq=seq, topk=min(2, seq), batch=2, group=64, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=2, seed=277 + seq)
    _both(wl)


@pytest.mark.parametrize("bits", [2, 4])
def test_chunked_appends_that_start_and_end_inside_tiles(bits):
    wl = TINY.scaled(seq=333, group=64, bits=bits, head_dim=128, n_q_heads=4, n_kv_heads=2, batch=2, topk=6, pfn_n=1, seed=56 + bits)
    _both(wl, chunks=(1, 14, 1, 33, 100, 1, 183))


@pytest.mark.parametrize("bits,group", [(2, 64), (2, 128), (4, 64), (4, 128), (3, 128)])
def test_chunks_through_the_bulk_quantizer(bits, group):
    # chunks that start on a multiple of the group size send their whole spans to the bulk kernel, the rest to the tile kernels
    G = group
    rep = 1 if bits == 3 else 2
    wl = TINY.scaled(seq=5 * G + 19, group=G, bits=bits, head_dim=128, n_q_heads=2 * rep, n_kv_heads=2, batch=2, topk=7, pfn_n=2, seed=83 + G + bits)
    _both(wl, chunks=(G, G + 6, G - 6, 2 * G, 19))


@pytest.mark.parametrize("bits,group,seq", [(2, 64, 101), (4, 128, 300), (3, 128, 77)])
def test_unwritten_cache_memory_never_reaches_a_result(bits, group, seq):
    rep = 1 if bits == 3 else 2
    wl = TINY.scaled(seq=seq, group=group, bits=bits, head_dim=128, n_q_heads=2 * rep, n_kv_heads=2, batch=2, topk=3, pfn_n=1, seed=71 + bits)
    _both(wl, poison=True)


def test_many_splits_and_clusters():
    # few units and a long sequence (merge kernel), then many units (cluster merge)
    _both(TINY.scaled(seq=64 * 40 + 5, group=64, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=1, batch=1, topk=20, seed=14))
    _both(TINY.scaled(seq=64 * 24 + 11, group=64, bits=4, head_dim=128, n_q_heads=16, n_kv_heads=16, batch=8, topk=6, pfn_n=1, seed=15))


def test_no_sink_tokens_at_all():
    wl = TINY.scaled(seq=150, group=64, bits=2, head_dim=128, n_q_heads=2, n_kv_heads=2, batch=1, topk=0, pfn_n=0, seed=16)
    _both(wl)


@pytest.mark.parametrize("kw", [dict(group=32), dict(head_dim=64, group=64), dict(n_q_heads=16, n_kv_heads=2), dict(bits=3, group=64),
                                dict(bits=3, n_q_heads=4, n_kv_heads=2)])
def test_unsupported_shapes_are_refused_on_the_host(kw):
    base = dict(seq=64, group=128, bits=2, head_dim=128, n_q_heads=2, n_kv_heads=2, batch=1)
    base.update(kw)
    wl = TINY.scaled(**base)
    _, gcfg = configs(wl)
    gc = kv.KVCache(gcfg, kv.SinkSet(gcfg), per_token_keys=True)
    x = torch.zeros((1, wl.n_kv_heads, 16, wl.head_dim), dtype=torch.float16, device="cuda")
    q = torch.zeros((1, wl.n_q_heads, wl.head_dim), dtype=torch.float16, device="cuda")
    with pytest.raises(kv.KvsinkError) as e:
        kv.quantize_append_pertoken(gcfg, gc, x, x)
    assert e.value.code == -3
    with pytest.raises(kv.KvsinkError) as e:
        kv.decode_attention_pertoken(gcfg, gc, q)
    assert e.value.code == -3
