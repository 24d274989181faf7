"""GPU parity of the prompt attention over the just-quantized cache (Algorithm 1's attention statement) against the CPU
oracle: |gpu - oracle| <= 2e-3 + 1e-2 |oracle| for every query row."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, configs, np16

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


def _both(wl, T, pos0, strided=False):
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    gc = kv.KVCache(gcfg, gs)
    kv.quantize_append(gcfg, gc, K, V)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    oc = oracle.Cache(ocfg, bm, pos, cnt)
    oracle.quantize_append(ocfg, oc, np16(K), np16(V))
    g = torch.Generator("cuda").manual_seed(wl.seed + T)
    q = torch.randn((wl.batch, wl.n_q_heads, T, wl.head_dim), device="cuda", generator=g).half()
    if T > 3:       # some queries look straight at a sink key
        p1 = int(pos[0, min(1, cnt[0] - 1)])
        q[0, :, 3] += (4.0 * K[0, :, p1].repeat_interleave(wl.n_q_heads // wl.n_kv_heads, dim=0)).half()
    if strided:     # [B, T, Hq, D] storage
        q = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    out, lse = kv.prefill_attention(gcfg, gc, q, pos0)
    ref, ref_lse = oracle.prefill_attention(ocfg, oc, np16(q), pos0)
    torch.cuda.synchronize()
    assert kv.read_status(gc) == 0
    assert_close(out.cpu().numpy(), ref, "prompt attention")
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-3 + 1e-3 * np.abs(ref_lse).max()


@pytest.mark.parametrize("bits,d,group", [(2, 128, 128), (3, 128, 64), (4, 128, 64), (2, 64, 32), (4, 64, 16)])
@pytest.mark.parametrize("hq,hkv", [(2, 2), (8, 2), (6, 2), (16, 2)])
def test_whole_prompt(bits, d, group, hq, hkv):
    # several groups and a ragged remainder in the fp16 tail; every token of the prompt is a query
    seq = 2 * group + 21
    wl = TINY.scaled(bits=bits, head_dim=d, group=group, n_q_heads=hq, n_kv_heads=hkv, batch=2, seq=seq, topk=4, pfn_n=2,
                     seed=11000 + bits * 100 + d + group + hq)
    _both(wl, seq, 0)


@pytest.mark.parametrize("T,pos0", [(1, 0), (1, 99), (7, 93), (40, 10), (33, 67)])
def test_chunks_of_queries(T, pos0):
    wl = TINY.scaled(bits=2, head_dim=128, group=32, n_q_heads=6, n_kv_heads=2, batch=2, seq=100, topk=5, pfn_n=1, seed=12000 + T)
    _both(wl, T, pos0, strided=True)


def test_queries_beyond_the_cache_are_refused():
    wl = TINY.scaled(seq=20, group=32, bits=2, head_dim=128, n_q_heads=2, n_kv_heads=2, batch=1)
    _, gcfg = configs(wl)
    gc = kv.KVCache(gcfg)
    gc.seq_len = 20
    q = torch.zeros((1, 2, 4, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(kv.KvsinkError) as e:
        kv.prefill_attention(gcfg, gc, q, 18)
    assert e.value.code == -1


@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("hq,hkv", [(2, 2), (8, 2)])
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_keys_with_a_wide_factor_range(bits, hq, hkv, seed):
    # the decode test's family of keys (a channel 300 times louder and one 1000 times quieter than the rest, ramps and noise far
    # from zero, constant channels) under N(0,1) queries at every position: 2 and 4 bit take the integer key side, whose sums
    # are exact whatever the spread of the factors; 3 bit stays on the fp16 key side (worst case 0.8 of the tolerance here)
    wl = TINY.scaled(seq=160, group=32, bits=bits, head_dim=128, batch=2, n_q_heads=hq, n_kv_heads=hkv, seed=500 + seed)
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    g = torch.Generator("cuda").manual_seed(seed)
    K[:, :, :, 3] = 2.5
    K[:, :, :, 4] = 0.0
    K[:, :, :, 6] *= 300.0
    K[:, :, :, 70] *= 1e-3
    K[:, :, :, 8] = 300.0 + torch.arange(160, device="cuda").half() * 0.25
    K[:, :, :, 100] = -40.0 + torch.randn(160, device="cuda", generator=g).half() * 0.01
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    gc, oc = kv.KVCache(gcfg, gs), oracle.Cache(ocfg, bm, pos, cnt)
    kv.quantize_append(gcfg, gc, K, V)
    oracle.quantize_append(ocfg, oc, np16(K), np16(V))
    gq = torch.Generator("cuda").manual_seed(seed + 100)
    q = torch.randn((2, hq, 160, 128), device="cuda", generator=gq).half()
    out, lse = kv.prefill_attention(gcfg, gc, q, 0)
    ref, ref_lse = oracle.prefill_attention(ocfg, oc, np16(q), 0)
    torch.cuda.synchronize()
    assert kv.read_status(gc) == 0
    assert_close(out.cpu().numpy(), ref, "prompt attention")
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-3 + 1e-3 * np.abs(ref_lse).max()
