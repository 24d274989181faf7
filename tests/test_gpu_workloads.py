"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

The oracle cannot redo a whole workload in seconds, so it is run one (sequence, KV head) unit at a time on
sampled units: sink prediction for the unit's whole sequence, the unit's packed codes / parameters / side buffer
bit for bit, then one appended token and the unit's attention outputs within tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, bits_equal, np16

pytestmark = pytest.mark.gpu


def _gpu_cfg(wl):
    return kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                     wl.channels)


def _unit_cfg(wl):
    rep = wl.n_q_heads // wl.n_kv_heads
    return oracle.Config(1, rep, 1, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n, wl.channels)


def _unit_slice(t, wl, b, h, per_unit):
    u = b * wl.n_kv_heads + h
    return t[u * per_unit:(u + 1) * per_unit].cpu().numpy()


def check_units(wl, H, layers, units, n_seq_checked=2):
    """layers: list of (K, V) device tensors; units: list of (b, h)."""
    gcfg, ucfg = _gpu_cfg(wl), _unit_cfg(wl)
    rep = wl.n_q_heads // wl.n_kv_heads
    sz = kv.cache_sizes(gcfg)
    nu = wl.batch * wl.n_kv_heads
    sinks = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, sinks)
    planted = synth.sink_positions(wl)
    cap = wl.topk + wl.pfn_n
    g_pos, g_cnt = sinks.pos.cpu().numpy().reshape(wl.batch, cap), sinks.count.cpu().numpy()
    g_bm = sinks.bitmask.cpu().numpy().view(np.uint32).reshape(wl.batch, -1)
    for b in range(wl.batch):                      # every sequence: the planted outliers (and token 0) are found
        want = sorted(set(planted[b].tolist()) | set(range(wl.pfn_n)))
        assert g_pos[b, :g_cnt[b]].tolist() == want
    seq_masks = {}
    for b in sorted({b for b, _ in units})[:max(n_seq_checked, 1)] + sorted({b for b, _ in units}):
        if b in seq_masks:
            continue
        bm, pos, cnt = oracle.predict_sinks(ucfg, np16(H[b:b + 1]))
        assert bits_equal(g_bm[b:b + 1], bm) and bits_equal(g_pos[b:b + 1], pos) and g_cnt[b] == cnt[0]
        seq_masks[b] = (bm, pos, cnt)
    worst = 0.0
    for li, (K, V) in enumerate(layers):
        cache = kv.KVCache(gcfg, sinks)
        kv.quantize_append(gcfg, cache, K, V)
        k1, v1 = synth.make_new_token(wl, li, 0, "cuda")
        pre = {name: getattr(cache, name).clone() for name in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero",
                                                                "sink_k", "sink_v")}
        kv.quantize_append(gcfg, cache, k1, v1)
        q = synth.make_query(wl, K, li)
        out, lse = kv.decode_attention(gcfg, cache, q)
        torch.cuda.synchronize()
        assert kv.read_status(cache) == 0
        for (b, h) in units:
            bm, pos, cnt = seq_masks[b]
            oc = oracle.Cache(ucfg, bm, pos, cnt)
            oracle.quantize_append(ucfg, oc, np16(K[b:b + 1, h:h + 1]), np16(V[b:b + 1, h:h + 1]))
            for name, per in (("k_codes", sz["k_codes_bytes"] // nu), ("v_codes", sz["v_codes_bytes"] // nu),
                              ("k_scale", sz["k_param_floats"] // nu), ("k_zero", sz["k_param_floats"] // nu),
                              ("v_scale", sz["v_param_floats"] // nu), ("v_zero", sz["v_param_floats"] // nu)):
                assert bits_equal(_unit_slice(pre[name], wl, b, h, per), getattr(oc, name)), f"layer {li} unit {(b, h)} {name}"
            per = sz["sink_halfs"] // nu
            for name in ("sink_k", "sink_v"):
                assert bits_equal(_unit_slice(pre[name], wl, b, h, per).view(np.uint16), getattr(oc, name)), f"unit {(b, h)} {name}"
            oracle.quantize_append(ucfg, oc, np16(k1[b:b + 1, h:h + 1]), np16(v1[b:b + 1, h:h + 1]))
            assert bits_equal(_unit_slice(cache.v_codes, wl, b, h, sz["v_codes_bytes"] // nu), oc.v_codes)
            assert bits_equal(_unit_slice(cache.k_tail, wl, b, h, wl.group * wl.head_dim)[:wl.head_dim].view(np.uint16),
                              oc.k_tail[:wl.head_dim])
            ref, ref_lse = oracle.decode_attention(ucfg, oc, np16(q[b:b + 1, h * rep:(h + 1) * rep]))
            worst = max(worst, assert_close(out[b:b + 1, h * rep:(h + 1) * rep].cpu().numpy(), ref, f"layer {li} unit {(b, h)} attention"))
            assert np.abs(lse[b, h * rep:(h + 1) * rep].cpu().numpy() - ref_lse[0]).max() < 2e-3 + 1e-3 * np.abs(ref_lse).max()
        del cache, pre
    return worst


def test_llama2_7b_layer_full_size():
    wl = synth.WORKLOADS["llama2_7b_layer"]
    H = synth.make_hidden(wl, "cuda")
    worst = check_units(wl, H, [synth.make_kv(wl, 0, "cuda")], [(0, 0), (3, 17), (7, 31), (5, 8)])
    print("config 2 worst attention error", worst)


def test_llama3_8b_gqa_full_size():
    wl = synth.WORKLOADS["llama3_8b_gqa"]
    H = synth.make_hidden(wl, "cuda")
    check_units(wl, H, [synth.make_kv(wl, 0, "cuda")], [(0, 0), (3, 7), (2, 4)])


def test_long_context_gqa_full_size():
    wl = synth.WORKLOADS["long_gqa"]
    H = synth.make_hidden(wl, "cuda")
    check_units(wl, H, [synth.make_kv(wl, 0, "cuda")], [(0, 0), (0, 5)])


@pytest.mark.parametrize("name", ["decode32_3bit", "decode32_4bit"])
def test_decode32_full_batch_two_layers(name):
    """Full batch and sequence of the 32-layer decode workload; two of the 32 layers (each 8.6 GB of fp16 input)."""
    wl = synth.WORKLOADS[name]
    H = synth.make_hidden(wl, "cuda")
    layers = [synth.make_kv(wl, 0, "cuda")]
    check_units(wl, H, layers, [(0, 0), (63, 31), (17, 5)])
    del layers
    torch.cuda.empty_cache()
    layers = [synth.make_kv(wl, 1, "cuda")]
    check_units(wl, H, layers, [(40, 12)])
