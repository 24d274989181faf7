"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

The single-layer workloads are compared in full: every (sequence, KV head) unit's packed codes, parameters, side
buffer and tail bit for bit, and every attention output within tolerance.  The 32-layer workload holds 2048 units of
8192 tokens per layer; there the oracle is run one unit at a time on 64 units spread over the whole index range, on
two of the layers: sink prediction for the unit's whole sequence, the unit's arrays bit for bit, then one appended
token and the unit's attention outputs within tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, bits_equal, np16, run_both

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


def check_units(wl, H, layers, units, n_seq_checked=2, layer0=0):
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
    for li, (K, V) in enumerate(layers, start=layer0):
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


def check_whole_workload(wl):
    """Every unit of a single-layer workload: prediction, prefill, one appended token, attention."""
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    r = run_both(wl, appends=1, H=H, K=K, V=V)
    planted = synth.sink_positions(wl)
    oc = r["oracle_cache"]
    cap = wl.topk + wl.pfn_n
    for b in range(wl.batch):                      # every sequence: the planted outliers (and the first N) are found
        want = sorted(set(planted[b].tolist()) | set(range(wl.pfn_n)))
        assert oc.sink_pos.reshape(wl.batch, cap)[b, :oc.sink_count[b]].tolist() == want
    return r["err"]


def test_llama2_7b_layer_full_size():
    print("config 2 worst attention error", check_whole_workload(synth.WORKLOADS["llama2_7b_layer"]))


def test_llama3_8b_gqa_full_size():
    print("config 3 worst attention error", check_whole_workload(synth.WORKLOADS["llama3_8b_gqa"]))


def test_long_context_gqa_full_size():
    print("config 5 worst attention error", check_whole_workload(synth.WORKLOADS["long_gqa"]))


def _spread_units(wl, n, shift):
    """n (sequence, KV head) units spread evenly over the unit index range, every KV head and many sequences among them."""
    nu = wl.batch * wl.n_kv_heads
    step = nu // n
    units = [(i * step + (i * 13 + shift) % step) for i in range(n)]
    return [(u // wl.n_kv_heads, u % wl.n_kv_heads) for u in units]


@pytest.mark.parametrize("name", ["decode32_3bit", "decode32_4bit"])
def test_decode32_full_batch_two_layers(name):
    """Full batch and sequence of the 32-layer decode workload; two of the 32 layers (each 8.6 GB of fp16 input), 64 units
    of each, the first and the last unit among them."""
    wl = synth.WORKLOADS[name]
    H = synth.make_hidden(wl, "cuda")
    for layer, shift in ((0, 0), (1, 5)):
        units = _spread_units(wl, 62, shift) + [(0, 0), (wl.batch - 1, wl.n_kv_heads - 1)]
        layers = [synth.make_kv(wl, layer, "cuda")]
        check_units(wl, H, layers, sorted(set(units)), layer0=layer)
        del layers
        torch.cuda.empty_cache()
