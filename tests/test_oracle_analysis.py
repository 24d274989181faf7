"""Pins for the oracle's analysis routines: the per-channel magnitude scan behind the paper's table of outlier
channels (Appendix D) and the quantization-error split of Table 1 (Section 4.1).

The scan is pinned to numpy's own reduction, planted outliers and the NaN rule.  The error split is pinned to a group
worked by hand from Eq. 8-11, to the round-to-nearest bound, to element bookkeeping, to the (separately pinned) cache
path -- the error of the tensors kvo_dequant_dense returns -- and to the direction of the paper's observation that
groups with sink tokens quantize worse.
"""
import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth

TINY = synth.WORKLOADS["tiny"]


def _cfg(wl, max_seq=None):
    return oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group,
                         wl.max_seq if max_seq is None else max_seq, wl.topk, wl.pfn_n, wl.channels)


def test_channel_scan_is_numpys_reduction_and_finds_planted_channels():
    wl = TINY.scaled(batch=3, seq=90)
    H = synth.make_hidden(wl).numpy()
    got = oracle.channel_absmax(H)
    want = np.abs(H.astype(np.float32)).max(axis=(0, 1))
    assert np.array_equal(got, want)
    top = set(np.argsort(-got)[:len(wl.channels)].tolist())
    assert top == set(wl.channels)                      # the planted outlier channels stand out
    assert got[list(wl.channels)].min() > 50 * np.delete(got, list(wl.channels)).max()


def test_channel_scan_ignores_nan_keeps_infinity_and_honours_strides():
    H = np.zeros((2, 5, 32), np.float16)
    H[0, 1, 3] = np.nan
    H[1, 2, 3] = -2.0
    H[0, 0, 4] = -np.inf
    H[1, 4, 5] = 7.5
    got = oracle.channel_absmax(H)
    assert got[3] == 2.0 and np.isinf(got[4]) and got[5] == 7.5 and got[0] == 0.0
    big = np.full((2, 7, 64), 100.0, np.float16)
    big[:, :5, :32] = H
    assert np.array_equal(oracle.channel_absmax(big[:, :5, :32]), got)


def test_error_of_a_group_worked_by_hand():
    # one token, 16 channels, 2 bit: min 0, max 3 -> scale 1, zero 0 (Eq. 10-11); 0.5, 1.5, 2.5 are ties and go to the
    # even integers 0, 2, 2 (Eq. 8), each off by 0.5; every other value is a code -> 3 * 0.25 in 16 elements
    cfg = oracle.Config(1, 1, 1, 16, 16, 2, 16, 16, 0, 0, ())
    x = np.zeros((1, 1, 1, 16), np.float16)
    x[0, 0, 0, :8] = [0, 0.5, 1.5, 2.5, 3, 1, 2, 3]
    bm = np.zeros((1, 1), np.uint32)
    out = oracle.quant_error(cfg, x, bm, per_channel=False, exclude_sinks=False)
    assert out.tolist() == [0.75, 16.0, 0.0, 0.0]
    # the same sixteen values down one channel of a 16-token key group
    xk = np.zeros((1, 1, 16, 16), np.float16)
    xk[0, 0, :, 5] = x[0, 0, 0]
    out = oracle.quant_error(cfg, xk, bm, per_channel=True, exclude_sinks=False)
    assert out.tolist() == [0.75, 256.0, 0.0, 0.0]     # the fifteen constant-zero channels reproduce themselves
    # token 2 (value 1.5) is a sink: with exclusion it is not counted, without it the whole group counts as "with sink"
    bm[0, 0] = 1 << 2
    assert oracle.quant_error(cfg, xk, bm, True, True).tolist() == [0.0, 0.0, 0.5, 240.0]
    assert oracle.quant_error(cfg, xk, bm, True, False).tolist() == [0.0, 0.0, 0.75, 256.0]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("per_channel", [True, False])
def test_error_bookkeeping_bound_and_the_cache_path(bits, per_channel):
    wl = TINY.scaled(bits=bits, batch=2, seq=96, group=32, head_dim=64, n_q_heads=4, n_kv_heads=2, topk=5, pfn_n=1, seed=77 + bits)
    cfg = _cfg(wl)
    H = synth.make_hidden(wl).numpy()
    K, V = (t.numpy() for t in synth.make_kv(wl))
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    x = K if per_channel else V
    n_all = x.size
    plain = oracle.quant_error(cfg, x, bm, per_channel, False)
    assert plain[1] + plain[3] == n_all                 # every element is in exactly one class
    excl = oracle.quant_error(cfg, x, bm, per_channel, True)
    n_sink_elems = int(cnt.sum()) * wl.n_kv_heads * wl.head_dim
    assert excl[1] + excl[3] == n_all - n_sink_elems     # sink tokens are not quantized
    # round to nearest: no element is off by more than half the largest step a group can have
    step_max = (float(np.abs(x.astype(np.float32)).max()) * 2) / ((1 << bits) - 1)
    assert plain[0] + plain[2] <= n_all * (step_max / 2) ** 2
    # the cache path (pinned by its own tests): the error of what attention would read, over the non-sink tokens
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    kd, vd = oracle.dequant_dense(cfg, cache)
    dense = kd if per_channel else vd
    keep = np.ones((wl.batch, wl.seq), bool)
    for b in range(wl.batch):
        keep[b, pos[b, :cnt[b]]] = False
    err = ((x.astype(np.float64) - dense) ** 2)[np.broadcast_to(keep[:, None, :, None], x.shape)].sum()
    assert np.isclose(excl[0] + excl[2], err, rtol=1e-12, atol=0)


def test_groups_with_sink_tokens_quantize_worse():
    # low-norm sink rows inside per-channel key groups with offsets widen the range of every channel of their group
    wl = synth.WORKLOADS["llama3_8b_gqa"].scaled(batch=1, seq=1024, n_q_heads=8, n_kv_heads=2, topk=6, group=32, bits=2)
    cfg = _cfg(wl)
    bm, pos, cnt = oracle.predict_sinks(cfg, synth.make_hidden(wl).numpy())
    K, _ = (t.numpy() for t in synth.make_kv(wl))
    K = (K.astype(np.float32) * 0.5 + 4.0).astype(np.float16)          # channels with an offset (Section 4.1: keys have them) ...
    for b, p in enumerate(synth.sink_positions(wl)):
        K[b, :, p, :] = (K[b, :, p, :].astype(np.float32) * 0.02).astype(np.float16)   # ... and small sink rows (Section 3.2)
    plain = oracle.quant_error(cfg, K, bm, True, False)
    excl = oracle.quant_error(cfg, K, bm, True, True)
    assert plain[3] > 0 and plain[2] / plain[3] > 1.05 * plain[0] / plain[1]     # Table 1, dynamic rows: "w/" above "w/o"
    assert excl[2] / excl[3] < plain[2] / plain[3]                               # excluding the sinks repairs those groups
