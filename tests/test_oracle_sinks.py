"""Pins for sink prediction (Algorithm 1 at the emergence layer; Section 4.3): planted outliers are found,
the selection equals a library sort on small inputs, ties go to the lower index, and the degenerate budgets."""
import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth


def _cfg(wl):
    return oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq,
                         wl.topk, wl.pfn_n, wl.channels)


def _bits(bm_row, n):
    return np.array([(bm_row[i // 32] >> (i % 32)) & 1 for i in range(n)], bool)


@pytest.mark.parametrize("name,scale", [("tiny", {}), ("llama2_7b_layer", dict(batch=2, seq=1024)),
                                        ("long_gqa", dict(seq=4096, topk=41))])
def test_planted_outliers_are_detected(name, scale):
    wl = synth.WORKLOADS[name].scaled(**scale)
    H = synth.make_hidden(wl).numpy()
    planted = synth.sink_positions(wl)
    bm, pos, cnt = oracle.predict_sinks(_cfg(wl), H)
    for b in range(wl.batch):
        want = sorted(set(planted[b].tolist()) | set(range(wl.pfn_n)))
        assert pos[b, :cnt[b]].tolist() == want
        assert np.flatnonzero(_bits(bm[b], wl.max_seq)).tolist() == want
        assert np.all(pos[b, cnt[b]:] == -1)


@pytest.mark.parametrize("n_channels", [0, 1, 3])
def test_equals_stable_library_sort(n_channels):
    rng = np.random.default_rng(n_channels)
    B, S, d, k, N = 3, 200, 48, 7, 2
    # few distinct magnitudes -> many ties
    H = (rng.integers(-6, 7, size=(B, S, d)) * 0.5).astype(np.float16)
    chans = tuple(int(c) for c in rng.choice(d, n_channels, replace=False))
    cfg = oracle.Config(B, 2, 2, 64, d, 4, 32, 224, k, N, chans)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    for b in range(B):
        a = np.abs(H[b].astype(np.float32))
        score = a.max(axis=1) if n_channels == 0 else a[:, list(chans)].max(axis=1)
        order = np.argsort(-score, kind="stable")          # descending score, ascending index among equals
        want = sorted(set(order[:k].tolist()) | set(range(N)))
        assert pos[b, :cnt[b]].tolist() == want


def test_degenerate_budgets():
    rng = np.random.default_rng(9)
    H = rng.standard_normal((1, 40, 16)).astype(np.float16)
    base = dict(batch=1, n_q_heads=1, n_kv_heads=1, head_dim=64, hidden=16, bits=4, group=16, max_seq=48, channels=(3,))
    bm, pos, cnt = oracle.predict_sinks(oracle.Config(topk=0, pfn_n=0, **base), H)
    assert cnt[0] == 0 and not bm.any()
    bm, pos, cnt = oracle.predict_sinks(oracle.Config(topk=0, pfn_n=3, **base), H)
    assert pos[0, :cnt[0]].tolist() == [0, 1, 2]
    bm, pos, cnt = oracle.predict_sinks(oracle.Config(topk=100, pfn_n=0, **base), H)
    assert cnt[0] == 40 and pos[0, :40].tolist() == list(range(40))          # k >= S keeps every token
    bm, pos, cnt = oracle.predict_sinks(oracle.Config(topk=1, pfn_n=100, **base), H)
    assert cnt[0] == 40
    bm, pos, cnt = oracle.predict_sinks(oracle.Config(topk=2, pfn_n=1, **base), H[:, :0])
    assert cnt[0] == 0 and not bm.any()


def test_strided_hidden_and_negative_outliers():
    wl = synth.WORKLOADS["tiny"]
    H = synth.make_hidden(wl).numpy()
    wide = np.zeros((wl.batch, wl.seq, wl.hidden + 24), np.float16)
    wide[:, :, :wl.hidden] = H
    a = oracle.predict_sinks(_cfg(wl), H)
    b = oracle.predict_sinks(_cfg(wl), wide[:, :, :wl.hidden])
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
