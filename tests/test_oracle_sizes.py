"""Pin: the size calculator reproduces the 24 memory figures the paper prints (Appendix F, Table 4)."""
import os

import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _rows():
    rows = []
    with open(os.path.join(HERE, "golden", "table4_memory.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            rows.append((p[0], int(p[1]), int(p[2]), int(p[3]), float(p[4]), [float(x) for x in p[5:8]]))
    return rows


def _round_like_paper(x, printed):
    digits = len(str(printed).split(".")[1]) if "." in str(printed) and not float(printed).is_integer() else 0
    return round(x + 1e-9, digits), digits


@pytest.mark.parametrize("row", _rows(), ids=lambda r: r[0])
def test_table4_memory_columns(row):
    name, layers, hkv, d, kv_mb, plus = row
    for k in (1, 5, 20):
        cfg = oracle.Config(batch=1, n_q_heads=hkv, n_kv_heads=hkv, head_dim=d, hidden=hkv * d, bits=2, group=128,
                            max_seq=4096, topk=k, pfn_n=0, channels=(0,))
        sz = oracle.cache_sizes(cfg)
        codes_mb = layers * (sz["k_codes_bytes"] + sz["v_codes_bytes"]) / 2**20
        assert codes_mb == kv_mb
        sink_mb = layers * 2 * sz["sink_halfs"] * 2 / 2**20
        printed = plus[(1, 5, 20).index(k)]
        got, digits = _round_like_paper(sink_mb, printed)
        # the paper rounds to two decimals (half-up); allow one unit in the last printed place
        assert abs(got - printed) <= 10.0 ** (-digits) * 0.51 + 1e-12, (name, k, sink_mb, printed)
        assert sz["sink_capacity"] == k


def test_bad_configs_are_rejected():
    good = dict(batch=1, n_q_heads=8, n_kv_heads=8, head_dim=64, hidden=512, bits=4, group=32, max_seq=256, topk=2,
                pfn_n=1, channels=(1,))
    oracle.cache_sizes(oracle.Config(**good))
    for bad in (dict(bits=5), dict(bits=1), dict(group=24), dict(max_seq=100), dict(n_q_heads=12), dict(head_dim=40),
                dict(bits=3, head_dim=32, group=32, hidden=256)):
        with pytest.raises(RuntimeError):
            oracle.cache_sizes(oracle.Config(**{**good, **bad}))
