"""The C-ABI library loads, exports every symbol include/kvsink.h declares, and rejects bad arguments on the
host (no GPU needed: argument checks come before any CUDA call)."""
import ctypes as C
import os
import re

import pytest

import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "kvsink.h")).read()
    return sorted(set(re.findall(r"\b(kvsink_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = binding.lib()
    names = _declared()
    assert set(binding.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_sizes_match_the_closed_forms():
    cfg = kv.Config(8, 32, 32, 128, 4096, 2, 128, 4096, 8, 1, (2533, 1415))
    s = kv.cache_sizes(cfg)
    assert s["k_codes_bytes"] == 8 * 32 * 4096 * 128 * 2 // 8
    assert s["k_param_floats"] == 8 * 32 * 32 * 128 and s["v_param_floats"] == 8 * 32 * 4096
    assert s["sink_capacity"] == 9 and s["sink_halfs"] == 8 * 32 * 9 * 128
    assert s["tile_bytes"] == 512 and s["v_group"] == 128
    # LLaMA2-7B, 32 layers, 2 bit, 4096 tokens, batch 1: 256 MiB of codes (the paper's efficiency table)
    one = kv.cache_sizes(kv.Config(1, 32, 32, 128, 4096, 2, 128, 4096, 1, 0, (2533,)))
    assert 32 * (one["k_codes_bytes"] + one["v_codes_bytes"]) == 256 * 2**20


@pytest.mark.parametrize("bad,code", [(dict(bits=5), -2), (dict(group=24), -2), (dict(max_seq=100), -2), (dict(n_q_heads=12), -2),
                                      (dict(head_dim=32), -3), (dict(bits=3, head_dim=64, hidden=512), -3),
                                      (dict(channels=(9999,)), -2)])
def test_bad_configs(bad, code):
    good = dict(batch=1, n_q_heads=8, n_kv_heads=8, head_dim=64, hidden=512, bits=4, group=32, max_seq=256, topk=2, pfn_n=1,
                channels=(1,))
    with pytest.raises(kv.KvsinkError) as e:
        kv.cache_sizes(kv.Config(**{**good, **bad}))
    assert e.value.code == code


def test_null_and_misaligned_pointers_are_refused_before_any_launch():
    lib = binding.lib()
    cfg = kv.Config(1, 8, 8, 64, 512, 4, 32, 256, 2, 1, (1,)).c()
    null = C.c_void_p(0)
    assert lib.kvsink_predict_sinks(C.byref(cfg), null, 10, C.c_int64(0), C.c_int64(512), null, null, null, null, C.c_size_t(0), null) == -1
    cache = binding._Cache()
    assert lib.kvsink_quantize_append(C.byref(cfg), C.byref(cache), null, null, 1, C.c_int64(0), C.c_int64(0), C.c_int64(64), null) == -1
    assert lib.kvsink_decode_attention(C.byref(cfg), C.byref(cache), null, null, null, null, C.c_size_t(0), null) == -1
    assert lib.kvsink_cache_sizes(None, None) == -1
    assert b"unknown" in lib.kvsink_strerror(12345)
