"""kvsink_decode_attention_static: decode attention for callers that cannot allocate device memory (an engine
plug-in living inside someone else's memory plan, a loop that forbids allocation after start-up).  It must give
what kvsink_decode_attention gives with a caller workspace, on repeated calls that reuse the library's built-in
scratch array, and must refuse configurations whose split partials would not fit in that array.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import binding, synth

from parity_util import ATOL, RTOL


@pytest.mark.gpu
def test_static_scratch_matches_the_workspace_entry_point_twice_in_a_row():
    # one KV head and a long sequence: many sequence splits, so the scratch array really carries partials
    wl = synth.WORKLOADS["tiny"].scaled(seq=32 * 60 + 9, group=32, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=1, batch=2,
                                         topk=12, pfn_n=1, seed=4242)
    cfg = kv.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq, wl.topk, wl.pfn_n,
                    wl.channels)
    assert kv.cache_sizes(cfg)["decode_workspace_bytes"] <= binding.STATIC_SCRATCH_BYTES
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    sinks = kv.SinkSet(cfg)
    kv.predict_sinks(cfg, H, sinks)
    cache = kv.KVCache(cfg, sinks)
    kv.quantize_append(cfg, cache, K, V)
    shape = (wl.batch, wl.n_q_heads, wl.head_dim)
    for call in range(2):                                   # the second call finds the first call's partials in the array
        q = synth.make_query(wl, K, 0, call)
        ref, ref_lse = kv.decode_attention(cfg, cache, q)
        out = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full(shape[:2], float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        if call == 1:       # the first call has made the one-time address lookup; from now on device memory must not move
            free_before, allocs_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_stats()["allocation.all.allocated"]
        kv.decode_attention_static(cfg, cache, q, out, lse)
        torch.cuda.synchronize()
        if call == 1:
            # no device memory was taken from the driver and no tensor was allocated during the call
            assert torch.cuda.mem_get_info()[0] >= free_before
            assert torch.cuda.memory_stats()["allocation.all.allocated"] == allocs_before
        o, r = out.cpu().numpy(), ref.cpu().numpy()
        assert np.all(np.isfinite(o))
        assert np.all(np.abs(o - r) <= ATOL + RTOL * np.abs(r)), f"call {call}: max diff {np.abs(o - r).max():.3e}"
        assert np.allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), atol=ATOL, rtol=1e-3)
    assert kv.read_status(cache) == 0


def test_static_scratch_refuses_what_does_not_fit():
    # 64 units (4 bit: eight query heads share a block) x up to 19 splits x 64 query heads x 130 floats > 4 MiB: refused on the
    # host, before any launch
    cfg = kv.Config(8, 64, 8, 128, 4096, 4, 128, 32768, 4, 1, (1,))
    assert kv.cache_sizes(cfg)["decode_workspace_bytes"] > binding.STATIC_SCRATCH_BYTES
    cache = binding._Cache()
    rc = binding.lib().kvsink_decode_attention_static(C.byref(cfg.c()), C.byref(cache), None, None, None, None)
    assert rc == -9
    assert "scratch" in kv.strerror(rc)
