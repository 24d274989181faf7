"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI.

Integer and byte results (mask, positions, counts, packed codes, scale / zero bit patterns, side buffer, tail)
must be identical; attention must satisfy |gpu - oracle| <= 2e-3 + 1e-2 |oracle|."""
import numpy as np
import pytest
import torch

import oracle
import paper_2508_04257_b200 as kv
from paper_2508_04257_b200 import synth

from parity_util import assert_close, bits_equal, compare_cache, compare_sinks, configs, np16, run_both

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


def test_tiny_workload_with_appends():
    r = run_both(TINY, appends=3)
    assert r["gpu_cache"].seq_len == TINY.seq + 3


@pytest.mark.parametrize("bits,d,group", [(2, 128, 128), (3, 128, 64), (4, 128, 64), (2, 64, 32), (4, 64, 32), (4, 64, 16),
                                          (2, 128, 32), (3, 128, 128), (4, 128, 256)])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (6, 2), (16, 2), (12, 1)])
def test_grid_of_shapes(bits, d, group, hq, hkv):
    # several groups and tiles plus a ragged remainder; sinks at token 0, mid sequence and inside the remainder
    seq = 3 * group + 37
    wl = TINY.scaled(bits=bits, head_dim=d, group=group, n_q_heads=hq, n_kv_heads=hkv, batch=2, seq=seq, topk=5, pfn_n=2,
                     seed=1000 + bits * 100 + d + group + hq)
    run_both(wl, appends=2)


@pytest.mark.parametrize("seq", [1, 15, 16, 17, 31, 32, 33, 64, 95, 96])
def test_short_and_ragged_lengths(seq):
    wl = TINY.scaled(seq=seq, topk=min(2, seq), batch=2, group=32, bits=2, seed=77 + seq)
    run_both(wl, appends=1, max_seq=128)


def test_appends_across_a_group_boundary():
    wl = TINY.scaled(seq=90, group=32, bits=3, head_dim=128, n_q_heads=4, n_kv_heads=2, batch=2, seed=5)
    r = run_both(wl, appends=8, max_seq=128)          # crosses 96 = 3 * 32
    assert r["gpu_cache"].seq_len == 98


@pytest.mark.parametrize("bits,group,chunks", [(2, 32, (50, 7, 1, 70, 33)), (4, 64, (10, 200, 5, 59, 1, 64)), (3, 64, (63, 1, 64, 65)),
                                               (2, 128, (100, 300, 28, 84))])
def test_chunked_prefill(bits, group, chunks):
    # chunks that start and end inside key groups, complete open groups, and span several groups: every state equals
    # the oracle's token-by-token cache
    total = sum(chunks)
    wl = TINY.scaled(seq=total, group=group, bits=bits, head_dim=128, n_q_heads=4, n_kv_heads=2, batch=2, topk=6, pfn_n=2, seed=31 + bits + group)
    ocfg, gcfg = configs(wl)
    H = synth.make_hidden(wl, "cuda")
    K, V = synth.make_kv(wl, 0, "cuda")
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    gc = kv.KVCache(gcfg, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    oc = oracle.Cache(ocfg, bm, pos, cnt)
    at = 0
    for n in chunks:
        kv.quantize_append(gcfg, gc, K[:, :, at:at + n], V[:, :, at:at + n])
        oracle.quantize_append(ocfg, oc, np16(K[:, :, at:at + n]), np16(V[:, :, at:at + n]))
        at += n
        compare_cache(gc, oc, wl, f"after {at} tokens: ")
    q = synth.make_query(wl, K)
    out, _ = kv.decode_attention(gcfg, gc, q)
    ref, _ = oracle.decode_attention(ocfg, oc, np16(q))
    assert_close(out.cpu().numpy(), ref, "attention")
    assert kv.read_status(gc) == 0


def test_append_from_an_empty_cache():
    wl = TINY.scaled(seq=0, topk=0, pfn_n=0, group=16, bits=4, batch=1, seed=6)
    ocfg, gcfg = configs(wl, 64)
    gc, oc = kv.KVCache(gcfg), oracle.Cache(ocfg)
    for step in range(35):
        k1, v1 = synth.make_new_token(wl, 0, step, "cuda")
        kv.quantize_append(gcfg, gc, k1, v1)
        oracle.quantize_append(ocfg, oc, np16(k1), np16(v1))
    compare_cache(gc, oc, wl)
    q = torch.randn((wl.batch, wl.n_q_heads, wl.head_dim), device="cuda", generator=torch.Generator("cuda").manual_seed(1)).half()
    out, lse = kv.decode_attention(gcfg, gc, q)
    ref, _ = oracle.decode_attention(ocfg, oc, np16(q))
    assert_close(out.cpu().numpy(), ref, "attention")


@pytest.mark.parametrize("topk,pfn", [(0, 0), (0, 4), (300, 0), (1, 300), (40, 3)])
def test_degenerate_sink_budgets(topk, pfn):
    wl = TINY.scaled(seq=150, topk=topk, pfn_n=pfn, group=32, bits=2, batch=2, seed=9 + topk)
    # planted outliers only make sense for small k; other budgets select among ordinary tokens (many near-ties)
    planted = TINY.scaled(seq=150, topk=min(topk, 3), pfn_n=pfn, group=32, bits=2, batch=2, seed=9 + topk)
    H = synth.make_hidden(planted, "cuda")
    K, V = synth.make_kv(planted, 0, "cuda")
    run_both(wl, appends=1, H=H, K=K, V=V, max_seq=160)


def test_ties_in_the_score_go_to_the_lower_index():
    wl = TINY.scaled(seq=200, topk=9, pfn_n=1, batch=3, seed=3)
    g = torch.Generator("cuda").manual_seed(4)
    H = (torch.randint(-5, 6, (wl.batch, wl.seq, wl.hidden), device="cuda", generator=g).half() * 0.5)
    run_both(wl, H=H)
    wl0 = wl.scaled(channels=())          # no listed channel: maximum over all d
    run_both(wl0, H=H)


@pytest.mark.parametrize("seq,topk,pfn", [(40000, 300, 3), (8193, 1, 0), (16384, 0, 5), (70001, 5000, 0), (262144, 17, 1), (300000, 40, 2)])
def test_long_sequences_with_many_ties(seq, topk, pfn):
    # sequences long enough for the multi-block selection (and one beyond it): small integer scores, so that the k-th
    # largest value is shared by thousands of tokens and the index tie-break decides across block boundaries
    wl = TINY.scaled(seq=seq, topk=topk, pfn_n=pfn, batch=2, hidden=64, channels=(5, 9), seed=seq)
    ocfg, gcfg = configs(wl)
    g = torch.Generator("cuda").manual_seed(seq)
    H = (torch.randint(-6, 7, (wl.batch, wl.seq, wl.hidden), device="cuda", generator=g).half() * 0.5)
    gs = kv.SinkSet(gcfg)
    kv.predict_sinks(gcfg, H, gs)
    bm, pos, cnt = oracle.predict_sinks(ocfg, np16(H))
    compare_sinks(gs, bm, pos, cnt, topk + pfn)


def test_nan_and_infinity_in_the_hidden_state():
    # an infinite value outranks every finite one; a NaN never raises a token's score (the comparison |x| > best is false)
    wl = TINY.scaled(seq=200, topk=4, pfn_n=1, batch=2, seed=21)
    H = synth.make_hidden(wl, "cuda")
    c0, c1 = wl.channels[0], wl.channels[1]
    H[0, 50, c0] = float("nan")
    H[0, 60, c1] = float("inf")
    H[1, 70, c0] = float("-inf")
    H[1, 71, c0] = float("nan")
    H[1, 71, c1] = 3.0
    r = run_both(wl, H=H)
    pos = r["oracle_cache"].sink_pos.reshape(wl.batch, -1)
    assert 60 in pos[0] and 50 not in pos[0] and 70 in pos[1]
    run_both(wl.scaled(channels=()), H=H)


def test_constant_groups_negative_zero_and_extremes():
    wl = TINY.scaled(seq=128, group=32, bits=4, batch=1, n_q_heads=2, n_kv_heads=2, seed=8)
    K, V = synth.make_kv(wl, 0, "cuda")
    K[:, :, :, 3] = 2.5            # constant channel
    K[:, :, :, 4] = 0.0
    K[:, :, 32:64, 5] = -0.0
    K[:, :, :, 6] = 60000.0
    K[:, :, 1::2, 6] = -60000.0    # widest range fp16 allows
    K[:, :, :, 7] = 6e-8           # subnormal
    V[:, :, 10, :] = -7.0          # constant row
    V[:, :, 11, :] = 0.0
    V[:, :, 12, ::2] = 1000.0
    K[:, :, :, 8] = 300.0 + torch.arange(128, device="cuda").half() * 0.25   # far from zero: large |zero|
    run_both(wl, K=K, V=V)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("hq,hkv", [(2, 2), (8, 2), (16, 2)])
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_wide_factor_range(bits, hq, hkv, seed):
    # head_dim 128; one, four and eight query heads per KV head (the three key-side paths): channels whose q * scale differ by several orders of magnitude
    # (one 300 times louder, one 1000 times quieter than the rest), large zero-points (a ramp far from zero, and seeded
    # noise of 0.01 around -40, |zero| ~ 1e4), constant and zero channels
    wl = TINY.scaled(seq=160, group=32, bits=bits, head_dim=128, batch=2, n_q_heads=hq, n_kv_heads=hkv, seed=500 + seed)
    K, V = synth.make_kv(wl, 0, "cuda")
    g = torch.Generator("cuda").manual_seed(seed)
    K[:, :, :, 3] = 2.5
    K[:, :, :, 4] = 0.0
    K[:, :, :, 6] *= 300.0
    K[:, :, :, 70] *= 1e-3
    K[:, :, :, 8] = 300.0 + torch.arange(160, device="cuda").half() * 0.25
    K[:, :, :, 100] = -40.0 + torch.randn(160, device="cuda", generator=g).half() * 0.01
    run_both(wl, K=K, V=V)


def test_bit_identical_across_runs_and_split_counts():
    wl = TINY.scaled(seq=32 * 40 + 5, group=32, bits=2, head_dim=128, n_q_heads=4, n_kv_heads=1, batch=1, topk=20, seed=12)
    r1 = run_both(wl)
    out2, lse2 = kv.decode_attention(configs(wl)[1], r1["gpu_cache"], r1["q"])
    assert bits_equal(out2.cpu().numpy(), r1["out"].cpu().numpy())      # deterministic merge
    # the same cache seen with more units (so fewer splits per unit): results agree to rounding
    wl8 = wl.scaled(batch=8)
    r8 = run_both(wl8)
    assert r8["err"] < 2e-3


def test_strided_inputs():
    wl = TINY.scaled(seq=100, group=32, bits=2, batch=2, seed=14)
    K, V = synth.make_kv(wl, 0, "cuda")
    big_k = torch.zeros((wl.batch, wl.n_kv_heads, wl.seq + 8, wl.head_dim + 64), dtype=torch.float16, device="cuda")
    big_v = torch.zeros_like(big_k)
    big_k[:, :, :wl.seq, :wl.head_dim] = K
    big_v[:, :, :wl.seq, :wl.head_dim] = V
    run_both(wl, K=big_k[:, :, :wl.seq, :wl.head_dim], V=big_v[:, :, :wl.seq, :wl.head_dim])
    # [B, S, H, D] storage viewed as [B, H, S, D]
    kt = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vt = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    run_both(wl, K=kt, V=vt)


@pytest.mark.parametrize("bits,group", [(2, 128), (2, 64), (3, 64), (4, 64), (4, 128)])
def test_bulk_append_kernel_strided_and_sink_dense(bits, group):
    # head_dim 128 with whole groups takes the tensor-map kernel: padded rows, [B, S, H, D] storage, and a prompt in
    # which a third of the tokens are sinks (runs that straddle tile and group boundaries, one group of sinks only)
    wl = TINY.scaled(bits=bits, head_dim=128, group=group, n_q_heads=6, n_kv_heads=3, batch=2, seq=5 * group + 9, topk=5,
                     pfn_n=2, seed=4000 + bits * 10 + group)
    K, V = synth.make_kv(wl, 0, "cuda")
    big_k = torch.zeros((wl.batch, wl.n_kv_heads, wl.seq + 8, wl.head_dim + 64), dtype=torch.float16, device="cuda")
    big_v = torch.zeros_like(big_k)
    big_k[:, :, :wl.seq, :wl.head_dim] = K
    big_v[:, :, :wl.seq, :wl.head_dim] = V
    run_both(wl, K=big_k[:, :, :wl.seq, :wl.head_dim], V=big_v[:, :, :wl.seq, :wl.head_dim], appends=1)
    kt = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vt = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    run_both(wl, K=kt, V=vt)
    dense = wl.scaled(topk=wl.seq // 3, pfn_n=group + 3, seed=wl.seed + 1)    # first-N covers the whole first group
    run_both(dense, appends=1)


@pytest.mark.parametrize("bits,group,n_groups", [(2, 128, 1), (2, 64, 2), (3, 64, 1), (4, 128, 2)])
def test_bulk_append_kernel_smallest_launches(bits, group, n_groups):
    # one sequence, one KV head: fewer work items than one block has warps, extents of 1 in the tensor map
    wl = TINY.scaled(bits=bits, head_dim=128, group=group, n_q_heads=1, n_kv_heads=1, batch=1, seq=n_groups * group, topk=3,
                     pfn_n=1, seed=5000 + bits * 10 + group)
    run_both(wl, appends=1)


@pytest.mark.parametrize("hq,hkv,batch,groups", [(16, 16, 8, 24), (8, 4, 12, 40), (4, 4, 3, 33)])
def test_decode_split_counts_that_merge_inside_a_cluster(hq, hkv, batch, groups):
    # enough (sequence, KV head) units that a unit gets two to eight sequence splits: those run as one thread-block
    # cluster and merge through distributed shared memory instead of the merge kernel
    wl = TINY.scaled(bits=2, head_dim=128, group=32, n_q_heads=hq, n_kv_heads=hkv, batch=batch, seq=32 * groups + 11, topk=6,
                     pfn_n=1, seed=6000 + hq + batch)
    r = run_both(wl, appends=1)
    out2, _ = kv.decode_attention(configs(wl)[1], r["gpu_cache"], r["q"])
    assert bits_equal(out2.cpu().numpy(), r["out"].cpu().numpy())      # the merge order is fixed
