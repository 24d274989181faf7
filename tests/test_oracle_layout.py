"""Pins for the physical order of packed codes.  The paper does not fix a byte order; the library stores a
16-token tile as the register image of the 16x16 A operand of the m16n8k16 tensor-core instruction.  The test
decodes the oracle's bytes lane by lane from the published fragment table (row = lane/4 (+8 for registers 1
and 3), col = 2*(lane%4) + half (+8 for registers 2 and 3)) and the documented bit positions, and must find
the codes it planted; plus pack/unpack identity through the oracle's own reader, and a committed hash."""
import hashlib
import os

import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


def _lane_word(tile_words, n_words, lane, i, base=0):
    """Word i of a lane inside a section of n_words per lane stored as planes of up to four words."""
    off, p = base, i // 4
    for pp in range(p):
        off += 32 * min(4, n_words - 4 * pp)
    u = min(4, n_words - 4 * p)
    return int(tile_words[off + u * lane + (i - 4 * p)])


def _fragment_decode(tile_words, D, bits):
    """[D/16][16][16] codes, indexed [matrix][row][col], read the way a warp's lanes own the A operand."""
    out = np.zeros((D // 16, 16, 16), np.int64)
    for lane in range(32):
        g, t = lane // 4, lane % 4
        for m in range(D // 16):
            for r in range(4):
                for e in range(2):
                    row, col = g + 8 * (r % 2), 2 * t + e + 8 * (r // 2)
                    s = 4 * m + r
                    if bits == 2:
                        w = _lane_word(tile_words, D // 32, lane, s // 8)
                        code = (w >> (16 * e + 2 * (s % 8))) & 3
                    elif bits == 4:
                        w = _lane_word(tile_words, D // 16, lane, s // 4)
                        code = (w >> (16 * e + 4 * (s % 4))) & 15
                    else:
                        i, k = s // 8, s % 8
                        lo = (_lane_word(tile_words, D // 32, lane, i) >> (16 * e + 2 * k)) & 3
                        hw = _lane_word(tile_words, D // 64, lane, i // 2, base=32 * (D // 32))
                        hi = (hw >> (16 * e + 4 * (k // 2) + 2 * (1 - i % 2) + k % 2)) & 1
                        code = lo | (hi << 2)
                    out[m, row, col] = code
    return out


def _planted(bits, group, d, seq, heads=2, batch=2, seed=0):
    """K and V whose codes are known in advance: integers 0..qmax with both extremes in every group."""
    rng = np.random.default_rng(seed)
    qmax = (1 << bits) - 1
    K = rng.integers(0, qmax + 1, size=(batch, heads, seq, d))
    V = rng.integers(0, qmax + 1, size=(batch, heads, seq, d))
    gv = min(group, d)
    for g0 in range(0, seq - group + 1, group):       # per channel, per token group: force 0 and qmax
        K[:, :, g0] = 0
        K[:, :, g0 + 1] = qmax
    for c0 in range(0, d, gv):                        # per token, per channel group
        V[..., c0] = 0
        V[..., c0 + 1] = qmax
    return K.astype(np.float16), V.astype(np.float16)


@pytest.mark.parametrize("bits,group,d", [(2, 32, 64), (2, 128, 128), (3, 64, 128), (4, 32, 64), (4, 64, 128)])
def test_tile_is_the_a_fragment_image(bits, group, d):
    batch, heads, seq = 2, 2, 2 * group
    cfg = oracle.Config(batch, heads, heads, d, 64, bits, group, seq, 0, 0, (0,))
    K, V = _planted(bits, group, d, seq, heads, batch, seed=bits * 7 + d)
    cache = oracle.Cache(cfg)
    oracle.quantize_append(cfg, cache, K, V)
    assert np.all(cache.k_scale == 1) and np.all(cache.k_zero == 0) and np.all(cache.v_scale == 1)
    tile_words = 16 * d * bits // 32
    kw = cache.k_codes.view(np.uint32).reshape(batch, heads, seq // 16, tile_words)
    vw = cache.v_codes.view(np.uint32).reshape(batch, heads, seq // 16, tile_words)
    for b in range(batch):
        for h in range(heads):
            for tile in range(seq // 16):
                kt = _fragment_decode(kw[b, h, tile], d, bits)        # [m][token][channel%16]
                want = K[b, h, 16 * tile:16 * tile + 16].astype(np.int64).reshape(16, d // 16, 16).transpose(1, 0, 2)
                assert np.array_equal(kt, want)
                vt = _fragment_decode(vw[b, h, tile], d, bits)        # [m][channel%16][token]
                want = V[b, h, 16 * tile:16 * tile + 16].astype(np.int64).reshape(16, d // 16, 16).transpose(1, 2, 0)
                assert np.array_equal(vt, want)
    # the oracle's own reader agrees (pack -> unpack identity)
    assert np.array_equal(oracle.unpack_codes(cfg, cache.k_codes, "k", seq), K.astype(np.int8))
    assert np.array_equal(oracle.unpack_codes(cfg, cache.v_codes, "v", seq), V.astype(np.int8))


def golden_digest():
    """sha256 over every oracle output for the tiny workload on integer-hash inputs (no torch RNG involved)."""
    wl = synth.WORKLOADS["tiny"]
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq,
                        wl.topk, wl.pfn_n, wl.channels)
    H = synth.hash_half((wl.batch, wl.seq, wl.hidden), 1)
    H[0, 0, list(wl.channels)] = np.float16(500.0)
    H[0, 97, list(wl.channels)] = np.float16(-512.0)
    K = synth.hash_half((wl.batch, wl.n_kv_heads, wl.seq, wl.head_dim), 2)
    V = synth.hash_half((wl.batch, wl.n_kv_heads, wl.seq, wl.head_dim), 3)
    q = synth.hash_half((wl.batch, wl.n_q_heads, wl.head_dim), 4)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    out, lse = oracle.decode_attention(cfg, cache, q)
    hsh = hashlib.sha256()
    for a in (bm, pos, cnt, cache.k_codes, cache.v_codes, cache.k_scale, cache.k_zero, cache.v_scale, cache.v_zero,
              cache.sink_k, cache.sink_v, cache.k_tail):
        hsh.update(np.ascontiguousarray(a).tobytes())
    hsh.update(np.round(out, 9).astype(np.float32).tobytes())   # attention: to 1e-9, immune to libm's last bit
    return hsh.hexdigest(), pos[0, :cnt[0]].tolist()


def test_committed_hash_of_the_tiny_workload():
    with open(os.path.join(HERE, "golden", "tiny_oracle_sha256.txt")) as f:
        lines = [l.strip() for l in f if l.strip() and not l.startswith("#")]
    digest, sinks = golden_digest()
    assert sinks == [0, 97]
    assert digest == lines[0]
