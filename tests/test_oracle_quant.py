"""Pins for the oracle's quantizer (Eq. 8-11, Appendix C) and its sink exclusion (Algorithm 1).

None of these re-types the oracle's binary32 formula: they check what the mathematics fixes -- the
round-to-nearest error bound, exact rational re-derivation of the parameters and of every code that is not
within rounding distance of a tie, the fate of the group's extremes, self-reproducing constant groups,
bit-exact preservation of sink rows -- plus the direction of the paper's observation that sink tokens inside
a per-channel key group raise the group's error (Section 4.1, Table 1).
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2508_04257_b200 import synth


def _f32_nearest(fr: Fraction) -> np.float32:
    """Correctly rounded binary32 of an exact rational (via candidates around the double approximation)."""
    c = np.float32(float(fr))
    cands = [np.nextafter(c, np.float32(-np.inf)), c, np.nextafter(c, np.float32(np.inf))]
    best = min(cands, key=lambda v: (abs(Fraction(float(v)) - fr), int(np.float32(v).view(np.uint32)) & 1))
    return np.float32(best)


def _round_half_even(fr: Fraction) -> int:
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2):
        return fl + 1
    if rem < Fraction(1, 2):
        return fl
    return fl if fl % 2 == 0 else fl + 1


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("kind", ["normal", "offset", "tiny_range", "wide"])
def test_group_against_exact_rationals(bits, kind):
    rng = np.random.default_rng(100 * bits + len(kind))
    qmax = (1 << bits) - 1
    checked = 0
    for trial in range(40):
        n = int(rng.choice([16, 32, 64, 128]))
        x = rng.standard_normal(n)
        if kind == "offset":
            x = x + rng.uniform(-40, 40)
        elif kind == "tiny_range":
            x = 3.0 + x * 1e-2
        elif kind == "wide":
            x = x * 3000.0
        x = x.astype(np.float16).astype(np.float32)
        member = (rng.random(n) > 0.1).astype(np.uint8)
        if member.sum() < 2:
            member[:2] = 1
        scale, zero, codes = oracle.quantize_group(x, member, bits)
        xm = x[member == 1]
        mn, mx = Fraction(float(xm.min())), Fraction(float(xm.max()))
        if mx == mn:
            continue
        # Eq. 10: scale is the binary32 nearest to fl32(max-min) / qmax
        r32 = _f32_nearest(mx - mn)
        assert scale == _f32_nearest(Fraction(float(r32)) / qmax)
        s = Fraction(float(scale))
        # Eq. 11: zero = -round(fl32(min/scale)), an integer
        assert zero == -_round_half_even(Fraction(float(_f32_nearest(mn / s))))
        z = int(zero)
        for j in range(n):
            if not member[j]:
                assert codes[j] == 0
                continue
            q = Fraction(float(x[j])) / s
            # Eq. 8 in exact arithmetic, wherever binary32 rounding of the quotient cannot move it across a tie
            dist_to_tie = abs(q - (Fraction(2 * (q.numerator // q.denominator) + 1, 2)))
            if dist_to_tie > abs(q) * Fraction(1, 1 << 22):
                want = min(max(_round_half_even(q) + z, 0), qmax)
                assert codes[j] == want, (x[j], float(scale), z, codes[j], want)
                checked += 1
            # Eq. 9 and the round-to-nearest bound |x - x'| <= scale/2 (+ binary32 rounding of the quotient)
            xr = s * (int(codes[j]) - z)
            assert abs(Fraction(float(x[j])) - xr) <= s / 2 + abs(Fraction(float(x[j]))) * Fraction(1, 1 << 22)
            assert 0 <= codes[j] <= qmax
        # the minimum maps to code 0 and the maximum to one of the two top codes
        assert codes[member == 1][np.argmin(xm)] == 0
        assert codes[member == 1][np.argmax(xm)] >= qmax - 1
    assert checked > 500


def test_tie_rounds_to_even_and_clamp_catches_the_extra_step():
    # min/scale = 0.5 exactly: scale = 1 (range 3, 2 bit), values 0.5, 1.5, 2.5, 3.5.
    x = np.array([0.5, 1.5, 2.5, 3.5], np.float32)
    scale, zero, codes = oracle.quantize_group(x, np.ones(4, np.uint8), 2)
    assert scale == 1.0 and zero == 0.0          # rint(0.5) = 0
    assert codes.tolist() == [0, 2, 2, 3]        # rint: 0, 2, 2, 4 -> clamp(4) = 3
    for xv, c in zip(x, codes):
        assert abs(xv - scale * (c - zero)) <= scale / 2


def test_constant_and_empty_groups():
    for v in (0.0, -0.0, 2.5, -7.0, 6.1e-5):
        x = np.full(32, v, np.float32)
        scale, zero, codes = oracle.quantize_group(x, np.ones(32, np.uint8), 4)
        assert scale > 0 and np.all(scale * (codes.astype(np.float32) - zero) == np.float32(v))
        assert np.signbit(zero) == False or zero != 0  # a zero zero-point is +0
    scale, zero, codes = oracle.quantize_group(np.arange(8, dtype=np.float32), np.zeros(8, np.uint8), 3)
    assert scale == 0 and zero == 0 and not codes.any()


def test_zero_point_is_unclamped_when_the_range_excludes_zero():
    x = np.linspace(10.0, 10.75, 16).astype(np.float16).astype(np.float32)
    scale, zero, codes = oracle.quantize_group(x, np.ones(16, np.uint8), 2)
    assert zero == -40.0 and scale == 0.25
    assert np.max(np.abs(scale * (codes - zero) - x)) <= scale / 2


def _tiny_case(bits=4, group=32, seq=256, topk=2, pfn=1, d=64, heads=2, batch=2, seed=3):
    wl = synth.WORKLOADS["tiny"].scaled(bits=bits, group=group, seq=seq, topk=topk, pfn_n=pfn, head_dim=d, n_q_heads=heads,
                                         n_kv_heads=heads, batch=batch, seed=seed)
    cfg = oracle.Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.hidden, wl.bits, wl.group, wl.max_seq,
                        wl.topk, wl.pfn_n, wl.channels)
    H = synth.make_hidden(wl).numpy()
    K, V = [t.numpy() for t in synth.make_kv(wl)]
    return wl, cfg, H, K, V


@pytest.mark.parametrize("bits,group,d", [(4, 32, 64), (2, 64, 128), (3, 64, 128), (2, 128, 128), (4, 16, 64)])
def test_cache_round_trip_error_bound_and_exact_sinks(bits, group, d):
    wl, cfg, H, K, V = _tiny_case(bits=bits, group=group, d=d, seq=4 * group + 21)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    cache = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, cache, K, V)
    assert cache.seq_len == wl.seq
    kd, vd = oracle.dequant_dense(cfg, cache)
    n_body = (wl.seq // group) * group
    gv = min(group, d)
    ks = cache.k_scale.reshape(wl.batch, wl.n_kv_heads, wl.max_seq // group, d)
    vs = cache.v_scale.reshape(wl.batch, wl.n_kv_heads, wl.max_seq, d // gv)
    for b in range(wl.batch):
        sinks = set(pos[b, :cnt[b]].tolist())
        assert 0 in sinks and len(sinks) == cnt[b]
        for p in range(wl.seq):
            k0, v0 = K[b, :, p].astype(np.float64), V[b, :, p].astype(np.float64)
            if p in sinks or p >= n_body:
                assert np.array_equal(kd[b, :, p], k0)          # fp16 rows come back bit for bit
            else:
                bound = ks[b, :, p // group] / 2 * (1 + 1e-6) + np.abs(k0) * 2.0**-22
                assert np.all(np.abs(kd[b, :, p] - k0) <= bound)
            if p in sinks:
                assert np.array_equal(vd[b, :, p], v0)
            else:
                bound = np.repeat(vs[b, :, p], gv, axis=-1) / 2 * (1 + 1e-6) + np.abs(v0) * 2.0**-22
                assert np.all(np.abs(vd[b, :, p] - v0) <= bound)
    # side buffer holds the exact rows in rank order
    cap = cfg.topk + cfg.pfn_n
    sk = cache.sink_k.reshape(wl.batch, wl.n_kv_heads, cap, d)
    for b in range(wl.batch):
        for j in range(cnt[b]):
            assert np.array_equal(sk[b, :, j], K[b, :, pos[b, j]].view(np.uint16))


def test_one_token_at_a_time_equals_bulk_prefill():
    wl, cfg, H, K, V = _tiny_case(bits=2, group=32, d=64, seq=75)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    a = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, a, K, V)
    b = oracle.Cache(cfg, bm, pos, cnt)
    for t in range(wl.seq):
        oracle.quantize_append(cfg, b, K[:, :, t:t + 1], V[:, :, t:t + 1])
    for name in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero", "sink_k", "sink_v"):
        assert np.array_equal(getattr(a, name), getattr(b, name)), name


def test_excluding_sinks_lowers_per_channel_key_error():
    """Direction of Section 4.1 / Table 1: key groups that contain a sink token quantize worse when the sink's
    small-norm row takes part in the channel statistics (keys have per-channel offsets)."""
    wl, cfg, H, K, V = _tiny_case(bits=2, group=32, d=64, seq=256, topk=6, batch=1)
    rng = np.random.default_rng(5)
    off = rng.uniform(3, 8, size=(1, wl.n_kv_heads, 1, wl.head_dim)) * rng.choice([-1, 1], size=(1, wl.n_kv_heads, 1, wl.head_dim))
    K = (K.astype(np.float32) + off).astype(np.float16)
    bm, pos, cnt = oracle.predict_sinks(cfg, H)
    for p in pos[0, :cnt[0]]:
        K[0, :, p] = (K[0, :, p].astype(np.float32) * 0.02).astype(np.float16)   # QKV suppression
    with_excl = oracle.Cache(cfg, bm, pos, cnt)
    oracle.quantize_append(cfg, with_excl, K, V)
    no_excl = oracle.Cache(cfg)     # empty mask: sinks take part in the statistics
    oracle.quantize_append(cfg, no_excl, K, V)
    ka, _ = oracle.dequant_dense(cfg, with_excl)
    kb, _ = oracle.dequant_dense(cfg, no_excl)
    sinks = pos[0, :cnt[0]]
    groups = np.unique(sinks // wl.group)
    err_a = err_b = 0.0
    for g in groups:
        toks = [p for p in range(g * wl.group, (g + 1) * wl.group) if p not in set(sinks.tolist())]
        ref = K[0][:, toks].astype(np.float64)
        err_a += np.mean((ka[0][:, toks] - ref) ** 2)
        err_b += np.mean((kb[0][:, toks] - ref) ** 2)
    assert err_a < 0.5 * err_b
