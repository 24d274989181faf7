// Whole-group quantization (Eq. 8-11 with Algorithm 1's sink exclusion) of a bulk append, fed by tensor-map bulk copies.
//
// One persistent block per SM whose warps never synchronise with one another.  Every warp owns one 8 KB stage of
// shared memory and walks over its own work items: lane 0 issues the item's bulk copies (hardware swizzle, completion
// on the warp's mbarrier), the warp waits for them, pulls the whole item into registers with ldmatrix, hands the stage
// to the copies of its next item at once, and then does statistics, parameters, coding and its global stores from
// registers while that item streams in.  Sixteen to twenty warps per SM keep 128-160 KB of copies in flight.
//
// An item is 4096 elements of one (sequence, KV head, token group):
//   keys   : 4096/G channels x G tokens   (per-channel statistics stay inside the warp)
//   values : 32 tokens x 128 channels     (per-token statistics stay inside the warp)
// ldmatrix (.trans for values, whose packed tiles are [channel x token]) gives each lane exactly the elements of its
// pair slots in the packed tile, so the registers that served the min/max pass are coded in place and the lane's
// packed words come out in the tile's own order.
//
// The copies are issued by one elected lane per warp.  (Issuing them from several lanes of one warp inside a
// divergent loop, and a ring of stages shared by all warps whose parity waits could run two phases ahead, were both
// tried and both faulted: every mbarrier here belongs to one warp and advances one phase per item.)
#include <cuda.h>   // CUtensorMap and its enums; the encoder itself is looked up through the runtime

#include <mutex>

#include "common.cuh"

namespace kvsink {
namespace {

constexpr int QB_D = 128;
constexpr int QB_STAGE_BYTES = 8192;
constexpr int QB_WAIT_LIMIT = 1 << 22;   // polls of an mbarrier before a warp gives up (far beyond any real latency)

__device__ __forceinline__ void qb_mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void qb_mbar_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool qb_mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool qb_wait(uint64_t *bar, unsigned parity)
{
    int polls = 0;
    while (!qb_mbar_try_wait(bar, parity))
        if (++polls > QB_WAIT_LIMIT) return false;
    return true;
}
// Tiled bulk copy global -> shared of one box of a rank-4 tensor map; completion is counted on `bar`.
// The innermost coordinate is a multiple of 8 elements (16 bytes).
__device__ __forceinline__ void qb_tma_load(void *dst, const CUtensorMap *tm, int c0, int c1, int c2, int c3, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(smem_addr(dst)), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void qb_ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void qb_ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// fp16 values in sorted order: sign-magnitude bit pattern <-> signed integer (both zeros map to 0).
constexpr int QB_OMAX = 0x7BFF;
__device__ __forceinline__ int qb_ord(unsigned b) { return (b & 0x8000u) ? -(int)(b & 0x7fffu) : (int)b; }
__device__ __forceinline__ unsigned qb_unord(int o) { return o >= 0 ? (unsigned)o : (0x8000u | (unsigned)(-o)); }
__device__ __forceinline__ float qb_val(int o) { return __half2float(__ushort_as_half((unsigned short)qb_unord(o))); }

// Bit pattern of the smallest finite fp16 value whose code reaches `level`, by bisection over all finite fp16 values
// with the literal formula; +inf if none does.  Only for the rare keys the closed form below cannot decide.
__device__ __noinline__ unsigned qb_threshold_search(float s, float z, float level, float qmax)
{
    int lo = -QB_OMAX, hi = QB_OMAX + 1;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((float)code_exact(qb_val(mid), s, z, qmax) >= level) hi = mid; else lo = mid + 1;
    }
    return lo > QB_OMAX ? 0x7C00u : qb_unord(lo);
}

// 2-bit coder by thresholds.  code(x) = clamp(rint(x / s) + z, 0, 3) is a non-decreasing step function of the fp16
// argument, so the smallest fp16 values t1 <= t2 <= t3 whose code reaches 1, 2, 3 describe it exactly and
// code(x) = [x >= t1] + [x >= t2] + [x >= t3].
//
// Threshold of one level, exactly and without a division.  With c = level - z (an integer) the code reaches the
// level iff rint(fl(x/s)) >= c.  The rounded quotient y = fl(x/s) is a binary32 number, so that holds iff y >= H with
// H = c - 1/2 when c is even (rint takes the tie to the even integer c) and H = the next binary32 number above
// c - 1/2 when c is odd.  Round-to-nearest division gives y >= H iff x/s lies above the midpoint M of H and its
// predecessor, or on it when H has an even mantissa.  M has 25 significant bits and s 24, so s * M is exact in
// binary64; the threshold is the first fp16 value at or above s * M, or the one after it when x/s == M is a tie
// that rounds down.
__device__ __forceinline__ unsigned qb_threshold(float s, double s_half, float z, float level, float qmax)
{
    if (s == 0.f) return 0x7C00u;                       // no member: every code is 0
    if (!(fabsf(z) < 4194304.f)) return qb_threshold_search(s, z, level, qmax);
    const float c = level - z, h = c - 0.5f, hc = c * 0.5f;     // all exact
    const unsigned hb = __float_as_uint(h);
    const float H = hc == rintf(hc) ? h : __uint_as_float(h > 0.f ? hb + 1u : hb - 1u);
    const unsigned Hb = __float_as_uint(H);
    const float H_dn = __uint_as_float(H > 0.f ? Hb - 1u : Hb + 1u);        // |H| >= 1/2: never zero
    const double sm = s_half * ((double)H + (double)H_dn);                  // s * M, exact
    const __half o = __float2half_ru(__double2float_ru(sm));                // first fp16 value >= s * M (+inf if none)
    unsigned t = __half_as_ushort(o);
    if ((double)__half2float(o) == sm && (Hb & 1u)) t = (t & 0x8000u) ? t - 1u : t + 1u;
    return t;
}

// acc + w * ([x >= t1] + [x >= t2] + [x >= t3]) on both halves.
__device__ __forceinline__ __half2 qb_thermo(__half2 acc, uint32_t x2, const __half2 (&t)[3], __half2 w)
{
    const __half2 x = *reinterpret_cast<const __half2 *>(&x2);
    const __half2 cnt = __hadd2(__hadd2(__hge2(x, t[0]), __hge2(x, t[1])), __hge2(x, t[2]));
    return __hfma2(cnt, w, acc);
}

__device__ __forceinline__ uint32_t qb_hmin2(uint32_t a, uint32_t b)
{
    __half2 r = __hmin2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}
__device__ __forceinline__ uint32_t qb_hmax2(uint32_t a, uint32_t b)
{
    __half2 r = __hmax2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}

// ---- 3- and 4-bit coder: rint(x / scale) + zero without a division per element ----
// y = fma(x, r, M + zero) with M = 1.5 * 2^23 rounds the product to an integer in the mantissa.  It is evaluated with
// r = 1/scale nudged down and up by 2^-22: where both agree no rounding of x/scale can fall on the other side of a tie
// and the agreed integer is the exact answer; where they differ the lane redoes that register with the IEEE division.
// The two elements of a register share one packed FMA per reciprocal; a matrix (four registers) is tested with one
// branch, and inside it only the registers that disagreed are redone.
constexpr float QB_MAGIC = 12582912.0f;   // 1.5 * 2^23
struct __align__(16) QbCoder {
    float r_lo, r_hi;   // 1/scale nudged down / up; r_lo = +inf forces the exact path
    float magic;        // M + zero
    float pad;
};
// mn, mx: the group's extremes.  The fast form is used only where it is provably exact: |x/scale| and |zero| far below
// 2^22 (integer in the mantissa) and the top code cannot exceed qmax (so no clamp is needed).
__device__ __forceinline__ QbCoder qb_make_coder(float scale, float zero, float mn, float mx, float qmax)
{
    QbCoder c;
    c.pad = 0.f;
    if (scale == 0.f) {   // no member, or sink token: code 0
        c.r_lo = c.r_hi = 0.f;
        c.magic = QB_MAGIC;
        return c;
    }
    const float r = __frcp_rn(scale);
    const float absmax = fmaxf(fabsf(mn), fabsf(mx));
    const bool top_fits = __fadd_rn(rintf(__fdiv_rn(mx, scale)), zero) <= qmax;
    const bool ok = absmax * r < 2097152.f && fabsf(zero) < 2097152.f && r < 3.0e38f && top_fits;
    c.r_lo = ok ? __fmul_rn(r, 1.f - 2.384185791015625e-07f) : __int_as_float(0x7f800000);
    c.r_hi = ok ? __fmul_rn(r, 1.f + 2.384185791015625e-07f) : r;
    c.magic = QB_MAGIC + (ok ? zero : 0.f);
    return c;
}
// Coder for a static pair (Eq. 8 with its clamp, values anywhere in fp16).  The argument is first clamped to fp16 bounds xl, xh
// whose own codes already saturate (unclamped code of xl <= -1, of xh >= qmax + 1: every value beyond them gets the same
// clamped code as the bound), which keeps the unclamped integer small enough for a signed 16-bit field; the packed codes are
// then clamped to [0, qmax] by one two-way 16-bit min/max.  Bounds beyond the fp16 range are infinite (no clamp needed).
__device__ __forceinline__ QbCoder qb_make_coder_static(float scale, float zero, float qmax, __half *xl, __half *xh)
{
    QbCoder c;
    c.pad = 0.f;
    *xl = __ushort_as_half((unsigned short)0xFC00);   // -inf
    *xh = __ushort_as_half((unsigned short)0x7C00);   // +inf
    if (scale == 0.f) {   // nothing was calibrated, or sink token: code 0
        c.r_lo = c.r_hi = 0.f;
        c.magic = QB_MAGIC;
        return c;
    }
    const float r = __frcp_rn(scale);
    const float lo_real = scale * (-zero - 2.f), hi_real = scale * (qmax - zero + 2.f);
    *xl = __float2half_rd(lo_real);
    *xh = __float2half_ru(hi_real);
    const float reach = fmaxf(fminf(fabsf(lo_real), 65504.f), fminf(fabsf(hi_real), 65504.f));   // largest |argument| after the clamp
    // NaN in any of these makes the comparison false: exact path
    const bool ok = reach * r + fabsf(zero) < 30000.f && r < 3.0e38f;
    c.r_lo = ok ? __fmul_rn(r, 1.f - 2.384185791015625e-07f) : __int_as_float(0x7f800000);
    c.r_hi = ok ? __fmul_rn(r, 1.f + 2.384185791015625e-07f) : r;
    c.magic = QB_MAGIC + (ok ? zero : 0.f);
    return c;
}
// The coders of two adjacent keys (the two elements of a half2 register), field by field, so that each field is the
// operand pair of one packed fp32 FMA.
struct __align__(16) QbCoder2 {
    float r_lo[2], r_hi[2];
    float magic[2], pad[2];
};
__device__ __forceinline__ unsigned long long qb_pair(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
// Codes of the two elements of a half2 register -> (code_lo | code_hi << 16); `differ` collects disagreement bits.
// Both elements go through one packed FMA per nudged reciprocal (fma.rn.f32x2: two IEEE FMAs, one instruction).
__device__ __forceinline__ uint32_t qb_code_pair(uint32_t h2, unsigned long long r_lo, unsigned long long r_hi, unsigned long long magic,
                                                 uint32_t &differ)
{
    const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const unsigned long long xx = qb_pair(x.x, x.y);
    unsigned long long a, b;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(a) : "l"(xx), "l"(r_lo), "l"(magic));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(b) : "l"(xx), "l"(r_hi), "l"(magic));
    uint32_t a0, a1, b0, b1;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a0), "=r"(a1) : "l"(a));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(b0), "=r"(b1) : "l"(b));
    differ |= (a0 ^ b0) | (a1 ^ b1);
    // low halves of the two results (the bit pattern of 1.5 * 2^23 has a zero low half)
    return __byte_perm(a0, a1, 0x5410);
}
__device__ __noinline__ uint32_t qb_code_pair_exact(uint32_t h2, float s0, float z0, float s1, float z1, float qmax)
{
    const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const uint32_t c0 = s0 == 0.f ? 0u : code_exact(x.x, s0, z0, qmax);
    const uint32_t c1 = s1 == 0.f ? 0u : code_exact(x.y, s1, z1, qmax);
    return c0 | (c1 << 16);
}
// Bits contributed by matrix m of a tile to a lane's words, from its four code pairs pc[r] (pair slots 4m + r).
//   4 bit: the whole word m in `lo`.
//   3 bit: the low two bits of the codes as a byte in each half of `lo` (byte m & 1 of each half of word m >> 1);
//          `hi` holds this matrix's bits of word m >> 2 of the second section, already in place.
template <int BITS>
__device__ __forceinline__ void qb_pack_matrix(const uint32_t (&pc)[4], int m, uint32_t *lo, uint32_t *hi)
{
    if constexpr (BITS == 4) {
        *lo = pc[0] | (pc[1] << 4) | (pc[2] << 8) | (pc[3] << 12);
        *hi = 0;
    } else {
        *lo = (pc[0] & 0x00030003u) | ((pc[1] & 0x00030003u) << 2) | ((pc[2] & 0x00030003u) << 4) | ((pc[3] & 0x00030003u) << 6);
        const uint32_t h = ((pc[0] >> 2) & 0x00010001u) | (((pc[1] >> 2) & 0x00010001u) << 1) | (((pc[2] >> 2) & 0x00010001u) << 4) |
                           (((pc[3] >> 2) & 0x00010001u) << 5);
        *hi = h << (8 * (m & 1) + 2 * (1 - ((m >> 1) & 1)));
    }
}

struct QbShape {
    int first_token, n_groups;
    unsigned n_items;
};

template <int G, int BITS = 2>
struct QbGeo {
    static constexpr int D = QB_D;
    static constexpr int KC = 4096 / G;           // channels of a key item
    static constexpr int MT = KC / 16;            // matrices per tile in a key item
    static constexpr int NT = G / 16;             // tiles per token group
    static constexpr int NK = D / KC;             // key items per group
    static constexpr int NV = G / 32;             // value items per group (32 tokens each)
    static constexpr int IPG = NK + NV;           // items per group
    static constexpr int Gv = G < D ? G : D, NGv = D / Gv;
    static constexpr int NS = 2 * D / G;          // statistic sets per item: MT for keys, 2 * NGv for values
    static constexpr int KPL = NS / 2;            // keys per lane
    static constexpr int KROWB = 2 * KC;          // bytes per row of a key item in shared memory
    // per warp and for each of the item's 16 * NS keys: three fp16 thresholds (2 bit), or a coder (stored by key pair)
    // and (scale, zero)
    // (static pairs: also the two fp16 clamp bounds of every key)
    static constexpr int SCRATCH = BITS == 2 ? 3 * 16 * NS * 2 : 8 * NS * (int)sizeof(QbCoder2) + 16 * NS * (int)sizeof(float2) + 2 * 16 * NS * 2;
    static constexpr int TILE_BYTES = 256 * BITS, ROW_BYTES = 16 * BITS;   // packed tile of 16 tokens x 128 channels
    // warps per block, each with one stage, one mbarrier and its scratch: 20 (96 registers per thread) for the 2-bit
    // coder; 16 (128 registers) for the 3- and 4-bit coder, which spills at 96 and measures 9 % faster this way
    static constexpr int WARPS = BITS == 2 ? 20 : 16;
    static_assert(G == 64 || G == 128, "group size");
    static_assert(BITS != 3 || G == 64, "a 3-bit key item must cover whole words of the high-bit section (64 channels)");
    static_assert(MT == NS && 2 * NGv == NS, "statistic sets");
};

// Position of an item: sequence, KV head, token group and sub-item (keys: channel slab, then values: 32-token slab).
struct QbPos { int sub, grp, h, b; };

template <int G>
__device__ __forceinline__ QbPos qb_decode(unsigned id, int n_groups, int Hkv)
{
    QbPos q;
    q.sub = (int)(id % QbGeo<G>::IPG);
    unsigned ug = id / QbGeo<G>::IPG;
    q.grp = (int)(ug % (unsigned)n_groups); ug /= (unsigned)n_groups;
    q.h = (int)(ug % (unsigned)Hkv);
    q.b = (int)(ug / (unsigned)Hkv);
    return q;
}
// q + step as mixed-radix digits (every digit of step is below its radix).
template <int G>
__device__ __forceinline__ QbPos qb_advance(QbPos q, const QbPos &step, int n_groups, int Hkv)
{
    q.sub += step.sub; int cy = q.sub >= QbGeo<G>::IPG; q.sub -= cy ? QbGeo<G>::IPG : 0;
    q.grp += step.grp + cy; cy = q.grp >= n_groups; q.grp -= cy ? n_groups : 0;
    q.h += step.h + cy; cy = q.h >= Hkv; q.h -= cy ? Hkv : 0;
    q.b += step.b + cy;
    return q;
}

// Sink bits of an item's tokens (up to 128): G/32 words for keys, one word for values; unused words are zero.
struct QbMask { uint32_t w0, w1, w2, w3; };
__device__ __forceinline__ uint32_t qb_mask_word(const QbMask &m, int i) { return i == 0 ? m.w0 : (i == 1 ? m.w1 : (i == 2 ? m.w2 : m.w3)); }

template <int G, bool KSLAB = false>
__device__ __forceinline__ void qb_load_mask(const Params &p, const kvsink_cache &c, int q_sub, int q_grp, int q_b, int first_token,
                                             QbMask &mw)
{
    const uint32_t *bm = c.sink_bitmask + (size_t)q_b * p.mask_words;
    const int p0 = first_token + q_grp * G;
    mw.w0 = mw.w1 = mw.w2 = mw.w3 = 0u;
    if (KSLAB && q_sub < QbGeo<G>::NK) {          // per-token keys: a key item is a 32-token slab like a value item
        mw.w0 = __ldg(bm + ((p0 + 32 * q_sub) >> 5));
    } else if (q_sub < QbGeo<G>::NK) {
        mw.w0 = __ldg(bm + (p0 >> 5));
        mw.w1 = __ldg(bm + (p0 >> 5) + 1);
        if (G == 128) { mw.w2 = __ldg(bm + (p0 >> 5) + 2); mw.w3 = __ldg(bm + (p0 >> 5) + 3); }
    } else {
        mw.w0 = __ldg(bm + ((p0 + 32 * (q_sub - QbGeo<G>::NK)) >> 5));
    }
}

// One stage refill: the bulk copies of item q into `dst`, counted on `bar` (one lane).
template <int G, bool KSLAB = false>
__device__ __forceinline__ void qb_issue(const CUtensorMap *tm_k, const CUtensorMap *tm_v, const QbPos &q, unsigned char *dst, uint64_t *bar)
{
    using Geo = QbGeo<G>;
    qb_mbar_expect_tx(bar, QB_STAGE_BYTES);
    if (KSLAB && q.sub < Geo::NK) {               // per-token keys: the key map has the value map's box
        const int tok = q.grp * G + 32 * q.sub;
        qb_tma_load(dst, tm_k, 0, tok, q.h, q.b, bar);
        qb_tma_load(dst + 4096, tm_k, 64, tok, q.h, q.b, bar);
    } else if (q.sub < Geo::NK) {
        qb_tma_load(dst, tm_k, q.sub * Geo::KC, q.grp * G, q.h, q.b, bar);
    } else {
        const int tok = q.grp * G + 32 * (q.sub - Geo::NK);
        qb_tma_load(dst, tm_v, 0, tok, q.h, q.b, bar);
        qb_tma_load(dst + 4096, tm_v, 64, tok, q.h, q.b, bar);
    }
}

// MODE 0: dynamic parameters (the statistics of every group are taken here).  MODE 1: static parameters `sp` (one pair per key
// channel and per value channel group of the KV head): no statistics pass, nothing written to the parameter arrays; the
// thresholds of the 2-bit coder describe Eq. 8's clamp exactly, so values outside the calibrated range need nothing more;
// the 3- and 4-bit coder clamps (qb_make_coder_static).
// MODE 2: per-token keys.  A key item is a 32-token slab like a value item (both maps have the value map's box) read with the
// plain ldmatrix, so that the registers are the pair slots of the KEY tiles (rows = tokens): the statistics of a token and
// channel group run over a row (registers 0, 2 or 1, 3, both halves, the four lanes of a quad), its pair goes to the
// key parameter arrays in the value parameters' shape, and both elements of a register share one key.
template <int BITS, int G, int MODE = 0>
__global__ void __launch_bounds__(32 * QbGeo<G, BITS>::WARPS, 1)
quantize_bulk_kernel(Params p, kvsink_cache c, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, QbShape sh,
                     kvsink_static_params sp)
{
    static_assert(QbGeo<G, BITS>::NK == QbGeo<G, BITS>::NV, "a group has as many 32-token slabs as 4096-element key items");
    using Geo = QbGeo<G, BITS>;
    constexpr int D = QB_D, NS = Geo::NS, KPL = Geo::KPL, MT = Geo::MT, NT = Geo::NT, NGv = Geo::NGv, NW = Geo::WARPS;
    constexpr int MPS = 16 / NS;                  // matrices per statistic set
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *stages = smem;                                               // [warps][8 KB], 1024-byte aligned
    uint64_t *full = (uint64_t *)(smem + NW * QB_STAGE_BYTES);                  // [warps]
    unsigned char *scratch = (unsigned char *)(full + NW);                      // [warps][SCRATCH], 16-byte aligned
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);                     // warp-uniform by construction
    const int g = lane >> 2, t4 = lane & 3, mj = lane >> 3, rr = lane & 7;
    const float qmax = (float)((1 << BITS) - 1);

    if (tid == 0) {
        for (int i = 0; i < NW; ++i) qb_mbar_init(&full[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();   // the only block-wide barrier
    pdl_wait();        // nothing before this line touches global memory
    if (!in_bounds(sh.first_token >= 0 && (long long)sh.first_token + (long long)sh.n_groups * G <= p.max_seq, c.status)) return;   // every thread alike
    if (smem_addr(smem) & 1023u) {   // the swizzle pattern of the stages assumes 1024-byte alignment
        if (tid == 0) atomicOr(c.status, KVSINK_STATUS_TIMEOUT);
        return;
    }

    // ldmatrix row addresses inside a stage: lane constants, the matrix index enters through one XOR and an offset.
    //   values: two boxes of 64 channels with 128-byte rows (token r at 128 r, 16-byte chunk k at k ^ (r & 7));
    //           matrix 8T + m = tile T x channels [16m, 16m+16): row 16T + rr + 8 (mj >> 1), chunk 2 (m & 3) + (mj & 1)
    //   keys:   KROWB-byte rows of KC channels; matrix NT*mi + T: row 16T + rr + 8 (mj & 1), chunk 2 mi + (mj >> 1)
    const uint32_t lane_v = (uint32_t)((rr + 8 * (mj >> 1)) * 128 + ((((mj & 1) ^ (rr & 1)) | (rr & 6)) << 4));
    const uint32_t lane_ks = (uint32_t)((rr + 8 * (mj & 1)) * 128 + ((((mj >> 1) ^ (rr & 1)) | (rr & 6)) << 4));   // key slabs (MODE 2): value layout, plain load
    const uint32_t lane_k = Geo::KROWB == 64 ? (uint32_t)((rr + 8 * (mj & 1)) * 64 + ((((mj >> 1) ^ ((rr >> 1) & 1)) | ((rr >> 1) & 2)) << 4))
                                             : (uint32_t)((rr + 8 * (mj & 1)) * 128 + ((((mj >> 1) ^ (rr & 1)) | (rr & 6)) << 4));

    __half *thr = (__half *)(scratch + (size_t)warp * Geo::SCRATCH);            // 2 bit: [3][16 * NS] thresholds
    QbCoder2 *coder = (QbCoder2 *)(scratch + (size_t)warp * Geo::SCRATCH);      // 3, 4 bit: [8 * NS] coders of key pairs ...
    float2 *sz = (float2 *)(coder + 8 * NS);                                   // ... and [16 * NS] (scale, zero)
    __half *xl_tab = (__half *)(sz + 16 * NS), *xh_tab = xl_tab + 16 * NS;      // ... and (static pairs) [16 * NS] lower / upper clamp bounds
    unsigned char *my_stage = stages + (size_t)warp * QB_STAGE_BYTES;
    uint64_t *my_full = full + warp;

    // the block's items: in round r the block takes NW consecutive items, one per warp
    const unsigned id_step = gridDim.x * NW;
    const QbPos step = qb_decode<G>(id_step, sh.n_groups, p.Hkv);
    unsigned id = blockIdx.x * NW + warp;
    QbPos cur = qb_decode<G>(id, sh.n_groups, p.Hkv);
    QbPos nxt = qb_advance<G>(cur, step, sh.n_groups, p.Hkv);
    QbMask mw;
    mw.w0 = mw.w1 = mw.w2 = mw.w3 = 0u;
    if (id < sh.n_items) {
        qb_load_mask<G, MODE == 2>(p, c, cur.sub, cur.grp, cur.b, sh.first_token, mw);
        if (lane == 0) qb_issue<G, MODE == 2>(&tm_k, &tm_v, cur, my_stage, my_full);
    }
    unsigned phase = 0;                           // parity of the stage's current use
    for (; id < sh.n_items; id += id_step, phase ^= 1u) {
        // sink bits of the warp's next item, fetched while this one is processed
        QbMask mw_next;
        mw_next.w0 = mw_next.w1 = mw_next.w2 = mw_next.w3 = 0u;
        if (id + id_step < sh.n_items) qb_load_mask<G, MODE == 2>(p, c, nxt.sub, nxt.grp, nxt.b, sh.first_token, mw_next);
        if (!__all_sync(0xffffffffu, qb_wait(my_full, phase))) {
            if (lane == 0) atomicOr(c.status, KVSINK_STATUS_TIMEOUT);
            break;
        }
        const uint32_t stage = smem_addr(my_stage);
        const bool is_v = cur.sub >= Geo::NK;     // warp-uniform
        const bool kslab = MODE == 2 && !is_v;    // a key item in the slab form
        const bool slab = is_v || kslab;          // 32 tokens x 128 channels, parameters per token
        const int sub = is_v ? cur.sub - Geo::NK : cur.sub;
        const int64_t unit = (int64_t)cur.b * p.Hkv + cur.h;
        const int p0 = sh.first_token + cur.grp * G;   // first token of the group (multiple of G)

        // ---- the item's elements, matrix by matrix in the register order of the packed tile; matrices
        //      [MPS*s, MPS*s + MPS) form statistic set s (keys: one 16-channel matrix column; values: one tile x channel group) ----
        uint32_t a[16][4];
        if (is_v) {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int T = u >> 3, m = u & 7;
                qb_ldmatrix_x4_trans(a[u], ((stage + lane_v) ^ ((m & 3) << 5)) + T * 2048 + (m >> 2) * 4096);
            }
        } else if (MODE == 2) {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int T = u >> 3, m = u & 7;
                qb_ldmatrix_x4(a[u], ((stage + lane_ks) ^ ((m & 3) << 5)) + T * 2048 + (m >> 2) * 4096);
            }
        } else {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int mi = u / NT, T = u % NT;
                qb_ldmatrix_x4(a[u], ((stage + lane_k) ^ (mi << 5)) + T * 16 * Geo::KROWB);
            }
        }
        const bool has_sink = (mw.w0 | mw.w1 | mw.w2 | mw.w3) != 0u;   // the same in every lane; false for almost every item

        // ---- sink rows: exact copies into the side buffer at the rank of their position.  One binary search finds
        //      the rank of the item's first sink token; the list is ascending and holds every masked token, so the
        //      item's other sink tokens follow it one by one ----
        if (has_sink) {
            const int count = min(c.sink_count[cur.b], p.cap);
            const int32_t *sp = c.sink_pos + (size_t)cur.b * p.cap;
            __half *side = (__half *)(is_v ? c.sink_v : c.sink_k);
            const int tok0 = slab ? p0 + 32 * sub : p0;
            int slot = -1;                        // rank of the next sink token of the item
#pragma unroll
            for (int wi = 0; wi < 4; ++wi)
            for (uint32_t rest = qb_mask_word(mw, wi); rest != 0u; rest &= rest - 1u) {   // the set bits only
                const int r = 32 * wi + __ffs((int)rest) - 1;
                if (slot < 0) {
                    int lo = 0, hi = count - 1;
                    while (lo <= hi) {
                        const int mid = (lo + hi) >> 1, v = sp[mid];
                        if (v == tok0 + r) { slot = mid; break; }
                        if (v < tok0 + r) lo = mid + 1; else hi = mid - 1;
                    }
                    if (slot < 0) slot = count;   // not in the list: reported below
                }
                const int my = slot++;
                if (my >= count || sp[my] != tok0 + r) {
                    if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
                    continue;
                }
                __half *dst = side + ((size_t)unit * p.cap + my) * D;
                uint32_t src;
                int n16, off;                     // 16-byte chunks of the row held by this item, first channel
                if (slab) {
                    src = stage + (lane >> 3) * 4096 + r * 128 + (((lane & 7) ^ (r & 7)) << 4);
                    n16 = 16; off = 0;
                } else {
                    const int sw = Geo::KROWB == 64 ? ((r >> 1) & 3) : (r & 7);
                    src = stage + r * Geo::KROWB + ((lane ^ sw) << 4);
                    n16 = Geo::KC / 8; off = sub * Geo::KC;
                }
                if (lane < n16) {
                    uint4 v;
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(src));
                    *(uint4 *)(dst + off + lane * 8) = v;
                }
            }
        }

        // ---- extremes: set s, side 0 covers registers 0,1 (keys: channels 2t,2t+1; values: tokens 2t,2t+1), side 1
        //      registers 2,3 (the same + 8); keys leave out the rows of sink tokens ----
        constexpr uint32_t PINF2 = 0x7C007C00u, NINF2 = 0xFC00FC00u;
        uint32_t mn[NS][2], mx[NS][2];
#pragma unroll
        for (int s = 0; s < NS; ++s) { mn[s][0] = mn[s][1] = PINF2; mx[s][0] = mx[s][1] = NINF2; }
        if constexpr (MODE == 1) {
            // static parameters: no statistics
        } else if (kslab) {
            // per-token keys: set s = tile x channel group, side 0 = the token of rows g (registers 0, 2), side 1 = that of rows g + 8
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int s = u / MPS;
                mn[s][0] = qb_hmin2(mn[s][0], qb_hmin2(a[u][0], a[u][2])); mx[s][0] = qb_hmax2(mx[s][0], qb_hmax2(a[u][0], a[u][2]));
                mn[s][1] = qb_hmin2(mn[s][1], qb_hmin2(a[u][1], a[u][3])); mx[s][1] = qb_hmax2(mx[s][1], qb_hmax2(a[u][1], a[u][3]));
            }
        } else if (is_v || !has_sink) {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int s = u / MPS;
                mn[s][0] = qb_hmin2(mn[s][0], qb_hmin2(a[u][0], a[u][1])); mx[s][0] = qb_hmax2(mx[s][0], qb_hmax2(a[u][0], a[u][1]));
                mn[s][1] = qb_hmin2(mn[s][1], qb_hmin2(a[u][2], a[u][3])); mx[s][1] = qb_hmax2(mx[s][1], qb_hmax2(a[u][2], a[u][3]));
            }
        } else {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int s = u / NT, T = u % NT;
                const uint32_t m16 = (qb_mask_word(mw, T >> 1) >> (16 * (T & 1))) & 0xffffu;
                if (!((m16 >> g) & 1u)) {
                    mn[s][0] = qb_hmin2(mn[s][0], a[u][0]); mx[s][0] = qb_hmax2(mx[s][0], a[u][0]);
                    mn[s][1] = qb_hmin2(mn[s][1], a[u][2]); mx[s][1] = qb_hmax2(mx[s][1], a[u][2]);
                }
                if (!((m16 >> (g + 8)) & 1u)) {
                    mn[s][0] = qb_hmin2(mn[s][0], a[u][1]); mx[s][0] = qb_hmax2(mx[s][0], a[u][1]);
                    mn[s][1] = qb_hmin2(mn[s][1], a[u][3]); mx[s][1] = qb_hmax2(mx[s][1], a[u][3]);
                }
            }
        }
        // every lane has consumed its ldmatrix results: the stage can take the warp's next item, which streams in
        // while this one is coded from registers
        const QbPos nn = qb_advance<G>(nxt, step, sh.n_groups, p.Hkv);
        __syncwarp();
        if (lane == 0 && id + id_step < sh.n_items) qb_issue<G, MODE == 2>(&tm_k, &tm_v, nxt, my_stage, my_full);

        if (kslab) {
            // the other channels of a token row live in the other half of the register and in the other lanes of the quad
#pragma unroll
            for (int s = 0; s < NS; ++s)
#pragma unroll
                for (int ab = 0; ab < 2; ++ab) {
                    uint32_t lo2 = qb_hmin2(mn[s][ab], __byte_perm(mn[s][ab], 0u, 0x1032)), hi2 = qb_hmax2(mx[s][ab], __byte_perm(mx[s][ab], 0u, 0x1032));
#pragma unroll
                    for (int o = 1; o < 4; o <<= 1) {
                        lo2 = qb_hmin2(lo2, __shfl_xor_sync(0xffffffffu, lo2, o));
                        hi2 = qb_hmax2(hi2, __shfl_xor_sync(0xffffffffu, hi2, o));
                    }
                    mn[s][ab] = lo2; mx[s][ab] = hi2;
                }
        } else if (NS == 4 && MODE != 1) {
            // The other rows of a column live in the lanes that differ in bits 2..4.  Eight (set, side) pairs for the eight
            // lanes of a column group: each exchange halves what a lane carries (it keeps the half its own bit names and sends
            // the other), so that lane g ends with the extremes of pair g alone -- both of its keys, one per half
            uint32_t vn[8], vx[8];
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) { vn[c8] = mn[(c8 >> 1) % NS][c8 & 1]; vx[c8] = mx[(c8 >> 1) % NS][c8 & 1]; }
#pragma unroll
            for (int w = 4; w >= 1; w >>= 1) {
                const bool up = (lane & (4 * w)) != 0;     // bit 4, 3, 2 of the lane = bit 2, 1, 0 of g
#pragma unroll
                for (int i = 0; i < w; ++i) {
                    const uint32_t sn = up ? vn[i] : vn[w + i], kn = up ? vn[w + i] : vn[i];
                    const uint32_t sx = up ? vx[i] : vx[w + i], kx = up ? vx[w + i] : vx[i];
                    vn[i] = qb_hmin2(kn, __shfl_xor_sync(0xffffffffu, sn, 4 * w));
                    vx[i] = qb_hmax2(kx, __shfl_xor_sync(0xffffffffu, sx, 4 * w));
                }
            }
            mn[0][0] = vn[0]; mx[0][0] = vx[0];
        } else {
        // the other rows of a column live in the lanes that differ in bits 2..4
#pragma unroll
        for (int o = 4; o < 32 && MODE != 1; o <<= 1)
#pragma unroll
            for (int s = 0; s < NS; ++s)
#pragma unroll
                for (int ab = 0; ab < 2; ++ab) {
                    mn[s][ab] = qb_hmin2(mn[s][ab], __shfl_xor_sync(0xffffffffu, mn[s][ab], o));
                    mx[s][ab] = qb_hmax2(mx[s][ab], __shfl_xor_sync(0xffffffffu, mx[s][ab], o));
                }
        }

        // ---- parameters (Eq. 10-11) and thresholds: the eight lanes of a column group share its 4 * NS keys ----
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            // the lane's j-th key.  Per-token keys: lane (g, t) takes the token of tile t >> 1, rows g + 8 (t & 1), channel group j
            // With eight (set, side) pairs (NS = 4) the exchange above left lane g with pair g: its keys are the two halves.
            const bool scat = NS == 4 && MODE != 1 && !kslab;
            const int kk = scat ? 2 * g + j : g + 8 * j;
            const int s_ = kslab ? (t4 >> 1) * NGv + j : kk >> 2, ab_ = kslab ? (t4 & 1) : (kk >> 1) & 1, e_ = kslab ? 0 : kk & 1;
            uint32_t smn = 0, smx = 0;
            if (scat) {
                smn = mn[0][0]; smx = mx[0][0];
            } else {
#pragma unroll
                for (int s = 0; s < NS; ++s)
#pragma unroll
                    for (int ab = 0; ab < 2; ++ab)
                        if (s_ == s && ab_ == ab) { smn = mn[s][ab]; smx = mx[s][ab]; }
            }
            const unsigned short lo16 = (unsigned short)(e_ ? smn >> 16 : smn & 0xffffu), hi16 = (unsigned short)(e_ ? smx >> 16 : smx & 0xffffu);
            const float fmn = __half2float(__ushort_as_half(lo16)), fmx = __half2float(__ushort_as_half(hi16));
            // values: token of the item (set = tile * NGv + channel group); keys: channel of the item (set = matrix)
            const int idx = kslab ? 16 * (t4 >> 1) + 8 * (t4 & 1) + g : 16 * (is_v ? s_ / NGv : s_) + 8 * ab_ + 2 * t4 + e_;
            const bool member = slab ? !((mw.w0 >> idx) & 1u) : (MODE == 1 || lo16 != 0x7C00);
            float s, z;
            if constexpr (MODE == 1) {
                // the pair of this key channel / of this token's value channel group; a sink token's values keep code 0
                const int pi = is_v ? cur.h * NGv + (s_ % NGv) : cur.h * D + sub * Geo::KC + idx;
                s = member ? __ldg((is_v ? sp.v_scale : sp.k_scale) + pi) : 0.f;
                z = member ? __ldg((is_v ? sp.v_zero : sp.k_zero) + pi) : 0.f;
            } else {
                group_params(member, fmn, fmx, qmax, &s, &z);
                const size_t ov = ((size_t)unit * p.max_seq + p0 + 32 * sub + idx) * NGv + (s_ % NGv);
                const size_t ok = ((size_t)unit * (p.max_seq / G) + p0 / G) * D + sub * Geo::KC + idx;
                float *ps = is_v ? c.v_scale + ov : c.k_scale + (kslab ? ov : ok), *pz = is_v ? c.v_zero + ov : c.k_zero + (kslab ? ov : ok);
                *ps = s;
                *pz = z;
            }
            // place of the key in the warp's table: (set, side) block of eight, then the lane coordinate that owns its elements
            const int pos = kslab ? 8 * (2 * s_ + ab_) + g : 8 * (kk >> 1) + 2 * t4 + e_;
            if constexpr (BITS == 2) {
                const double s_half = 0.5 * (double)s;
#pragma unroll
                for (int l = 0; l < 3; ++l)
                    thr[l * (16 * NS) + pos] = __ushort_as_half((unsigned short)qb_threshold(s, s_half, z, (float)(l + 1), qmax));
            } else {
                QbCoder cc;
                if constexpr (MODE == 1) {
                    __half xl, xh;
                    cc = qb_make_coder_static(s, z, qmax, &xl, &xh);
                    xl_tab[pos] = xl;
                    xh_tab[pos] = xh;
                } else {
                    cc = qb_make_coder(s, z, fmn, fmx, qmax);
                }
                QbCoder2 *c2 = coder + (pos >> 1);
                c2->r_lo[pos & 1] = cc.r_lo;
                c2->r_hi[pos & 1] = cc.r_hi;
                c2->magic[pos & 1] = cc.magic;
                sz[pos] = make_float2(s, z);
            }
        }
        __syncwarp();

        const size_t tile0 = (size_t)unit * (p.max_seq / KVSINK_TILE) + p0 / KVSINK_TILE + (slab ? 2 * sub : 0);
        uint8_t *codes = (is_v ? c.v_codes : c.k_codes) + tile0 * Geo::TILE_BYTES;
        if constexpr (BITS == 2) {
            // ---- coding: every register becomes its byte of packed fields (in both halves) ----
            const __half2 base = __half2half2(__float2half(1024.f));
            const __half2 w0 = __half2half2(__float2half(1.f)), w1 = __half2half2(__float2half(4.f));
            const __half2 w2 = __half2half2(__float2half(16.f)), w3 = __half2half2(__float2half(64.f));
            uint32_t bits[16];
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                // thresholds of the keys of registers 0, 1 (side 0) and 2, 3 (side 1); per-token keys: of registers 0, 2 and 1, 3,
                // one key for both halves
                __half2 tq[2][3], tq1[3], tq2[3];
#pragma unroll
                for (int ab = 0; ab < 2; ++ab)
#pragma unroll
                    for (int l = 0; l < 3; ++l)
                        tq[ab][l] = kslab ? __half2half2(thr[l * (16 * NS) + 8 * (2 * s + ab) + g])
                                          : *reinterpret_cast<const __half2 *>(thr + l * (16 * NS) + 8 * (2 * s + ab) + 2 * t4);
#pragma unroll
                for (int l = 0; l < 3; ++l) { tq1[l] = kslab ? tq[1][l] : tq[0][l]; tq2[l] = kslab ? tq[0][l] : tq[1][l]; }
#pragma unroll
                for (int i = 0; i < MPS; ++i) {
                    const int u = s * MPS + i;
                    __half2 acc = base;
                    acc = qb_thermo(acc, a[u][0], tq[0], w0);
                    acc = qb_thermo(acc, a[u][1], tq1, w1);
                    acc = qb_thermo(acc, a[u][2], tq2, w2);
                    acc = qb_thermo(acc, a[u][3], tq[1], w3);
                    bits[u] = *reinterpret_cast<uint32_t *>(&acc);   // 0x6400 | byte in each half
                }
            }
            __syncwarp();   // the scratch is rewritten by the next item
            if (has_sink && !slab) {
                // sink tokens keep code 0: fields 0, 2 of a byte are row g, fields 1, 3 row g + 8 (items with per-token
                // parameters need nothing: the thresholds of a sink token are +inf)
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const int T = u % NT;
                    const uint32_t m16 = (qb_mask_word(mw, T >> 1) >> (16 * (T & 1))) & 0xffffu;
                    if ((m16 >> g) & 1u) bits[u] &= 0xffccffccu;
                    if ((m16 >> (g + 8)) & 1u) bits[u] &= 0xff33ff33u;
                }
            }
            // ---- packed words: bytes (even matrix lo, odd matrix lo, even matrix hi, odd matrix hi) ----
            if (slab) {
#pragma unroll
                for (int T = 0; T < 2; ++T) {
                    uint4 w;
                    w.x = __byte_perm(bits[8 * T + 0], bits[8 * T + 1], 0x6240); w.y = __byte_perm(bits[8 * T + 2], bits[8 * T + 3], 0x6240);
                    w.z = __byte_perm(bits[8 * T + 4], bits[8 * T + 5], 0x6240); w.w = __byte_perm(bits[8 * T + 6], bits[8 * T + 7], 0x6240);
                    *(uint4 *)(codes + T * Geo::TILE_BYTES + lane * 16) = w;
                }
            } else {
#pragma unroll
                for (int T = 0; T < NT; ++T) {
                    uint8_t *dst = codes + T * Geo::TILE_BYTES + lane * 16 + (sub * MT / 2) * 4;
                    if constexpr (MT == 2) {
                        *(uint32_t *)dst = __byte_perm(bits[T], bits[NT + T], 0x6240);
                    } else {
                        uint2 w;
                        w.x = __byte_perm(bits[T], bits[NT + T], 0x6240);
                        w.y = __byte_perm(bits[2 * NT + T], bits[3 * NT + T], 0x6240);
                        *(uint2 *)dst = w;
                    }
                }
            }
        } else {
            // ---- coding, 3 and 4 bit: set by set (its four keys' coders from the scratch), matrix by matrix ----
            uint32_t lo[16], hi[16];
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                unsigned long long k_lo[2], k_hi[2], k_magic[2];   // key pairs of this lane's columns (side 0, side 1)
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    if (kslab) {                                   // one key (token row g + 8 q) for both elements
                        const QbCoder2 *c2 = coder + 4 * (2 * s + q) + (g >> 1);
                        const float rl = c2->r_lo[g & 1], rh = c2->r_hi[g & 1], mg = c2->magic[g & 1];
                        k_lo[q] = qb_pair(rl, rl);
                        k_hi[q] = qb_pair(rh, rh);
                        k_magic[q] = qb_pair(mg, mg);
                    } else {
                        const QbCoder2 *c2 = coder + 4 * (2 * s + q) + t4;
                        const float4 rr = *reinterpret_cast<const float4 *>(c2->r_lo);
                        const float2 mm = *reinterpret_cast<const float2 *>(c2->magic);
                        k_lo[q] = qb_pair(rr.x, rr.y);
                        k_hi[q] = qb_pair(rr.z, rr.w);
                        k_magic[q] = qb_pair(mm.x, mm.y);
                    }
                }
                // registers 0, 1 take side 0 and 2, 3 side 1; with per-token keys registers 0, 2 take side 0 and 1, 3 side 1
                const unsigned long long kl[4] = {k_lo[0], kslab ? k_lo[1] : k_lo[0], kslab ? k_lo[0] : k_lo[1], k_lo[1]};
                const unsigned long long kh[4] = {k_hi[0], kslab ? k_hi[1] : k_hi[0], kslab ? k_hi[0] : k_hi[1], k_hi[1]};
                const unsigned long long km[4] = {k_magic[0], kslab ? k_magic[1] : k_magic[0], kslab ? k_magic[0] : k_magic[1], k_magic[1]};
                uint32_t xl2[2] = {0u, 0u}, xh2[2] = {0u, 0u};   // static pairs: clamp bounds of the two keys of side 0 / side 1
                if constexpr (MODE == 1) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        xl2[q] = *reinterpret_cast<const uint32_t *>(xl_tab + 8 * (2 * s + q) + 2 * t4);
                        xh2[q] = *reinterpret_cast<const uint32_t *>(xh_tab + 8 * (2 * s + q) + 2 * t4);
                    }
                }
#pragma unroll
                for (int i = 0; i < MPS; ++i) {
                    const int u = s * MPS + i;
                    const int m = slab ? (u & 7) : sub * MT + u / NT;   // matrix of the tile
                    uint32_t pc[4];
                    uint32_t differ[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        uint32_t x2 = a[u][r];
                        if constexpr (MODE == 1) x2 = qb_hmin2(qb_hmax2(x2, xl2[r >> 1]), xh2[r >> 1]);
                        pc[r] = qb_code_pair(x2, kl[r], kh[r], km[r], differ[r]);
                    }
                    if (differ[0] | differ[1] | differ[2] | differ[3]) {
                        // a value too close to a rounding tie (fp16 inputs land on exact ties often): redo those registers
#pragma unroll
                        for (int r = 0; r < 4; ++r)
                            if (differ[r]) {
                                const int zi = kslab ? 8 * (2 * s + (r & 1)) + g : 8 * (2 * s + (r >> 1)) + 2 * t4;
                                const float2 z0 = sz[zi], z1 = sz[kslab ? zi : zi + 1];
                                pc[r] = qb_code_pair_exact(a[u][r], z0.x, z0.y, z1.x, z1.y, qmax);
                            }
                    }
                    if constexpr (MODE == 1) {   // Eq. 8's clamp on both 16-bit fields (an exact redo is inside the range already)
                        const uint32_t q2 = (uint32_t)((1 << BITS) - 1) * 0x00010001u;
#pragma unroll
                        for (int r = 0; r < 4; ++r) pc[r] = __vimin_s16x2_relu(pc[r], q2);
                    }
                    if (has_sink && !slab) {   // sink tokens keep code 0: pair slots 0, 2 are row g, slots 1, 3 row g + 8
                        const int T = u % NT;
                        const uint32_t m16 = (qb_mask_word(mw, T >> 1) >> (16 * (T & 1))) & 0xffffu;
                        if ((m16 >> g) & 1u) pc[0] = pc[2] = 0;
                        if ((m16 >> (g + 8)) & 1u) pc[1] = pc[3] = 0;
                    }
                    qb_pack_matrix<BITS>(pc, m, &lo[u], &hi[u]);
                }
            }
            __syncwarp();   // the scratch is rewritten by the next item
            // ---- packed words.  4 bit: word m of a lane is matrix m, planes of four words.  3 bit: low section as for
            //      2 bit (word m >> 1, byte m & 1 of each half), high section at 512 bytes (word m >> 2, two per lane) ----
            if (slab) {
#pragma unroll
                for (int T = 0; T < 2; ++T) {
                    uint8_t *dst = codes + T * Geo::TILE_BYTES;
                    if constexpr (BITS == 4) {
                        *(uint4 *)(dst + lane * 16) = make_uint4(lo[8 * T], lo[8 * T + 1], lo[8 * T + 2], lo[8 * T + 3]);
                        *(uint4 *)(dst + 512 + lane * 16) = make_uint4(lo[8 * T + 4], lo[8 * T + 5], lo[8 * T + 6], lo[8 * T + 7]);
                    } else {
                        uint4 w;
                        w.x = lo[8 * T + 0] | (lo[8 * T + 1] << 8); w.y = lo[8 * T + 2] | (lo[8 * T + 3] << 8);
                        w.z = lo[8 * T + 4] | (lo[8 * T + 5] << 8); w.w = lo[8 * T + 6] | (lo[8 * T + 7] << 8);
                        *(uint4 *)(dst + lane * 16) = w;
                        uint2 h;
                        h.x = hi[8 * T + 0] | hi[8 * T + 1] | hi[8 * T + 2] | hi[8 * T + 3];
                        h.y = hi[8 * T + 4] | hi[8 * T + 5] | hi[8 * T + 6] | hi[8 * T + 7];
                        *(uint2 *)(dst + 512 + lane * 8) = h;
                    }
                }
            } else {
#pragma unroll
                for (int T = 0; T < NT; ++T) {
                    uint8_t *dst = codes + T * Geo::TILE_BYTES;
                    if constexpr (BITS == 4 && MT == 4) {          // matrices 4 sub .. 4 sub + 3: plane `sub`
                        *(uint4 *)(dst + sub * 512 + lane * 16) = make_uint4(lo[T], lo[NT + T], lo[2 * NT + T], lo[3 * NT + T]);
                    } else if constexpr (BITS == 4) {              // matrices 2 sub, 2 sub + 1: half of a lane's plane entry
                        *(uint2 *)(dst + (sub >> 1) * 512 + lane * 16 + (sub & 1) * 8) = make_uint2(lo[T], lo[NT + T]);
                    } else {                                       // 3 bit, 64 channels: two low words and one whole high word
                        uint2 w;
                        w.x = lo[T] | (lo[NT + T] << 8);
                        w.y = lo[2 * NT + T] | (lo[3 * NT + T] << 8);
                        *(uint2 *)(dst + lane * 16 + sub * 8) = w;
                        *(uint32_t *)(dst + 512 + lane * 8 + sub * 4) = hi[T] | hi[NT + T] | hi[2 * NT + T] | hi[3 * NT + T];
                    }
                }
            }
        }
        cur = nxt;
        nxt = nn;
        mw = mw_next;
    }
}

// ---- host side ----
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                   const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    });
    return fn;
}

// fp16 tensor [B][Hkv][T][D] with element strides (sb, sh, stt, 1); box = box_ch channels x box_tok tokens.
bool make_map(CUtensorMap *tm, const __half *base, const Params &p, int T, int64_t sb, int64_t sh, int64_t stt, int box_ch, int box_tok,
              CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)p.D, (cuuint64_t)T, (cuuint64_t)p.Hkv, (cuuint64_t)p.B};
    // a dimension of extent 1 never advances: any valid stride will do
    const int64_t s_h = p.Hkv > 1 ? sh : stt * T, s_b = p.B > 1 ? sb : stt * T;
    if (stt <= 0 || s_h <= 0 || s_b <= 0) return false;
    const cuuint64_t strides[3] = {(cuuint64_t)stt * 2, (cuuint64_t)s_h * 2, (cuuint64_t)s_b * 2};
    const cuuint32_t box[4] = {(cuuint32_t)box_ch, (cuuint32_t)box_tok, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BITS, int G, int MODE = 0>
int launch_bulk(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src, int first_token,
                int n_groups, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    using Geo = QbGeo<G, BITS>;
    CUtensorMap tm_k, tm_v;
    const int T = n_groups * G;
    if (MODE == 2) {
        if (!make_map(&tm_k, k_src, p, T, sb, sh, stt, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return KVSINK_ERR_UNSUPPORTED;
    } else if (!make_map(&tm_k, k_src, p, T, sb, sh, stt, Geo::KC, G, Geo::KROWB == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B))
        return KVSINK_ERR_UNSUPPORTED;
    if (!make_map(&tm_v, v_src, p, T, sb, sh, stt, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return KVSINK_ERR_UNSUPPORTED;
    constexpr int NW = Geo::WARPS;
    constexpr size_t smem = (size_t)NW * (QB_STAGE_BYTES + 8 + Geo::SCRATCH);
    static_assert(smem <= 227 * 1024, "stages too large");
    auto kern = quantize_bulk_kernel<BITS, G, MODE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    QbShape shp;
    shp.first_token = first_token;
    shp.n_groups = n_groups;
    const long n_items = (long)p.B * p.Hkv * n_groups * Geo::IPG;
    if (n_items >= (1L << 30)) return KVSINK_ERR_UNSUPPORTED;
    shp.n_items = (unsigned)n_items;
    long blocks = (n_items + NW - 1) / NW;
    if (blocks > 148) blocks = 148;
    return launch_pdl(kern, dim3((unsigned)blocks), dim3(32 * NW), smem, st, p, c, tm_k, tm_v, shp, sp) == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

}  // namespace

// Whole groups of a bulk append (keys, values and sink rows).  Returns KVSINK_ERR_UNSUPPORTED when the shape has no
// kernel of this kind or the inputs cannot be described by a tensor map; the caller then uses another kernel.
int launch_quantize_groups_bulk(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                                int n_groups, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (p.D != QB_D || n_groups < 1) return KVSINK_ERR_UNSUPPORTED;
    const kvsink_static_params none = {nullptr, nullptr, nullptr, nullptr};
    if (p.bits == 2 && p.G == 128) return launch_bulk<2, 128>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 2 && p.G == 64) return launch_bulk<2, 64>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 3 && p.G == 64) return launch_bulk<3, 64>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 128) return launch_bulk<4, 128>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 64) return launch_bulk<4, 64>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    return KVSINK_ERR_UNSUPPORTED;
}

// The same for static parameters: n_groups spans of G tokens (G only sets the shape of the work items here), the first at a
// multiple of G.  Shapes without a bulk kernel return KVSINK_ERR_UNSUPPORTED and the caller uses the tile kernels.
int launch_quantize_static_bulk(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                                int first_token, int n_groups, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (p.D != QB_D || n_groups < 1 || first_token % p.G) return KVSINK_ERR_UNSUPPORTED;
    if (p.bits == 2 && p.G == 128) return launch_bulk<2, 128, 1>(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 2 && p.G == 64) return launch_bulk<2, 64, 1>(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 3 && p.G == 64) return launch_bulk<3, 64, 1>(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 128) return launch_bulk<4, 128, 1>(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 64) return launch_bulk<4, 64, 1>(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    return KVSINK_ERR_UNSUPPORTED;
}

// The same for per-token keys (keys quantized like values; the pairs go to the key parameter arrays in the value parameters' shape).
// 3 bit has no form here: its bulk items need 64-token spans, which give two channel groups per row, and the decode side of
// per-token keys takes one group at 3 bit.
int launch_quantize_pertoken_bulk(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                                  int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (p.D != QB_D || n_groups < 1 || first_token % p.G) return KVSINK_ERR_UNSUPPORTED;
    const kvsink_static_params none = {nullptr, nullptr, nullptr, nullptr};
    if (p.bits == 2 && p.G == 128) return launch_bulk<2, 128, 2>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 2 && p.G == 64) return launch_bulk<2, 64, 2>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 128) return launch_bulk<4, 128, 2>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    if (p.bits == 4 && p.G == 64) return launch_bulk<4, 64, 2>(p, c, none, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
    return KVSINK_ERR_UNSUPPORTED;
}

}  // namespace kvsink
