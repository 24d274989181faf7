// Whole-group quantization (Eq. 8-11 with Algorithm 1's sink exclusion) at streaming speed.
//
// Persistent blocks walk over work items; an item is the keys or the values of one (token group, KV head, sequence).
// The item's G x D fp16 tile is staged once in shared memory with cp.async into XOR-swizzled 16-byte chunks (double
// buffered, so the next item streams in while this one is coded; HBM is read exactly once).  After one barrier every
// warp works alone: ldmatrix (ldmatrix.trans for values, whose packed tiles are [channel x token]) hands each lane
// exactly the elements of its pair slots, and the same registers serve the min/max pass (fp16, exact), the
// parameters (IEEE binary32) and the coding pass, which therefore emits words in the packed tile's own layout.  The literal  rint(x / scale) + zero  is reproduced bit for bit without a division per
// element: y = fma(x, r, M + zero) with r = 1/scale nudged down and up by 2^-22 and M = 1.5 * 2^23 rounds the
// product to an integer in the mantissa; if both nudged results agree, no rounding of x/scale can land on the other
// side of a tie and the agreed integer is the exact answer; if they differ (about one element in 10^5) the lane
// recomputes its batch with the IEEE division.
#include "common.cuh"

namespace kvsink {

constexpr float MAGIC = 12582912.0f;   // 1.5 * 2^23

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *smem_row)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void *smem_row)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(smem_row)));
}

// Per channel (keys) or per (token, channel group) (values): what the fast coder needs.
struct __align__(16) Coder {
    float r_lo, r_hi;   // 1/scale nudged down / up; r_lo = +inf forces the exact path
    float magic;        // M + zero
    float pad;
};

// mn, mx: the group's extremes.  The fast coder is used only where it is provably exact: |x/scale| and |zero| far
// below 2^22 (integer-in-mantissa), and the top code cannot exceed qmax (so no clamp is needed).
__device__ __forceinline__ Coder make_coder(float scale, float zero, float mn, float mx, float qmax)
{
    Coder c;
    c.pad = 0.f;
    if (scale == 0.f) {   // no member, or sink token: code 0
        c.r_lo = c.r_hi = 0.f;
        c.magic = MAGIC;
        return c;
    }
    const float r = __frcp_rn(scale);
    const float absmax = fmaxf(fabsf(mn), fabsf(mx));
    const bool top_fits = __fadd_rn(rintf(__fdiv_rn(mx, scale)), zero) <= qmax;
    const bool ok = absmax * r < 2097152.f && fabsf(zero) < 2097152.f && r < 3.0e38f && top_fits;
    c.r_lo = ok ? __fmul_rn(r, 1.f - 2.384185791015625e-07f) : __int_as_float(0x7f800000);
    c.r_hi = ok ? __fmul_rn(r, 1.f + 2.384185791015625e-07f) : r;
    c.magic = MAGIC + (ok ? zero : 0.f);
    return c;
}

// Codes of the two elements of a half2 register -> (code_lo | code_hi << 16); `differ` collects disagreement bits.
template <int BITS>
__device__ __forceinline__ uint32_t code_pair(uint32_t h2, const Coder &c0, const Coder &c1, uint32_t &differ)
{
    const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const float a0 = fmaf(x.x, c0.r_lo, c0.magic), b0 = fmaf(x.x, c0.r_hi, c0.magic);
    const float a1 = fmaf(x.y, c1.r_lo, c1.magic), b1 = fmaf(x.y, c1.r_hi, c1.magic);
    differ |= (__float_as_uint(a0) ^ __float_as_uint(b0)) | (__float_as_uint(a1) ^ __float_as_uint(b1));
    // low halves of the two results (the bit pattern of 1.5 * 2^23 has a zero low half)
    return __byte_perm(__float_as_uint(a0), __float_as_uint(a1), 0x5410);
}

template <int BITS>
__device__ __noinline__ uint32_t code_pair_exact(uint32_t h2, float s0, float z0, float s1, float z1)
{
    const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const float qmax = (float)((1 << BITS) - 1);
    const uint32_t c0 = s0 == 0.f ? 0u : code_exact(x.x, s0, z0, qmax);
    const uint32_t c1 = s1 == 0.f ? 0u : code_exact(x.y, s1, z1, qmax);
    return c0 | (c1 << 16);
}

// Bits contributed by one matrix (index m) of a tile to a lane's words, from its four code pairs pc[r].
//   2 bit: 8 bits in each half of `lo` (to be placed at byte m&1 of each half of word m>>1).
//   4 bit: the whole word m in `lo`.
//   3 bit: low two bits as 2 bit in `lo`; `hi` holds this matrix's bits of hi word m>>2, already in place.
template <int BITS>
__device__ __forceinline__ void pack_matrix(const uint32_t (&pc)[4], int m, uint32_t *lo, uint32_t *hi)
{
    if constexpr (BITS == 2) {
        *lo = pc[0] | (pc[1] << 2) | (pc[2] << 4) | (pc[3] << 6);
        *hi = 0;
    } else if constexpr (BITS == 4) {
        *lo = pc[0] | (pc[1] << 4) | (pc[2] << 8) | (pc[3] << 12);
        *hi = 0;
    } else {
        *lo = (pc[0] & 0x00030003u) | ((pc[1] & 0x00030003u) << 2) | ((pc[2] & 0x00030003u) << 4) | ((pc[3] & 0x00030003u) << 6);
        const uint32_t h = ((pc[0] >> 2) & 0x00010001u) | (((pc[1] >> 2) & 0x00010001u) << 1) | (((pc[2] >> 2) & 0x00010001u) << 4) |
                           (((pc[3] >> 2) & 0x00010001u) << 5);
        *hi = h << (8 * (m & 1) + 2 * (1 - ((m >> 1) & 1)));
    }
}

// ---- 2-bit coder by thresholds ----
// code(x) = clamp(rint(x / scale) + zero, 0, 3) is a non-decreasing step function of x, and x is fp16: three fp16
// thresholds t1 <= t2 <= t3 (the smallest values whose code reaches 1, 2, 3) describe it exactly, and
// code(x) = [x >= t1] + [x >= t2] + [x >= t3] needs no division, no rounding guard and no conversion.
// fp16 values in sorted order: sign-magnitude bit pattern -> signed integer (both zeros map to 0).
__device__ __forceinline__ int h_ord(unsigned b) { return (b & 0x8000u) ? -(int)(b & 0x7fffu) : (int)b; }
__device__ __forceinline__ unsigned h_unord(int o) { return o >= 0 ? (unsigned)o : (0x8000u | (unsigned)(-o)); }
__device__ __forceinline__ float h_val(int o) { return __half2float(__ushort_as_half((unsigned short)h_unord(o))); }

// Bit pattern of the smallest finite fp16 value whose code under (scale, zero) is at least `level` (1..qmax), found by
// evaluating the literal formula around a closed-form estimate; +inf if no finite value reaches it.
__device__ __noinline__ unsigned code_threshold(float s, float z, int level, float qmax)
{
    constexpr int OMAX = 0x7BFF;
    if (s == 0.f) return 0x7C00u;
    float est = s * ((float)level - 0.5f - z);
    est = fminf(fmaxf(est, -65504.f), 65504.f);
    int o = h_ord(__half_as_ushort(__float2half_ru(est)));
    bool done = false;
#pragma unroll 1
    for (int it = 0; it < 6 && !done; ++it) {
        if (o > OMAX) return 0x7C00u;
        if ((int)code_exact(h_val(o), s, z, qmax) >= level) done = true; else ++o;
    }
    if (done) {
        done = false;
#pragma unroll 1
        for (int it = 0; it < 6 && !done; ++it) {
            if (o - 1 < -OMAX || (int)code_exact(h_val(o - 1), s, z, qmax) < level) done = true; else --o;
        }
    }
    if (!done) {   // estimate far off (does not happen for sane parameters): bisection over all finite fp16 values
        int lo = -OMAX, hi = OMAX + 1;   // invariant: code(lo - 1) < level (vacuous at the bottom), code(hi) >= level or hi beyond the top
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((int)code_exact(h_val(mid), s, z, qmax) >= level) hi = mid; else lo = mid + 1;
        }
        o = lo;
        if (o > OMAX) return 0x7C00u;
    }
    return h_unord(o);
}

// The three thresholds of each of a warp's 16 keys with every lane busy.  The lanes g and g + 4 of a column group hold
// the same key's (s, z): the lower one resolves level 1, the upper one level 2, and they share level 3.
// Let T = level - zero - 1/2 and o the first fp16 value at or above est = fl(s * T).  Every value below o lies below
// s * T, so its code stays under the level unless its quotient rounds onto T (checked: `below`).  The value o itself
// reaches the level unless its quotient is exactly the tie T and rounds to the even neighbour below (common at 2 bit,
// where scale = range / 3 makes s * T an fp16 value for a third of the groups); its successor is then the threshold,
// because one fp16 step (>= 2^-12 relative, or 2^-24 absolute next to zero) moves the quotient past T by far more than
// the 2^-24 relative error of est and the half ulp the rounded quotient can lose.  Estimates outside the finite range,
// and the rare `below` hit, go to the search above.
// `th` points at the key's half of thr[t4][column half][0]; consecutive levels are two halves apart.
__device__ __forceinline__ void warp_thresholds(float s, float z, int g, float qmax, __half *th)
{
    constexpr int OMAX = 0x7BFF;
    const bool upper = g >= 4;
    // clamp(q, 0, qmax) >= level  <=>  q >= level  for 1 <= level <= qmax
    auto reaches = [&](int o, float level) { return __fadd_rn(rintf(__fdiv_rn(h_val(o), s)), z) >= level; };
    const float own = upper ? 2.f : 1.f;
    const float est_own = s * (own - 0.5f - z), est3 = s * (3.f - 0.5f - z);
    const int o_own = h_ord(__half_as_ushort(__float2half_ru(fminf(fmaxf(est_own, -65504.f), 65504.f))));
    const int o3 = h_ord(__half_as_ushort(__float2half_ru(fminf(fmaxf(est3, -65504.f), 65504.f))));
    const bool own_at = reaches(o_own, own);
    const bool own_below = o_own > -OMAX && reaches(max(o_own - 1, -OMAX), own);
    const bool r3 = upper ? (o3 > -OMAX && reaches(max(o3 - 1, -OMAX), 3.f)) : reaches(o3, 3.f);
    const bool below3 = __shfl_xor_sync(0xffffffffu, (int)r3, 16) != 0;   // meaningful in the lower lane
    unsigned t_own = h_unord(o_own + (own_at ? 0 : 1));
    if (s == 0.f) t_own = 0x7C00u;
    else if (own_below || !(fabsf(est_own) < 65504.f)) t_own = code_threshold(s, z, upper ? 2 : 1, qmax);
    th[upper ? 2 : 0] = __ushort_as_half((unsigned short)t_own);
    if (!upper) {
        unsigned t3 = h_unord(o3 + (r3 ? 0 : 1));
        if (s == 0.f) t3 = 0x7C00u;
        else if (below3 || !(fabsf(est3) < 65504.f)) t3 = code_threshold(s, z, 3, qmax);
        th[4] = __ushort_as_half((unsigned short)t3);
    }
}

// Codes of the two elements of a half2 register, positioned: returns acc + w * ([x>=t1] + [x>=t2] + [x>=t3]) per half.
__device__ __forceinline__ __half2 thermo_accumulate(__half2 acc, uint32_t x2, const __half2 (&t)[3], __half2 w)
{
    const __half2 x = *reinterpret_cast<const __half2 *>(&x2);
    const __half2 cnt = __hadd2(__hadd2(__hge2(x, t[0]), __hge2(x, t[1])), __hge2(x, t[2]));
    return __hfma2(cnt, w, acc);
}

// Reduces the lane's pairwise extremes over the eight lanes that hold the other rows (lane bits 2..4).
__device__ __forceinline__ void reduce_rows(__half2 &mn, __half2 &mx)
{
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        uint32_t a = __shfl_xor_sync(0xffffffffu, *reinterpret_cast<uint32_t *>(&mn), o);
        uint32_t b = __shfl_xor_sync(0xffffffffu, *reinterpret_cast<uint32_t *>(&mx), o);
        mn = __hmin2(mn, *reinterpret_cast<__half2 *>(&a));
        mx = __hmax2(mx, *reinterpret_cast<__half2 *>(&b));
    }
}

// Per-warp scratch: the 16 keys (channels for K, tokens for V) a warp is coding, indexed [lane&3][key 0..3] where
// key 0,1 are the two halves of pair slots with column half 0 and key 2,3 those with column half 1.
struct WarpScratch {
    Coder coder[16];
    float2 sz[16];   // (scale, zero) for the exact path
    __half2 thr[4][2][4];   // 2 bit: thresholds [lane&3][column half][level-1]; the halves are the pair's two keys
};

template <int BITS, int D, int G>
__global__ void __launch_bounds__(32 * (D / 16), (D == 128) ? 3 : 4)
quantize_groups_stream(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src, int first_token,
                       int n_groups, int64_t sb, int64_t sh, int64_t stt, int kinds)
{
    constexpr int CH = D / 8;            // 16-byte chunks per row
    constexpr int NM = D / 16;           // 16x16 matrices per tile = warps per block
    constexpr int NW = NM, THREADS = 32 * NW;
    constexpr int NT = G / KVSINK_TILE;  // tiles per group
    constexpr int Gv = G < D ? G : D, NGv = D / Gv, MPG = Gv / 16;
    constexpr int W = D * BITS / 64;     // words per lane per tile
    constexpr int NLO = (BITS == 3) ? D / 32 : W, NHI = (BITS == 3) ? D / 64 : 0;
    constexpr int TILE_WORDS = 32 * W;
    const float qmax = (float)((1 << BITS) - 1);
    const __half2 H_PINF = __half2half2(__ushort_as_half(0x7C00)), H_NINF = __half2half2(__ushort_as_half(0xFC00));
    if (!in_bounds(first_token >= 0 && (long long)first_token + (long long)n_groups * G <= p.max_seq, c.status)) return;   // every thread alike

    extern __shared__ __align__(128) unsigned char smem[];
    __half *Xbuf = (__half *)smem;                                 // [2][G][D] swizzled 16-byte chunks (double buffer)
    uint32_t *xout = (uint32_t *)(Xbuf + 2 * (size_t)G * D);       // [NT][TILE_WORDS] packed words of the item
    WarpScratch *scr_all = (WarpScratch *)(xout + NT * TILE_WORDS);
    uint32_t *tmask = (uint32_t *)(scr_all + NW);                  // [2][NT] sink bits of each tile

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const int mj = lane >> 3, rr = lane & 7;      // ldmatrix: this lane addresses row rr of 8x8 block mj
    WarpScratch &scr = scr_all[warp];
    const long n_items = (long)p.B * p.Hkv * n_groups * kinds;

    // item -> (kind, group, head, sequence) as mixed-radix digits; advancing by gridDim.x is a digit-wise add with carry
    struct ItemPos { int kind, grp, h, b; };
    auto decode_item = [&](long item) {
        ItemPos q;
        q.kind = (int)(item % kinds); item /= kinds;
        q.grp = (int)(item % n_groups); item /= n_groups;
        q.h = (int)(item % p.Hkv);
        q.b = (int)(item / p.Hkv);
        return q;
    };
    const ItemPos step = decode_item((long)gridDim.x);
    auto advance = [&](ItemPos q) {
        q.kind += step.kind; int cy = q.kind >= kinds; q.kind -= cy ? kinds : 0;
        q.grp += step.grp + cy; cy = q.grp >= n_groups; q.grp -= cy ? n_groups : 0;
        q.h += step.h + cy; cy = q.h >= p.Hkv; q.h -= cy ? p.Hkv : 0;
        q.b += step.b + cy;
        return q;
    };
    auto stage = [&](const ItemPos &q, int buf) {
        const int b = q.b, h = q.h, grp = q.grp, kind = q.kind;
        const __half *xbase = (kind == 0 ? k_src : v_src) + b * sb + h * sh + (int64_t)(grp * G) * stt;
        __half *Xt = Xbuf + (size_t)buf * G * D;
        constexpr int RPI = THREADS / CH;             // rows per iteration: 16, so (t & 7) is the same every iteration
        const int ch = tid % CH, t0 = tid / CH;
        const __half *src = xbase + (int64_t)t0 * stt + ch * 8;
        __half *dst = Xt + (size_t)t0 * D + (ch ^ (t0 & 7)) * 8;
#pragma unroll
        for (int i = 0; i < G / RPI; ++i) cp_async16(dst + (size_t)i * RPI * D, src + (int64_t)i * RPI * stt);
        if (tid < NT) {
            const int tok = first_token + grp * G + tid * KVSINK_TILE;   // multiple of 16
            tmask[buf * NT + tid] = (c.sink_bitmask[(size_t)b * p.mask_words + (tok >> 5)] >> (tok & 31)) & 0xffffu;
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    long item = blockIdx.x;
    ItemPos cur = decode_item(item);
    if (item < n_items) stage(cur, 0);
    for (int it = 0; item < n_items; item += gridDim.x, ++it) {
        const int buf = it & 1;
        const ItemPos nxt = advance(cur);
        if (item + gridDim.x < n_items) {
            stage(nxt, buf ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();   // the item's tile is in shared memory; everyone is done with the previous item's xout
        const int b = cur.b, h = cur.h, grp = cur.grp, kind = cur.kind;
        cur = nxt;
        const __half *Xt = Xbuf + (size_t)buf * G * D;
        const uint32_t *tm = tmask + buf * NT;
        const int64_t unit = (int64_t)b * p.Hkv + h;
        const int p0 = first_token + grp * G;
        bool has_sink = false;   // block-uniform; false for almost every item
#pragma unroll
        for (int T = 0; T < NT; ++T) has_sink |= tm[T] != 0;

        if (kind == 0) {
            // ================= keys: warp m owns channels [16m, 16m+16) of every tile =================
            const int m = warp;
            uint32_t a[NT][4];
            {
                const int row = rr + 8 * (mj & 1);
                const __half *src = Xt + (size_t)row * D + (((2 * m + (mj >> 1)) ^ (row & 7)) * 8);
#pragma unroll
                for (int T = 0; T < NT; ++T) ldmatrix_x4(a[T], src + (size_t)T * 16 * D);
            }
            // extremes per channel over the non-sink tokens: registers 0,1 hold channels (2t, 2t+1), registers 2,3 (2t+8, 2t+9)
            __half2 mnA = H_PINF, mxA = H_NINF, mnB = H_PINF, mxB = H_NINF;
            if (!has_sink) {
#pragma unroll
                for (int T = 0; T < NT; ++T) {
                    const __half2 *h = reinterpret_cast<const __half2 *>(a[T]);
                    mnA = __hmin2(mnA, __hmin2(h[0], h[1])); mxA = __hmax2(mxA, __hmax2(h[0], h[1]));
                    mnB = __hmin2(mnB, __hmin2(h[2], h[3])); mxB = __hmax2(mxB, __hmax2(h[2], h[3]));
                }
            } else {
#pragma unroll
                for (int T = 0; T < NT; ++T) {
                    const uint32_t m16 = tm[T];
                    const __half2 *h = reinterpret_cast<const __half2 *>(a[T]);
                    if (!((m16 >> g) & 1u)) { mnA = __hmin2(mnA, h[0]); mxA = __hmax2(mxA, h[0]); mnB = __hmin2(mnB, h[2]); mxB = __hmax2(mxB, h[2]); }
                    if (!((m16 >> (g + 8)) & 1u)) { mnA = __hmin2(mnA, h[1]); mxA = __hmax2(mxA, h[1]); mnB = __hmin2(mnB, h[3]); mxB = __hmax2(mxB, h[3]); }
                }
            }
            reduce_rows(mnA, mxA);
            reduce_rows(mnB, mxB);
            // parameters (Eq. 10-11): the lanes of a column group share its four channels (key g & 3)
            {
                const int kq = g & 3;
                const __half2 mn2 = (kq & 2) ? mnB : mnA, mx2 = (kq & 2) ? mxB : mxA;
                const __half lo = (kq & 1) ? __high2half(mn2) : __low2half(mn2), hi = (kq & 1) ? __high2half(mx2) : __low2half(mx2);
                const bool any = __half_as_ushort(lo) != 0x7C00;
                const float mn = __half2float(lo), mx = __half2float(hi);
                float s, z;
                group_params(any, mn, mx, qmax, &s, &z);
                if (g < 4) {
                    if constexpr (BITS != 2) scr.coder[4 * t4 + kq] = make_coder(s, z, mn, mx, qmax);
                    scr.sz[4 * t4 + kq] = make_float2(s, z);
                    const int ch = 16 * m + 2 * t4 + (kq & 1) + 8 * (kq >> 1);
                    const size_t o = ((size_t)unit * (p.max_seq / G) + p0 / G) * D + ch;
                    c.k_scale[o] = s;
                    c.k_zero[o] = z;
                }
                if constexpr (BITS == 2) warp_thresholds(s, z, g, qmax, reinterpret_cast<__half *>(&scr.thr[t4][kq >> 1][0]) + (kq & 1));
            }
            __syncwarp();
            const int lo_word = (BITS == 4) ? section_word_offset(NLO, lane, m) : section_word_offset(NLO, lane, m >> 1);
            if constexpr (BITS == 2) {
                __half2 tA[3], tB[3];
#pragma unroll
                for (int j = 0; j < 3; ++j) { tA[j] = scr.thr[t4][0][j]; tB[j] = scr.thr[t4][1][j]; }
                const __half2 base = __half2half2(__float2half(1024.f));
                const __half2 w0 = __half2half2(__float2half(1.f)), w1 = __half2half2(__float2half(4.f));
                const __half2 w2 = __half2half2(__float2half(16.f)), w3 = __half2half2(__float2half(64.f));
                const __half2 zero2 = __half2half2(__float2half(0.f));
                uint8_t *wb0 = (uint8_t *)(xout + lo_word) + (m & 1);
                if (!has_sink) {
#pragma unroll
                    for (int T = 0; T < NT; ++T) {
                        __half2 acc = base;
                        acc = thermo_accumulate(acc, a[T][0], tA, w0);
                        acc = thermo_accumulate(acc, a[T][1], tA, w1);
                        acc = thermo_accumulate(acc, a[T][2], tB, w2);
                        acc = thermo_accumulate(acc, a[T][3], tB, w3);
                        const uint32_t bits = *reinterpret_cast<uint32_t *>(&acc);   // 0x6400 | byte in each half
                        uint8_t *wb = wb0 + T * TILE_WORDS * 4;
                        wb[0] = (uint8_t)bits;
                        wb[2] = (uint8_t)(bits >> 16);
                    }
                } else {
#pragma unroll
                    for (int T = 0; T < NT; ++T) {   // sink tokens keep code 0: pair slots 0, 2 are row g, slots 1, 3 row g + 8
                        const uint32_t m16 = tm[T];
                        const bool s0 = (m16 >> g) & 1u, s1 = (m16 >> (g + 8)) & 1u;
                        __half2 acc = base;
                        acc = thermo_accumulate(acc, a[T][0], tA, s0 ? zero2 : w0);
                        acc = thermo_accumulate(acc, a[T][1], tA, s1 ? zero2 : w1);
                        acc = thermo_accumulate(acc, a[T][2], tB, s0 ? zero2 : w2);
                        acc = thermo_accumulate(acc, a[T][3], tB, s1 ? zero2 : w3);
                        const uint32_t bits = *reinterpret_cast<uint32_t *>(&acc);
                        uint8_t *wb = wb0 + T * TILE_WORDS * 4;
                        wb[0] = (uint8_t)bits;
                        wb[2] = (uint8_t)(bits >> 16);
                    }
                }
            } else {
                Coder kc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) kc[q] = scr.coder[4 * t4 + q];
                const int hi_word = (BITS == 3) ? 32 * NLO + section_word_offset(NHI > 0 ? NHI : 1, lane, m >> 2) : 0;
                if constexpr (BITS == 3) {   // hi words are OR-ed together by the four warps that share them
                    for (int i = tid; i < 32 * NHI * NT; i += THREADS) xout[(i / (32 * NHI)) * TILE_WORDS + 32 * NLO + i % (32 * NHI)] = 0;
                    __syncthreads();
                }
#pragma unroll
                for (int T = 0; T < NT; ++T) {
                    uint32_t pc[4], differ = 0;
#pragma unroll
                    for (int r = 0; r < 4; ++r) pc[r] = code_pair<BITS>(a[T][r], kc[2 * (r >> 1)], kc[2 * (r >> 1) + 1], differ);
                    const uint32_t m16 = tm[T];
                    if (differ | m16) {   // rare: a value too close to a rounding tie, or a tile with sink tokens
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const float2 z0 = scr.sz[4 * t4 + 2 * (r >> 1)], z1 = scr.sz[4 * t4 + 2 * (r >> 1) + 1];
                            pc[r] = code_pair_exact<BITS>(a[T][r], z0.x, z0.y, z1.x, z1.y);
                        }
                        // sink tokens keep code 0 in the packed stream: pair slots 0, 2 are row g, slots 1, 3 row g + 8
                        if ((m16 >> g) & 1u) pc[0] = pc[2] = 0;
                        if ((m16 >> (g + 8)) & 1u) pc[1] = pc[3] = 0;
                    }
                    uint32_t lo, hi;
                    pack_matrix<BITS>(pc, m, &lo, &hi);
                    uint32_t *tile = xout + T * TILE_WORDS;
                    if constexpr (BITS == 4) {
                        tile[lo_word] = lo;
                    } else {
                        uint8_t *wb = (uint8_t *)(tile + lo_word);
                        wb[m & 1] = (uint8_t)lo;
                        wb[2 + (m & 1)] = (uint8_t)(lo >> 16);
                        if constexpr (BITS == 3) atomicOr(&tile[hi_word], hi);
                    }
                }
            }
        } else {
            // ================= values: a warp owns a tile (16 tokens x D channels), or one channel group of a tile
            //                    when there are fewer tiles than warps =================
            constexpr int JG = (NT < NW && !(BITS == 3 && MPG < 4)) ? NGv : 1;   // jobs per tile (3-bit hi words span 4 matrices)
            for (int job = warp; job < NT * JG; job += NW) {
                const int T = job / JG, my_jg = job % JG;
                const uint32_t m16 = tm[T];
                uint32_t wl[NLO], wh[NHI > 0 ? NHI : 1];
#pragma unroll
                for (int i = 0; i < NLO; ++i) wl[i] = 0;
#pragma unroll
                for (int i = 0; i < (NHI > 0 ? NHI : 1); ++i) wh[i] = 0;
                const int row = 16 * T + rr + 8 * (mj >> 1);
                const __half *rowp = Xt + (size_t)row * D;
#pragma unroll
                for (int jg = 0; jg < NGv; ++jg) {
                    if (JG > 1 && jg != my_jg) continue;   // warp-uniform
                    uint32_t a[MPG][4];
#pragma unroll
                    for (int mi = 0; mi < MPG; ++mi)
                        ldmatrix_x4_trans(a[mi], rowp + (((2 * (jg * MPG + mi) + (mj & 1)) ^ (row & 7)) * 8));
                    // extremes per token over the group's channels: registers 0,1 hold tokens (2t, 2t+1), registers 2,3 (2t+8, 2t+9)
                    __half2 mnA = H_PINF, mxA = H_NINF, mnB = H_PINF, mxB = H_NINF;
#pragma unroll
                    for (int mi = 0; mi < MPG; ++mi) {
                        const __half2 *h = reinterpret_cast<const __half2 *>(a[mi]);
                        mnA = __hmin2(mnA, __hmin2(h[0], h[1])); mxA = __hmax2(mxA, __hmax2(h[0], h[1]));
                        mnB = __hmin2(mnB, __hmin2(h[2], h[3])); mxB = __hmax2(mxB, __hmax2(h[2], h[3]));
                    }
                    reduce_rows(mnA, mxA);
                    reduce_rows(mnB, mxB);
                    {
                        const int kq = g & 3;
                        const __half2 mn2 = (kq & 2) ? mnB : mnA, mx2 = (kq & 2) ? mxB : mxA;
                        const __half lo = (kq & 1) ? __high2half(mn2) : __low2half(mn2), hi = (kq & 1) ? __high2half(mx2) : __low2half(mx2);
                        const int tk = 2 * t4 + (kq & 1) + 8 * (kq >> 1);      // token within the tile
                        const bool member = !((m16 >> tk) & 1u);
                        const float mn = __half2float(lo), mx = __half2float(hi);
                        float s, z;
                        group_params(member, mn, mx, qmax, &s, &z);
                        if (g < 4) {
                            if constexpr (BITS != 2) scr.coder[4 * t4 + kq] = make_coder(s, z, mn, mx, qmax);
                            scr.sz[4 * t4 + kq] = make_float2(s, z);
                            const size_t o = ((size_t)unit * p.max_seq + p0 + 16 * T + tk) * NGv + jg;
                            c.v_scale[o] = s;
                            c.v_zero[o] = z;
                        }
                        if constexpr (BITS == 2)
                            warp_thresholds(s, z, g, qmax, reinterpret_cast<__half *>(&scr.thr[t4][kq >> 1][0]) + (kq & 1));
                    }
                    __syncwarp();
                    if constexpr (BITS == 2) {
                        __half2 tA[3], tB[3];
#pragma unroll
                        for (int j = 0; j < 3; ++j) { tA[j] = scr.thr[t4][0][j]; tB[j] = scr.thr[t4][1][j]; }
                        const __half2 base = __half2half2(__float2half(1024.f));
                        const __half2 w0 = __half2half2(__float2half(1.f)), w1 = __half2half2(__float2half(4.f));
                        const __half2 w2 = __half2half2(__float2half(16.f)), w3 = __half2half2(__float2half(64.f));
#pragma unroll
                        for (int mi = 0; mi < MPG; ++mi) {
                            const int m = jg * MPG + mi;
                            __half2 acc = base;
                            acc = thermo_accumulate(acc, a[mi][0], tA, w0);
                            acc = thermo_accumulate(acc, a[mi][1], tA, w1);
                            acc = thermo_accumulate(acc, a[mi][2], tB, w2);
                            acc = thermo_accumulate(acc, a[mi][3], tB, w3);
                            const uint32_t bits = *reinterpret_cast<uint32_t *>(&acc) & 0x00ff00ffu;
                            wl[m >> 1] |= bits << (8 * (m & 1));
                        }
                    } else {
                        Coder vc[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) vc[q] = scr.coder[4 * t4 + q];
#pragma unroll
                        for (int mi = 0; mi < MPG; ++mi) {
                            const int m = jg * MPG + mi;
                            uint32_t pc[4], differ = 0;
#pragma unroll
                            for (int r = 0; r < 4; ++r) pc[r] = code_pair<BITS>(a[mi][r], vc[2 * (r >> 1)], vc[2 * (r >> 1) + 1], differ);
                            if (differ) {   // rare: a value too close to a rounding tie
#pragma unroll
                                for (int r = 0; r < 4; ++r) {
                                    const float2 z0 = scr.sz[4 * t4 + 2 * (r >> 1)], z1 = scr.sz[4 * t4 + 2 * (r >> 1) + 1];
                                    pc[r] = code_pair_exact<BITS>(a[mi][r], z0.x, z0.y, z1.x, z1.y);
                                }
                            }
                            uint32_t lo, hi;
                            pack_matrix<BITS>(pc, m, &lo, &hi);
                            if constexpr (BITS == 4) {
                                wl[m] = lo;
                            } else {
                                wl[m >> 1] |= lo << (8 * (m & 1));
                                if constexpr (BITS == 3) wh[m >> 2] |= hi;
                            }
                        }
                    }
                    __syncwarp();   // the scratch is rewritten for the next channel group / tile
                }
                uint32_t *tile = xout + T * TILE_WORDS;
#pragma unroll
                for (int i = 0; i < NLO; ++i) {
                    const int word_jg = ((BITS == 4) ? i : 2 * i) / MPG;   // channel group of the word's matrices
                    if (JG == 1 || word_jg == my_jg) tile[section_word_offset(NLO, lane, i)] = wl[i];
                }
                if constexpr (BITS == 3) {
#pragma unroll
                    for (int i = 0; i < NHI; ++i)
                        if (JG == 1 || (4 * i) / MPG == my_jg) tile[32 * NLO + section_word_offset(NHI, lane, i)] = wh[i];
                }
            }
        }

        // ---- sink rows: exact copies into the side buffer at the rank of their position (prefill only) ----
        if (kinds == 2) {
            if (has_sink) {
                const int count = min(c.sink_count[b], p.cap);
                const int32_t *sp = c.sink_pos + (size_t)b * p.cap;
                __half *side = (__half *)(kind == 0 ? c.sink_k : c.sink_v);
                for (int t = warp; t < G; t += NW) {
                    if (!((tm[t >> 4] >> (t & 15)) & 1u)) continue;
                    int lo = 0, hi = count - 1, slot = -1;
                    while (lo <= hi) {
                        const int mid = (lo + hi) >> 1, v = sp[mid];
                        if (v == p0 + t) { slot = mid; break; }
                        if (v < p0 + t) lo = mid + 1; else hi = mid - 1;
                    }
                    if (slot < 0) {
                        if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
                        continue;
                    }
                    if (lane < CH)
                        *(uint4 *)(side + ((size_t)unit * p.cap + slot) * D + lane * 8) =
                            *(const uint4 *)(Xt + (size_t)t * D + ((lane ^ (t & 7)) * 8));
                }
            }
        }
        __syncthreads();   // all words of the item are in xout; nobody reads this tile buffer any more

        // ---- store the group's tiles (contiguous in memory) ----
        {
            uint8_t *codes = kind == 0 ? c.k_codes : c.v_codes;
            uint4 *dst = (uint4 *)(codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)(p0 / KVSINK_TILE) * p.tile_bytes);
            constexpr int N16 = NT * TILE_WORDS / 4;
            for (int i = tid; i < N16; i += THREADS) dst[i] = ((const uint4 *)xout)[i];
        }
    }
}

template <int BITS, int D, int G>
static int launch_stream(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                         int64_t sb, int64_t sh, int64_t stt, bool do_v, cudaStream_t st)
{
    constexpr int NT = G / KVSINK_TILE, W = D * BITS / 64, NW = D / 16;
    constexpr size_t smem = 2 * (size_t)G * D * 2 + (size_t)NT * 32 * W * 4 + NW * sizeof(WarpScratch) + 2 * NT * 4 + 16;
    static_assert(smem <= 227 * 1024, "tile too large");
    auto kern = quantize_groups_stream<BITS, D, G>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    const int kinds = do_v ? 2 : 1;
    const long n_items = (long)p.B * p.Hkv * n_groups * kinds;
    int per_sm = (int)((227 * 1024) / (smem + 1024));
    const int cap = (D == 128) ? 3 : 4;
    if (per_sm > cap) per_sm = cap;
    long blocks = 148L * per_sm;
    if (blocks > n_items) blocks = n_items;
    note_launch();
    kern<<<(unsigned)blocks, 32 * NW, smem, st>>>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, kinds);
    return cudaGetLastError() == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

template <int BITS, int D>
static int launch_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                       int64_t sb, int64_t sh, int64_t stt, bool do_v, cudaStream_t st)
{
    switch (p.G) {
    case 32: return launch_stream<BITS, D, 32>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    case 64: return launch_stream<BITS, D, 64>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    case 128: return launch_stream<BITS, D, 128>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    default: return KVSINK_ERR_UNSUPPORTED;
    }
}

// Returns KVSINK_ERR_UNSUPPORTED when the shape has no streaming kernel (the caller then uses the generic one).
int launch_quantize_groups_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                                int n_groups, int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st)
{
    if (p.D == 128) {
        if (p.bits == 2) return launch_fast<2, 128>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
        if (p.bits == 3) return launch_fast<3, 128>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
        if (p.bits == 4) return launch_fast<4, 128>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
    } else if (p.D == 64) {
        if (p.bits == 2) return launch_fast<2, 64>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
        if (p.bits == 4) return launch_fast<4, 64>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
    }
    return KVSINK_ERR_UNSUPPORTED;
}

}  // namespace kvsink
