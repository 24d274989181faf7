// Whole-group quantization (Eq. 8-11 with Algorithm 1's sink exclusion) at streaming speed.
//
// One block per (token group, KV head, sequence).  The group's K and V tiles (G x D fp16 each) are staged once in
// shared memory with cp.async into XOR-swizzled 16-byte chunks, so HBM is read exactly once.  Statistics run in
// fp16 (exact), parameters in IEEE binary32.  Codes are produced in the register layout of the packed tile:
// ldmatrix hands every lane exactly the elements of its pair slots (ldmatrix.trans for V, whose tiles are
// [channel x token]).  The literal  rint(x / scale) + zero  is reproduced bit for bit without a division per
// element: y = fma(x, r, M + zero) with r = 1/scale nudged down and up by 2^-22 and M = 1.5 * 2^23 rounds the
// product to an integer in the mantissa; if both nudged results agree, no rounding of x/scale can land on the other
// side of a tie and the agreed integer is the exact answer; if they differ (about one element in 10^5) the lane
// recomputes its batch with the IEEE division.
#include "common.cuh"

namespace kvsink {

constexpr int QF_THREADS = 256;
constexpr int QF_WARPS = QF_THREADS / 32;
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

// Field masks of matrix row g (pair slots r = 0, 2) in the forms pack_matrix returns, before placement.
template <int BITS> struct RowMask;
template <> struct RowMask<2> { static constexpr uint32_t LO = 0x00330033u, HI = 0u; };
template <> struct RowMask<4> { static constexpr uint32_t LO = 0x0f0f0f0fu, HI = 0u; };
template <> struct RowMask<3> { static constexpr uint32_t LO = 0x00330033u, HI = 0x00110011u; };

// Codes of one value tile (16 tokens x D channels) in the tile's register layout, written to `tile` (shared memory).
// The lane's four tokens are 2*t4, 2*t4+1, 2*t4+8, 2*t4+9.  Returns (warp-uniform) whether any lane's fast result
// is not certain; with EXACT those matrices are recomputed with the IEEE division.
template <int BITS, int D, int NGv, bool EXACT>
__device__ __forceinline__ bool encode_v_tile(const __half *Xt, const Coder *coder, const float *xscale, const float *xzero, int T,
                                              int lane, uint32_t *tile)
{
    constexpr int W = D * BITS / 64;
    constexpr int NLO = (BITS == 3) ? D / 32 : W, NHI = (BITS == 3) ? D / 64 : 0;
    constexpr int mpg = (D / NGv) / 16;      // matrices per channel group
    const int t4 = lane & 3, mj = lane >> 3, rr = lane & 7;
    const int tok = 16 * T + rr + 8 * (mj >> 1), tk0 = 16 * T + 2 * t4;
    const __half *rowp = Xt + (size_t)tok * D;
    const int sw = tok & 7;
    uint32_t wl[NLO], wh[NHI > 0 ? NHI : 1], differ_all = 0;
#pragma unroll
    for (int i = 0; i < NLO; ++i) wl[i] = 0;
#pragma unroll
    for (int i = 0; i < (NHI > 0 ? NHI : 1); ++i) wh[i] = 0;
#pragma unroll
    for (int jg = 0; jg < NGv; ++jg) {
        Coder vc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) vc[q] = coder[(tk0 + (q & 1) + 8 * (q >> 1)) * NGv + jg];
#pragma unroll
        for (int mi = 0; mi < mpg; ++mi) {
            const int m = jg * mpg + mi;
            uint32_t a[4], pc[4], differ = 0;
            ldmatrix_x4_trans(a, rowp + (((2 * m + (mj & 1)) ^ sw) * 8));
#pragma unroll
            for (int r = 0; r < 4; ++r) pc[r] = code_pair<BITS>(a[r], vc[2 * (r >> 1)], vc[2 * (r >> 1) + 1], differ);
            if (EXACT && differ) {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i0 = (tk0 + 8 * (r >> 1)) * NGv + jg;
                    pc[r] = code_pair_exact<BITS>(a[r], xscale[i0], xzero[i0], xscale[i0 + NGv], xzero[i0 + NGv]);
                }
            }
            differ_all |= differ;
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
    if (!EXACT && __any_sync(0xffffffffu, differ_all != 0)) return true;
#pragma unroll
    for (int i = 0; i < NLO; ++i) tile[section_word_offset(NLO, lane, i)] = wl[i];
    if constexpr (BITS == 3) {
#pragma unroll
        for (int i = 0; i < NHI; ++i) tile[32 * NLO + section_word_offset(NHI, lane, i)] = wh[i];
    }
    return false;
}

template <int BITS, int D, int NGv>
__global__ void __launch_bounds__(QF_THREADS, 3)
quantize_groups_fast(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src, int first_token,
                     int n_groups, int64_t sb, int64_t sh, int64_t stt, int kinds)
{
    constexpr int CH = D / 8;            // 16-byte chunks per row
    constexpr int NM = D / 16;           // 16x16 matrices per tile
    constexpr int NSET = D / 32;         // 32-channel sets per row
    constexpr int W = D * BITS / 64;     // words per lane per tile
    constexpr int NLO = (BITS == 3) ? D / 32 : W, NHI = (BITS == 3) ? D / 64 : 0;
    constexpr int TILE_WORDS = 32 * W;
    const float qmax = (float)((1 << BITS) - 1);
    constexpr int Gv = D / NGv;
    const int G = p.G, n_tiles = G / KVSINK_TILE;

    extern __shared__ __align__(128) unsigned char smem[];
    __half *Xbuf = (__half *)smem;                                 // [2][G][D] swizzled 16-byte chunks (double buffer)
    Coder *coder = (Coder *)(Xbuf + 2 * (size_t)G * D);            // keys: [D]; values: [G][NGv]
    const int max_coders = D > G * NGv ? D : G * NGv;
    float *xscale = (float *)(coder + max_coders);                 // same indexing as coder
    float *xzero = xscale + max_coders;
    uint32_t *tmask = (uint32_t *)(xzero + max_coders);            // [2][n_tiles] sink bits of each tile
    uint32_t *stat = tmask + 2 * n_tiles;                          // keys: [warps][D]; values: [G][NSET]  (min | max << 16)
    uint32_t *xout = stat;                                         // [n_tiles][TILE_WORDS], reuses the statistics area

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const int mj = lane >> 3, rr = lane & 7;      // ldmatrix: this lane addresses row rr of 8x8 block mj
    const long n_items = (long)p.B * p.Hkv * n_groups * kinds;

    // item -> (sequence, head, group, kind); a block quantizes the keys (kind 0) or the values (kind 1) of a group
    auto decode_item = [&](long item, int *b, int *h, int *grp, int *kind) {
        *kind = (int)(item % kinds); item /= kinds;
        *grp = (int)(item % n_groups); item /= n_groups;
        *h = (int)(item % p.Hkv);
        *b = (int)(item / p.Hkv);
    };
    auto stage = [&](long item, int buf) {
        int b, h, grp, kind;
        decode_item(item, &b, &h, &grp, &kind);
        const __half *xbase = (kind == 0 ? k_src : v_src) + b * sb + h * sh + (int64_t)(grp * G) * stt;
        __half *Xt = Xbuf + (size_t)buf * G * D;
        {
            constexpr int RPI = QF_THREADS / CH;          // rows per iteration (a multiple of 8, so t & 7 is fixed)
            const int ch = tid % CH, t0 = tid / CH;
            const __half *src = xbase + (int64_t)t0 * stt + ch * 8;
            __half *dst = Xt + (size_t)t0 * D + (ch ^ (t0 & 7)) * 8;
            for (int t = t0; t < G; t += RPI, src += (int64_t)RPI * stt, dst += (size_t)RPI * D) cp_async16(dst, src);
        }
        if (tid < n_tiles) {
            const int tok = first_token + grp * G + tid * KVSINK_TILE;   // multiple of 16
            tmask[buf * n_tiles + tid] = (c.sink_bitmask[(size_t)b * p.mask_words + (tok >> 5)] >> (tok & 31)) & 0xffffu;
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    long item = blockIdx.x;
    if (item < n_items) stage(item, 0);
    for (int it = 0; item < n_items; item += gridDim.x, ++it) {
        const int buf = it & 1;
        if (item + gridDim.x < n_items) {
            stage(item + gridDim.x, buf ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        int b, h, grp, kind;
        decode_item(item, &b, &h, &grp, &kind);
        const __half *Xt = Xbuf + (size_t)buf * G * D;
        const uint32_t *tm = tmask + buf * n_tiles;
        const int64_t unit = (int64_t)b * p.Hkv + h;
        const int p0 = first_token + grp * G;
        auto is_sink = [&](int t) { return (tm[t >> 4] >> (t & 15)) & 1u; };

        if (kind == 0) {
            // ---- keys: per-channel statistics over the non-sink tokens (column slices) ----
            {
                constexpr int NS = QF_THREADS / CH;      // token slices
                const int cidx = tid % CH, slice = tid / CH;
                __half2 mn[4], mx[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { mn[i] = __half2half2(__ushort_as_half(0x7C00)); mx[i] = __half2half2(__ushort_as_half(0xFC00)); }
                for (int t = slice; t < G; t += NS) {
                    if (is_sink(t)) continue;
                    const uint4 v = *(const uint4 *)(Xt + (size_t)t * D + ((cidx ^ (t & 7)) * 8));
                    const __half2 *hv = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
                    for (int i = 0; i < 4; ++i) { mn[i] = __hmin2(mn[i], hv[i]); mx[i] = __hmax2(mx[i], hv[i]); }
                }
#pragma unroll
                for (int o = CH; o < 32; o <<= 1)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t a = __shfl_xor_sync(0xffffffffu, *reinterpret_cast<uint32_t *>(&mn[i]), o);
                        uint32_t bb = __shfl_xor_sync(0xffffffffu, *reinterpret_cast<uint32_t *>(&mx[i]), o);
                        mn[i] = __hmin2(mn[i], *reinterpret_cast<__half2 *>(&a));
                        mx[i] = __hmax2(mx[i], *reinterpret_cast<__half2 *>(&bb));
                    }
                if (lane < CH) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t a = *reinterpret_cast<uint32_t *>(&mn[i]), bb = *reinterpret_cast<uint32_t *>(&mx[i]);
                        stat[warp * D + cidx * 8 + 2 * i] = (a & 0xffffu) | (bb << 16);
                        stat[warp * D + cidx * 8 + 2 * i + 1] = (a >> 16) | (bb & 0xffff0000u);
                    }
                }
            }
            __syncthreads();
            // ---- parameters (Eq. 10-11) and coders ----
            for (int ch = tid; ch < D; ch += QF_THREADS) {
                __half lo = __ushort_as_half(0x7C00), hi = __ushort_as_half(0xFC00);
#pragma unroll
                for (int w = 0; w < QF_WARPS; ++w) {
                    const uint32_t v = stat[w * D + ch];
                    lo = __hmin(lo, __ushort_as_half((unsigned short)(v & 0xffffu)));
                    hi = __hmax(hi, __ushort_as_half((unsigned short)(v >> 16)));
                }
                const bool any = __half_as_ushort(lo) != 0x7C00;
                const float mn = __half2float(lo), mx = __half2float(hi);
                float s, z;
                group_params(any, mn, mx, qmax, &s, &z);
                xscale[ch] = s;
                xzero[ch] = z;
                coder[ch] = make_coder(s, z, mn, mx, qmax);
                const size_t o = ((size_t)unit * (p.max_seq / G) + p0 / G) * D + ch;
                c.k_scale[o] = s;
                c.k_zero[o] = z;
            }
            __syncthreads();   // parameters visible; statistics no longer needed (xout reuses their space)
            if constexpr (BITS == 3)
                for (int i = tid; i < 32 * NHI * n_tiles; i += QF_THREADS) xout[(i / (32 * NHI)) * TILE_WORDS + 32 * NLO + i % (32 * NHI)] = 0;
            if constexpr (BITS == 3) __syncthreads();
            // ---- codes in the tile's register layout: a warp takes one matrix over a range of tiles ----
            {
                constexpr int CHUNKS = QF_WARPS / NM;
                const int m = warp % NM, part = warp / NM;
                const int tb = (n_tiles * part) / CHUNKS, te = (n_tiles * (part + 1)) / CHUNKS;
                Coder kc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) kc[q] = coder[16 * m + 2 * t4 + (q & 1) + 8 * (q >> 1)];
                const int lo_word = (BITS == 4) ? section_word_offset(NLO, lane, m) : section_word_offset(NLO, lane, m >> 1);
                const int hi_word = (BITS == 3) ? 32 * NLO + section_word_offset(NHI > 0 ? NHI : 1, lane, m >> 2) : 0;
                const int row_in_tile = rr + 8 * (mj & 1), chunk = 2 * m + (mj >> 1);
                for (int T = tb; T < te; ++T) {
                    uint32_t a[4], pc[4], differ = 0;
                    const int tok = 16 * T + row_in_tile;
                    ldmatrix_x4(a, Xt + (size_t)tok * D + ((chunk ^ (tok & 7)) * 8));
#pragma unroll
                    for (int r = 0; r < 4; ++r) pc[r] = code_pair<BITS>(a[r], kc[2 * (r >> 1)], kc[2 * (r >> 1) + 1], differ);
                    const uint32_t m16 = tm[T];
                    if (differ | m16) {   // rare: a value too close to a rounding tie, or a tile with sink tokens
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const int ch = 16 * m + 2 * t4 + 8 * (r >> 1);
                            pc[r] = code_pair_exact<BITS>(a[r], xscale[ch], xzero[ch], xscale[ch + 1], xzero[ch + 1]);
                        }
                    }
                    uint32_t lo, hi;
                    pack_matrix<BITS>(pc, m, &lo, &hi);
                    if (m16) {   // sink tokens keep code 0 in the packed stream
                        uint32_t keep = 0xffffffffu, keeph = 0xffffffffu;
                        const int hsh = 8 * (m & 1) + 2 * (1 - ((m >> 1) & 1));
                        if ((m16 >> g) & 1u) { keep &= ~RowMask<BITS>::LO; keeph &= ~(RowMask<BITS>::HI << hsh); }
                        if ((m16 >> (g + 8)) & 1u) { keep &= ~(RowMask<BITS>::LO << (BITS == 4 ? 4 : 2)); keeph &= ~(RowMask<BITS>::HI << (hsh + 1)); }
                        lo &= keep;
                        hi &= keeph;
                    }
                    uint32_t *tile = xout + (size_t)T * TILE_WORDS;
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
            // ---- values: per-token statistics over 32-channel sets, two threads per token ----
            {
                constexpr int SPT = (D == 128) ? 2 : 1;      // sets per thread
                for (int i2 = tid; i2 < 2 * G; i2 += QF_THREADS) {
                    const int t = i2 >> 1, hh = i2 & 1;
#pragma unroll
                    for (int sidx = 0; sidx < SPT; ++sidx) {
                        const int set = (D == 128) ? (hh + 2 * sidx) : hh;
                        __half2 mn = __half2half2(__ushort_as_half(0x7C00)), mx = __half2half2(__ushort_as_half(0xFC00));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int ch = 4 * set + j;
                            const uint4 v = *(const uint4 *)(Xt + (size_t)t * D + ((ch ^ (t & 7)) * 8));
                            const __half2 *hv = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
                            for (int i = 0; i < 4; ++i) { mn = __hmin2(mn, hv[i]); mx = __hmax2(mx, hv[i]); }
                        }
                        const __half lo = __hmin(__low2half(mn), __high2half(mn)), hi = __hmax(__low2half(mx), __high2half(mx));
                        stat[t * NSET + set] = (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
                    }
                }
            }
            __syncthreads();
            {
                constexpr int spg = Gv / 32;     // sets per channel group
                for (int i2 = tid; i2 < G * NGv; i2 += QF_THREADS) {
                    const int t = i2 / NGv, j = i2 % NGv;
                    float s = 0.f, z = 0.f, gmn = 0.f, gmx = 0.f;
                    if (!is_sink(t)) {
                        __half lo = __ushort_as_half(0x7C00), hi = __ushort_as_half(0xFC00);
                        for (int q = 0; q < spg; ++q) {
                            const uint32_t v = stat[t * NSET + j * spg + q];
                            lo = __hmin(lo, __ushort_as_half((unsigned short)(v & 0xffffu)));
                            hi = __hmax(hi, __ushort_as_half((unsigned short)(v >> 16)));
                        }
                        gmn = __half2float(lo);
                        gmx = __half2float(hi);
                        group_params(true, gmn, gmx, qmax, &s, &z);
                    }
                    xscale[i2] = s;
                    xzero[i2] = z;
                    coder[i2] = make_coder(s, z, gmn, gmx, qmax);
                    const size_t o = ((size_t)unit * p.max_seq + p0 + t) * NGv + j;
                    c.v_scale[o] = s;
                    c.v_zero[o] = z;
                }
            }
            __syncthreads();
            // ---- codes: a warp takes whole tiles ----
            for (int T = warp; T < n_tiles; T += QF_WARPS) {
                uint32_t *tile = xout + (size_t)T * TILE_WORDS;
                // everything through the fast coder; if any lane saw a value too close to a rounding tie (rare), the whole
                // warp repeats the tile with the exact division where a lane's matrix needs it
                if (encode_v_tile<BITS, D, NGv, false>(Xt, coder, xscale, xzero, T, lane, tile))
                    encode_v_tile<BITS, D, NGv, true>(Xt, coder, xscale, xzero, T, lane, tile);
            }
        }
        __syncthreads();

        // ---- store the group's tiles (contiguous in memory) ----
        {
            uint8_t *codes = kind == 0 ? c.k_codes : c.v_codes;
            uint4 *dst = (uint4 *)(codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)(p0 / KVSINK_TILE) * p.tile_bytes);
            const int n16 = n_tiles * TILE_WORDS / 4;
            for (int i = tid; i < n16; i += QF_THREADS) dst[i] = ((const uint4 *)xout)[i];
        }

        // ---- sink rows: exact copies into the side buffer at the rank of their position (prefill only) ----
        if (kinds == 2) {
            bool any = false;
            for (int T = 0; T < n_tiles; ++T) any |= tm[T] != 0;
            if (any) {
                const int count = min(c.sink_count[b], p.cap);
                const int32_t *sp = c.sink_pos + (size_t)b * p.cap;
                __half *side = (__half *)(kind == 0 ? c.sink_k : c.sink_v);
                for (int t = warp; t < G; t += QF_WARPS) {
                    if (!is_sink(t)) continue;
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
        __syncthreads();   // the next iteration's prefetch overwrites this buffer's neighbour; xout and coders are reused
    }
}

template <int BITS, int D, int NGV>
static int launch_fast_n(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                         int64_t sb, int64_t sh, int64_t stt, bool do_v, cudaStream_t st)
{
    const int G = p.G, n_tiles = G / KVSINK_TILE;
    constexpr int W = D * BITS / 64;
    const size_t max_coders = (size_t)(D > G * NGV ? D : G * NGV);
    size_t stat_words = (size_t)(QF_WARPS * D > G * (D / 32) ? QF_WARPS * D : G * (D / 32));
    if (stat_words < (size_t)n_tiles * 32 * W) stat_words = (size_t)n_tiles * 32 * W;
    const size_t smem = 2 * (size_t)G * D * 2 + max_coders * (16 + 8) + stat_words * 4 + 2 * (size_t)n_tiles * 4 + 16;
    if (smem > 227 * 1024) return KVSINK_ERR_UNSUPPORTED;
    auto kern = quantize_groups_fast<BITS, D, NGV>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    const int kinds = do_v ? 2 : 1;
    const long n_items = (long)p.B * p.Hkv * n_groups * kinds;
    int per_sm = (int)((227 * 1024) / (smem + 1024));
    if (per_sm > 3) per_sm = 3;
    if (per_sm < 1) per_sm = 1;
    long blocks = 148L * per_sm;
    if (blocks > n_items) blocks = n_items;
    kern<<<(unsigned)blocks, QF_THREADS, smem, st>>>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, kinds);
    return cudaGetLastError() == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

template <int BITS, int D>
static int launch_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                       int64_t sb, int64_t sh, int64_t stt, bool do_v, cudaStream_t st)
{
    if (p.NGv == 1) return launch_fast_n<BITS, D, 1>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    if (p.NGv == 2) return launch_fast_n<BITS, D, 2>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    if constexpr (D == 128)
        if (p.NGv == 4) return launch_fast_n<BITS, D, 4>(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, do_v, st);
    return KVSINK_ERR_UNSUPPORTED;
}

// Returns KVSINK_ERR_UNSUPPORTED when the shape has no streaming kernel (the caller then uses the generic one).
int launch_quantize_groups_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                                int n_groups, int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st)
{
    if (p.Gv < 32 || p.G > 512) return KVSINK_ERR_UNSUPPORTED;
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
