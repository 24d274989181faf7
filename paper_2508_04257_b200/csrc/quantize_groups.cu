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
    float r_lo, r_hi;   // 1/scale nudged down / up; +inf forces the exact path
    float magic;        // M + zero
    float ymax;         // M + zero clamp: M + qmax
};

__device__ __forceinline__ Coder make_coder(float scale, float zero, float absmax, float qmax)
{
    Coder c;
    if (scale == 0.f) {   // no member, or sink token: code 0
        c.r_lo = c.r_hi = 0.f;
        c.magic = MAGIC;
        c.ymax = MAGIC + qmax;
        return c;
    }
    const float r = __frcp_rn(scale);
    // the integer-in-mantissa trick needs |x/scale| and |zero| well below 2^22
    const bool ok = absmax * r < 2097152.f && fabsf(zero) < 2097152.f && r < 3.0e38f;
    c.r_lo = ok ? __fmul_rn(r, 1.f - 2.384185791015625e-07f) : __int_as_float(0x7f800000);
    c.r_hi = ok ? __fmul_rn(r, 1.f + 2.384185791015625e-07f) : r;
    c.magic = MAGIC + (ok ? zero : 0.f);
    c.ymax = MAGIC + qmax;
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
    const uint32_t u0 = __float_as_uint(fminf(a0, c0.ymax)), u1 = __float_as_uint(fminf(a1, c1.ymax));
    // low halves of u0 and u1 (the bit pattern of 1.5 * 2^23 has a zero low half); the mask only matters for rows that are discarded
    return __byte_perm(u0, u1, 0x5410) & (((1u << BITS) - 1u) * 0x00010001u);
}

template <int BITS>
__device__ __forceinline__ uint32_t code_pair_exact(uint32_t h2, float s0, float z0, float s1, float z1)
{
    const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    const float qmax = (float)((1 << BITS) - 1);
    const uint32_t c0 = s0 == 0.f ? 0u : code_exact(x.x, s0, z0, qmax);
    const uint32_t c1 = s1 == 0.f ? 0u : code_exact(x.y, s1, z1, qmax);
    return c0 | (c1 << 16);
}

// Words of one lane for a pair of matrices (2m0, 2m0+1) of a tile from the eight code pairs pc[mm][r].
// 2 bit: one word.  4 bit: two words.  3 bit: one lo word and this pair's bits of the shared hi word.
template <int BITS>
__device__ __forceinline__ void pack_pair(const uint32_t (&pc)[2][4], int pair_index, uint32_t *w0, uint32_t *w1)
{
    if constexpr (BITS == 2) {
        uint32_t w = 0;
#pragma unroll
        for (int mm = 0; mm < 2; ++mm)
#pragma unroll
            for (int r = 0; r < 4; ++r) w |= pc[mm][r] << (2 * (4 * mm + r));
        *w0 = w;
        *w1 = 0;
    } else if constexpr (BITS == 4) {
        uint32_t a = 0, b = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) { a |= pc[0][r] << (4 * r); b |= pc[1][r] << (4 * r); }
        *w0 = a;
        *w1 = b;
    } else {
        uint32_t lo = 0, hi = 0;
        const int wsel = pair_index & 1;
#pragma unroll
        for (int mm = 0; mm < 2; ++mm)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int k = 4 * mm + r;
                lo |= (pc[mm][r] & 0x00030003u) << (2 * k);
                hi |= ((pc[mm][r] >> 2) & 0x00010001u) << (4 * (k >> 1) + (k & 1));
            }
        *w0 = lo;
        *w1 = hi << (2 * (1 - wsel));
    }
}

template <int BITS, int D>
__global__ void __launch_bounds__(QF_THREADS)
quantize_groups_fast(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src, int first_token,
                     int64_t sb, int64_t sh, int64_t stt, int kinds)
{
    constexpr int CH = D / 8;            // 16-byte chunks per row
    constexpr int NM = D / 16, NP = NM / 2;
    constexpr int NSET = D / 32;         // 32-channel sets per row
    constexpr int W = D * BITS / 64;     // words per lane per tile
    constexpr int NLO = (BITS == 3) ? D / 32 : W, NHI = (BITS == 3) ? D / 64 : 0;
    constexpr int TILE_WORDS = 32 * W;
    const float qmax = (float)((1 << BITS) - 1);
    const int G = p.G, NGv = p.NGv, Gv = p.Gv, n_tiles = G / KVSINK_TILE;
    // a block quantizes either the keys (kind 0) or the values (kind 1) of one group
    const int grp = blockIdx.x / kinds, kind = blockIdx.x % kinds, h = blockIdx.y, b = blockIdx.z;

    extern __shared__ __align__(128) unsigned char smem[];
    __half *Xt = (__half *)smem;                                   // [G][D] swizzled 16-byte chunks
    Coder *coder = (Coder *)(Xt + (size_t)G * D);                  // keys: [D]; values: [G][NGv]
    const int max_coders = D > G * NGv ? D : G * NGv;
    float *xscale = (float *)(coder + max_coders);                 // same indexing as coder
    float *xzero = xscale + max_coders;
    uint32_t *stat = (uint32_t *)(xzero + max_coders);             // keys: [warps][D]; values: [G][NSET]  (min | max << 16)
    const int stat_words = QF_WARPS * D > G * NSET ? QF_WARPS * D : G * NSET;
    uint32_t *xout = stat + stat_words;                            // [n_tiles][TILE_WORDS]
    uint32_t *tmask = xout + (size_t)n_tiles * TILE_WORDS;         // [n_tiles] sink bits of each tile

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const int64_t unit = (int64_t)b * p.Hkv + h;
    const int p0 = first_token + grp * G;
    const uint32_t *bm = c.sink_bitmask + (size_t)b * p.mask_words;

    // ---- stage the tile ----
    const __half *xbase = (kind == 0 ? k_src : v_src) + b * sb + h * sh + (int64_t)(grp * G) * stt;
    for (int idx = tid; idx < G * CH; idx += QF_THREADS) {
        const int t = idx / CH, ch = idx % CH;
        cp_async16(Xt + (size_t)t * D + (ch ^ (t & 7)) * 8, xbase + (int64_t)t * stt + ch * 8);
    }
    if (tid < n_tiles) {
        const int tok = p0 + tid * KVSINK_TILE;   // multiple of 16
        tmask[tid] = (bm[tok >> 5] >> (tok & 31)) & 0xffffu;
    }
    if constexpr (BITS == 3)
        for (int i = tid; i < n_tiles * TILE_WORDS; i += QF_THREADS) xout[i] = 0;   // hi words are OR-ed in
    cp_async_wait_all();
    __syncthreads();
    auto is_sink = [&](int t) { return (tmask[t >> 4] >> (t & 15)) & 1u; };
    constexpr uint32_t ROW0 = (BITS == 4) ? 0x0f0f0f0fu : 0x33333333u;   // fields of matrix row g (r = 0, 2)
    const int mj = lane >> 3, rr = lane & 7;      // ldmatrix: this lane addresses row rr of 8x8 block mj

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
            coder[ch] = make_coder(s, z, fmaxf(fabsf(mn), fabsf(mx)), qmax);
            const size_t o = ((size_t)unit * (p.max_seq / G) + p0 / G) * D + ch;
            c.k_scale[o] = s;
            c.k_zero[o] = z;
        }
        __syncthreads();
        // ---- codes in the tile's register layout: a warp takes one matrix pair over a range of tiles ----
        {
            constexpr int CHUNKS = QF_WARPS / NP;
            const int pair = warp % NP, part = warp / NP;
            const int tb = (n_tiles * part) / CHUNKS, te = (n_tiles * (part + 1)) / CHUNKS;
            Coder kc[2][4];
#pragma unroll
            for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                for (int q = 0; q < 4; ++q) kc[mm][q] = coder[16 * (2 * pair + mm) + 2 * t4 + (q & 1) + 8 * (q >> 1)];
            for (int T = tb; T < te; ++T) {
                uint32_t a[2][4], pc[2][4], differ = 0;
#pragma unroll
                for (int mm = 0; mm < 2; ++mm) {
                    const int tok = 16 * T + rr + 8 * (mj & 1), chunk = 2 * (2 * pair + mm) + (mj >> 1);
                    ldmatrix_x4(a[mm], Xt + (size_t)tok * D + ((chunk ^ (tok & 7)) * 8));
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        pc[mm][r] = code_pair<BITS>(a[mm][r], kc[mm][2 * (r >> 1)], kc[mm][2 * (r >> 1) + 1], differ);
                }
                if (differ) {
#pragma unroll
                    for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const int ch = 16 * (2 * pair + mm) + 2 * t4 + 8 * (r >> 1);
                            pc[mm][r] = code_pair_exact<BITS>(a[mm][r], xscale[ch], xzero[ch], xscale[ch + 1], xzero[ch + 1]);
                        }
                }
                uint32_t w0, w1;
                pack_pair<BITS>(pc, pair, &w0, &w1);
                const uint32_t m16 = tmask[T];
                if (m16) {   // sink tokens keep code 0 in the packed stream
                    uint32_t keep = 0xffffffffu, keeph = 0xffffffffu;
                    if ((m16 >> g) & 1u) { keep &= ~ROW0; keeph &= ~0x55555555u; }
                    if ((m16 >> (g + 8)) & 1u) { keep &= ROW0; keeph &= 0x55555555u; }
                    w0 &= keep;
                    w1 &= (BITS == 3) ? keeph : keep;
                }
                uint32_t *tile = xout + (size_t)T * TILE_WORDS;
                if constexpr (BITS == 2) {
                    tile[section_word_offset(NLO, lane, pair)] = w0;
                } else if constexpr (BITS == 4) {
                    tile[section_word_offset(NLO, lane, 2 * pair)] = w0;
                    tile[section_word_offset(NLO, lane, 2 * pair + 1)] = w1;
                } else {
                    tile[section_word_offset(NLO, lane, pair)] = w0;
                    atomicOr(&tile[32 * NLO + section_word_offset(NHI, lane, pair >> 1)], w1);
                }
            }
        }
    } else {
        // ---- values: per-token statistics over 32-channel sets, two threads per token ----
        {
            constexpr int SPT = (D == 128) ? 2 : 1;      // sets per thread
            for (int it = tid; it < 2 * G; it += QF_THREADS) {
                const int t = it >> 1, hh = it & 1;
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
            const int spg = Gv / 32;     // sets per channel group
            for (int it = tid; it < G * NGv; it += QF_THREADS) {
                const int t = it / NGv, j = it % NGv;
                float s = 0.f, z = 0.f, amax = 0.f;
                if (!is_sink(t)) {
                    __half lo = __ushort_as_half(0x7C00), hi = __ushort_as_half(0xFC00);
                    for (int q = 0; q < spg; ++q) {
                        const uint32_t v = stat[t * NSET + j * spg + q];
                        lo = __hmin(lo, __ushort_as_half((unsigned short)(v & 0xffffu)));
                        hi = __hmax(hi, __ushort_as_half((unsigned short)(v >> 16)));
                    }
                    const float mn = __half2float(lo), mx = __half2float(hi);
                    group_params(true, mn, mx, qmax, &s, &z);
                    amax = fmaxf(fabsf(mn), fabsf(mx));
                }
                xscale[it] = s;
                xzero[it] = z;
                coder[it] = make_coder(s, z, amax, qmax);
                const size_t o = ((size_t)unit * p.max_seq + p0 + t) * NGv + j;
                c.v_scale[o] = s;
                c.v_zero[o] = z;
            }
        }
        __syncthreads();
        {
            const int mpg = Gv / 16;
            for (int T = warp; T < n_tiles; T += QF_WARPS) {
                uint32_t *tile = xout + (size_t)T * TILE_WORDS;
#pragma unroll
                for (int pair = 0; pair < NP; ++pair) {
                    uint32_t a[2][4], pc[2][4], differ = 0;
#pragma unroll
                    for (int mm = 0; mm < 2; ++mm) {
                        const int m = 2 * pair + mm, jg = m / mpg;
                        const int tok = 16 * T + rr + 8 * (mj >> 1), chunk = 2 * m + (mj & 1);
                        ldmatrix_x4_trans(a[mm], Xt + (size_t)tok * D + ((chunk ^ (tok & 7)) * 8));
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const int tk = 16 * T + 2 * t4 + 8 * (r >> 1);
                            pc[mm][r] = code_pair<BITS>(a[mm][r], coder[tk * NGv + jg], coder[(tk + 1) * NGv + jg], differ);
                        }
                    }
                    if (differ) {
#pragma unroll
                        for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                            for (int r = 0; r < 4; ++r) {
                                const int jg = (2 * pair + mm) / mpg, i0 = (16 * T + 2 * t4 + 8 * (r >> 1)) * NGv + jg;
                                pc[mm][r] = code_pair_exact<BITS>(a[mm][r], xscale[i0], xzero[i0], xscale[i0 + NGv], xzero[i0 + NGv]);
                            }
                    }
                    uint32_t w0, w1;
                    pack_pair<BITS>(pc, pair, &w0, &w1);
                    if constexpr (BITS == 2) {
                        tile[section_word_offset(NLO, lane, pair)] = w0;
                    } else if constexpr (BITS == 4) {
                        tile[section_word_offset(NLO, lane, 2 * pair)] = w0;
                        tile[section_word_offset(NLO, lane, 2 * pair + 1)] = w1;
                    } else {
                        tile[section_word_offset(NLO, lane, pair)] = w0;
                        atomicOr(&tile[32 * NLO + section_word_offset(NHI, lane, pair >> 1)], w1);
                    }
                }
            }
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
        for (int T = 0; T < n_tiles; ++T) any |= tmask[T] != 0;
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
}

template <int BITS, int D>
static int launch_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                       int64_t sb, int64_t sh, int64_t stt, bool do_v, cudaStream_t st)
{
    const int G = p.G, n_tiles = G / KVSINK_TILE;
    constexpr int W = D * BITS / 64;
    const size_t max_coders = (size_t)(D > G * p.NGv ? D : G * p.NGv);
    const size_t stat_words = (size_t)(QF_WARPS * D > G * (D / 32) ? QF_WARPS * D : G * (D / 32));
    const size_t smem = (size_t)G * D * 2 + max_coders * (16 + 8) + stat_words * 4 + (size_t)n_tiles * 32 * W * 4 + (size_t)n_tiles * 4 + 16;
    if (smem > 227 * 1024) return KVSINK_ERR_UNSUPPORTED;
    auto kern = quantize_groups_fast<BITS, D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    const int kinds = do_v ? 2 : 1;
    dim3 grid(n_groups * kinds, p.Hkv, p.B);
    kern<<<grid, QF_THREADS, smem, st>>>(p, c, k_src, v_src, first_token, sb, sh, stt, kinds);
    return cudaGetLastError() == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
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
