// Static (calibrated) parameters: the paper's per-channel-key / per-token-value scheme with fixed parameters (Section 5.1),
// sink tokens left out of the calibration as well as of the quantization (Algorithm 1's remark on calibration, Section 4.1,
// Appendix C "Dynamic and static quantization").
//   calibration : global min / max per key channel and per value channel group of every KV head over all sequences and
//                 non-sink tokens, then Eq. 10-11
//   append      : every token is coded on arrival with the fixed pairs (Eq. 8, values outside the calibrated range clamp);
//                 no key tail, no per-group parameters; sink rows go to the side buffer
// The same two append kernels serve per-token keys (PT; Section 4.1 "Per-token quantization", Section 5.1's per-token Key and
// Value dynamic scheme): keys and values alike get one (scale, zero) per token and channel group, computed on arrival from
// the token's own extremes (Eq. 10-11) and stored in the cache's parameter arrays, sink tokens (0, 0).
#include "common.cuh"
#include "tile_words.cuh"

namespace kvsink {
namespace {

// fp16 bit pattern <-> integer in value order (both zeros map to 0).
__device__ __forceinline__ int ordered(unsigned b) { return (b & 0x8000u) ? -(int)(b & 0x7fffu) : (int)b; }
__device__ __forceinline__ float unordered(int o)
{
    const unsigned b = o >= 0 ? (unsigned)o : (0x8000u | (unsigned)(-o));
    return __half2float(__ushort_as_half((unsigned short)b));
}
constexpr int NO_MIN = 0x7fffffff, NO_MAX = -0x7fffffff - 1;

// workspace: int [4][Hkv][D] = key min, key max, value min, value max per channel, in value order
__global__ void calibrate_init_kernel(int *__restrict__ ws, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (i < n) { ws[i] = NO_MIN; ws[n + i] = NO_MAX; ws[2 * n + i] = NO_MIN; ws[3 * n + i] = NO_MAX; }
}

constexpr int CAL_THREADS = 128, CAL_SLICE = 256;   // tokens per block

// grid (token slices, Hkv, B); thread = eight channels of one of 128 / (D / 8) token lanes.
__global__ void __launch_bounds__(CAL_THREADS)
calibrate_scan_kernel(Params p, const __half *__restrict__ k, const __half *__restrict__ v, int T, int64_t sb, int64_t sh, int64_t stt,
                      const uint32_t *__restrict__ bitmask, int *__restrict__ ws)
{
    __shared__ int s_mm[4][128];
    const int D = p.D, tid = threadIdx.x, oct = D / 8, co = tid % oct, tl = tid / oct, lanes = CAL_THREADS / oct;
    const int h = blockIdx.y, b = blockIdx.z;
    const uint32_t *bm = bitmask + (size_t)b * p.mask_words;
    if (tid < D) { s_mm[0][tid] = NO_MIN; s_mm[1][tid] = NO_MAX; s_mm[2][tid] = NO_MIN; s_mm[3][tid] = NO_MAX; }
    pdl_wait();
    __syncthreads();
    constexpr uint32_t PINF2 = 0x7C007C00u, NINF2 = 0xFC00FC00u;
    uint32_t kmn[4] = {PINF2, PINF2, PINF2, PINF2}, kmx[4] = {NINF2, NINF2, NINF2, NINF2};
    uint32_t vmn[4] = {PINF2, PINF2, PINF2, PINF2}, vmx[4] = {NINF2, NINF2, NINF2, NINF2};
    bool any = false;
    const int t_end = min(T, (int)(blockIdx.x + 1) * CAL_SLICE);
    for (int t = blockIdx.x * CAL_SLICE + tl; t < t_end; t += lanes) {
        if (mask_bit(bm, t)) continue;
        const int64_t off = b * sb + h * sh + (int64_t)t * stt + co * 8;
        const uint4 a = __ldg(reinterpret_cast<const uint4 *>(k + off)), c = __ldg(reinterpret_cast<const uint4 *>(v + off));
        const uint32_t ka[4] = {a.x, a.y, a.z, a.w}, va[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            __half2 x = *reinterpret_cast<const __half2 *>(&ka[j]), y = *reinterpret_cast<const __half2 *>(&va[j]);
            __half2 r;
            r = __hmin2(*reinterpret_cast<__half2 *>(&kmn[j]), x); kmn[j] = *reinterpret_cast<uint32_t *>(&r);
            r = __hmax2(*reinterpret_cast<__half2 *>(&kmx[j]), x); kmx[j] = *reinterpret_cast<uint32_t *>(&r);
            r = __hmin2(*reinterpret_cast<__half2 *>(&vmn[j]), y); vmn[j] = *reinterpret_cast<uint32_t *>(&r);
            r = __hmax2(*reinterpret_cast<__half2 *>(&vmx[j]), y); vmx[j] = *reinterpret_cast<uint32_t *>(&r);
        }
        any = true;
    }
    if (any) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ch = co * 8 + 2 * j + e, shft = 16 * e;
                atomicMin(&s_mm[0][ch], ordered((kmn[j] >> shft) & 0xffffu));
                atomicMax(&s_mm[1][ch], ordered((kmx[j] >> shft) & 0xffffu));
                atomicMin(&s_mm[2][ch], ordered((vmn[j] >> shft) & 0xffffu));
                atomicMax(&s_mm[3][ch], ordered((vmx[j] >> shft) & 0xffffu));
            }
    }
    __syncthreads();
    if (tid < D && s_mm[0][tid] != NO_MIN) {
        const int n = p.Hkv * D, o = h * D + tid;
        atomicMin(ws + o, s_mm[0][tid]);
        atomicMax(ws + n + o, s_mm[1][tid]);
        atomicMin(ws + 2 * n + o, s_mm[2][tid]);
        atomicMax(ws + 3 * n + o, s_mm[3][tid]);
    }
}

// One thread per key channel, then one per value channel group: Eq. 10-11 from the extremes.
__global__ void calibrate_finish_kernel(Params p, const int *__restrict__ ws, kvsink_static_params sp)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x, n = p.Hkv * p.D;
    const float qmax = (float)((1 << p.bits) - 1);
    pdl_wait();
    if (i < n) {
        const bool any = ws[i] != NO_MIN;
        group_params(any, any ? unordered(ws[i]) : 0.f, any ? unordered(ws[n + i]) : 0.f, qmax, sp.k_scale + i, sp.k_zero + i);
    }
    if (i < p.Hkv * p.NGv) {
        const int h = i / p.NGv, j = i % p.NGv;
        int mn = NO_MIN, mx = NO_MAX;
        for (int e = 0; e < p.Gv; ++e) {
            mn = min(mn, ws[2 * n + h * p.D + j * p.Gv + e]);
            mx = max(mx, ws[3 * n + h * p.D + j * p.Gv + e]);
        }
        const bool any = mn != NO_MIN;
        group_params(any, any ? unordered(mn) : 0.f, any ? unordered(mx) : 0.f, qmax, sp.v_scale + i, sp.v_zero + i);
    }
}

// Eq. 8 with fixed parameters; scale 0 (nothing was calibrated) gives code 0.
__device__ __forceinline__ uint32_t code_static(float x, float s, float z, float qmax) { return s == 0.f ? 0u : code_exact(x, s, z, qmax); }

// One block per (tile touched, KV head, sequence): the new tokens' key and value codes are inserted into their tiles
// (fields of earlier tokens keep their bits; a tile whose first token arrives is written whole).
constexpr int CQ_THREADS = 128;

template <bool PT>
__global__ void __launch_bounds__(CQ_THREADS)
quantize_calibrated_kernel(Params p, kvsink_cache c, kvsink_static_params sp, const __half *__restrict__ k_src, const __half *__restrict__ v_src,
                           int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt)
{
    __shared__ uint8_t kcode[KVSINK_TILE * 128], vcode[KVSINK_TILE * 128];
    __shared__ uint8_t present[KVSINK_TILE];
    const int D = p.D;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = blockIdx.y, b = blockIdx.z;
    const int64_t unit = (int64_t)b * p.Hkv + h;
    const int tile = first_token / KVSINK_TILE + blockIdx.x;
    const int t_lo = max(first_token, tile * KVSINK_TILE), t_hi = min(first_token + n_tokens, (tile + 1) * KVSINK_TILE);
    const float qmax = (float)((1 << p.bits) - 1);
    const uint32_t *bm = c.sink_bitmask + (size_t)b * p.mask_words;
    if (tid < KVSINK_TILE) present[tid] = (tile * KVSINK_TILE + tid >= t_lo && tile * KVSINK_TILE + tid < t_hi) ? 1 : 0;
    pdl_wait();
    if (!in_bounds(first_token >= 0 && first_token + n_tokens <= p.max_seq && (tile + 1) * KVSINK_TILE <= p.max_seq, c.status)) return;

    const int cpl = D / 32;   // channels per lane (2 or 4)
    float ks[4], kz[4], vs[4], vz[4];
    for (int e = 0; e < cpl; ++e) {
        const int ch = lane * cpl + e;
        ks[e] = kz[e] = vs[e] = vz[e] = 0.f;
        if constexpr (!PT) {
            ks[e] = sp.k_scale[h * D + ch]; kz[e] = sp.k_zero[h * D + ch];
            vs[e] = sp.v_scale[h * p.NGv + ch / p.Gv]; vz[e] = sp.v_zero[h * p.NGv + ch / p.Gv];
        }
    }
    for (int pos = t_lo + warp; pos < t_hi; pos += CQ_THREADS / 32) {
        const int64_t src = b * sb + h * sh + (int64_t)(pos - first_token) * stt;
        const bool sink = mask_bit(bm, pos);
        __half kx[4], vx[4];
        for (int e = 0; e < cpl; ++e) { kx[e] = k_src[src + lane * cpl + e]; vx[e] = v_src[src + lane * cpl + e]; }
        if (sink) {
            const int count = min(c.sink_count[b], p.cap);
            const int slot = find_slot(c.sink_pos + (size_t)b * p.cap, count, pos);
            if (slot < 0) {
                if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
            } else {
                __half *dk = (__half *)c.sink_k + ((size_t)unit * p.cap + slot) * D;
                __half *dv = (__half *)c.sink_v + ((size_t)unit * p.cap + slot) * D;
                for (int e = 0; e < cpl; ++e) { dk[lane * cpl + e] = kx[e]; dv[lane * cpl + e] = vx[e]; }
            }
        }
        if constexpr (PT) {
            // the token's own parameters: min / max over the lanes of each channel group, keys and values alike
            float kmn = __half2float(kx[0]), kmx = kmn, vmn = __half2float(vx[0]), vmx = vmn;
            for (int e = 1; e < cpl; ++e) {
                kmn = fminf(kmn, __half2float(kx[e])); kmx = fmaxf(kmx, __half2float(kx[e]));
                vmn = fminf(vmn, __half2float(vx[e])); vmx = fmaxf(vmx, __half2float(vx[e]));
            }
            const int lanes_per_group = p.Gv / cpl;
            for (int o = 1; o < lanes_per_group; o <<= 1) {
                kmn = fminf(kmn, __shfl_xor_sync(0xffffffffu, kmn, o)); kmx = fmaxf(kmx, __shfl_xor_sync(0xffffffffu, kmx, o));
                vmn = fminf(vmn, __shfl_xor_sync(0xffffffffu, vmn, o)); vmx = fmaxf(vmx, __shfl_xor_sync(0xffffffffu, vmx, o));
            }
            float s0, z0, s1, z1;
            group_params(!sink, kmn, kmx, qmax, &s0, &z0);
            group_params(!sink, vmn, vmx, qmax, &s1, &z1);
            for (int e = 0; e < cpl; ++e) { ks[e] = s0; kz[e] = z0; vs[e] = s1; vz[e] = z1; }
            if (lane % lanes_per_group == 0) {
                const size_t o = ((size_t)unit * p.max_seq + pos) * p.NGv + lane / lanes_per_group;
                c.k_scale[o] = s0; c.k_zero[o] = z0;
                c.v_scale[o] = s1; c.v_zero[o] = z1;
            }
        }
        for (int e = 0; e < cpl; ++e) {
            const int o = (pos % KVSINK_TILE) * D + lane * cpl + e;
            kcode[o] = sink ? 0 : (uint8_t)code_static(__half2float(kx[e]), ks[e], kz[e], qmax);
            vcode[o] = sink ? 0 : (uint8_t)code_static(__half2float(vx[e]), vs[e], vz[e], qmax);
        }
    }
    __syncthreads();

    const int tile_words = p.tile_bytes / 4;
    const size_t tile_off = (size_t)unit * p.max_seq * p.row_bytes + (size_t)tile * p.tile_bytes;
    uint32_t *kout = (uint32_t *)(c.k_codes + tile_off), *vout = (uint32_t *)(c.v_codes + tile_off);
    const bool fresh = (t_lo % KVSINK_TILE) == 0;   // no earlier token lives in this tile
    for (int word = tid; word < tile_words; word += CQ_THREADS) {
        uint32_t fieldmask;
        // key tile: matrix element (row, col) = (token, channel); value tile: (channel, token)
        uint32_t newbits = assemble_word_masked(p.bits, D, word, [&](int m, int row, int col) {
            return present[row] ? (uint32_t)kcode[row * D + 16 * m + col] : 0x100u; }, &fieldmask);
        if (fieldmask || fresh) kout[word] = ((fresh ? 0u : kout[word]) & ~fieldmask) | newbits;
        newbits = assemble_word_masked(p.bits, D, word, [&](int m, int row, int col) {
            return present[col] ? (uint32_t)vcode[col * D + 16 * m + row] : 0x100u; }, &fieldmask);
        if (fieldmask || fresh) vout[word] = ((fresh ? 0u : vout[word]) & ~fieldmask) | newbits;
    }
}

// Eq. 8 with fixed parameters without a division per element: r is the rounded reciprocal of the scale, so x * r is within
// 2^-22 |x / scale| of the quotient; unless it lies that close to a rounding tie, its nearest integer is that of the IEEE
// quotient.  Near a tie (fp16 inputs hit exact ties often), for huge quotients and for a reciprocal that is not finite the
// literal formula is evaluated.
__device__ __forceinline__ uint32_t code_static_fast(float x, float s, float r, float z, float qmax)
{
    const float q = x * r, c = rintf(q);
    const float room = 0.5f - fabsf(q - c);                    // distance to the nearest tie
    if (!(room > fabsf(q) * 4.76837158203125e-07f)) return code_static(x, s, z, qmax);
    return (uint32_t)(int)fminf(fmaxf(c + z, 0.f), qmax);
}

// Whole fresh tiles (a bulk append that starts on a tile boundary): one warp per 16-token tile.  The warp stages the
// tile's key and value rows in shared memory and every lane codes exactly the elements of its own pair slots of the packed
// tiles, so the lane's words come out in the tile's own order and are stored with one 16-byte (or 8-byte) store per plane.
constexpr int CF_WARPS = 4;

template <int BITS, bool PT>
__global__ void __launch_bounds__(32 * CF_WARPS)
quantize_calibrated_tiles_kernel(Params p, kvsink_cache c, kvsink_static_params sp, const __half *__restrict__ k_src,
                                 const __half *__restrict__ v_src, int first_token, int n_tiles, int64_t sb, int64_t sh, int64_t stt)
{
    constexpr int D = 128, W = D * BITS / 64, NLO = BITS == 3 ? D / 32 : W, NHI = BITS == 3 ? D / 64 : 0;
    constexpr int ROW = D + 8;                                 // padded row (halves): conflict-free column reads
    __shared__ __align__(16) __half s_k[CF_WARPS][KVSINK_TILE * ROW], s_v[CF_WARPS][KVSINK_TILE * ROW];
    __shared__ float4 s_kp[D];                                 // (scale, 1 / scale, zero) of the KV head's key channels
    __shared__ float4 s_pt[PT ? CF_WARPS : 1][2][KVSINK_TILE][4];   // per-token keys: the same per (K / V, token, 32-channel block)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int h = blockIdx.y, b = blockIdx.z;
    const int64_t unit = (int64_t)b * p.Hkv + h;
    const float qmax = (float)((1 << BITS) - 1);
    const uint32_t *bm = c.sink_bitmask + (size_t)b * p.mask_words;
    pdl_wait();
    for (int i = tid; i < D && !PT; i += 32 * CF_WARPS) {
        const float sc = sp.k_scale[h * D + i];
        s_kp[i] = make_float4(sc, sc == 0.f ? 0.f : __frcp_rn(sc), sp.k_zero[h * D + i], 0.f);
    }
    __syncthreads();
    const int ti = blockIdx.x * CF_WARPS + warp;               // tile of this append
    if (ti >= n_tiles) return;
    const int tok0 = first_token + ti * KVSINK_TILE, src0 = ti * KVSINK_TILE;
    if (!in_bounds(tok0 >= 0 && tok0 + KVSINK_TILE <= p.max_seq, c.status)) return;
    __half *mk = s_k[warp], *mv = s_v[warp];
    for (int i = lane; i < KVSINK_TILE * (D / 8); i += 32) {
        const int r = i / (D / 8), c8 = i % (D / 8);
        const int64_t off = b * sb + h * sh + (int64_t)(src0 + r) * stt + c8 * 8;
        *reinterpret_cast<uint4 *>(mk + r * ROW + c8 * 8) = __ldg(reinterpret_cast<const uint4 *>(k_src + off));
        *reinterpret_cast<uint4 *>(mv + r * ROW + c8 * 8) = __ldg(reinterpret_cast<const uint4 *>(v_src + off));
    }
    const uint32_t mask16 = (bm[tok0 >> 5] >> (tok0 & 31)) & 0xffffu;   // sink bits of the tile's tokens
    __syncwarp();
    if (mask16) {   // exact rows to the side buffer at the rank of their position
        const int count = min(c.sink_count[b], p.cap);
        for (uint32_t rest = mask16; rest; rest &= rest - 1u) {
            const int r = __ffs((int)rest) - 1;
            const int slot = find_slot(c.sink_pos + (size_t)b * p.cap, count, tok0 + r);
            if (slot < 0) {
                if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
                continue;
            }
            __half *dk = (__half *)c.sink_k + ((size_t)unit * p.cap + slot) * D, *dv = (__half *)c.sink_v + ((size_t)unit * p.cap + slot) * D;
            if (lane < D / 8) {
                *reinterpret_cast<uint4 *>(dk + lane * 8) = *reinterpret_cast<const uint4 *>(mk + r * ROW + lane * 8);
                *reinterpret_cast<uint4 *>(dv + lane * 8) = *reinterpret_cast<const uint4 *>(mv + r * ROW + lane * 8);
            }
        }
    }
    if constexpr (PT) {
        // per-token parameters: lane -> token lane / 2, channels 64 (lane % 2) ... + 63 as two 32-channel blocks, combined to
        // the channel group (32, 64 or 128 channels) and written to the parameter arrays by the group's first lane
        const int tk = lane >> 1, hf = lane & 1;
        const bool sink = (mask16 >> tk) & 1u;
#pragma unroll
        for (int kind = 0; kind < 2; ++kind) {
            const __half *row = (kind ? mv : mk) + tk * ROW + 64 * hf;
            float mn[2], mx[2];
#pragma unroll
            for (int sbk = 0; sbk < 2; ++sbk) {
                __half2 lo = *reinterpret_cast<const __half2 *>(row + 32 * sbk), hi = lo;
#pragma unroll
                for (int i = 1; i < 16; ++i) {
                    const __half2 x = *reinterpret_cast<const __half2 *>(row + 32 * sbk + 2 * i);
                    lo = __hmin2(lo, x); hi = __hmax2(hi, x);
                }
                mn[sbk] = fminf(__low2float(lo), __high2float(lo)); mx[sbk] = fmaxf(__low2float(hi), __high2float(hi));
            }
            if (p.Gv >= 64) { mn[0] = mn[1] = fminf(mn[0], mn[1]); mx[0] = mx[1] = fmaxf(mx[0], mx[1]); }
            if (p.Gv >= 128) {
                mn[0] = mn[1] = fminf(mn[0], __shfl_xor_sync(0xffffffffu, mn[0], 1));
                mx[0] = mx[1] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], 1));
            }
            float *ps = kind ? c.v_scale : c.k_scale, *pz = kind ? c.v_zero : c.k_zero;
#pragma unroll
            for (int sbk = 0; sbk < 2; ++sbk) {
                float sc, ze;
                group_params(!sink, mn[sbk], mx[sbk], qmax, &sc, &ze);
                const int ch0 = 64 * hf + 32 * sbk;
                s_pt[warp][kind][tk][2 * hf + sbk] = make_float4(sc, sc == 0.f ? 0.f : __frcp_rn(sc), ze, 0.f);
                if (ch0 % p.Gv == 0) {
                    const size_t o = ((size_t)unit * p.max_seq + tok0 + tk) * p.NGv + ch0 / p.Gv;
                    ps[o] = sc; pz[o] = ze;
                }
            }
        }
        __syncwarp();
    }
    // codes of pair slot s = 4m + r, half e: keys (token, channel) = (g + 8(r&1), 16m + 8(r>>1) + 2t + e),
    //                                        values (channel, token) = (16m + g + 8(r&1), 8(r>>1) + 2t + e)
    uint32_t kw[W], vw[W];
#pragma unroll
    for (int i = 0; i < W; ++i) kw[i] = vw[i] = 0u;
#pragma unroll
    for (int m = 0; m < D / 16; ++m) {
        const int vj = (16 * m) / p.Gv;   // value channel group of this matrix (groups are multiples of 16 channels)
        float vs = 0.f, vz = 0.f, vr = 0.f;
        if constexpr (!PT) { vs = sp.v_scale[h * p.NGv + vj]; vz = sp.v_zero[h * p.NGv + vj]; vr = vs == 0.f ? 0.f : __frcp_rn(vs); }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int s_ = 4 * m + r;
                const int ktok = g + 8 * (r & 1), kch = 16 * m + 8 * (r >> 1) + 2 * t + e;
                const int vch = 16 * m + g + 8 * (r & 1), vtok = 8 * (r >> 1) + 2 * t + e;
                const float4 kp = PT ? s_pt[PT ? warp : 0][0][ktok][kch >> 5] : s_kp[kch];
                const float4 vp = PT ? s_pt[PT ? warp : 0][1][vtok][vch >> 5] : make_float4(vs, vr, vz, 0.f);
                const uint32_t kc = ((mask16 >> ktok) & 1u) || kp.x == 0.f ? 0u : code_static_fast(__half2float(mk[ktok * ROW + kch]), kp.x, kp.y, kp.z, qmax);
                const uint32_t vc = ((mask16 >> vtok) & 1u) || vp.x == 0.f ? 0u : code_static_fast(__half2float(mv[vtok * ROW + vch]), vp.x, vp.y, vp.z, qmax);
                if constexpr (BITS == 2) {
                    kw[s_ / 8] |= kc << (16 * e + 2 * (s_ % 8)); vw[s_ / 8] |= vc << (16 * e + 2 * (s_ % 8));
                } else if constexpr (BITS == 4) {
                    kw[s_ / 4] |= kc << (16 * e + 4 * (s_ % 4)); vw[s_ / 4] |= vc << (16 * e + 4 * (s_ % 4));
                } else {
                    const int i = s_ / 8, k = s_ % 8, hb = 16 * e + 4 * (k / 2) + 2 * (1 - (i % 2)) + (k % 2);
                    kw[i] |= (kc & 3u) << (16 * e + 2 * k); vw[i] |= (vc & 3u) << (16 * e + 2 * k);
                    kw[NLO + i / 2] |= (kc >> 2) << hb; vw[NLO + i / 2] |= (vc >> 2) << hb;
                }
            }
    }
    // a section of n words per lane is stored as planes of up to four words per lane
    const size_t tile_off = (size_t)unit * p.max_seq * p.row_bytes + (size_t)(tok0 / KVSINK_TILE) * p.tile_bytes;
    uint32_t *ko = (uint32_t *)(c.k_codes + tile_off), *vo = (uint32_t *)(c.v_codes + tile_off);
    auto store_section = [&](uint32_t *dst, const uint32_t *w, int n) {
        for (int pl = 0; pl * 4 < n; ++pl) {
            const int u = n - 4 * pl > 4 ? 4 : n - 4 * pl;
            uint32_t *d = dst + u * lane;
            if (u == 4) *reinterpret_cast<uint4 *>(d) = make_uint4(w[4 * pl], w[4 * pl + 1], w[4 * pl + 2], w[4 * pl + 3]);
            else if (u == 2) *reinterpret_cast<uint2 *>(d) = make_uint2(w[4 * pl], w[4 * pl + 1]);
            else for (int i = 0; i < u; ++i) d[i] = w[4 * pl + i];
            dst += 32 * u;
        }
    };
    store_section(ko, kw, NLO);
    store_section(vo, vw, NLO);
    if constexpr (BITS == 3) { store_section(ko + 32 * NLO, kw + NLO, NHI); store_section(vo + 32 * NLO, vw + NLO, NHI); }
}

}  // namespace

size_t calibrate_workspace_bytes(const Params &p) { return (size_t)4 * p.Hkv * p.D * sizeof(int) + 16; }

int launch_calibrate(const Params &p, const __half *k, const __half *v, int T, int64_t sb, int64_t sh, int64_t stt, const uint32_t *bitmask,
                     const kvsink_static_params &sp, void *workspace, cudaStream_t st)
{
    int *ws = (int *)workspace;
    const int n = p.Hkv * p.D;
    if (launch_pdl(calibrate_init_kernel, dim3((n + 255) / 256), dim3(256), 0, st, ws, n) != cudaSuccess) return KVSINK_ERR_CUDA;
    if (T > 0) {
        const dim3 grid((T + CAL_SLICE - 1) / CAL_SLICE, p.Hkv, p.B);
        if (launch_pdl(calibrate_scan_kernel, grid, dim3(CAL_THREADS), 0, st, p, k, v, T, sb, sh, stt, bitmask, ws) != cudaSuccess)
            return KVSINK_ERR_CUDA;
    }
    return launch_pdl(calibrate_finish_kernel, dim3((n + 255) / 256), dim3(256), 0, st, p, (const int *)ws, sp) == cudaSuccess ? KVSINK_OK
                                                                                                                                : KVSINK_ERR_CUDA;
}

template <bool PT>
static int launch_tokens(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                         int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (n_tokens <= 0) return KVSINK_OK;
    // whole fresh tiles of a head-size-128 cache take the tile kernel, the ragged rest (at most 15 tokens) the general one
    if (p.D == 128 && first_token % KVSINK_TILE == 0 && n_tokens >= KVSINK_TILE && ((uintptr_t)k_src & 15u) == 0 && ((uintptr_t)v_src & 15u) == 0) {
        const int n_tiles = n_tokens / KVSINK_TILE;
        const dim3 grid((n_tiles + CF_WARPS - 1) / CF_WARPS, p.Hkv, p.B);
        cudaError_t e = p.bits == 2 ? launch_pdl(quantize_calibrated_tiles_kernel<2, PT>, grid, dim3(32 * CF_WARPS), 0, st, p, c, sp, k_src, v_src, first_token, n_tiles, sb, sh, stt)
                      : p.bits == 3 ? launch_pdl(quantize_calibrated_tiles_kernel<3, PT>, grid, dim3(32 * CF_WARPS), 0, st, p, c, sp, k_src, v_src, first_token, n_tiles, sb, sh, stt)
                                    : launch_pdl(quantize_calibrated_tiles_kernel<4, PT>, grid, dim3(32 * CF_WARPS), 0, st, p, c, sp, k_src, v_src, first_token, n_tiles, sb, sh, stt);
        if (e != cudaSuccess) return KVSINK_ERR_CUDA;
        const int done = n_tiles * KVSINK_TILE;
        return launch_tokens<PT>(p, c, sp, k_src + (int64_t)done * stt, v_src + (int64_t)done * stt, first_token + done, n_tokens - done, sb, sh, stt, st);
    }
    const int tiles = (first_token + n_tokens - 1) / KVSINK_TILE - first_token / KVSINK_TILE + 1;
    const dim3 grid(tiles, p.Hkv, p.B);
    return launch_pdl(quantize_calibrated_kernel<PT>, grid, dim3(CQ_THREADS), 0, st, p, c, sp, k_src, v_src, first_token, n_tokens, sb, sh, stt) ==
                   cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

int launch_quantize_calibrated(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                               int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    // whole G-token spans from a multiple of G go to the bulk quantizer where it has a static form (G only shapes its work items)
    if (n_tokens >= p.G && first_token % p.G == 0) {
        const int n_groups = n_tokens / p.G;
        const int rc = launch_quantize_static_bulk(p, c, sp, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
        if (rc == KVSINK_OK) {
            const int done = n_groups * p.G;
            return launch_tokens<false>(p, c, sp, k_src + (int64_t)done * stt, v_src + (int64_t)done * stt, first_token + done, n_tokens - done, sb, sh,
                                        stt, st);
        }
        if (rc != KVSINK_ERR_UNSUPPORTED) return rc;
    }
    return launch_tokens<false>(p, c, sp, k_src, v_src, first_token, n_tokens, sb, sh, stt, st);
}

int launch_quantize_pertoken(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_tokens,
                             int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    const kvsink_static_params none = {nullptr, nullptr, nullptr, nullptr};
    // whole G-token spans from a multiple of G go to the bulk quantizer where it has this form (G only shapes its work items)
    if (n_tokens >= p.G && first_token % p.G == 0) {
        const int n_groups = n_tokens / p.G;
        const int rc = launch_quantize_pertoken_bulk(p, c, k_src, v_src, first_token, n_groups, sb, sh, stt, st);
        if (rc == KVSINK_OK) {
            const int done = n_groups * p.G;
            return launch_tokens<true>(p, c, none, k_src + (int64_t)done * stt, v_src + (int64_t)done * stt, first_token + done, n_tokens - done, sb, sh,
                                       stt, st);
        }
        if (rc != KVSINK_ERR_UNSUPPORTED) return rc;
    }
    return launch_tokens<true>(p, c, none, k_src, v_src, first_token, n_tokens, sb, sh, stt, st);
}

}  // namespace kvsink
