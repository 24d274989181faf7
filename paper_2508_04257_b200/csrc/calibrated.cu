// Static (calibrated) parameters: the paper's per-channel-key / per-token-value scheme with fixed parameters (Section 5.1),
// sink tokens left out of the calibration as well as of the quantization (Algorithm 1's remark on calibration, Section 4.1,
// Appendix C "Dynamic and static quantization").
//   calibration : global min / max per key channel and per value channel group of every KV head over all sequences and
//                 non-sink tokens, then Eq. 10-11
//   append      : every token is coded on arrival with the fixed pairs (Eq. 8, values outside the calibrated range clamp);
//                 no key tail, no per-group parameters; sink rows go to the side buffer
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

    const int cpl = D / 32;   // channels per lane (2 or 4)
    float ks[4], kz[4], vs[4], vz[4];
    for (int e = 0; e < cpl; ++e) {
        const int ch = lane * cpl + e;
        ks[e] = sp.k_scale[h * D + ch]; kz[e] = sp.k_zero[h * D + ch];
        vs[e] = sp.v_scale[h * p.NGv + ch / p.Gv]; vz[e] = sp.v_zero[h * p.NGv + ch / p.Gv];
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

int launch_quantize_calibrated(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                               int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (n_tokens <= 0) return KVSINK_OK;
    const int tiles = (first_token + n_tokens - 1) / KVSINK_TILE - first_token / KVSINK_TILE + 1;
    const dim3 grid(tiles, p.Hkv, p.B);
    return launch_pdl(quantize_calibrated_kernel, grid, dim3(CQ_THREADS), 0, st, p, c, sp, k_src, v_src, first_token, n_tokens, sb, sh, stt) ==
                   cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

}  // namespace kvsink
