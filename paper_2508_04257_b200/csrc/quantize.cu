// Asymmetric group quantization (Eq. 8-11) with sink exclusion (Algorithm 1), bit-packing into the tile
// layout, side-buffer compaction of sink rows, and the append path (Eq. 6).
#include "common.cuh"
#include "tile_words.cuh"

namespace kvsink {

// ---------------------------------------------------------------------------------------------------------
// Whole groups: one block per (token group, KV head, sequence).  Keys per channel over the group's non-sink
// tokens, values per token, sink rows to the side buffer.
// ---------------------------------------------------------------------------------------------------------
constexpr int QG_THREADS = 256;

__global__ void __launch_bounds__(QG_THREADS)
quantize_groups_kernel(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src,
                       int first_token, int64_t sb, int64_t sh, int64_t stt, int do_v_and_sinks)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int D = p.D, G = p.G, RS = D + 8;      // padded row stride in halves
    if (!in_bounds(first_token >= 0 && first_token + ((int)blockIdx.x + 1) * G <= p.max_seq, c.status)) return;   // every thread of the block alike
    __half *Kt = (__half *)smem;                  // [G][RS]
    __half *Vt = Kt + (size_t)G * RS;             // [G][RS]
    uint8_t *kcode = (uint8_t *)(Vt + (size_t)G * RS);   // [G][D]
    uint8_t *vcode = kcode + (size_t)G * D;               // [G][D]
    float *ks = (float *)(vcode + (size_t)G * D);         // [D] scale
    float *kz = ks + D;                                   // [D] zero
    float *vs = kz + D;                                   // [G][NGv]
    float *vz = vs + G * p.NGv;
    uint8_t *flag = (uint8_t *)(vz + G * p.NGv);          // [G] sink flags

    const int tid = threadIdx.x;
    const int grp = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int64_t unit = (int64_t)b * p.Hkv + h;
    const int p0 = first_token + grp * G;         // absolute position of the group's first token
    const int gidx = p0 / G;
    const float qmax = (float)((1 << p.bits) - 1);
    const uint32_t *bm = c.sink_bitmask + (size_t)b * p.mask_words;

    // load the tiles (16-byte chunks)
    const int chunks = D / 8;
    const __half *kbase = k_src + b * sb + h * sh + (int64_t)(grp * G) * stt;
    const __half *vbase = v_src + b * sb + h * sh + (int64_t)(grp * G) * stt;
    for (int idx = tid; idx < G * chunks; idx += QG_THREADS) {
        int t = idx / chunks, ch = (idx % chunks) * 8;
        *(uint4 *)(Kt + (size_t)t * RS + ch) = __ldg((const uint4 *)(kbase + (int64_t)t * stt + ch));
        if (do_v_and_sinks) *(uint4 *)(Vt + (size_t)t * RS + ch) = __ldg((const uint4 *)(vbase + (int64_t)t * stt + ch));
    }
    for (int t = tid; t < G; t += QG_THREADS) flag[t] = mask_bit(bm, p0 + t) ? 1 : 0;
    __syncthreads();

    // key parameters: one thread per channel
    for (int ch = tid; ch < D; ch += QG_THREADS) {
        bool any = false;
        float mn = 0.f, mx = 0.f;
        for (int t = 0; t < G; ++t) {
            if (flag[t]) continue;
            float x = __half2float(Kt[(size_t)t * RS + ch]);
            if (!any) { mn = mx = x; any = true; }
            else { mn = fminf(mn, x); mx = fmaxf(mx, x); }
        }
        float s, z;
        group_params(any, mn, mx, qmax, &s, &z);
        ks[ch] = s;
        kz[ch] = z;
        size_t o = ((size_t)unit * (p.max_seq / G) + gidx) * D + ch;
        c.k_scale[o] = s;
        c.k_zero[o] = z;
    }
    // value parameters: one thread per (token, channel group)
    if (do_v_and_sinks) {
        for (int it = tid; it < G * p.NGv; it += QG_THREADS) {
            int t = it / p.NGv, j = it % p.NGv;
            float s = 0.f, z = 0.f;
            if (!flag[t]) {
                const __half *row = Vt + (size_t)t * RS + j * p.Gv;
                float mn = __half2float(row[0]), mx = mn;
                for (int e = 1; e < p.Gv; ++e) {
                    float x = __half2float(row[e]);
                    mn = fminf(mn, x);
                    mx = fmaxf(mx, x);
                }
                group_params(true, mn, mx, qmax, &s, &z);
            }
            vs[it] = s;
            vz[it] = z;
            size_t o = ((size_t)unit * p.max_seq + p0 + t) * p.NGv + j;
            c.v_scale[o] = s;
            c.v_zero[o] = z;
        }
    }
    __syncthreads();

    // codes
    for (int idx = tid; idx < G * D; idx += QG_THREADS) {
        int t = idx / D, ch = idx % D;
        uint32_t kc = 0, vc = 0;
        if (!flag[t]) {
            kc = code_exact(__half2float(Kt[(size_t)t * RS + ch]), ks[ch], kz[ch], qmax);
            if (do_v_and_sinks) {
                int j = ch / p.Gv;
                vc = code_exact(__half2float(Vt[(size_t)t * RS + ch]), vs[t * p.NGv + j], vz[t * p.NGv + j], qmax);
            }
        }
        kcode[idx] = (uint8_t)kc;
        vcode[idx] = (uint8_t)vc;
    }
    __syncthreads();

    // pack: the group's tiles are contiguous in memory; one thread per 32-bit word
    const int tile_words = p.tile_bytes / 4, n_tiles = G / KVSINK_TILE;
    uint32_t *kout = (uint32_t *)(c.k_codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)(p0 / KVSINK_TILE) * p.tile_bytes);
    uint32_t *vout = (uint32_t *)(c.v_codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)(p0 / KVSINK_TILE) * p.tile_bytes);
    for (int idx = tid; idx < n_tiles * tile_words; idx += QG_THREADS) {
        int tile = idx / tile_words, word = idx % tile_words;
        const uint8_t *kc = kcode + (size_t)tile * KVSINK_TILE * D;
        kout[idx] = assemble_word(p.bits, D, word, [&](int m, int row, int col) { return (uint32_t)kc[row * D + 16 * m + col]; });
        if (do_v_and_sinks) {
            const uint8_t *vc = vcode + (size_t)tile * KVSINK_TILE * D;
            vout[idx] = assemble_word(p.bits, D, word, [&](int m, int row, int col) { return (uint32_t)vc[col * D + 16 * m + row]; });
        }
    }

    // sink rows: exact fp16 copies into the side buffer at the rank of their position
    if (do_v_and_sinks) {
        const int count = min(c.sink_count[b], p.cap);
        for (int t = 0; t < G; ++t) {
            if (!flag[t]) continue;
            int slot = find_slot(c.sink_pos + (size_t)b * p.cap, count, p0 + t);
            if (slot < 0) {
                if (tid == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
                continue;
            }
            __half *dk = (__half *)c.sink_k + ((size_t)unit * p.cap + slot) * D;
            __half *dv = (__half *)c.sink_v + ((size_t)unit * p.cap + slot) * D;
            for (int ch = tid; ch < chunks; ch += QG_THREADS) {
                *(uint4 *)(dk + ch * 8) = *(const uint4 *)(Kt + (size_t)t * RS + ch * 8);
                *(uint4 *)(dv + ch * 8) = *(const uint4 *)(Vt + (size_t)t * RS + ch * 8);
            }
        }
    }
}

static size_t groups_smem_bytes(const Params &p)
{
    size_t RS = p.D + 8;
    return 2 * (size_t)p.G * RS * 2 + 2 * (size_t)p.G * p.D + 2 * (size_t)p.D * 4 + 2 * (size_t)p.G * p.NGv * 4 + p.G + 16;
}

int launch_quantize_groups(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                           int n_groups, int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st)
{
    if (n_groups <= 0) return KVSINK_OK;
    size_t smem = groups_smem_bytes(p);
    if (smem > 227 * 1024) return KVSINK_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(quantize_groups_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return KVSINK_ERR_CUDA;
    dim3 grid(n_groups, p.Hkv, p.B);
    note_launch();
    quantize_groups_kernel<<<grid, QG_THREADS, smem, st>>>(p, c, k_src, v_src, first_token, sb, sh, stt, do_v_and_sinks ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------------------
// Single tokens (decode-time append, and the remainder of a prefill that does not fill a group): values are
// quantized per token and inserted into their tile, keys go to the fp16 tail, sink rows to the side buffer.
// One block per (tile touched, KV head, sequence).
// ---------------------------------------------------------------------------------------------------------
constexpr int QT_THREADS = 128;

__global__ void __launch_bounds__(QT_THREADS)
quantize_tokens_kernel(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src, int src_offset,
                       int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt)
{
    __shared__ uint8_t vcode[KVSINK_TILE * 128];
    __shared__ uint8_t present[KVSINK_TILE];
    const int D = p.D, G = p.G;
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
    for (int pos = t_lo + warp; pos < t_hi; pos += QT_THREADS / 32) {
        const int64_t src = b * sb + h * sh + (int64_t)(src_offset + pos - first_token) * stt;
        const bool sink = mask_bit(bm, pos);
        float x[4];
        __half kx[4], vx[4];
        for (int e = 0; e < cpl; ++e) {
            vx[e] = v_src[src + lane * cpl + e];
            x[e] = __half2float(vx[e]);
            kx[e] = k_src[src + lane * cpl + e];
        }
        // key row -> tail
        __half *tail = (__half *)c.k_tail + ((size_t)unit * G + pos % G) * D;
        for (int e = 0; e < cpl; ++e) tail[lane * cpl + e] = kx[e];
        if (sink) {
            const int count = min(c.sink_count[b], p.cap);
            int slot = find_slot(c.sink_pos + (size_t)b * p.cap, count, pos);
            if (slot < 0) {
                if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
            } else {
                __half *dk = (__half *)c.sink_k + ((size_t)unit * p.cap + slot) * D;
                __half *dv = (__half *)c.sink_v + ((size_t)unit * p.cap + slot) * D;
                for (int e = 0; e < cpl; ++e) {
                    dk[lane * cpl + e] = kx[e];
                    dv[lane * cpl + e] = vx[e];
                }
            }
        }
        // value row: min / max over the lanes of each channel group
        float mn = x[0], mx = x[0];
        for (int e = 1; e < cpl; ++e) { mn = fminf(mn, x[e]); mx = fmaxf(mx, x[e]); }
        const int lanes_per_group = p.Gv / cpl;
        for (int o = 1; o < lanes_per_group; o <<= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        float s, z;
        group_params(!sink, mn, mx, qmax, &s, &z);
        const int j = lane / lanes_per_group;
        if (lane % lanes_per_group == 0) {
            size_t o = ((size_t)unit * p.max_seq + pos) * p.NGv + j;
            c.v_scale[o] = s;
            c.v_zero[o] = z;
        }
        for (int e = 0; e < cpl; ++e)
            vcode[(pos % KVSINK_TILE) * D + lane * cpl + e] = sink ? 0 : (uint8_t)code_exact(x[e], s, z, qmax);
    }
    __syncthreads();

    // insert the new tokens' fields into the tile; fields of other tokens keep their bits
    const int tile_words = p.tile_bytes / 4;
    uint32_t *vout = (uint32_t *)(c.v_codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)tile * p.tile_bytes);
    const bool fresh = (t_lo % KVSINK_TILE) == 0;   // no earlier token lives in this tile
    for (int word = tid; word < tile_words; word += QT_THREADS) {
        uint32_t keep = fresh ? 0u : vout[word];
        uint32_t fieldmask;
        const uint32_t newbits = assemble_word_masked(p.bits, D, word, [&](int m, int row, int col) {
            return present[col] ? (uint32_t)vcode[col * D + 16 * m + row] : 0x100u; }, &fieldmask);
        if (fieldmask || fresh) vout[word] = (keep & ~fieldmask) | newbits;   // a fresh tile is written whole
    }
}

// ---------------------------------------------------------------------------------------------------------
// One token per sequence (the decode-time append): one warp per (sequence, KV head).  The value row is coded and its
// fields go straight into the tile's words: every channel's field has its own place (lane, word, bit) in the tile, so
// the lanes clear and set their fields with word atomics and nothing but the token's own fields is touched.
// ---------------------------------------------------------------------------------------------------------
constexpr int QA_WARPS = 4;

// Word (index among the tile's 32-bit words) and bit position of the field of matrix element (m, row, col); for 3 bit
// the low two bits, and through *hi_word / *hi_shift the high bit.
__device__ __forceinline__ void field_place(int bits, int D, int m, int row, int col, int *word, int *shift, int *hi_word, int *hi_shift)
{
    const int lane = 4 * (row & 7) + ((col & 7) >> 1), e = col & 1;
    const int s = 4 * m + (row >> 3) + 2 * (col >> 3);
    if (bits == 3) {
        const int nlo = D / 32, nhi = D / 64, i = s >> 3, k = s & 7;
        *word = section_word_offset(nlo, lane, i);
        *shift = 16 * e + 2 * k;
        *hi_word = 32 * nlo + section_word_offset(nhi, lane, i >> 1);
        *hi_shift = 16 * e + 4 * (k >> 1) + 2 * (1 - (i & 1)) + (k & 1);
    } else {
        const int n = D * bits / 64, fields = 16 / bits;
        *word = section_word_offset(n, lane, s / fields);
        *shift = 16 * e + bits * (s % fields);
        *hi_word = *hi_shift = 0;
    }
}

__global__ void __launch_bounds__(32 * QA_WARPS)
append_one_kernel(Params p, kvsink_cache c, const __half *__restrict__ k_src, const __half *__restrict__ v_src, int src_token, int pos,
                  int64_t sb, int64_t sh, int64_t stt)
{
    const int D = p.D, G = p.G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t unit = (int64_t)blockIdx.x * QA_WARPS + warp;
    pdl_wait();
    if (unit >= (int64_t)p.B * p.Hkv) return;
    if (!in_bounds(pos >= 0 && pos < p.max_seq, c.status)) return;
    const int b = (int)(unit / p.Hkv), h = (int)(unit % p.Hkv);
    const float qmax = (float)((1 << p.bits) - 1);
    const int cpl = D / 32;   // channels per lane (2 or 4)
    const int64_t src = b * sb + h * sh + (int64_t)src_token * stt;
    const bool sink = mask_bit(c.sink_bitmask + (size_t)b * p.mask_words, pos);
    float x[4];
    __half kx[4], vx[4];
    for (int e = 0; e < cpl; ++e) {
        vx[e] = v_src[src + lane * cpl + e];
        x[e] = __half2float(vx[e]);
        kx[e] = k_src[src + lane * cpl + e];
    }
    // key row -> tail
    __half *tail = (__half *)c.k_tail + ((size_t)unit * G + pos % G) * D;
    for (int e = 0; e < cpl; ++e) tail[lane * cpl + e] = kx[e];
    if (sink) {
        const int count = min(c.sink_count[b], p.cap);
        const int slot = find_slot(c.sink_pos + (size_t)b * p.cap, count, pos);
        if (slot < 0) {
            if (lane == 0) atomicOr(c.status, KVSINK_STATUS_SINK_MISMATCH);
        } else {
            __half *dk = (__half *)c.sink_k + ((size_t)unit * p.cap + slot) * D;
            __half *dv = (__half *)c.sink_v + ((size_t)unit * p.cap + slot) * D;
            for (int e = 0; e < cpl; ++e) {
                dk[lane * cpl + e] = kx[e];
                dv[lane * cpl + e] = vx[e];
            }
        }
    }
    // value row: min / max over the lanes of each channel group, parameters, codes
    float mn = x[0], mx = x[0];
    for (int e = 1; e < cpl; ++e) { mn = fminf(mn, x[e]); mx = fmaxf(mx, x[e]); }
    const int lanes_per_group = p.Gv / cpl;
    for (int o = 1; o < lanes_per_group; o <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    float s, z;
    group_params(!sink, mn, mx, qmax, &s, &z);
    if (lane % lanes_per_group == 0) {
        const size_t o = ((size_t)unit * p.max_seq + pos) * p.NGv + lane / lanes_per_group;
        c.v_scale[o] = s;
        c.v_zero[o] = z;
    }
    // the token's fields in its tile; a tile whose first token this is is written whole (zeros elsewhere)
    const int tile = pos / KVSINK_TILE, col = pos % KVSINK_TILE;
    uint32_t *vout = (uint32_t *)(c.v_codes + (size_t)unit * p.max_seq * p.row_bytes + (size_t)tile * p.tile_bytes);
    const bool fresh = col == 0;
    if (fresh) {
        for (int w = lane; w < p.tile_bytes / 4; w += 32) vout[w] = 0u;
        __syncwarp();
    }
    for (int e = 0; e < cpl; ++e) {
        const int ch = lane * cpl + e;
        const uint32_t code = sink ? 0u : code_exact(x[e], s, z, qmax);
        int word, shift, hi_word, hi_shift;
        field_place(p.bits, D, ch >> 4, ch & 15, col, &word, &shift, &hi_word, &hi_shift);
        const uint32_t lo_mask = p.bits == 3 ? 3u : (1u << p.bits) - 1u;
        if (!fresh) atomicAnd(&vout[word], ~(lo_mask << shift));
        if (code & lo_mask) atomicOr(&vout[word], (code & lo_mask) << shift);
        if (p.bits == 3) {
            if (!fresh) atomicAnd(&vout[hi_word], ~(1u << hi_shift));
            if (code >> 2) atomicOr(&vout[hi_word], 1u << hi_shift);
        }
    }
}

int launch_quantize_tokens(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int src_offset,
                           int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st)
{
    if (n_tokens <= 0) return KVSINK_OK;
    if (n_tokens == 1) {
        const long units = (long)p.B * p.Hkv;
        return launch_pdl(append_one_kernel, dim3((unsigned)((units + QA_WARPS - 1) / QA_WARPS)), dim3(32 * QA_WARPS), 0, st, p, c, k_src, v_src,
                          src_offset, first_token, sb, sh, stt) == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
    }
    int tiles = (first_token + n_tokens - 1) / KVSINK_TILE - first_token / KVSINK_TILE + 1;
    dim3 grid(tiles, p.Hkv, p.B);
    return launch_pdl(quantize_tokens_kernel, grid, dim3(QT_THREADS), 0, st, p, c, k_src, v_src, src_offset, first_token, n_tokens, sb, sh,
                      stt) == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

}  // namespace kvsink
