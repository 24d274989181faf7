// Sink-token prediction: per-token outlier score, exact per-sequence top-k with index tie-break,
// Preserve-First-N, bitmask + ascending position list (Algorithm 1 at the emergence layer; Section 4.3).
#include <cooperative_groups.h>

#include "common.cuh"

namespace kvsink {

struct ChannelList {
    int n;
    int c[8];
};

// Magnitude key of an fp16 value: its 15-bit pattern, which orders finite values and infinity as |x| does.  A NaN
// (pattern above 0x7c00) compares false against everything in the reference comparison `|x| > best`, so it never raises
// a score: its key is 0.
__device__ __forceinline__ unsigned magnitude_key(uint16_t h)
{
    const unsigned a = h & 0x7fffu;
    return a > 0x7c00u ? 0u : a;
}

// score = max over listed channels of |H| as the 15-bit magnitude pattern of the fp16 value (order-preserving).
__global__ void sink_score_listed(const uint16_t *__restrict__ H, int S, int64_t sb, int64_t ss, ChannelList cl,
                                  uint16_t *__restrict__ score, int score_stride)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int b = blockIdx.y;
    pdl_wait();
    if (i >= S) return;
    const uint16_t *row = H + b * sb + i * ss;
    // the listed channels sit in different sectors of a row: all loads are issued before the first one is used
    uint16_t v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = j < cl.n ? __ldg(row + cl.c[j]) : (uint16_t)0;
    unsigned best = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const unsigned a = magnitude_key(v[j]);
        best = a > best ? a : best;
    }
    score[(size_t)b * score_stride + i] = (uint16_t)best;
}

// All d channels: one warp per token.
__global__ void sink_score_all(const uint16_t *__restrict__ H, int S, int d, int64_t sb, int64_t ss,
                               uint16_t *__restrict__ score, int score_stride)
{
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int b = blockIdx.y;
    pdl_wait();
    if (warp >= S) return;
    const uint16_t *row = H + b * sb + warp * ss;
    unsigned best = 0;
    for (int c = lane; c < d; c += 32) {
        unsigned a = magnitude_key(__ldg(row + c));
        best = a > best ? a : best;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned x = __shfl_xor_sync(0xffffffffu, best, o);
        best = x > best ? x : best;
    }
    if (lane == 0) score[(size_t)b * score_stride + warp] = (uint16_t)best;
}

constexpr int SEL_THREADS = 1024;

// Exclusive prefix sum of `v` over the block in thread order; *total = the sum over the block.
__device__ __forceinline__ int block_excl_sum(int v, int *total, unsigned *warp_tot)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    if (lane == 31) warp_tot[w] = (unsigned)incl;
    __syncthreads();
    const unsigned t = warp_tot[lane];           // SEL_THREADS / 32 == 32 warps
    unsigned tincl = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned x = __shfl_up_sync(0xffffffffu, tincl, o);
        if (lane >= o) tincl += x;
    }
    const int before = (int)__shfl_sync(0xffffffffu, tincl - t, w);
    *total = (int)__shfl_sync(0xffffffffu, tincl, 31);
    __syncthreads();
    return before + incl - v;
}

// Largest bin index whose suffix count (keys in bins >= it) reaches `need`, and how many of that bin's keys are still
// needed, from a 256-bin histogram; one warp, eight bins per lane.  need >= 1; if the histogram holds fewer than
// `need` keys the answer is bin 0.
__device__ __forceinline__ void find_bin(const unsigned *hist, int need, int *bin_out, int *rest_out)
{
    const int lane = threadIdx.x & 31;
    // lane l owns bins 255 - 8l ... 248 - 8l (descending), so that a prefix over lanes is a suffix over bins
    unsigned h[8], mine = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { h[j] = hist[255 - 8 * lane - j]; mine += h[j]; }
    unsigned incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    const unsigned before = incl - mine;                         // keys in the bins above this lane's
    const unsigned hit = __ballot_sync(0xffffffffu, (int)incl >= need);
    const int owner = hit ? __ffs((int)hit) - 1 : 31;            // first lane whose bins reach the count
    if (lane == owner) {
        int cum = (int)before, bin = 255 - 8 * lane;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            bin = 255 - 8 * lane - j;
            if (cum + (int)h[j] >= need || bin == 0) break;
            cum += (int)h[j];
        }
        *bin_out = bin;
        *rest_out = need - cum;
    }
}

// One more key in a shared-memory histogram.  (Electing one lane per bin with a warp match was measured: slower than the
// atomics it saves.)
__device__ __forceinline__ void hist_add(unsigned *hist, unsigned bin, bool valid)
{
    if (valid) atomicAdd(&hist[bin], 1u);
}

// One block per sequence: 2-pass radix select of the k-th largest 16-bit score, then an ordered pass that
// breaks ties by index, ORs the first N tokens in and emits mask words and ascending positions.
__global__ void __launch_bounds__(SEL_THREADS)
sink_select(const uint16_t *__restrict__ score, int score_stride, int S, int k, int N, int mask_words, int cap,
            uint32_t *__restrict__ bitmask, int32_t *__restrict__ sink_pos, int32_t *__restrict__ sink_count)
{
    __shared__ unsigned hist[256];
    __shared__ unsigned warp_tot[32];
    __shared__ int s_hi, s_need, s_lo, s_r;
    const int b = blockIdx.x, tid = threadIdx.x;
    const uint16_t *sc = score + (size_t)b * score_stride;
    const int kk = k < S ? k : S;
    pdl_wait();
    int vstar = 0x10000, r = 0;   // no score exceeds 0x10000: no top-k selection when kk == 0
    if (kk > 0) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        // eight independent loads per thread and trip, so that their latencies overlap
        constexpr int HB = 8;
        for (int base = 0; base < S; base += HB * SEL_THREADS) {
            unsigned v[HB];
#pragma unroll
            for (int j = 0; j < HB; ++j) { const int i = base + j * SEL_THREADS + tid; v[j] = i < S ? sc[i] : 0xffffffffu; }
#pragma unroll
            for (int j = 0; j < HB; ++j) hist_add(hist, (v[j] >> 8) & 0xffu, v[j] != 0xffffffffu);
        }
        __syncthreads();
        if (tid < 32) find_bin(hist, kk, &s_hi, &s_need);
        __syncthreads();
        const int hi = s_hi;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int base = 0; base < S; base += HB * SEL_THREADS) {
            unsigned v[HB];
#pragma unroll
            for (int j = 0; j < HB; ++j) { const int i = base + j * SEL_THREADS + tid; v[j] = i < S ? sc[i] : 0xffffffffu; }
#pragma unroll
            for (int j = 0; j < HB; ++j) hist_add(hist, v[j] & 0xffu, v[j] != 0xffffffffu && (int)(v[j] >> 8) == hi);
        }
        __syncthreads();
        if (tid < 32) find_bin(hist, s_need, &s_lo, &s_r);
        __syncthreads();
        vstar = (hi << 8) | s_lo;
        r = s_r;
    }
    // Ordered pass, TPT consecutive tokens per thread and step: two block scans per TPT * 1024 tokens.
    constexpr int TPT = 4;
    int run_eq = 0, run_sel = 0;
    const int lane = tid & 31;
    const int step = SEL_THREADS * TPT;
    const int S_round = (S + step - 1) / step * step;
    for (int base = 0; base < S_round; base += step) {
        const int i0 = base + TPT * tid;
        int key[TPT];
        if (i0 + TPT <= S) {   // the score rows are 16-byte aligned and i0 is a multiple of 4
            const uint2 v = *reinterpret_cast<const uint2 *>(sc + i0);
            key[0] = (int)(v.x & 0xffffu); key[1] = (int)(v.x >> 16); key[2] = (int)(v.y & 0xffffu); key[3] = (int)(v.y >> 16);
        } else {
#pragma unroll
            for (int j = 0; j < TPT; ++j) key[j] = i0 + j < S ? (int)sc[i0 + j] : -1;
        }
        int n_eq = 0;
#pragma unroll
        for (int j = 0; j < TPT; ++j) n_eq += key[j] == vstar;
        int tot_eq;
        int eq_rank = run_eq + block_excl_sum(n_eq, &tot_eq, warp_tot);
        unsigned nib = 0;
#pragma unroll
        for (int j = 0; j < TPT; ++j) {
            const bool eq = key[j] == vstar;
            const bool sel = i0 + j < S && (i0 + j < N || key[j] > vstar || (eq && eq_rank < r));
            eq_rank += eq;
            nib |= (unsigned)sel << j;
        }
        // eight threads share a mask word
        unsigned word = nib << (4 * (lane & 7));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        word |= __shfl_xor_sync(0xffffffffu, word, 4);
        if ((lane & 7) == 0 && (i0 >> 5) < mask_words) bitmask[(size_t)b * mask_words + (i0 >> 5)] = word;
        int tot_sel;
        int rank = run_sel + block_excl_sum(__popc(nib), &tot_sel, warp_tot);
#pragma unroll
        for (int j = 0; j < TPT; ++j)
            if ((nib >> j) & 1u) {
                if (rank < cap) sink_pos[(size_t)b * cap + rank] = i0 + j;
                ++rank;
            }
        run_eq += tot_eq;
        run_sel += tot_sel;
    }
    for (int w = S_round / 32 + tid; w < mask_words; w += SEL_THREADS) bitmask[(size_t)b * mask_words + w] = 0u;
    for (int j = run_sel + tid; j < cap; j += SEL_THREADS) sink_pos[(size_t)b * cap + j] = -1;
    if (tid == 0) sink_count[b] = run_sel < cap ? run_sel : cap;
}

// Long sequences: the blocks of one thread-block cluster share a sequence.  Block r owns the tokens
// [r * slice, (r + 1) * slice), slice a multiple of 4096; the blocks add their histograms up through distributed shared
// memory (both radix passes), count their keys equal to the k-th largest, and take the ranks of their selected tokens from
// the counts of the blocks before them, so that the result is the one sink_select gives.
constexpr int SELC_MAX_STEPS = 8;   // 4096-token steps per block

__global__ void __launch_bounds__(SEL_THREADS)
sink_select_cluster(const uint16_t *__restrict__ score, int score_stride, int S, int k, int N, int mask_words, int cap, int slice,
                    uint32_t *__restrict__ bitmask, int32_t *__restrict__ sink_pos, int32_t *__restrict__ sink_count)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cl = cg::this_cluster();
    __shared__ unsigned hist[256], ghist[256];
    __shared__ unsigned warp_tot[32];
    __shared__ int s_hi, s_need, s_lo, s_r, s_neq, s_nsel;
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int rk = (int)cl.block_rank(), C = (int)cl.num_blocks();
    const uint16_t *sc = score + (size_t)b * score_stride;
    const int kk = k < S ? k : S;
    const int lo = min(S, rk * slice), hi = min(S, lo + slice);
    pdl_wait();
    int vstar = 0x10000, r = 0;   // no score exceeds 0x10000: no top-k selection when kk == 0
    if (tid == 0) { s_neq = 0; s_nsel = 0; }
    // keys of this block's steps (TPT consecutive tokens per thread and step), loaded once (all loads in flight together) and
    // kept in registers for the histograms and both passes below; a token slot beyond the block's slice carries 0xffff,
    // which no key equals (keys are 15-bit magnitudes)
    constexpr int TPT = 4, STEP = SEL_THREADS * TPT;
    uint2 keys[SELC_MAX_STEPS];
#pragma unroll
    for (int st = 0; st < SELC_MAX_STEPS; ++st) {
        const int i0 = lo + st * STEP + TPT * tid;
        keys[st] = make_uint2(0xffffffffu, 0xffffffffu);
        if (st * STEP < slice && i0 < hi) {
            if (i0 + TPT <= hi) keys[st] = *reinterpret_cast<const uint2 *>(sc + i0);   // rows are 16-byte aligned, i0 a multiple of 4
            else {
                unsigned kq[4];
                for (int j = 0; j < TPT; ++j) kq[j] = i0 + j < hi ? sc[i0 + j] : 0xffffu;
                keys[st] = make_uint2(kq[0] | (kq[1] << 16), kq[2] | (kq[3] << 16));
            }
        }
    }
    auto key_of = [&](int st, int j) { return ((j < 2 ? keys[st].x : keys[st].y) >> (16 * (j & 1))) & 0xffffu; };
    if (kk > 0) {
        // the cluster's histogram of a key byte: every block sums the blocks' histograms for itself
        auto global_bin = [&](int need, int *bin_out, int *rest_out) {
            cl.sync();                                  // every block's histogram is complete
            if (tid < 256) {
                unsigned g = 0;
                for (int j = 0; j < C; ++j) g += cl.map_shared_rank(hist, j)[tid];
                ghist[tid] = g;
            }
            __syncthreads();
            if (tid < 32) find_bin(ghist, need, bin_out, rest_out);
            cl.sync();                                  // every block has read every histogram: they may be reused
        };
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
#pragma unroll
        for (int st = 0; st < SELC_MAX_STEPS; ++st)
            if (st * STEP < slice) {                    // block-uniform
#pragma unroll
                for (int j = 0; j < TPT; ++j) { const unsigned v = key_of(st, j); hist_add(hist, (v >> 8) & 0xffu, v != 0xffffu); }
            }
        global_bin(kk, &s_hi, &s_need);
        const int hi_byte = s_hi;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
#pragma unroll
        for (int st = 0; st < SELC_MAX_STEPS; ++st)
            if (st * STEP < slice) {
#pragma unroll
                for (int j = 0; j < TPT; ++j) { const unsigned v = key_of(st, j); hist_add(hist, v & 0xffu, v != 0xffffu && (int)(v >> 8) == hi_byte); }
            }
        global_bin(s_need, &s_lo, &s_r);
        vstar = (hi_byte << 8) | s_lo;
        r = s_r;
    }
    int my_eq = 0;
#pragma unroll
    for (int st = 0; st < SELC_MAX_STEPS; ++st)
#pragma unroll
        for (int j = 0; j < TPT; ++j) my_eq += (int)key_of(st, j) == vstar;
    // keys equal to the k-th largest in the blocks before this one
    if (my_eq) atomicAdd(&s_neq, my_eq);
    cl.sync();
    int run_eq = 0;
    for (int j = 0; j < rk; ++j) run_eq += *cl.map_shared_rank(&s_neq, j);
    // ordered pass over the block's tokens: selection bits and local ranks
    unsigned nib[SELC_MAX_STEPS];
    int lrank[SELC_MAX_STEPS];
    int run_sel = 0;
#pragma unroll
    for (int st = 0; st < SELC_MAX_STEPS; ++st) {
        nib[st] = 0; lrank[st] = 0;
        if (st * STEP < slice && lo + st * STEP < hi) {         // block-uniform
            const int i0 = lo + st * STEP + TPT * tid;
            int key[TPT], n_eq = 0;
#pragma unroll
            for (int j = 0; j < TPT; ++j) {
                key[j] = i0 + j < hi ? (int)(((j < 2 ? keys[st].x : keys[st].y) >> (16 * (j & 1))) & 0xffffu) : -1;
                n_eq += key[j] == vstar;
            }
            int tot_eq;
            int eq_rank = run_eq + block_excl_sum(n_eq, &tot_eq, warp_tot);
            unsigned nb = 0;
#pragma unroll
            for (int j = 0; j < TPT; ++j) {
                const bool eq = key[j] == vstar;
                const bool sel = i0 + j < hi && (i0 + j < N || key[j] > vstar || (eq && eq_rank < r));
                eq_rank += eq;
                nb |= (unsigned)sel << j;
            }
            unsigned word = nb << (4 * (lane & 7));           // eight threads share a mask word
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            word |= __shfl_xor_sync(0xffffffffu, word, 4);
            if ((lane & 7) == 0 && (i0 >> 5) < mask_words) bitmask[(size_t)b * mask_words + (i0 >> 5)] = word;
            int tot_sel;
            lrank[st] = run_sel + block_excl_sum(__popc(nb), &tot_sel, warp_tot);
            nib[st] = nb;
            run_eq += tot_eq;
            run_sel += tot_sel;
        }
    }
    if (tid == 0) s_nsel = run_sel;
    cl.sync();
    int base = 0, total = 0;
    for (int j = 0; j < C; ++j) {
        const int nj = *cl.map_shared_rank(&s_nsel, j);
        base += j < rk ? nj : 0;
        total += nj;
    }
#pragma unroll
    for (int st = 0; st < SELC_MAX_STEPS; ++st) {
        int rank = base + lrank[st];
        const int i0 = lo + st * STEP + TPT * tid;
#pragma unroll
        for (int j = 0; j < TPT; ++j)
            if ((nib[st] >> j) & 1u) {
                if (rank < cap) sink_pos[(size_t)b * cap + rank] = i0 + j;
                ++rank;
            }
    }
    if (rk == C - 1) {    // mask words beyond the last slice, unused positions, the count
        const int w0 = (min(S, C * slice) + STEP - 1) / STEP * STEP / 32;   // words the ordered pass has written
        for (int w = w0 + tid; w < mask_words; w += SEL_THREADS) bitmask[(size_t)b * mask_words + w] = 0u;
        for (int j = total + tid; j < cap; j += SEL_THREADS) sink_pos[(size_t)b * cap + j] = -1;
        if (tid == 0) sink_count[b] = total < cap ? total : cap;
    }
    cl.sync();   // nobody's shared memory goes away while another block reads it
}

size_t predict_workspace_bytes(const Params &p)
{
    size_t stride = ((size_t)p.max_seq + 7) / 8 * 8;
    return (size_t)p.B * stride * sizeof(uint16_t) + 16;
}

int launch_predict_sinks(const Params &p, const __half *hidden, int S, int64_t sb, int64_t ss, uint32_t *bitmask, int32_t *sink_pos,
                         int32_t *sink_count, void *workspace, cudaStream_t st)
{
    uint16_t *score = (uint16_t *)workspace;
    const int stride = (p.max_seq + 7) / 8 * 8;
    if (S > 0) {
        if (p.n_channels > 0) {
            ChannelList cl;
            cl.n = p.n_channels;
            for (int i = 0; i < 8; ++i) cl.c[i] = p.channels[i];
            dim3 grid((S + 255) / 256, p.B);
            if (launch_pdl(sink_score_listed, grid, dim3(256), 0, st, (const uint16_t *)hidden, S, sb, ss, cl, score, stride) != cudaSuccess)
                return KVSINK_ERR_CUDA;
        } else {
            dim3 grid((S + 7) / 8, p.B);
            if (launch_pdl(sink_score_all, grid, dim3(256), 0, st, (const uint16_t *)hidden, S, p.hidden, sb, ss, score, stride) != cudaSuccess)
                return KVSINK_ERR_CUDA;
        }
    }
    // long sequences: a cluster of 2, 4 or 8 blocks per sequence (slices of at least 8192 tokens, at most 32768)
    int C = 1;
    while (C < 8 && S > C * 8192) C *= 2;
    if (C > 1) {
        const int step = SEL_THREADS * 4;
        const int slice = ((S + C - 1) / C + step - 1) / step * step;
        if (slice <= SELC_MAX_STEPS * step) {
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = C; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(C, p.B);
            cfg.blockDim = dim3(SEL_THREADS);
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            if (cudaLaunchKernelEx(&cfg, sink_select_cluster, (const uint16_t *)score, stride, S, p.topk, p.pfn_n, p.mask_words, p.cap, slice,
                                   bitmask, sink_pos, sink_count) == cudaSuccess) {
                note_launch();
                return KVSINK_OK;
            }
            (void)cudaGetLastError();   // a cluster that cannot be placed: the one-block kernel below
        }
    }
    return launch_pdl(sink_select, dim3(p.B), dim3(SEL_THREADS), 0, st, (const uint16_t *)score, stride, S, p.topk, p.pfn_n, p.mask_words,
                      p.cap, bitmask, sink_pos, sink_count) == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

}  // namespace kvsink
