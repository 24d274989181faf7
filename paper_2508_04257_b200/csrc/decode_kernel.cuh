// Single-token decode attention over the packed cache (Eq. 3 with Eq. 7's split into sink and non-sink sums).
//
// A packed tile is the register image of the m16n8k16 A operand, so a lane's 128-bit load IS its fragment.
// Codes are never converted: a b-bit field masked in place is an fp16 subnormal (code * 2^k * 2^-24), which the
// tensor core multiplies exactly; the power-of-two position factors are folded into the B operand (column half)
// and into the fp32 epilogue (row half).
//   scores   S[token, head] = sum_c code[token, c] * (q[head, c] * scale[c]) - sum_c q*scale*zero      (keys)
//   outputs  O[c, head]     = sum_t code[c, t] * (p[t, head] * scale[t])  - sum_t p*scale*zero         (values)
// with M = 16 tokens (keys) or 16 channels (values), N = 8 query heads of one KV head, fp32 accumulation.
// Each warp streams whole key groups of one (sequence, KV head) unit; sequence splits are merged by a second
// kernel.  Sink tokens are masked out of the packed stream and added from the fp16 side buffer under the same
// softmax; keys of the open group come from the fp16 tail.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace kvsink {

constexpr int DEC_THREADS = DEC_WARPS * 32;
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movm_trans(uint32_t v)
{
    uint32_t o;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(o) : "r"(v));
    return o;
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}

// floor(log2(x)) of a positive normal float; -127 for zero and subnormals.
__device__ __forceinline__ int floor_log2(float x) { return (int)((__float_as_uint(x) >> 23) & 0xffu) - 127; }
// 2^e for -126 <= e <= 127.
__device__ __forceinline__ float pow2i(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <int BITS, int D>
struct Geo {
    static constexpr int W = D * BITS / 64;                  // 32-bit words per lane per tile
    static constexpr int NLO = (BITS == 3) ? D / 32 : W;     // words per lane in the first section
    static constexpr int NHI = (BITS == 3) ? D / 64 : 0;
    static constexpr int NM = D / 16;                        // 16x16 matrices per tile
    // value of a masked field = code * ROWF^(row half) * COLF^(col half) * 2^-24
    static constexpr float ROWF = (BITS == 2) ? 4.f : (BITS == 3 ? 1.f : 16.f);
    static constexpr float COLF = (BITS == 4) ? 1.f : 16.f;
};

// A lane's words of one tile: section planes of up to four words per lane.
template <int N>
__device__ __forceinline__ void load_section(const uint32_t *__restrict__ sec, int lane, uint32_t *w)
{
#pragma unroll
    for (int p = 0; p * 4 < N; ++p) {
        const int u = (N - 4 * p) > 4 ? 4 : (N - 4 * p);
        const uint32_t *src = sec + u * lane;
        if (u == 4) {
            uint4 v = __ldg((const uint4 *)src);
            w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
        } else if (u == 2) {
            uint2 v = __ldg((const uint2 *)src);
            w[4 * p] = v.x; w[4 * p + 1] = v.y;
        } else {
#pragma unroll
            for (int i = 0; i < u; ++i) w[4 * p + i] = __ldg(src + i);
        }
        sec += 32 * u;
    }
}

// The same from a tile image in shared memory.
template <int N>
__device__ __forceinline__ void load_section_shared(const uint32_t *sec, int lane, uint32_t *w)
{
#pragma unroll
    for (int p = 0; p * 4 < N; ++p) {
        const int u = (N - 4 * p) > 4 ? 4 : (N - 4 * p);
        const uint32_t *src = sec + u * lane;
        if (u == 4) {
            uint4 v = *(const uint4 *)src;
            w[4 * p] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
        } else if (u == 2) {
            uint2 v = *(const uint2 *)src;
            w[4 * p] = v.x; w[4 * p + 1] = v.y;
        } else {
#pragma unroll
            for (int i = 0; i < u; ++i) w[4 * p + i] = src[i];
        }
        sec += 32 * u;
    }
}

template <int BITS, int D>
__device__ __forceinline__ void load_tile_shared(const uint32_t *tile, int lane, uint32_t (&w)[Geo<BITS, D>::W])
{
    using G_ = Geo<BITS, D>;
    load_section_shared<G_::NLO>(tile, lane, w);
    if constexpr (BITS == 3) load_section_shared<G_::NHI>(tile + 32 * G_::NLO, lane, w + G_::NLO);
}

template <int BITS, int D>
__device__ __forceinline__ void load_tile(const uint32_t *__restrict__ tile, int lane, uint32_t (&w)[Geo<BITS, D>::W])
{
    using G_ = Geo<BITS, D>;
    load_section<G_::NLO>(tile, lane, w);
    if constexpr (BITS == 3) load_section<G_::NHI>(tile + 32 * G_::NLO, lane, w + G_::NLO);
}

// Masked fields of a lane's words as the A registers of the tile's NM matrices.
template <int BITS, int D>
__device__ __forceinline__ void tile_frags(const uint32_t (&w)[Geo<BITS, D>::W], uint32_t (&a)[Geo<BITS, D>::NM][4])
{
    using G_ = Geo<BITS, D>;
    if constexpr (BITS == 2) {
#pragma unroll
        for (int i = 0; i < G_::W; ++i) {
            const uint32_t x = w[i], y = x >> 8;
            a[2 * i][0] = x & 0x00030003u; a[2 * i][1] = x & 0x000c000cu; a[2 * i][2] = x & 0x00300030u; a[2 * i][3] = x & 0x00c000c0u;
            a[2 * i + 1][0] = y & 0x00030003u; a[2 * i + 1][1] = y & 0x000c000cu; a[2 * i + 1][2] = y & 0x00300030u; a[2 * i + 1][3] = y & 0x00c000c0u;
        }
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < G_::W; ++i) {
            const uint32_t x = w[i], y = x >> 8;
            a[i][0] = x & 0x000f000fu; a[i][1] = x & 0x00f000f0u; a[i][2] = y & 0x000f000fu; a[i][3] = y & 0x00f000f0u;
        }
    } else {
#pragma unroll
        for (int i = 0; i < G_::NLO; ++i) {
            const uint32_t x = w[i];
            const uint32_t hh = (i & 1) ? (w[G_::NLO + i / 2] << 2) : w[G_::NLO + i / 2];
            const uint32_t me = (x & 0x33333333u) | (hh & 0xccccccccu);                 // even fields, 3 bits at 4j
            const uint32_t mo = ((x >> 2) & 0x33333333u) | ((hh >> 1) & 0xccccccccu);   // odd fields
            const uint32_t me8 = me >> 8, mo8 = mo >> 8;
            a[2 * i][0] = me & 0x00070007u; a[2 * i][1] = mo & 0x00070007u; a[2 * i][2] = me & 0x00700070u; a[2 * i][3] = mo & 0x00700070u;
            a[2 * i + 1][0] = me8 & 0x00070007u; a[2 * i + 1][1] = mo8 & 0x00070007u; a[2 * i + 1][2] = me8 & 0x00700070u; a[2 * i + 1][3] = mo8 & 0x00700070u;
        }
    }
}

// ---- per-warp bulk-copy ring (TMA, cp.async.bulk) ----
// Barriers and copy destinations are passed as 32-bit shared-window addresses, converted once per warp.
__device__ __forceinline__ void mbar_init(uint32_t bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Global -> shared bulk copy; addresses and size are multiples of 16 bytes; completion is counted on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, unsigned bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

constexpr int DEC_WAIT_LIMIT = 1 << 22;   // polls of a full-barrier before a warp gives up (far beyond any real latency)

// Shared-memory plan of a decode block, shared by the kernel and the launcher.  CT = tiles per ring chunk, NQMAX = the
// most query heads a block of this instantiation serves (1 on the integer key side, 4 with the pair layout, else 8).
template <int BITS, int D, int NGv, int CT, int NQMAX, bool KTOK = false>
struct DecodePlan {
    static constexpr int W = D * BITS / 64, TILE_BYTES = 128 * W;
    static constexpr int BST = D + 8;                                   // padded row stride of the key B tables (bank spread)
    static constexpr int KV_BYTES = CT * TILE_BYTES, SZ_BYTES = CT * 16 * NGv * 4;
    // K words, V words, V scales, V zeros of CT tiles; with per-token keys (KTOK) also the K scales and K zeros
    static constexpr int SLOT_BYTES = 2 * KV_BYTES + (KTOK ? 4 : 2) * SZ_BYTES;
    static constexpr int NSLOT = (9216 / SLOT_BYTES >= 4) ? 4 : 2;      // power of two
    static constexpr int KP_BYTES = 2 * D * 4;                          // key scale + zero of one group
    static constexpr int WARP_RING = NSLOT * SLOT_BYTES + KP_BYTES;
    static constexpr int PS = D + 2;                                    // partial record: o[D], m, l
    // query tables (fp32 scaled, fp16 as given); the same space later holds the block's record for a cluster merge
    static constexpr int Q_BYTES = (NQMAX * D * 6 > NQMAX * PS * 4 ? NQMAX * D * 6 : NQMAX * PS * 4);
    static constexpr int B_BYTES = 2 * NQMAX * BST * 2;                 // per warp: key B operand rows (>= 512 for the limb tables)
    static constexpr int FIXED = (Q_BYTES + DEC_WARPS * B_BYTES + DEC_WARPS * 8 * 8 + 127) / 128 * 128;
    static constexpr int RING = DEC_WARPS * WARP_RING, PART = 2 * DEC_WARPS * NQMAX * PS * 4;
    static constexpr int BYTES = FIXED + (RING > PART ? RING : PART);
};

// PL ("pair layout", for at most four query heads per KV head): query head h owns accumulator columns 2h and 2h+1;
// column 2h multiplies by the fp16 factor q*scale and column 2h+1 by its fp16 rounding residual, so every score carries
// the factor to ~22 bits at no extra instruction.  Without PL (five to eight heads) head h owns column h and the
// residual of channels with large factors goes through a second multiply.
// I8 (one query head per KV head): the key side runs on the integer tensor path.  The four bytes of a stored
// word are four channels of one token row.  2 bit: the word masked with 0x03.., 0x0c.., 0x30.., 0xc0.. is the u8 A
// fragment of one m16n8k32 (fields in place: x1, x4 for the rows g + 8, x16 for the upper contraction slots, x64 for
// both).  4 bit: a word masked with 0x0f.. and 0xf0.. gives the registers of rows g and g + 8 (x16), two words (two
// matrices) make one fragment.  The B operand holds the factor q * scale * 2^sh of each channel as three signed 7-bit
// limbs in four accumulator columns (2, 3 bit: divided by 16 beforehand for the upper slots); sums are exact in int32.
// 3 bit: the low two bits as for 2 bit, the high bits of the second section (same byte structure) through four more
// MMAs with the same B operands into accumulators of their own.
// I8 = 2 (two to four query heads per KV head, 2 and 4 bit): the same with two B operands per word, which hold the upper
// and the lower byte pair of every head's factors in the pair layout's columns.
// I8 = 3 (five to eight rows: query heads, or the rows of a block of prompt queries; 2 and 4 bit): two operand tables of the
// I8 = 2 kind, one for the even rows and one for the odd rows, multiplied with the same masked words, so that lane t finds
// rows 2t and 2t+1 in its accumulators: the two columns it owns on the (eight-column, fp16) value side.  The key sums are
// exact integers, which the fp16 key side cannot offer when one channel is far louder than the rest.
//
// CAL (static, calibrated parameters): one (scale, zero) per key channel and per value channel group of the KV head for every
// token.  There are no token groups: the key B operand is prepared once per block, a ring chunk holds code words only, the
// stream covers every tile up to the sequence length (tokens beyond it are masked) and there is no fp16 tail.
//
// KT (per-token keys, PM = 2): keys carry one (scale, zero) per token and channel group like the values, so the key B operand
// holds the query alone (prepared once per block) and a token's parameters are applied to its dot products afterwards:
// score = sum over channel groups j of scale[t][j] * (dot_j - zero[t][j] * sum of the query over group j).  The parameters
// of a chunk's tokens arrive with the chunk.  Like CAL there are no token groups and no tail.  Integer key side only.
//
// PRE (attention of a chunk of prompt queries over the cache, Algorithm 1's attention statement): the eight accumulator
// columns of a block are eight (query token, query head) rows of one KV head, token-major; query token t sits at position
// q_pos0 + t and sees the cached tokens up to its own position, so every column has its own length limit.  One block streams
// the cache up to its last row's limit; there are no sequence splits.
struct PrefillShape {
    int T, q_pos0;               // queries in the chunk (0: single-token decode), position of the first
    int64_t q_sb, q_sh, q_st;    // element strides of q [B][Hq][T][D]
};

template <int BITS, int D, int NGv, int CT, bool PL, int I8 = 0, int PM = 0, bool PRE = false>
__global__ void __launch_bounds__(DEC_THREADS, 4)
decode_kernel(Params p, kvsink_cache c, kvsink_static_params sp, const __half *__restrict__ q, float *__restrict__ out, float *__restrict__ lse,
              float *__restrict__ part_ws, int nsplit, int groups_per_split, int qchunks, int seq_len, int cluster_merge, PrefillShape pre)
{
    using G_ = Geo<BITS, D>;
    constexpr int NQMAX = I8 == 1 ? 1 : (PL ? 4 : 8);
    using Plan = DecodePlan<BITS, D, NGv, CT, NQMAX, PM == 2>;
    constexpr int NM = G_::NM, W = G_::W, BST = Plan::BST, TILE_WORDS = 32 * W;
    constexpr int NSLOT = Plan::NSLOT, SLOT_BYTES = Plan::SLOT_BYTES, KV_BYTES = Plan::KV_BYTES, SZ_BYTES = Plan::SZ_BYTES;
    constexpr int mpg = (D / NGv) / 16;                              // value matrices per channel group
    constexpr int ST = CT >= 4 ? 4 : (CT >= 2 ? 2 : 1);                              // tiles per softmax step
    constexpr int CPL = D / 32;                                      // channels per lane in per-channel passes
    constexpr float LOG2E = 1.4426950408889634f;
    constexpr float QMAX = (float)((1 << BITS) - 1);
    constexpr float R1 = 1.f / G_::ROWF, C1 = 1.f / G_::COLF;

    const int tid = threadIdx.x, lane = tid & 31, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), g = lane >> 2, t = lane & 3;
    constexpr bool CAL = PM == 1, KT = PM == 2, FLAT = PM != 0;    // static parameters / per-token keys / either: no token groups
    constexpr int NGK = KT ? NGv : 1;                              // separate dot products per tile on the key side
    static_assert(!PRE || (!PL && (I8 == 0 || I8 == 3) && !FLAT), "prompt queries take an eight-column path");
    static_assert(I8 != 3 || (!PL && !KT && D == 128 && BITS != 3), "eight rows on the integer key side: 2 and 4 bit, head size 128");
    static_assert(!KT || (I8 != 0 && NGv <= 2 && (BITS != 3 || NGv == 1)), "per-token keys: integer key side, one or two channel groups");
    // decode: grid (splits, KV heads x blocks of eight query heads, sequences); prompt queries: grid (row blocks, KV heads, sequences)
    const int split = PRE ? 0 : blockIdx.x, h = PRE ? blockIdx.y : blockIdx.y / qchunks, qc = PRE ? blockIdx.x : blockIdx.y % qchunks, b = blockIdx.z;
    const int nq = I8 == 1 ? 1 : (PRE ? min(NQMAX, pre.T * p.rep - 8 * qc) : min(NQMAX, p.rep - NQMAX * qc)), hq0 = h * p.rep + (PRE ? 0 : NQMAX * qc);
    // prompt queries: row i of the block is query token (8 qc + i) / rep, query head (8 qc + i) % rep of this KV head
    auto row_token = [&](int i) { return (8 * qc + i) / p.rep; };
    auto row_limit = [&](int i) { return i < nq ? pre.q_pos0 + row_token(i) + 1 : 0; };    // cached tokens the row sees
    const int64_t unit = (int64_t)b * p.Hkv + h;
    // with static parameters a "group" of the loops below is one ring chunk, and every token belongs to one
    const int G = FLAT ? CT * KVSINK_TILE : p.G;
    const int n = PRE ? min(seq_len, row_limit(nq - 1)) : seq_len;                        // tokens this block looks at
    const int n_groups = FLAT ? (n + G - 1) / G : (PRE ? min(seq_len / G, (n + G - 1) / G) : n / G);
    const int n_body = FLAT ? n : (seq_len / G) * G;                                       // where the fp16 tail begins
    // limits of this lane's accumulator columns 2t, 2t+1 and the smallest limit of the block (prompt queries only)
    const int lim0 = PRE ? row_limit(2 * t) : 0, lim1 = PRE ? row_limit(2 * t + 1) : 0, lim_min = PRE ? row_limit(0) : 0;
    if (PRE) groups_per_split = n_groups;
    const int TPG = G / KVSINK_TILE, CPG = TPG / CT;                 // tiles and ring chunks per key group
    const uint32_t *bm = c.sink_bitmask + (size_t)b * p.mask_words;
    const float qscale = LOG2E * rsqrtf((float)D);

    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *qs = (float *)smem_raw;                                   // [NQMAX][D] q * log2e/sqrt(D)
    __half *q16 = (__half *)(qs + NQMAX * D);                        // [NQMAX][D] q as given
    __half *Bs_all = (__half *)(smem_raw + Plan::Q_BYTES);           // [warps][2][NQMAX][BST] key B operand (hi, lo) of the group
    uint64_t *bars = (uint64_t *)(smem_raw + Plan::Q_BYTES + DEC_WARPS * Plan::B_BYTES);   // [warps][8]: 4 chunk slots, 2 parameter slots
    unsigned char *ring_all = smem_raw + Plan::FIXED;                // [warps][WARP_RING]; later reused for the partials
    float *part = (float *)ring_all;                                 // [2*warps][nq][D+2]

    // chunk full-barriers (one per ring slot) and the parameter full-barrier of this warp, as shared-window addresses
    const uint32_t cbar = smem_addr(bars + warp * 8), pbar = cbar + 4 * 8;
    if (lane == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(cbar + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // launched with programmatic stream serialization: everything above overlaps the tail of the kernel before this
    // one in the stream; nothing it may have written (the query, the cache) is read before this point
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the next kernel in the stream may be scheduled from now on: its blocks take whatever room this grid leaves, set
    // themselves up, and wait at the same point until this grid has completed
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Sink rows of the side buffer are shared out over all warps of all splits and handled after the stream; the
    // first row of this warp is fetched now, so that its latency hides behind the stream.
    const int sink_n = min(c.sink_count[b], p.cap);
    const int sink_worker = split * DEC_WARPS + warp, sink_workers = nsplit * DEC_WARPS;
    int sink_pos_next = -1;
    uint32_t sink_k_next[CPL / 2], sink_v_next[CPL / 2];
    auto fetch_sink = [&](int j) {
        sink_pos_next = -1;
#pragma unroll
        for (int e = 0; e < CPL / 2; ++e) sink_k_next[e] = sink_v_next[e] = 0u;
        if (j < sink_n) {
            sink_pos_next = c.sink_pos[(size_t)b * p.cap + j];
            const uint32_t *kr = (const uint32_t *)((const __half *)c.sink_k + ((size_t)unit * p.cap + j) * D + lane * CPL);
            const uint32_t *vr = (const uint32_t *)((const __half *)c.sink_v + ((size_t)unit * p.cap + j) * D + lane * CPL);
#pragma unroll
            for (int e = 0; e < CPL / 2; ++e) { sink_k_next[e] = kr[e]; sink_v_next[e] = vr[e]; }
        }
    };
    fetch_sink(sink_worker);

    // ---------------- packed stream ----------------
    float m0 = M_INIT, m1 = M_INIT, l0 = 0.f, l1 = 0.f;             // running max / sum of query heads 2t and 2t+1
    float O[NM][4];
    float bv[NGv][2];                     // sum p*scale*zero per value channel group and head
    int ev = 60;                          // the value B operand is p * scale * 2^ev; lowered so that it fits fp16
    float evf = pow2i(60);
#pragma unroll
    for (int m = 0; m < NM; ++m)
#pragma unroll
        for (int i = 0; i < 4; ++i) O[m][i] = 0.f;
#pragma unroll
    for (int j = 0; j < NGv; ++j) bv[j][0] = bv[j][1] = 0.f;

    __half *Bs = Bs_all + (size_t)warp * 2 * NQMAX * BST, *Bl = Bs + (size_t)NQMAX * BST;
    const uint8_t *kc_base = c.k_codes + (size_t)unit * p.max_seq * p.row_bytes;
    const uint8_t *vc_base = c.v_codes + (size_t)unit * p.max_seq * p.row_bytes;
    const float *vs_base = c.v_scale + (size_t)unit * p.max_seq * NGv;
    const float *vz_base = c.v_zero + (size_t)unit * p.max_seq * NGv;
    const float *ktok_s_base = c.k_scale + (size_t)unit * p.max_seq * NGv;    // per-token keys: [unit][max_seq][NGv]
    const float *ktok_z_base = c.k_zero + (size_t)unit * p.max_seq * NGv;
    const float *ks_base = c.k_scale + (size_t)unit * (p.max_seq / G) * D;
    const float *kz_base = c.k_zero + (size_t)unit * (p.max_seq / G) * D;

    // Lowers ev so that p * scale * 2^ev stays below 2^13 for the largest |scale| mx any lane has seen.
    // ev_limit = 2^(13 - ev): scales below it need no action, which is the common case and costs one vote.
    float ev_limit = 0.f;
    auto fit_value_scale = [&](float mx) {
        if (!__any_sync(0xffffffffu, mx >= ev_limit)) return;
        mx = warp_max(mx);
        int need = 12 - floor_log2(mx);
        need = need > 60 ? 60 : (need < -60 ? -60 : need);
        if (need < ev) {     // warp-uniform: every quad column holds the same tokens
            const float f = pow2i(need - ev);
#pragma unroll
            for (int m = 0; m < NM; ++m)
#pragma unroll
                for (int i = 0; i < 4; ++i) O[m][i] *= f;
            ev = need;
            evf = pow2i(ev);
            ev_limit = pow2i(13 - ev);
        }
    };
    // New running maxima after a batch of scores with per-lane maxima tm0 / tm1; rescales the accumulators if needed.
    // Once the running maxima have settled no lane exceeds them and the step costs one vote.
    auto advance_max = [&](float tm0, float tm1) {
        if (PL) tm1 = M_INIT;
        if (!__any_sync(0xffffffffu, tm0 > m0 || tm1 > m1)) return;
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            tm0 = fmaxf(tm0, __shfl_xor_sync(0xffffffffu, tm0, o));
            tm1 = fmaxf(tm1, __shfl_xor_sync(0xffffffffu, tm1, o));
        }
        const float mn0 = fmaxf(m0, tm0), mn1 = fmaxf(m1, tm1);
        const float c0 = ex2(m0 - mn0), c1 = ex2(m1 - mn1);
        l0 *= c0; l1 *= c1;
#pragma unroll
        for (int j = 0; j < NGv; ++j) { bv[j][0] *= c0; bv[j][1] *= c1; }
#pragma unroll
        for (int m = 0; m < NM; ++m) { O[m][0] *= c0; O[m][2] *= c0; O[m][1] *= PL ? c0 : c1; O[m][3] *= PL ? c0 : c1; }
        m0 = mn0; m1 = mn1;
    };
    // Value products of one tile: scores s (log2 units, relative maxima already advanced), value words vw, and the
    // (scale, zero) of tokens g (sv0, zv0) and g+8 (sv1, zv1) per channel group.
    auto tile_values = [&](const float (&s)[4], const uint32_t (&vw)[W], const float (&sv0)[NGv], const float (&zv0)[NGv],
                           const float (&sv1)[NGv], const float (&zv1)[NGv]) {
        const float p0 = ex2(s[0] - m0), p1 = PL ? 0.f : ex2(s[1] - m1), p2 = ex2(s[2] - m0), p3 = PL ? 0.f : ex2(s[3] - m1);
        l0 += p0 + p2;
        if (!PL) l1 += p1 + p3;
        uint32_t va[NM][4];
        tile_frags<BITS, D>(vw, va);
        const float evc = evf * C1;
#pragma unroll
        for (int j = 0; j < NGv; ++j) {
            const float e0 = sv0[j] * evf, e1 = sv1[j] * evc, sz0 = sv0[j] * zv0[j], sz1 = sv1[j] * zv1[j];
            bv[j][0] = fmaf(p0, sz0, fmaf(p2, sz1, bv[j][0]));
            if (!PL) bv[j][1] = fmaf(p1, sz0, fmaf(p3, sz1, bv[j][1]));
            uint32_t b0, b1;
            if constexpr (PL) {
                // the odd columns carry the fp16 rounding residual of the weight p * scale: the outputs keep the weight
                // to ~22 bits (columns 2h and 2h+1 are added at the end)
                const float x0 = p0 * e0, x1 = p2 * e1;
                const float r0 = x0 - __half2float(__float2half_rn(x0)), r1 = x1 - __half2float(__float2half_rn(x1));
                b0 = movm_trans(pack_half2(x0, r0));
                b1 = movm_trans(pack_half2(x1, r1));
            } else {
                // every column is a row of its own: the fp16 rounding residuals of the four weights go through a second
                // multiply of the same value fragments (no further masks), which keeps the weights to ~22 bits here too
                const float x0 = p0 * e0, x1 = p1 * e0, x2 = p2 * e1, x3 = p3 * e1;
                const __half2 h01 = __floats2half2_rn(x0, x1), h23 = __floats2half2_rn(x2, x3);
                const float2 f01 = __half22float2(h01), f23 = __half22float2(h23);
                b0 = movm_trans(*reinterpret_cast<const uint32_t *>(&h01));
                b1 = movm_trans(*reinterpret_cast<const uint32_t *>(&h23));
                const uint32_t r0 = movm_trans(pack_half2(x0 - f01.x, x1 - f01.y)), r1 = movm_trans(pack_half2(x2 - f23.x, x3 - f23.y));
#pragma unroll
                for (int mi = 0; mi < mpg; ++mi) mma16816(O[j * mpg + mi], va[j * mpg + mi], r0, r1);
            }
#pragma unroll
            for (int mi = 0; mi < mpg; ++mi) mma16816(O[j * mpg + mi], va[j * mpg + mi], b0, b1);
        }
    };

    // ---- complete key groups of this split: the warps take contiguous, nearly equal ranges of its groups.  A warp's
    //      chunks (CT tiles each) are consecutive in memory and arrive through a ring of NSLOT bulk-copy slots filled
    //      NSLOT - 1 chunks ahead by lane 0; the key parameters of a group arrive one group ahead through one more slot. ----
    const int g_begin = split * groups_per_split, g_end = min(n_groups, g_begin + groups_per_split);
    const int g_cnt = max(g_end - g_begin, 0);
    const int w_begin = g_begin + (g_cnt * warp) / DEC_WARPS, w_end = g_begin + (g_cnt * (warp + 1)) / DEC_WARPS;
    const int my_groups = w_end - w_begin;
    unsigned char *ring = ring_all + (size_t)warp * Plan::WARP_RING;
    float *kp_ring = (float *)(ring + NSLOT * SLOT_BYTES);           // [scale D | zero D] of the next group to prepare
    // Every lane keeps the issue bookkeeping (so that addresses and counters stay warp-uniform values); lane 0 alone
    // issues the copies.  Byte offsets inside the unit's arrays fit 32 bits.
    const int n_chunks = my_groups * CPG;
    int iss = 0;                                                     // chunks issued so far
    uint32_t iss_kv = (uint32_t)w_begin * TPG * Plan::TILE_BYTES;    // byte offset of the next chunk in the code arrays
    uint32_t iss_sz = (uint32_t)w_begin * TPG * 16 * NGv * 4;        // and in the value parameter arrays
    const uint32_t ring_s = smem_addr(ring), kp_s = smem_addr(kp_ring);
    auto issue_chunk = [&]() {
        const int slot = iss & (NSLOT - 1);
        // debug builds: the chunk must lie inside the unit's code arrays (a skipped copy ends in the wait's time-out)
        const bool inside = in_bounds((size_t)iss_kv + KV_BYTES <= (size_t)p.max_seq * p.row_bytes, c.status);
        const uint32_t dst = ring_s + slot * SLOT_BYTES, bar = cbar + 8 * slot;
        if (lane == 0 && inside) {
            mbar_expect_tx(bar, CAL ? 2 * KV_BYTES : SLOT_BYTES);
            bulk_g2s(dst, kc_base + iss_kv, KV_BYTES, bar);
            bulk_g2s(dst + KV_BYTES, vc_base + iss_kv, KV_BYTES, bar);
            if constexpr (!CAL) {
                bulk_g2s(dst + 2 * KV_BYTES, (const unsigned char *)vs_base + iss_sz, SZ_BYTES, bar);
                bulk_g2s(dst + 2 * KV_BYTES + SZ_BYTES, (const unsigned char *)vz_base + iss_sz, SZ_BYTES, bar);
            }
            if constexpr (KT) {   // the tokens' key parameters (same shape as the value parameters) follow them in the slot
                bulk_g2s(dst + 2 * KV_BYTES + 2 * SZ_BYTES, (const unsigned char *)ktok_s_base + iss_sz, SZ_BYTES, bar);
                bulk_g2s(dst + 2 * KV_BYTES + 3 * SZ_BYTES, (const unsigned char *)ktok_z_base + iss_sz, SZ_BYTES, bar);
            }
        }
        ++iss;
        iss_kv += KV_BYTES;
        iss_sz += SZ_BYTES;
    };
    auto issue_params = [&](int gi) {
        if (lane == 0) {
            mbar_expect_tx(pbar, Plan::KP_BYTES);
            bulk_g2s(kp_s, ks_base + (size_t)(w_begin + gi) * D, D * 4, pbar);
            bulk_g2s(kp_s + D * 4, kz_base + (size_t)(w_begin + gi) * D, D * 4, pbar);
        }
    };
    auto wait_bar = [&](uint32_t bar, unsigned parity) {
        int polls = 0;
        bool ok = true;
        while (!mbar_try_wait(bar, parity)) {
            if (++polls > DEC_WAIT_LIMIT) { ok = false; break; }
        }
        return __all_sync(0xffffffffu, ok);
    };
    if (my_groups > 0) {
        if (!FLAT) issue_params(0);
        for (int i = 0; i < NSLOT - 1 && iss < n_chunks; ++i) issue_chunk();
    }
    // static value parameters of the KV head: the same for every token
    float cal_sv[NGv], cal_zv[NGv];
#pragma unroll
    for (int j = 0; j < NGv; ++j) { cal_sv[j] = cal_zv[j] = 0.f; }
    if constexpr (CAL) {
        float mx = 0.f;
#pragma unroll
        for (int j = 0; j < NGv; ++j) {
            cal_sv[j] = sp.v_scale[h * NGv + j]; cal_zv[j] = sp.v_zero[h * NGv + j];
            mx = fmaxf(mx, fabsf(cal_sv[j]));
        }
        fit_value_scale(mx);
    }
    // the first copies are in flight: now the query tables (the copies do not depend on them)
    for (int i = tid; i < NQMAX * D; i += DEC_THREADS) {
        const int qh = i / D, ch = i % D;
        __half v = __float2half(0.f);
        if (qh < nq)
            v = PRE ? q[b * pre.q_sb + (int64_t)(hq0 + (8 * qc + qh) % p.rep) * pre.q_sh + (int64_t)row_token(qh) * pre.q_st + ch]
                    : q[((size_t)b * p.Hq + hq0 + qh) * D + ch];
        q16[i] = v;
        qs[i] = __half2float(v) * qscale;
    }
    __syncthreads();

    constexpr int PS = D + 2;                                        // partial record: o[D], m, l

    // Integer key side: lane l prepares the B operand bytes of one group of four contraction slots, (MMA l/8, lower or
    // upper slots (l/4)%2, slots 4(l%4) ... +3); these are its four channels and their query values.
    int i8_ch[4] = {0, 0, 0, 0};
    float i8_q[4] = {0.f, 0.f, 0.f, 0.f};
    if constexpr (I8) {
        const int mi = lane >> 3, c2 = (lane >> 2) & 1, tq = lane & 3;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            i8_ch[e] = BITS != 4 ? 16 * (2 * mi + (e & 1)) + 8 * c2 + 2 * tq + (e >> 1)
                                 : 16 * (2 * mi + c2) + 8 * (e & 1) + 2 * tq + (e >> 1);
            if (I8 == 1) i8_q[e] = qs[i8_ch[e]];
        }
    }

    // sink bits of the CT tiles starting at tile T: one 32-bit word covers two tiles
    auto load_mask_words = [&](int T) {
        uint2 w;
        w.x = __ldg(bm + (T >> 1));
        w.y = CT == 4 ? __ldg(bm + (T >> 1) + 1) : 0u;
        return w;
    };
    uint2 mword_next = my_groups > 0 ? load_mask_words(w_begin * TPG) : make_uint2(0u, 0u);
    bool stream_ok = true;
    int ci = 0;                                                      // running chunk index of this warp

    // ---- tokens of the open group: keys from the fp16 tail (last split only).  They come first, while the warp's first
    //      chunks are on their way (the order of the softmax steps does not matter) ----
    if (!FLAT && split == nsplit - 1) {
        const __half *tail = (const __half *)c.k_tail + (size_t)unit * G * D;
        const int T_begin = n_body / KVSINK_TILE, T_end = (n + KVSINK_TILE - 1) / KVSINK_TILE;
        for (int T = T_begin + warp; T < T_end; T += DEC_WARPS) {
            const int tok0 = T * KVSINK_TILE + g, tok1 = tok0 + 8;
            const bool in0 = tok0 < n, in1 = tok1 < n;
            const __half *r0 = tail + (size_t)(tok0 % G) * D, *r1 = tail + (size_t)(tok1 % G) * D;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int m = 0; m < NM; ++m) {
                uint32_t a[4];
                a[0] = in0 ? *(const uint32_t *)(r0 + 16 * m + 2 * t) : 0u;
                a[1] = in1 ? *(const uint32_t *)(r1 + 16 * m + 2 * t) : 0u;
                a[2] = in0 ? *(const uint32_t *)(r0 + 16 * m + 2 * t + 8) : 0u;
                a[3] = in1 ? *(const uint32_t *)(r1 + 16 * m + 2 * t + 8) : 0u;
                const int qrow = PL ? (g >> 1) : g;          // query head in accumulator column g
                const bool qcol = PL ? (!(g & 1) && qrow < NQMAX) : true;
                const uint32_t b0 = qcol ? *(const uint32_t *)(q16 + qrow * D + 16 * m + 2 * t) : 0u;
                const uint32_t b1 = qcol ? *(const uint32_t *)(q16 + qrow * D + 16 * m + 2 * t + 8) : 0u;
                mma16816(acc, a, b0, b1);
            }
            const bool v0 = in0 && !mask_bit(bm, in0 ? tok0 : 0), v1 = in1 && !mask_bit(bm, in1 ? tok1 : 0);
            float s[4];
            s[0] = v0 ? acc[0] * qscale : -INFINITY; s[1] = (v0 && !PL) ? acc[1] * qscale : -INFINITY;
            s[2] = v1 ? acc[2] * qscale : -INFINITY; s[3] = (v1 && !PL) ? acc[3] * qscale : -INFINITY;
            if constexpr (PRE) {   // every column sees the tokens up to its own query
                if (tok0 >= lim0) s[0] = -INFINITY;
                if (tok0 >= lim1) s[1] = -INFINITY;
                if (tok1 >= lim0) s[2] = -INFINITY;
                if (tok1 >= lim1) s[3] = -INFINITY;
            }
            advance_max(fmaxf(s[0], s[2]), fmaxf(s[1], s[3]));
            uint32_t vw[W];
            load_tile<BITS, D>((const uint32_t *)(vc_base + (size_t)T * p.tile_bytes), lane, vw);
            float sv0[NGv], zv0[NGv], sv1[NGv], zv1[NGv];
            float mx = 0.f;
#pragma unroll
            for (int j = 0; j < NGv; ++j) {   // tokens beyond the sequence have no parameters yet
                sv0[j] = v0 ? __ldg(vs_base + (size_t)tok0 * NGv + j) : 0.f; zv0[j] = v0 ? __ldg(vz_base + (size_t)tok0 * NGv + j) : 0.f;
                sv1[j] = v1 ? __ldg(vs_base + (size_t)tok1 * NGv + j) : 0.f; zv1[j] = v1 ? __ldg(vz_base + (size_t)tok1 * NGv + j) : 0.f;
                mx = fmaxf(mx, fmaxf(fabsf(sv0[j]), fabsf(sv1[j])));
            }
            fit_value_scale(mx);
            tile_values(s, vw, sv0, zv0, sv1, zv1);
        }
    }

    // state of the current key group (with static parameters: of the KV head, set up on the first trip)
    float bias0 = 0.f, bias1 = 0.f, ks0 = 0.f, ks1 = 0.f;
    uint32_t need_lo = 0;     // bit m: matrix m also gets the low half of the split factor (warp-uniform)
    uint32_t bk[NM][2];
#pragma unroll
    for (int m = 0; m < NM; ++m) bk[m][0] = bk[m][1] = 0u;
#pragma unroll 1
    for (int gi = 0; gi < my_groups && stream_ok; ++gi) {
        const int grp = w_begin + gi;
        // ---- B operand of the group: fp16(q * scale * 2^sh) per channel and head (sh puts the largest factor of the
        //      head in [2^13, 2^14)), column half pre-divided by COLF; bias = sum_c of the same rounded factors * zero ----
        if (!FLAT || gi == 0) {
        bias0 = bias1 = ks0 = ks1 = 0.f;
        need_lo = 0;
        {
            float scv[CPL], zev[CPL];
            if constexpr (CAL) {
#pragma unroll
                for (int e = 0; e < CPL; ++e) {
                    const int ch = I8 ? i8_ch[e] : lane * CPL + e;
                    scv[e] = sp.k_scale[h * D + ch]; zev[e] = sp.k_zero[h * D + ch];
                }
            } else if constexpr (KT) {
                // the operand is the query itself; with zero = 1 the "zero-point term" below is the sum of the query
#pragma unroll
                for (int e = 0; e < CPL; ++e) { scv[e] = 1.f; zev[e] = 1.f; }
            } else {
                if (!wait_bar(pbar, (unsigned)gi & 1u)) { stream_ok = false; break; }
                const float *kp = kp_ring;
#pragma unroll
                for (int e = 0; e < CPL; ++e) {
                    const int ch = I8 ? i8_ch[e] : lane * CPL + e;
                    scv[e] = kp[ch]; zev[e] = kp[D + ch];
                }
                __syncwarp();   // the parameters are in registers: the slot can take the next group's while this one streams
                if (gi + 1 < my_groups) issue_params(gi + 1);
            }
            if constexpr (I8 == 1) {
                // limbs of the one head's factors: F = rint(q * scale * 2^sh) with the largest |F| in [2^29, 2^30), cut into
                // four signed bytes (radix 256): every factor is kept to 2^-30 of the group's largest one (2^-26 where the
                // factor is pre-divided for the upper contraction slots), finer than binary32 keeps the factor itself.
                // Adding 0x808080 propagates the carries of the signed digits and the exclusive-or removes the offset again.
                float v[4], amax = 0.f, bsum = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[e] = i8_q[e] * scv[e];
                    amax = fmaxf(amax, fabsf(v[e]));
                    // the zero-point term takes the unrounded factor: the limbs' rounding then meets the codes (at most
                    // qmax) only, not code - zero, which is large for a channel far from zero with a narrow range
                    bsum = fmaf(v[e], zev[e], bsum);
                }
                amax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(amax)));   // non-negative floats order as integers
                int sh = 29 - floor_log2(amax);
                sh = sh > 60 ? 60 : (sh < -60 ? -60 : sh);
                const bool upper = BITS != 4 && (lane & 4) != 0;   // 2, 3 bit: this lane's channels sit in the upper contraction slots (x16 in place)
                const float pre = upper ? pow2i(sh - 4) : pow2i(sh);
                uint32_t d[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) d[e] = ((uint32_t)__float2int_rn(v[e] * pre) + 0x00808080u) ^ 0x00808080u;
                // byte transpose: word j = byte j of the four channels, in contraction-slot order
                const uint32_t t0 = __byte_perm(d[0], d[1], 0x5140), t1 = __byte_perm(d[0], d[1], 0x7362);
                const uint32_t t2 = __byte_perm(d[2], d[3], 0x5140), t3 = __byte_perm(d[2], d[3], 0x7362);
                // table [MMA][lower / upper slots][limb, most significant first][t][byte]: this lane owns one 4-byte slot group
                uint32_t *tab = reinterpret_cast<uint32_t *>(Bs) + (lane >> 2) * 16 + (lane & 3);
                tab[0] = __byte_perm(t1, t3, 0x7632);
                tab[4] = __byte_perm(t1, t3, 0x5410);
                tab[8] = __byte_perm(t0, t2, 0x7632);
                tab[12] = __byte_perm(t0, t2, 0x5410);
                if constexpr (KT && NGv == 2) {
                    // per-token keys, two channel groups: the query's sum over each (lanes 0-15 hold channels 0-63)
                    const float b0s = warp_sum(lane < 16 ? bsum : 0.f), b1s = warp_sum(lane < 16 ? 0.f : bsum);
                    if (t == 0) { bias0 = b0s; bias1 = b1s; ks0 = pow2i(-sh); }
                } else {
                    bsum = warp_sum(bsum);
                    if (t == 0) { bias0 = bsum; ks0 = pow2i(-sh); }
                }
            } else if constexpr (I8 >= 2) {
                // up to four heads: the same four signed bytes per factor and head, each head with its own power of two.
                // The two most significant bytes of every head fill the eight columns of one B operand (head h in columns
                // 2h, 2h+1), the two less significant ones those of a second: lane t then finds both halves of head t's sum
                // in its own accumulators.  Table [MMA][lower / upper slots][operand][column][t] in 32-bit words.
                // I8 = 3 (five to eight rows): two such tables, the first for the even rows and the second for the odd rows, so
                // that lane t finds rows 2t and 2t+1 -- the two columns it owns on the value side -- in its accumulators.
                constexpr int NROW = I8 == 3 ? 8 : 4;
                const bool upper = BITS != 4 && (lane & 4) != 0;
#pragma unroll
                for (int row = 0; row < NROW; ++row) {
                    const int hh = I8 == 3 ? row >> 1 : row, set = I8 == 3 ? row & 1 : 0;
                    uint32_t *tab = reinterpret_cast<uint32_t *>(Bs) + set * 512 + (lane >> 2) * 64 + (lane & 3);
                    uint32_t w3 = 0u, w2 = 0u, w1 = 0u, w0 = 0u;
                    if (row < nq) {
                        float v[4], amax = 0.f, bsum = 0.f;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            v[e] = qs[row * D + i8_ch[e]] * scv[e];
                            amax = fmaxf(amax, fabsf(v[e]));
                            bsum = fmaf(v[e], zev[e], bsum);
                        }
                        amax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(amax)));
                        int sh = 29 - floor_log2(amax);
                        sh = sh > 60 ? 60 : (sh < -60 ? -60 : sh);
                        const float pre = upper ? pow2i(sh - 4) : pow2i(sh);
                        uint32_t d[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) d[e] = ((uint32_t)__float2int_rn(v[e] * pre) + 0x00808080u) ^ 0x00808080u;
                        const uint32_t t0 = __byte_perm(d[0], d[1], 0x5140), t1 = __byte_perm(d[0], d[1], 0x7362);
                        const uint32_t t2 = __byte_perm(d[2], d[3], 0x5140), t3 = __byte_perm(d[2], d[3], 0x7362);
                        w3 = __byte_perm(t1, t3, 0x7632); w2 = __byte_perm(t1, t3, 0x5410);
                        w1 = __byte_perm(t0, t2, 0x7632); w0 = __byte_perm(t0, t2, 0x5410);
                        if constexpr (KT && NGv == 2) {
                            const float b0s = warp_sum(lane < 16 ? bsum : 0.f), b1s = warp_sum(lane < 16 ? 0.f : bsum);
                            if (t == hh) { bias0 = b0s; bias1 = b1s; ks0 = pow2i(-sh); }
                        } else {
                            bsum = warp_sum(bsum);
                            if (t == hh) {
                                if (set == 0) { bias0 = bsum; ks0 = pow2i(-sh); } else { bias1 = bsum; ks1 = pow2i(-sh); }
                            }
                        }
                    }
                    tab[(2 * hh) * 4] = w3;
                    tab[(2 * hh + 1) * 4] = w2;
                    tab[(8 + 2 * hh) * 4] = w1;
                    tab[(8 + 2 * hh + 1) * 4] = w0;
                }
            } else {
            // one power-of-two scaling for all heads of the group: the largest factor lands in [2^13, 2^14)
            constexpr int NQL = PL ? 4 : 8;
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < NQL; ++i)
                if (i < nq) {
#pragma unroll
                    for (int e = 0; e < CPL; ++e) amax = fmaxf(amax, fabsf(qs[i * D + lane * CPL + e] * scv[e]));
                }
            amax = warp_max(amax);
            int sh = 13 - floor_log2(amax);
            sh = sh > 60 ? 60 : (sh < -60 ? -60 : sh);
            const float f = pow2i(sh), finv = pow2i(-sh), ksc = pow2i(24 - sh);
            const bool scaled_col = ((lane * CPL) & 8) && G_::COLF != 1.f;   // this lane's channels sit in the column half
            const __half2 colf = __half2half2(__float2half(scaled_col ? C1 : 1.f));
            bool big = false;
#pragma unroll
            for (int i = 0; i < NQL; ++i) {
                if (i < nq) {
                    float bsum = 0.f;
                    __half2 hb[CPL / 2], lb[CPL / 2];
#pragma unroll
                    for (int e = 0; e < CPL; e += 2) {
                        const float v0 = qs[i * D + lane * CPL + e] * scv[e], v1 = qs[i * D + lane * CPL + e + 1] * scv[e + 1];
                        const float f0 = v0 * f, f1 = v1 * f;
                        // fp16 keeps 11 bits of a factor; its rounding residual is kept as a second factor (always with PL,
                        // else where it could move a score by more than ~4e-4: factor * largest |code - zero| * 2^-12)
                        const __half2 h = __floats2half2_rn(f0, f1);
                        const float2 hf = __half22float2(h);
                        const __half2 l = __floats2half2_rn(f0 - hf.x, f1 - hf.y);
                        const float2 lf = __half22float2(l);
                        bsum += (hf.x + lf.x) * zev[e] + (hf.y + lf.y) * zev[e + 1];
                        if (!PL)
                            big |= fabsf(v0) * fmaxf(fabsf(zev[e]), fabsf(QMAX - zev[e])) > 1.6f ||
                                   fabsf(v1) * fmaxf(fabsf(zev[e + 1]), fabsf(QMAX - zev[e + 1])) > 1.6f;
                        hb[e / 2] = __hmul2(h, colf);
                        lb[e / 2] = __hmul2(l, colf);
                    }
                    __half *hrow = PL ? Bs + (2 * i) * BST : Bs + i * BST, *lrow = PL ? Bs + (2 * i + 1) * BST : Bl + i * BST;
                    if constexpr (CPL == 4) {
                        *reinterpret_cast<uint2 *>(hrow + lane * CPL) = make_uint2(*reinterpret_cast<uint32_t *>(&hb[0]), *reinterpret_cast<uint32_t *>(&hb[1]));
                        *reinterpret_cast<uint2 *>(lrow + lane * CPL) = make_uint2(*reinterpret_cast<uint32_t *>(&lb[0]), *reinterpret_cast<uint32_t *>(&lb[1]));
                    } else {
                        *reinterpret_cast<__half2 *>(hrow + lane * CPL) = hb[0];
                        *reinterpret_cast<__half2 *>(lrow + lane * CPL) = lb[0];
                    }
                    bsum = warp_sum(bsum) * finv;
                    if (PL) {
                        if (i == t) { bias0 = bsum; ks0 = ksc; }
                    } else {
                        if (i == 2 * t) { bias0 = bsum; ks0 = ksc; }
                        if (i == 2 * t + 1) { bias1 = bsum; ks1 = ksc; }
                    }
                }
            }
            if (!PL) {
                const uint32_t bal = __ballot_sync(0xffffffffu, big);
                constexpr int LPM = 16 / CPL;     // lanes per 16-channel matrix
#pragma unroll
                for (int m = 0; m < NM; ++m)
                    if ((bal >> (LPM * m)) & ((1u << LPM) - 1u)) need_lo |= 1u << m;
            }
            }
            __syncwarp();
        }
        if constexpr (I8 >= 2) {
            // (I8 = 3: those of the even rows; the odd rows' are read from the table tile by tile)
            // B fragments of the four words, first operand (bk[0..3]) and second (bk[4..7]): column g, slots 4t .. 4t + 3
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    const uint32_t *e = reinterpret_cast<const uint32_t *>(Bs) + (i * 2 + c2) * 64 + g * 4 + t;
                    bk[i][c2] = e[0];
                    bk[4 + i][c2] = e[32];
                }
        } else if constexpr (I8 == 1) {
            // B fragments of the four words: column g = limb g, contraction slots 4t .. 4t + 3 (lower, upper)
#pragma unroll
            for (int m = 0; m < NM; ++m) bk[m][0] = bk[m][1] = 0u;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2)
                    bk[i][c2] = g < 4 ? *reinterpret_cast<const uint32_t *>(reinterpret_cast<const signed char *>(Bs) + (i * 2 + c2) * 64 + g * 16 + 4 * t) : 0u;
        } else {
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const bool col_used = PL ? g < 2 * nq : g < nq;
            bk[m][0] = col_used ? *(const uint32_t *)(Bs + g * BST + 16 * m + 2 * t) : 0u;
            bk[m][1] = col_used ? *(const uint32_t *)(Bs + g * BST + 16 * m + 2 * t + 8) : 0u;
        }
        }
        }
        const float ks0r = ks0 * R1, ks1r = ks1 * R1;

#pragma unroll 1
        for (int cj = 0; cj < CPG; ++cj, ++ci) {
            const int slot = ci & (NSLOT - 1);
            // refill the slot freed by the previous chunk, then wait for this chunk's bytes
            __syncwarp();
            if (iss < n_chunks) issue_chunk();
            if (!wait_bar(cbar + 8 * slot, (unsigned)(ci / NSLOT) & 1u)) { stream_ok = false; break; }
            const uint2 mwords = mword_next;
            {   // sink bits of the warp's next chunk, fetched one chunk ahead
                if (ci + 1 < n_chunks) mword_next = load_mask_words(grp * TPG + (cj + 1) * CT);   // the warp's chunks are consecutive
            }
            const uint32_t *kt0 = (const uint32_t *)(ring + slot * SLOT_BYTES), *vt0 = kt0 + KV_BYTES / 4;
            const float *ssv0 = (const float *)(vt0 + KV_BYTES / 4), *szv0 = ssv0 + SZ_BYTES / 4;
#pragma unroll
            for (int sub = 0; sub < CT / ST; ++sub) {   // softmax steps of ST tiles inside the chunk
            const uint32_t *kt = kt0 + sub * ST * TILE_WORDS, *vt = vt0 + sub * ST * TILE_WORDS;
            const float *ssv = ssv0 + sub * ST * 16 * NGv, *szv = szv0 + sub * ST * 16 * NGv;
            const int T0 = grp * TPG + cj * CT + sub * ST;
            const uint32_t mword = ST == 4 ? (mwords.x | mwords.y) : (sub == 0 ? mwords.x : mwords.y);

            // per-token keys: (scale, zero) of the chunk's tokens, token-major, delivered with the chunk
            const float *kts = ssv0 + 2 * (SZ_BYTES / 4) + sub * ST * 16 * NGv, *ktz = kts + SZ_BYTES / 4;
            // score of a token from its group dot products d[j] (already in query units): sum_j scale_j * (d_j - zero_j * qsum_j)
            auto token_score = [&](const float (&d)[NGK], int tok) {
                float r = 0.f;
#pragma unroll
                for (int j = 0; j < NGK; ++j) r = fmaf(kts[tok * NGv + j], fmaf(-ktz[tok * NGv + j], j == 0 ? bias0 : bias1, d[j]), r);
                return r;
            };
            // scores of the chunk's tiles
            float s[ST][4];
#pragma unroll
            for (int k = 0; k < ST; ++k) {
                if constexpr (I8 >= 2) {
                    uint32_t kw[W];
                    load_tile_shared<BITS, D>(kt + k * TILE_WORDS, lane, kw);
                    // upper / lower byte pair of the heads' sums; per-token keys: one set per channel group (MMA i covers
                    // channels 32 i ... 32 i + 31)
                    int ia[NGK][4], ib[NGK][4];
                    int ic[4] = {0, 0, 0, 0}, id[4] = {0, 0, 0, 0};   // I8 = 3: the same for the odd rows
#pragma unroll
                    for (int j = 0; j < NGK; ++j)
#pragma unroll
                        for (int x = 0; x < 4; ++x) ia[j][x] = ib[j][x] = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int jg = NGK == 2 ? (i >> 1) : 0;
                        uint32_t a0, a1, a2, a3;
                        if constexpr (BITS != 4) {
                            const uint32_t x = kw[i];
                            a0 = x & 0x03030303u; a1 = x & 0x0c0c0c0cu; a2 = x & 0x30303030u; a3 = x & 0xc0c0c0c0u;
                        } else {
                            const uint32_t x = kw[2 * i], y = kw[2 * i + 1];
                            a0 = x & 0x0f0f0f0fu; a1 = x & 0xf0f0f0f0u; a2 = y & 0x0f0f0f0fu; a3 = y & 0xf0f0f0f0u;
                        }
                        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                     : "+r"(ia[jg][0]), "+r"(ia[jg][1]), "+r"(ia[jg][2]), "+r"(ia[jg][3])
                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bk[i][0]), "r"(bk[i][1]));
                        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                     : "+r"(ib[jg][0]), "+r"(ib[jg][1]), "+r"(ib[jg][2]), "+r"(ib[jg][3])
                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bk[4 + i][0]), "r"(bk[4 + i][1]));
                        if constexpr (I8 == 3) {   // the odd rows' operands from the second table, the same masked words
                            const uint32_t *e0 = reinterpret_cast<const uint32_t *>(Bs) + 512 + (i * 2) * 64 + g * 4 + t;
                            const uint32_t c00 = e0[0], c01 = e0[64], c10 = e0[32], c11 = e0[96];
                            asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                         : "+r"(ic[0]), "+r"(ic[1]), "+r"(ic[2]), "+r"(ic[3])
                                         : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(c00), "r"(c01));
                            asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                         : "+r"(id[0]), "+r"(id[1]), "+r"(id[2]), "+r"(id[3])
                                         : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(c10), "r"(c11));
                        }
                    }
                    // lane t holds head t: bytes 3, 2 of its sum in the first accumulators, bytes 1, 0 in the second
                    float tg[NGK], th[NGK];
#pragma unroll
                    for (int j = 0; j < NGK; ++j) {
                        tg[j] = fmaf(fmaf((float)ia[j][0], 256.f, (float)ia[j][1]), 65536.f, fmaf((float)ib[j][0], 256.f, (float)ib[j][1]));
                        th[j] = fmaf(fmaf((float)ia[j][2], 256.f, (float)ia[j][3]), 65536.f, fmaf((float)ib[j][2], 256.f, (float)ib[j][3]));
                    }
                    if constexpr (KT) {
#pragma unroll
                        for (int j = 0; j < NGK; ++j) { tg[j] *= ks0; th[j] *= ks0 * (BITS == 4 ? 0.0625f : 0.25f); }
                        s[k][0] = token_score(tg, k * 16 + g); s[k][1] = -INFINITY;
                        s[k][2] = token_score(th, k * 16 + g + 8); s[k][3] = -INFINITY;
                    } else if constexpr (I8 == 3) {   // rows 2t (even table) and 2t + 1 (odd table): this lane's two columns
                        const float ug = fmaf(fmaf((float)ic[0], 256.f, (float)ic[1]), 65536.f, fmaf((float)id[0], 256.f, (float)id[1]));
                        const float uh = fmaf(fmaf((float)ic[2], 256.f, (float)ic[3]), 65536.f, fmaf((float)id[2], 256.f, (float)id[3]));
                        s[k][0] = fmaf(tg[0], ks0, -bias0); s[k][1] = fmaf(ug, ks1, -bias1);
                        s[k][2] = fmaf(th[0], ks0 * (BITS == 4 ? 0.0625f : 0.25f), -bias0);
                        s[k][3] = fmaf(uh, ks1 * (BITS == 4 ? 0.0625f : 0.25f), -bias1);
                    } else {
                        s[k][0] = fmaf(tg[0], ks0, -bias0); s[k][1] = -INFINITY;
                        s[k][2] = fmaf(th[0], ks0 * (BITS == 4 ? 0.0625f : 0.25f), -bias0); s[k][3] = -INFINITY;
                    }
                    continue;
                }
                if constexpr (I8 == 1) {
                    uint32_t kw[W];
                    load_tile_shared<BITS, D>(kt + k * TILE_WORDS, lane, kw);
                    int iag[NGK][4];                                    // per-token keys: one set per channel group
#pragma unroll
                    for (int j = 0; j < NGK; ++j)
#pragma unroll
                        for (int x = 0; x < 4; ++x) iag[j][x] = 0;
                    int ih0[4] = {0, 0, 0, 0}, ih1[4] = {0, 0, 0, 0};   // 3 bit: the high bits of the even / odd words
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int (&ia)[4] = iag[NGK == 2 ? (i >> 1) : 0];
                        uint32_t a0, a1, a2, a3;
                        if constexpr (BITS == 3) {
                            // the second section has the byte structure of the first: the high bits of word i sit at bits
                            // 2, 3, 6, 7 (even i) or 0, 1, 4, 5 (odd i) of the bytes of word 4 + i / 2
                            const uint32_t hw = kw[4 + (i >> 1)];
                            if ((i & 1) == 0) {
                                asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                             : "+r"(ih0[0]), "+r"(ih0[1]), "+r"(ih0[2]), "+r"(ih0[3])
                                             : "r"(hw & 0x04040404u), "r"(hw & 0x08080808u), "r"(hw & 0x40404040u), "r"(hw & 0x80808080u), "r"(bk[i][0]), "r"(bk[i][1]));
                            } else {
                                asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                             : "+r"(ih1[0]), "+r"(ih1[1]), "+r"(ih1[2]), "+r"(ih1[3])
                                             : "r"(hw & 0x01010101u), "r"(hw & 0x02020202u), "r"(hw & 0x10101010u), "r"(hw & 0x20202020u), "r"(bk[i][0]), "r"(bk[i][1]));
                            }
                        }
                        if constexpr (BITS != 4) {
                            const uint32_t x = kw[i];
                            a0 = x & 0x03030303u; a1 = x & 0x0c0c0c0cu; a2 = x & 0x30303030u; a3 = x & 0xc0c0c0c0u;
                        } else {
                            const uint32_t x = kw[2 * i], y = kw[2 * i + 1];
                            a0 = x & 0x0f0f0f0fu; a1 = x & 0xf0f0f0f0u; a2 = y & 0x0f0f0f0fu; a3 = y & 0xf0f0f0f0u;
                        }
                        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                     : "+r"(ia[0]), "+r"(ia[1]), "+r"(ia[2]), "+r"(ia[3])
                                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bk[i][0]), "r"(bk[i][1]));
                    }
                    if constexpr (BITS == 3) {
                        // code = low + 4 * high; in place the high bits weigh 4, 8 (rows g, g + 8) in even words and 1, 2 in
                        // odd ones, the low fields 1, 4: rows g in units of 1, rows g + 8 in units of 4
                        int (&ia)[4] = iag[0];
                        ia[0] += ih0[0] + 4 * ih1[0]; ia[1] += ih0[1] + 4 * ih1[1];
                        ia[2] += 2 * ih0[2] + 8 * ih1[2]; ia[3] += 2 * ih0[3] + 8 * ih1[3];
                    }
                    // lane t = 0 holds limbs 0, 1 (columns 0, 1), its neighbour limbs 2, 3 (columns 2, 3): each lane combines
                    // its pair (every column sum is below 2^24, exact in binary32), then the pairs combine
                    float tg[NGK], th[NGK];
#pragma unroll
                    for (int j = 0; j < NGK; ++j) {
                        const float xg = fmaf((float)iag[j][0], 256.f, (float)iag[j][1]), xh = fmaf((float)iag[j][2], 256.f, (float)iag[j][3]);
                        const float yg = __shfl_down_sync(0xffffffffu, xg, 1), yh = __shfl_down_sync(0xffffffffu, xh, 1);
                        tg[j] = fmaf(xg, 65536.f, yg);
                        th[j] = fmaf(xh, 65536.f, yh);
                    }
                    // lanes t != 0 hold no head: their factor and bias are zero, their columns are never read
                    if constexpr (KT) {
#pragma unroll
                        for (int j = 0; j < NGK; ++j) { tg[j] *= ks0; th[j] *= ks0 * (BITS == 4 ? 0.0625f : 0.25f); }
                        s[k][0] = token_score(tg, k * 16 + g); s[k][1] = -INFINITY;
                        s[k][2] = token_score(th, k * 16 + g + 8); s[k][3] = -INFINITY;
                    } else {
                        s[k][0] = fmaf(tg[0], ks0, -bias0); s[k][1] = -INFINITY;
                        s[k][2] = fmaf(th[0], ks0 * (BITS == 4 ? 0.0625f : 0.25f), -bias0); s[k][3] = -INFINITY;
                    }
                    continue;
                }
                uint32_t kw[W], ka[NM][4];
                load_tile_shared<BITS, D>(kt + k * TILE_WORDS, lane, kw);
                tile_frags<BITS, D>(kw, ka);
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                if (PL || need_lo == 0) {
#pragma unroll
                    for (int m = 0; m < NM; ++m) mma16816(acc, ka[m], bk[m][0], bk[m][1]);
                } else {
#pragma unroll
                    for (int m = 0; m < NM; ++m) {
                        mma16816(acc, ka[m], bk[m][0], bk[m][1]);
                        if (need_lo & (1u << m)) {
                            const uint32_t h0 = g < nq ? *(const uint32_t *)(Bl + g * BST + 16 * m + 2 * t) : 0u;
                            const uint32_t h1 = g < nq ? *(const uint32_t *)(Bl + g * BST + 16 * m + 2 * t + 8) : 0u;
                            mma16816(acc, ka[m], h0, h1);
                        }
                    }
                }
                if (PL) {   // column 2t: rounded factors, column 2t+1: their residuals
                    s[k][0] = fmaf(acc[0] + acc[1], ks0, -bias0); s[k][1] = -INFINITY;
                    s[k][2] = fmaf(acc[2] + acc[3], ks0r, -bias0); s[k][3] = -INFINITY;
                } else {
                    s[k][0] = fmaf(acc[0], ks0, -bias0); s[k][1] = fmaf(acc[1], ks1, -bias1);
                    s[k][2] = fmaf(acc[2], ks0r, -bias0); s[k][3] = fmaf(acc[3], ks1r, -bias1);
                }
            }
            if (mword) {   // sink tokens are not part of the packed stream (their value parameters are zero)
#pragma unroll
                for (int k = 0; k < ST; ++k) {
                    // a chunk of an even number of tiles starts on an even tile: the half of the word is known at compile time
                    const int half = (CT % 2 == 0) ? (k & 1) : ((T0 + k) & 1);
                    const uint32_t mask16 = ((ST == 4 ? (k < 2 ? mwords.x : mwords.y) : mword) >> (16 * half)) & 0xffffu;
                    if ((mask16 >> g) & 1u) s[k][0] = s[k][1] = -INFINITY;
                    if ((mask16 >> (g + 8)) & 1u) s[k][2] = s[k][3] = -INFINITY;
                }
            }
            if constexpr (PRE) {
                if ((T0 + ST) * KVSINK_TILE > lim_min) {   // tiles that reach beyond the earliest query of the block
#pragma unroll
                    for (int k = 0; k < ST; ++k) {
                        const int tok = (T0 + k) * KVSINK_TILE + g;
                        if (tok >= lim0) s[k][0] = -INFINITY;
                        if (tok >= lim1) s[k][1] = -INFINITY;
                        if (tok + 8 >= lim0) s[k][2] = -INFINITY;
                        if (tok + 8 >= lim1) s[k][3] = -INFINITY;
                    }
                }
            }
            if constexpr (FLAT) {
                if ((T0 + ST) * KVSINK_TILE > n) {   // the last tiles reach beyond the sequence: those tokens do not exist
#pragma unroll
                    for (int k = 0; k < ST; ++k) {
                        const int tok = (T0 + k) * KVSINK_TILE + g;
                        if (tok >= n) s[k][0] = s[k][1] = -INFINITY;
                        if (tok + 8 >= n) s[k][2] = s[k][3] = -INFINITY;
                    }
                }
            }
            // one softmax step for the whole chunk
            {
                float tm0 = fmaxf(s[0][0], s[0][2]), tm1 = fmaxf(s[0][1], s[0][3]);
#pragma unroll
                for (int k = 1; k < ST; ++k) { tm0 = fmaxf(tm0, fmaxf(s[k][0], s[k][2])); tm1 = fmaxf(tm1, fmaxf(s[k][1], s[k][3])); }
                advance_max(tm0, tm1);
            }
            // value scales of this lane's tokens; their maximum bounds the fp16 range needed
            float sv0[ST][NGv], zv0[ST][NGv], sv1[ST][NGv], zv1[ST][NGv];
            if constexpr (CAL) {
#pragma unroll
                for (int k = 0; k < ST; ++k)
#pragma unroll
                    for (int j = 0; j < NGv; ++j) { sv0[k][j] = sv1[k][j] = cal_sv[j]; zv0[k][j] = zv1[k][j] = cal_zv[j]; }
            } else {
                float mx = 0.f;
#pragma unroll
                for (int k = 0; k < ST; ++k)
#pragma unroll
                    for (int j = 0; j < NGv; ++j) {
                        sv0[k][j] = ssv[(k * 16 + g) * NGv + j]; zv0[k][j] = szv[(k * 16 + g) * NGv + j];
                        sv1[k][j] = ssv[(k * 16 + g + 8) * NGv + j]; zv1[k][j] = szv[(k * 16 + g + 8) * NGv + j];
                        if constexpr (KT) {   // tokens beyond the sequence: whatever the arrays hold there must not reach the sums
                            if ((T0 + k) * KVSINK_TILE + g >= n) sv0[k][j] = zv0[k][j] = 0.f;
                            if ((T0 + k) * KVSINK_TILE + g + 8 >= n) sv1[k][j] = zv1[k][j] = 0.f;
                        }
                        mx = fmaxf(mx, fmaxf(fabsf(sv0[k][j]), fabsf(sv1[k][j])));
                    }
                fit_value_scale(mx);
            }
#pragma unroll
            for (int k = 0; k < ST; ++k) {
                uint32_t vw[W];
                load_tile_shared<BITS, D>(vt + k * TILE_WORDS, lane, vw);
                tile_values(s[k], vw, sv0[k], zv0[k], sv1[k], zv1[k]);
            }
            }
        }
    }
    if (!stream_ok && lane == 0) atomicOr(c.status, KVSINK_STATUS_TIMEOUT);

    // ---- this warp's packed partial: finish the reductions over the token lanes, convert units ----
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
#pragma unroll
        for (int j = 0; j < NGv; ++j) {
            bv[j][0] += __shfl_xor_sync(0xffffffffu, bv[j][0], o);
            bv[j][1] += __shfl_xor_sync(0xffffffffu, bv[j][1], o);
        }
    }
    __syncthreads();   // every warp has drained its ring: the space now holds the block's partials
    float *my_part = part + (size_t)(2 * warp) * nq * PS;
    {
        const float OS0 = pow2i(24 - ev), OS1 = OS0 * R1;
#pragma unroll
        for (int m = 0; m < NM; ++m) {
            const float bj0 = bv[m / mpg][0], bj1 = bv[m / mpg][1];
            const int ch0 = 16 * m + g, ch1 = ch0 + 8;
            if (PL) {
                if (t < nq) {
                    my_part[t * PS + ch0] = (O[m][0] + O[m][1]) * OS0 - bj0;
                    my_part[t * PS + ch1] = (O[m][2] + O[m][3]) * OS1 - bj0;
                }
                continue;
            }
            if (2 * t < nq) {
                my_part[(2 * t) * PS + ch0] = O[m][0] * OS0 - bj0;
                my_part[(2 * t) * PS + ch1] = O[m][2] * OS1 - bj0;
            }
            if (2 * t + 1 < nq) {
                my_part[(2 * t + 1) * PS + ch0] = O[m][1] * OS0 - bj1;
                my_part[(2 * t + 1) * PS + ch1] = O[m][3] * OS1 - bj1;
            }
        }
        if (g == 0 && PL) {
            if (t < nq) { my_part[t * PS + D] = m0; my_part[t * PS + D + 1] = l0; }
        } else if (g == 0) {
            if (2 * t < nq) { my_part[(2 * t) * PS + D] = m0; my_part[(2 * t) * PS + D + 1] = l0; }
            if (2 * t + 1 < nq) { my_part[(2 * t + 1) * PS + D] = m1; my_part[(2 * t + 1) * PS + D + 1] = l1; }
        }
    }

    // ---------------- sink rows (fp16 side buffer), plain fp32 arithmetic ----------------
    {
        float ms[NQMAX], ls[NQMAX], os[NQMAX][CPL];
#pragma unroll
        for (int i = 0; i < NQMAX; ++i) {
            ms[i] = M_INIT; ls[i] = 0.f;
#pragma unroll
            for (int e = 0; e < CPL; ++e) os[i][e] = 0.f;
        }
        for (int j = sink_worker; j < sink_n; j += sink_workers) {
            const int pos = sink_pos_next;
            float kf[CPL], vf[CPL];
#pragma unroll
            for (int e = 0; e < CPL / 2; ++e) {
                const float2 k2 = __half22float2(*reinterpret_cast<const __half2 *>(&sink_k_next[e]));
                const float2 v2 = __half22float2(*reinterpret_cast<const __half2 *>(&sink_v_next[e]));
                kf[2 * e] = k2.x; kf[2 * e + 1] = k2.y; vf[2 * e] = v2.x; vf[2 * e + 1] = v2.y;
            }
            fetch_sink(j + sink_workers);   // the next row streams in while this one is used
            if (pos < 0 || pos >= n) continue;
#pragma unroll
            for (int i = 0; i < NQMAX; ++i) {
                if (i < nq && (!PRE || pos < row_limit(i))) {
                    float d = 0.f;
#pragma unroll
                    for (int e = 0; e < CPL; ++e) d += qs[i * D + lane * CPL + e] * kf[e];
                    const float sc = warp_sum(d);
                    const float mnew = fmaxf(ms[i], sc);
                    const float corr = ex2(ms[i] - mnew), pp = ex2(sc - mnew);
                    ls[i] = ls[i] * corr + pp;
#pragma unroll
                    for (int e = 0; e < CPL; ++e) os[i][e] = os[i][e] * corr + pp * vf[e];
                    ms[i] = mnew;
                }
            }
        }
        float *sp = my_part + (size_t)nq * PS;
#pragma unroll
        for (int i = 0; i < NQMAX; ++i) {
            if (i < nq) {
#pragma unroll
                for (int e = 0; e < CPL; ++e) sp[i * PS + lane * CPL + e] = os[i][e];
                if (lane == 0) { sp[i * PS + D] = ms[i]; sp[i * PS + D + 1] = ls[i]; }
            }
        }
    }
    __syncthreads();

    // ---- merge the block's partials; write the result or this split's partial ----
    for (int idx = tid; idx < nq * D; idx += DEC_THREADS) {
        const int qh = idx / D, ch = idx % D;
        float M = M_INIT;
        for (int w = 0; w < 2 * DEC_WARPS; ++w) M = fmaxf(M, part[((size_t)w * nq + qh) * PS + D]);
        float acc = 0.f, L = 0.f;
        for (int w = 0; w < 2 * DEC_WARPS; ++w) {
            const float *pr = part + ((size_t)w * nq + qh) * PS;
            const float f = ex2(pr[D] - M);
            acc += pr[ch] * f;
            L += pr[D + 1] * f;
        }
        const size_t oq = PRE ? ((size_t)b * p.Hq + hq0 + (8 * qc + qh) % p.rep) * pre.T + row_token(qh) : (size_t)b * p.Hq + hq0 + qh;
        if (nsplit == 1) {
            out[oq * D + ch] = L > 0.f ? acc / L : 0.f;
            if (lse && ch == 0) lse[oq] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
        } else {
            // the split's record: to the workspace for the merge kernel, or, when the splits of a unit form a thread-block
            // cluster, to this block's shared memory (the query tables are no longer needed) for the cluster's first block
            float *wsr = cluster_merge ? qs + (size_t)qh * PS : part_ws + (oq * nsplit + split) * PS;
            wsr[ch] = acc;
            if (ch == 0) { wsr[D] = M; wsr[D + 1] = L; }
        }
    }
    if (cluster_merge) {
        // the splits of a unit are the blocks of one cluster: its first block reads the records of the others through
        // distributed shared memory and merges them in split order (the same arithmetic as the merge kernel)
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        if (split == 0) {
            for (int idx = tid; idx < nq * D; idx += DEC_THREADS) {
                const int qh = idx / D, ch = idx % D;
                float M = M_INIT;
                for (int sp = 0; sp < nsplit; ++sp) M = fmaxf(M, cluster.map_shared_rank(qs, sp)[(size_t)qh * PS + D]);
                float acc = 0.f, L = 0.f;
                for (int sp = 0; sp < nsplit; ++sp) {
                    const float *pr = cluster.map_shared_rank(qs, sp) + (size_t)qh * PS;
                    const float f = ex2(pr[D] - M);
                    acc += pr[ch] * f;
                    L += pr[D + 1] * f;
                }
                const size_t oq = (size_t)b * p.Hq + hq0 + qh;
                out[oq * D + ch] = L > 0.f ? acc / L : 0.f;
                if (lse && ch == 0) lse[oq] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
            }
        }
        cluster.sync();   // nobody's shared memory goes away while the first block reads it
    }
}

// ---- launch: one instantiation per (bits, head size, value groups per row, chunk size, key-side variant) ----
template <int BITS, int D, int NGV, int CT, bool PL, int I8 = 0, int PM = 0>
static int launch_decode_p(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                           cudaStream_t st)
{
    // the units the sequence is split in: key groups, or ring chunks when the parameters are static
    const int n_groups = PM != 0 ? (c.seq_len + CT * KVSINK_TILE - 1) / (CT * KVSINK_TILE) : c.seq_len / p.G;
    const kvsink_static_params sp = PM == 1 ? *cal : kvsink_static_params{nullptr, nullptr, nullptr, nullptr};
    const int nsplit = choose_splits(p, n_groups);
    const int gps = n_groups > 0 ? (n_groups + nsplit - 1) / nsplit : 0;
    const int qchunks = decode_qchunks(p);      // blocks per KV head; each serves up to NQMAX query heads
    if (qchunks * (I8 == 1 ? 1 : (PL ? 4 : 8)) < p.rep) return KVSINK_ERR_UNSUPPORTED;
    const size_t smem = DecodePlan<BITS, D, NGV, CT, I8 == 1 ? 1 : (PL ? 4 : 8), PM == 2>::BYTES;
    auto kern = decode_kernel<BITS, D, NGV, CT, PL, I8, PM>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    cudaLaunchAttribute pdl[2];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    // up to eight splits (the portable cluster size): the splits of a unit are launched as one thread-block cluster and
    // merged inside the kernel through distributed shared memory; more splits go through the workspace and the merge kernel
    bool cluster_merge = nsplit > 1 && nsplit <= 8;
    for (;;) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(nsplit, p.Hkv * qchunks, p.B);
        cfg.blockDim = dim3(DEC_THREADS);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cfg.attrs = pdl;
        cfg.numAttrs = 1;
        if (cluster_merge) {
            pdl[1].id = cudaLaunchAttributeClusterDimension;
            pdl[1].val.clusterDim.x = nsplit;
            pdl[1].val.clusterDim.y = 1;
            pdl[1].val.clusterDim.z = 1;
            cfg.numAttrs = 2;
        }
        if (cudaLaunchKernelEx(&cfg, kern, p, c, sp, q, out, lse, ws, nsplit, gps, qchunks, (int)c.seq_len, (int)cluster_merge, PrefillShape{0, 0, 0, 0, 0}) == cudaSuccess) {
            note_launch();
            break;
        }
        (void)cudaGetLastError();
        if (!cluster_merge) return KVSINK_ERR_CUDA;
        cluster_merge = false;   // a cluster that cannot be placed: the same launch without one, merged by the second kernel
    }
    if (nsplit > 1 && !cluster_merge) return launch_decode_merge(ws, nsplit, D, p.B * p.Hq, out, lse, st);
    return KVSINK_OK;
}

// Prompt queries (the eight-column fp16 path): one block per eight (query token, query head) rows of a KV head.
template <int BITS, int D, int NGV, int CT>
static int launch_prefill_p(const Params &p, const kvsink_cache &c, const __half *q, const PrefillShape &pre, float *out, float *lse, cudaStream_t st)
{
    const size_t smem = DecodePlan<BITS, D, NGV, CT, 8>::BYTES;
    auto kern = decode_kernel<BITS, D, NGV, CT, false, (D == 128 && BITS != 3) ? 3 : 0, 0, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVSINK_ERR_CUDA;
    const long long blocks = ((long long)pre.T * p.rep + 7) / 8;
    if (blocks > 0x7fffffffLL) return KVSINK_ERR_UNSUPPORTED;
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, p.Hkv, p.B);
    cfg.blockDim = dim3(DEC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    const kvsink_static_params none = {nullptr, nullptr, nullptr, nullptr};
    if (cudaLaunchKernelEx(&cfg, kern, p, c, none, q, out, lse, (float *)nullptr, 1, 0, (int)blocks, (int)c.seq_len, 0, pre) != cudaSuccess)
        return KVSINK_ERR_CUDA;
    note_launch();
    return KVSINK_OK;
}

template <int BITS, int D, int NGV>
static int launch_prefill_n(const Params &p, const kvsink_cache &c, const __half *q, const PrefillShape &pre, float *out, float *lse, cudaStream_t st)
{
    // several channel groups per row mean G = D / NGV tokens per group: only chunk sizes that divide such a group are built;
    // four groups per row take one tile per chunk (their parameter registers would spill otherwise)
    constexpr int TPG_MAX = NGV == 1 ? 4 : D / NGV / KVSINK_TILE;
    if constexpr (TPG_MAX % 4 == 0 && 4 * (2 * 128 * (D * BITS / 64) + 2 * 16 * NGV * 4) <= 4800)
        if ((p.G / KVSINK_TILE) % 4 == 0) return launch_prefill_p<BITS, D, NGV, 4>(p, c, q, pre, out, lse, st);
    if constexpr (TPG_MAX % 2 == 0 && NGV < 4)
        if ((p.G / KVSINK_TILE) % 2 == 0) return launch_prefill_p<BITS, D, NGV, 2>(p, c, q, pre, out, lse, st);
    return launch_prefill_p<BITS, D, NGV, 1>(p, c, q, pre, out, lse, st);
}

template <int BITS, int D>
static int launch_prefill_t(const Params &p, const kvsink_cache &c, const __half *q, const PrefillShape &pre, float *out, float *lse, cudaStream_t st)
{
    if (p.NGv == 1) return launch_prefill_n<BITS, D, 1>(p, c, q, pre, out, lse, st);
    if (p.NGv == 2) return launch_prefill_n<BITS, D, 2>(p, c, q, pre, out, lse, st);
    if (p.NGv == 4) return launch_prefill_n<BITS, D, 4>(p, c, q, pre, out, lse, st);
    return KVSINK_ERR_UNSUPPORTED;
}

template <int BITS>
static int launch_prefill_bits(const Params &p, const kvsink_cache &c, const __half *q, int T, int q_pos0, int64_t sb, int64_t sh, int64_t stt,
                               float *out, float *lse, cudaStream_t st)
{
    const PrefillShape pre = {T, q_pos0, sb, sh, stt};
    if (p.D == 128) return launch_prefill_t<BITS, 128>(p, c, q, pre, out, lse, st);
    if constexpr (BITS != 3)
        if (p.D == 64) return launch_prefill_t<BITS, 64>(p, c, q, pre, out, lse, st);
    return KVSINK_ERR_UNSUPPORTED;
}

template <int BITS, int D, int NGV, int CT, int PM>
static int launch_decode_c(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                           cudaStream_t st)
{
    // key side by head size, code width and query heads per KV head; only the reachable kernels are built
    if constexpr (D == 128)
        if (p.rep == 1) return launch_decode_p<BITS, D, NGV, CT, true, 1, PM>(p, c, cal, q, out, lse, ws, st);
    if constexpr (D == 128 && BITS != 3) {
        if (p.rep <= 4) return launch_decode_p<BITS, D, NGV, CT, true, 2, PM>(p, c, cal, q, out, lse, ws, st);
        if constexpr (PM != 2) return launch_decode_p<BITS, D, NGV, CT, false, 3, PM>(p, c, cal, q, out, lse, ws, st);
        else return KVSINK_ERR_UNSUPPORTED;      // per-token keys: at most four query heads per KV head
    } else if constexpr (PM == 2) {
        return KVSINK_ERR_UNSUPPORTED;           // per-token keys run on the integer key side only
    } else if constexpr (D == 128) {
        return launch_decode_p<BITS, D, NGV, CT, true, 0, PM>(p, c, cal, q, out, lse, ws, st);   // 3 bit: pair layout, four heads at a time
    } else {
        if (p.rep <= 4) return launch_decode_p<BITS, D, NGV, CT, true, 0, PM>(p, c, cal, q, out, lse, ws, st);
        return launch_decode_p<BITS, D, NGV, CT, false, 0, PM>(p, c, cal, q, out, lse, ws, st);
    }
}

template <int BITS, int D, int NGV, int PM>
static int launch_decode_n(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                           cudaStream_t st)
{
    // ring chunks of four tiles where a key group divides into them and two slots of that size stay below ~9 KB per
    // warp, else of two tiles (G a multiple of 32), else of one
    // several channel groups per row mean G = D / NGV tokens per group: only chunk sizes that divide such a group are built;
    // four groups per row take one tile per chunk (their parameter registers would spill otherwise)
    constexpr int TPG_MAX = NGV == 1 ? 4 : D / NGV / KVSINK_TILE;
    if constexpr (TPG_MAX % 4 == 0 && 4 * (2 * 128 * (D * BITS / 64) + (PM == 2 ? 4 : 2) * 16 * NGV * 4) <= (PM == 2 ? 5200 : 4800))
        if ((p.G / KVSINK_TILE) % 4 == 0) return launch_decode_c<BITS, D, NGV, 4, PM>(p, c, cal, q, out, lse, ws, st);
    if constexpr (TPG_MAX % 2 == 0 && NGV < 4)
        if ((p.G / KVSINK_TILE) % 2 == 0) return launch_decode_c<BITS, D, NGV, 2, PM>(p, c, cal, q, out, lse, ws, st);
    return launch_decode_c<BITS, D, NGV, 1, PM>(p, c, cal, q, out, lse, ws, st);
}

template <int BITS, int D, int PM>
static int launch_decode_t(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                           cudaStream_t st)
{
    if (p.NGv == 1) return launch_decode_n<BITS, D, 1, PM>(p, c, cal, q, out, lse, ws, st);
    if constexpr (PM != 2 || BITS != 3)
        if (p.NGv == 2) return launch_decode_n<BITS, D, 2, PM>(p, c, cal, q, out, lse, ws, st);
    if constexpr (PM == 0)
        if (p.NGv == 4) return launch_decode_n<BITS, D, 4, PM>(p, c, cal, q, out, lse, ws, st);
    return KVSINK_ERR_UNSUPPORTED;
}

// Dispatch over head size for one code width; each width is compiled in a translation unit of its own.  mode 0: dynamic
// per-channel key parameters (`cal` null); 1: static parameters `cal`; 2: per-token key parameters.  Modes 1 and 2 are
// built for head size 128 with one or two channel groups per row; mode 2 for at most four query heads per KV head
// (3 bit: one, with one channel group).
template <int BITS>
static int launch_decode_bits(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out,
                              float *lse, float *ws, cudaStream_t st)
{
    if (mode == 2) return p.D == 128 ? launch_decode_t<BITS, 128, 2>(p, c, cal, q, out, lse, ws, st) : KVSINK_ERR_UNSUPPORTED;
    if (mode == 1) return p.D == 128 && cal ? launch_decode_t<BITS, 128, 1>(p, c, cal, q, out, lse, ws, st) : KVSINK_ERR_UNSUPPORTED;
    if (p.D == 128) return launch_decode_t<BITS, 128, 0>(p, c, cal, q, out, lse, ws, st);
    if constexpr (BITS != 3)
        if (p.D == 64) return launch_decode_t<BITS, 64, 0>(p, c, cal, q, out, lse, ws, st);
    return KVSINK_ERR_UNSUPPORTED;
}

}  // namespace kvsink
