/*
 * KVSink reference oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, sequential CPU restatement of the KVSink hot path (sink-token prediction,
 * asymmetric group quantization with sink exclusion, packed KV cache with an fp16 side buffer,
 * single-token decode attention).  It exists so that the CUDA library can be checked against
 * something obviously correct.  It shares no code with the CUDA path, is never linked into the
 * product, and must only be called from tests, the smoke check and the CPU-baseline leg of the
 * benchmark.
 *
 * Every function cites the passage of the paper (arXiv 2508.04257) it follows:
 *   Eq. 3        softmax attention                         (Section 2)
 *   Eq. 6        KV-cache append                           (Section 2)
 *   Eq. 7        attention split into sink / non-sink sums (Section 4.2)
 *   Eq. 8-11     asymmetric n-bit integer quantization     (Appendix C)
 *   Algorithm 1  prefill with KVSink (sink exclusion, top-k sink prediction) (Appendix G)
 *   Section 4.3  items (1)-(4): top-k on a pre-identified outlier channel, once, at prefill
 *   Section 4.1  Table 1: quantization error with / without sink tokens; static calibration without them
 *   Section 5.1, Appendix C  static per-channel-key / per-token-value parameters
 *   Appendix D   outlier channels (the per-channel magnitude scan)
 *
 * Pins (see tests/test_oracle_*.py): Table 4 memory columns (closed form), |x - x'| <= scale/2,
 * exact rational re-derivation of codes, bit-exact round trip of sink / first-N rows, planted
 * outliers, brute-force sort for top-k, textbook fp64 softmax attention on the dequantised
 * tensors, Eq. 7 log-sum-exp merge identity, and the published m16n8k16 A-fragment ownership
 * table for the physical code order.  The routines at the end of the file (channel scan, error
 * split of Table 1, static calibration / quantization / attention, prompt attention) are pinned by
 * tests/test_oracle_analysis.py, test_oracle_static.py and test_oracle_prefill.py: numpy's own
 * reductions, a group worked by hand, exact rationals with the clamp, the pinned group routine on
 * numpy's extremes, textbook (causal) attention in numpy, reduction to the pinned decode attention.
 *
 * Parity unpinned: none of the arithmetic.  The physical order of codes inside a 16-token tile is a
 * design choice the paper does not fix; it is pinned only against the published tensor-core
 * fragment table and by pack/unpack identity.
 *
 * Floating point: quantization parameters and codes follow Eq. 8-11 in IEEE binary32 with
 * round-to-nearest-even and no fused multiply-add (build with -ffp-contract=off); attention is
 * evaluated in binary64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define KVO_OK 0
#define KVO_ERR_BAD_ARG (-1)
#define KVO_ERR_BAD_CONFIG (-2)
#define KVO_ERR_SEQ_OVERFLOW (-5)

#define KVO_TILE 16

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, hidden;
    int32_t bits, group, max_seq, topk, pfn_n;
    int32_t n_channels;
    int32_t channels[8];
} kvo_config;

typedef struct {
    uint8_t *k_codes, *v_codes;
    float *k_scale, *k_zero, *v_scale, *v_zero;
    uint16_t *k_tail;
    uint16_t *sink_k, *sink_v;
    uint32_t *sink_bitmask;
    int32_t *sink_pos, *sink_count;
    int32_t seq_len;
} kvo_cache;

typedef struct {
    int64_t k_codes_bytes, v_codes_bytes;    /* per cache (one layer) */
    int64_t k_param_floats, v_param_floats;  /* floats in EACH of scale and zero */
    int64_t k_tail_halfs, sink_halfs;        /* fp16 elements; sink_halfs is for EACH of sink_k, sink_v */
    int64_t bitmask_words, sink_pos_ints;
    int32_t sink_capacity, v_group, v_groups_per_row, tile_bytes;
} kvo_sizes;

/* Threads the independent-unit loops run on (1 when built without OpenMP). */
int kvo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
void kvo_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---------- binary16 <-> binary32 (exact widening) ---------- */
static float half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) << 31;
    uint32_t ex = (h >> 10) & 0x1f;
    uint32_t man = h & 0x3ff;
    uint32_t bits;
    if (ex == 0) {
        if (man == 0) {
            bits = sign;
        } else { /* subnormal: man * 2^-24 */
            float f = (float)man * 5.9604644775390625e-08f;
            memcpy(&bits, &f, 4);
            bits |= sign;
        }
    } else if (ex == 31) {
        bits = sign | 0x7f800000u | (man << 13);
    } else {
        bits = sign | ((ex + 112) << 23) | (man << 13);
    }
    float out;
    memcpy(&out, &bits, 4);
    return out;
}

/* ---------- sizes: Table 4 memory columns are codes_bytes and sink row bytes ---------- */
static int check_config(const kvo_config *c)
{
    if (!c) return KVO_ERR_BAD_ARG;
    if (c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return KVO_ERR_BAD_CONFIG;
    if (c->n_q_heads % c->n_kv_heads) return KVO_ERR_BAD_CONFIG;
    if (c->head_dim < 16 || c->head_dim % 16) return KVO_ERR_BAD_CONFIG;
    if (c->bits < 2 || c->bits > 4) return KVO_ERR_BAD_CONFIG;
    if (c->bits == 3 && c->head_dim % 64) return KVO_ERR_BAD_CONFIG;
    if (c->group < 16 || c->group % 16) return KVO_ERR_BAD_CONFIG;
    if (c->max_seq < c->group || c->max_seq % c->group) return KVO_ERR_BAD_CONFIG;
    if (c->topk < 0 || c->pfn_n < 0) return KVO_ERR_BAD_CONFIG;
    if (c->n_channels < 0 || c->n_channels > 8) return KVO_ERR_BAD_CONFIG;
    int gv = c->group < c->head_dim ? c->group : c->head_dim;
    if (c->head_dim % gv) return KVO_ERR_BAD_CONFIG;
    return KVO_OK;
}

static int v_group_of(const kvo_config *c) { return c->group < c->head_dim ? c->group : c->head_dim; }
static int sink_cap_of(const kvo_config *c) { return c->topk + c->pfn_n; }

int kvo_cache_sizes(const kvo_config *c, kvo_sizes *s)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!s) return KVO_ERR_BAD_ARG;
    int64_t units = (int64_t)c->batch * c->n_kv_heads;
    int gv = v_group_of(c);
    s->v_group = gv;
    s->v_groups_per_row = c->head_dim / gv;
    s->tile_bytes = KVO_TILE * c->head_dim * c->bits / 8;
    s->k_codes_bytes = units * c->max_seq * c->head_dim * c->bits / 8;
    s->v_codes_bytes = s->k_codes_bytes;
    s->k_param_floats = units * (c->max_seq / c->group) * c->head_dim;
    s->v_param_floats = units * c->max_seq * s->v_groups_per_row;
    s->k_tail_halfs = units * c->group * c->head_dim;
    s->sink_capacity = sink_cap_of(c);
    s->sink_halfs = units * s->sink_capacity * c->head_dim;
    s->bitmask_words = (int64_t)c->batch * ((c->max_seq + 31) / 32);
    s->sink_pos_ints = (int64_t)c->batch * s->sink_capacity;
    return KVO_OK;
}

/* ---------- physical order of codes inside a 16-token tile ----------
 * A tile of K is a stack of head_dim/16 matrices [16 tokens x 16 channels]; a tile of V is a stack
 * of head_dim/16 matrices [16 channels x 16 tokens].  Matrix element (row, col) of matrix m belongs
 * to "lane" 4*(row%8) + (col%8)/2, pair slot r = row/8 + 2*(col/8), half e = col%2 -- the
 * ownership table of the 16x16 A operand of the m16n8k16 tensor-core instruction.  Lane words are
 * little-endian 32-bit; slot s = 4*m + r.
 *   2 bit: word s/8, field k = s%8 at bit 16e + 2k.
 *   4 bit: word s/4, field k = s%4 at bit 16e + 4k.
 *   3 bit: the low two bits as in 2 bit ("lo" section); the high bit in a "hi" section with one
 *          word per two lo words: hi word (s/8)/2, bit 16e + 4*(k/2) + 2*(1 - (s/8)%2) + k%2.
 * A section of n words per lane is stored as planes of up to four words per lane: plane p holds
 * words [4p, min(4p+4, n)); a plane of width u puts lane l's words at word offset u*l.
 */
static int section_word_offset(int n_words, int lane, int i)
{
    int off = 0, p = i / 4;
    for (int pp = 0; pp < p; ++pp) {
        int u = n_words - 4 * pp;
        if (u > 4) u = 4;
        off += 32 * u;
    }
    int u = n_words - 4 * p;
    if (u > 4) u = 4;
    return off + u * lane + (i - 4 * p);
}

/* Writes / reads the b-bit code of matrix element (m,row,col) in a tile of `tile_words`. */
static void tile_put(uint32_t *tile, int D, int bits, int m, int row, int col, uint32_t code)
{
    int lane = 4 * (row % 8) + (col % 8) / 2;
    int r = row / 8 + 2 * (col / 8);
    int e = col % 2;
    int s = 4 * m + r;
    if (bits == 2) {
        int n = D / 32, i = s / 8, k = s % 8;
        uint32_t *w = &tile[section_word_offset(n, lane, i)];
        int sh = 16 * e + 2 * k;
        *w = (*w & ~(3u << sh)) | ((code & 3u) << sh);
    } else if (bits == 4) {
        int n = D / 16, i = s / 4, k = s % 4;
        uint32_t *w = &tile[section_word_offset(n, lane, i)];
        int sh = 16 * e + 4 * k;
        *w = (*w & ~(15u << sh)) | ((code & 15u) << sh);
    } else {
        int nlo = D / 32, nhi = D / 64, i = s / 8, k = s % 8;
        uint32_t *w = &tile[section_word_offset(nlo, lane, i)];
        int sh = 16 * e + 2 * k;
        *w = (*w & ~(3u << sh)) | ((code & 3u) << sh);
        uint32_t *h = &tile[32 * nlo + section_word_offset(nhi, lane, i / 2)];
        int hb = 16 * e + 4 * (k / 2) + 2 * (1 - (i % 2)) + (k % 2);
        *h = (*h & ~(1u << hb)) | (((code >> 2) & 1u) << hb);
    }
}

static uint32_t tile_get(const uint32_t *tile, int D, int bits, int m, int row, int col)
{
    int lane = 4 * (row % 8) + (col % 8) / 2;
    int r = row / 8 + 2 * (col / 8);
    int e = col % 2;
    int s = 4 * m + r;
    if (bits == 2) {
        int n = D / 32, i = s / 8, k = s % 8;
        return (tile[section_word_offset(n, lane, i)] >> (16 * e + 2 * k)) & 3u;
    } else if (bits == 4) {
        int n = D / 16, i = s / 4, k = s % 4;
        return (tile[section_word_offset(n, lane, i)] >> (16 * e + 4 * k)) & 15u;
    } else {
        int nlo = D / 32, nhi = D / 64, i = s / 8, k = s % 8;
        uint32_t lo = (tile[section_word_offset(nlo, lane, i)] >> (16 * e + 2 * k)) & 3u;
        int hb = 16 * e + 4 * (k / 2) + 2 * (1 - (i % 2)) + (k % 2);
        uint32_t hi = (tile[32 * nlo + section_word_offset(nhi, lane, i / 2)] >> hb) & 1u;
        return lo | (hi << 2);
    }
}

static uint32_t *tile_ptr(uint8_t *codes, const kvo_config *c, int b, int h, int token)
{
    int64_t row_bytes = (int64_t)c->head_dim * c->bits / 8;
    int64_t unit = ((int64_t)b * c->n_kv_heads + h) * c->max_seq * row_bytes;
    return (uint32_t *)(codes + unit + (int64_t)(token / KVO_TILE) * KVO_TILE * row_bytes);
}

static void k_code_put(uint8_t *codes, const kvo_config *c, int b, int h, int token, int ch, uint32_t code)
{
    tile_put(tile_ptr(codes, c, b, h, token), c->head_dim, c->bits, ch / 16, token % 16, ch % 16, code);
}
static uint32_t k_code_get(const uint8_t *codes, const kvo_config *c, int b, int h, int token, int ch)
{
    return tile_get(tile_ptr((uint8_t *)codes, c, b, h, token), c->head_dim, c->bits, ch / 16, token % 16, ch % 16);
}
static void v_code_put(uint8_t *codes, const kvo_config *c, int b, int h, int token, int ch, uint32_t code)
{
    tile_put(tile_ptr(codes, c, b, h, token), c->head_dim, c->bits, ch / 16, ch % 16, token % 16, code);
}
static uint32_t v_code_get(const uint8_t *codes, const kvo_config *c, int b, int h, int token, int ch)
{
    return tile_get(tile_ptr((uint8_t *)codes, c, b, h, token), c->head_dim, c->bits, ch / 16, ch % 16, token % 16);
}

/* Logical codes of every token < seq (int8, [B,Hkv,seq,D]); kind 0 = K, 1 = V. */
int kvo_unpack_codes(const kvo_config *c, const uint8_t *codes, int kind, int seq, int8_t *out)
{
    int rc = check_config(c);
    if (rc) return rc;
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < c->n_kv_heads; ++h)
            for (int t = 0; t < seq; ++t)
                for (int ch = 0; ch < c->head_dim; ++ch) {
                    uint32_t v = kind ? v_code_get(codes, c, b, h, t, ch) : k_code_get(codes, c, b, h, t, ch);
                    out[(((int64_t)b * c->n_kv_heads + h) * seq + t) * c->head_dim + ch] = (int8_t)v;
                }
    return KVO_OK;
}

/* ---------- sink mask ---------- */
static int mask_bit(const uint32_t *bitmask, const kvo_config *c, int b, int pos)
{
    int words = (c->max_seq + 31) / 32;
    return (bitmask[(int64_t)b * words + pos / 32] >> (pos % 32)) & 1u;
}

typedef struct { float score; int32_t idx; } scored;
static int by_score_desc_then_index(const void *pa, const void *pb)
{
    const scored *a = (const scored *)pa, *b = (const scored *)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/*
 * Algorithm 1, the two statements under "if l = l_E", and Section 4.3 items (1)-(4):
 * S_sink = token indices of Top-k |H[i,c]|.  With several listed channels the score of a token is
 * the largest |H[i,c]| over them; with none listed it is the largest over all d channels.
 * Ties go to the lower token index.  The first pfn_n tokens are OR'd in (Preserve-First-N).
 * Outputs: bitmask (bit i%32 of word i/32, row of ceil(max_seq/32) words per sequence, rewritten
 * in full), ascending positions, and their count.
 */
int kvo_predict_sinks(const kvo_config *c, const uint16_t *hidden, int32_t S, int64_t stride_b, int64_t stride_s,
                      uint32_t *bitmask, int32_t *sink_pos, int32_t *sink_count)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!hidden || !bitmask || !sink_pos || !sink_count || S < 0 || S > c->max_seq) return KVO_ERR_BAD_ARG;
    for (int i = 0; i < c->n_channels; ++i)
        if (c->channels[i] < 0 || c->channels[i] >= c->hidden) return KVO_ERR_BAD_CONFIG;
    int words = (c->max_seq + 31) / 32;
    int cap = sink_cap_of(c);
    scored *sc = (scored *)malloc(sizeof(scored) * (size_t)(S > 0 ? S : 1));
    for (int b = 0; b < c->batch; ++b) {
        uint32_t *bm = bitmask + (int64_t)b * words;
        memset(bm, 0, sizeof(uint32_t) * (size_t)words);
        for (int i = 0; i < S; ++i) {
            const uint16_t *row = hidden + b * stride_b + i * stride_s;
            float best = 0.0f;
            if (c->n_channels == 0) {
                for (int ch = 0; ch < c->hidden; ++ch) {
                    float a = fabsf(half_to_float(row[ch]));
                    if (a > best) best = a;
                }
            } else {
                for (int j = 0; j < c->n_channels; ++j) {
                    float a = fabsf(half_to_float(row[c->channels[j]]));
                    if (a > best) best = a;
                }
            }
            sc[i].score = best;
            sc[i].idx = i;
        }
        qsort(sc, (size_t)S, sizeof(scored), by_score_desc_then_index);
        int k = c->topk < S ? c->topk : S;
        for (int j = 0; j < k; ++j) bm[sc[j].idx / 32] |= 1u << (sc[j].idx % 32);
        int n = c->pfn_n < S ? c->pfn_n : S;
        for (int i = 0; i < n; ++i) bm[i / 32] |= 1u << (i % 32);
        int cnt = 0;
        for (int i = 0; i < S; ++i)
            if ((bm[i / 32] >> (i % 32)) & 1u) sink_pos[(int64_t)b * cap + cnt++] = i;
        for (int j = cnt; j < cap; ++j) sink_pos[(int64_t)b * cap + j] = -1;
        sink_count[b] = cnt;
    }
    free(sc);
    return KVO_OK;
}

/* ---------- Eq. 8-11 on one group ----------
 * x: the group's values; member[j] != 0 marks the values that take part (non-sink tokens).
 * scale = (max - min) / (2^n - 1)                     Eq. 10 (no clipping: plain min / max)
 * zero  = -round(min / scale)                         Eq. 11
 * Q     = clamp(round(x / scale) + zero, 0, 2^n - 1)  Eq. 8
 * round = to nearest, ties to even.  A group whose members are all equal takes scale = |min|
 * (1 if min is 0) so that it reproduces itself; a group without members takes scale = zero = 0.
 * Non-members get code 0.
 */
void kvo_quantize_group(const float *x, const uint8_t *member, int n, int bits, float *scale_out, float *zero_out,
                        int32_t *codes)
{
    const float qmax = (float)((1 << bits) - 1);
    int any = 0;
    float mn = 0.0f, mx = 0.0f;
    for (int j = 0; j < n; ++j) {
        if (!member[j]) continue;
        if (!any) { mn = mx = x[j]; any = 1; }
        else { if (x[j] < mn) mn = x[j]; if (x[j] > mx) mx = x[j]; }
    }
    if (!any) {
        *scale_out = 0.0f;
        *zero_out = 0.0f;
        for (int j = 0; j < n; ++j) codes[j] = 0;
        return;
    }
    float r = mx - mn;
    float scale;
    if (r == 0.0f) scale = (mn == 0.0f) ? 1.0f : fabsf(mn);
    else scale = r / qmax;
    float zero = 0.0f - rintf(mn / scale);
    for (int j = 0; j < n; ++j) {
        if (!member[j]) { codes[j] = 0; continue; }
        float q = rintf(x[j] / scale) + zero;
        q = fminf(fmaxf(q, 0.0f), qmax);
        codes[j] = (int32_t)q;
    }
    *scale_out = scale;
    *zero_out = zero;
}

/* Eq. 9: X' = scale * (Q - zero), in binary32. */
static float dequant(float scale, float zero, uint32_t code) { return scale * ((float)code - zero); }

/* ---------- append (Eq. 6) with sink exclusion (Algorithm 1, the two "quantize" statements) ----------
 * Tokens are appended one by one at positions seq_len, seq_len+1, ...  For the token at position p of
 * sequence b (all KV heads alike):
 *   - if bit p of the sink mask is set, its K and V rows are copied bit for bit into the side buffer at
 *     slot = rank of p in sink_pos[b]; its packed V codes and V parameters are 0;
 *   - otherwise V is quantized per token, one group per v_group channels (Eq. 8-11), and stored;
 *   - its K row goes to k_tail[p % group]; when p completes a group of `group` tokens, that group is
 *     quantized per channel over its non-sink tokens (Eq. 8-11) and stored; sink tokens get code 0.
 * new tokens: fp16 [B, Hkv, T, D] with element strides stride_b, stride_h, stride_t (D contiguous).
 */
int kvo_quantize_append(const kvo_config *c, kvo_cache *cache, const uint16_t *k_new, const uint16_t *v_new, int32_t T,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !k_new || !v_new || T < 0) return KVO_ERR_BAD_ARG;
    if (cache->seq_len < 0 || (int64_t)cache->seq_len + T > c->max_seq) return KVO_ERR_SEQ_OVERFLOW;
    const int D = c->head_dim, G = c->group, gv = v_group_of(c), ngv = D / gv, cap = sink_cap_of(c);
    const int Hk = c->n_kv_heads;
    const int buf = G > D ? G : D;
    int bad = 0;
    /* (sequence, KV head) units are independent; the loop over them may run on several threads */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t unit = 0; unit < (int64_t)c->batch * Hk; ++unit) {
        const int b = (int)(unit / Hk), h = (int)(unit % Hk);
        float *xs = (float *)malloc(sizeof(float) * (size_t)buf);
        uint8_t *mem = (uint8_t *)malloc((size_t)buf);
        int32_t *codes = (int32_t *)malloc(sizeof(int32_t) * (size_t)buf);
        uint16_t *tail = cache->k_tail + unit * G * D;
        for (int i = 0; i < T; ++i) {
            int p = cache->seq_len + i;
            const uint16_t *krow = k_new + b * stride_b + h * stride_h + i * stride_t;
            const uint16_t *vrow = v_new + b * stride_b + h * stride_h + i * stride_t;
            int sink = mask_bit(cache->sink_bitmask, c, b, p);
            if (sink) {
                int slot = -1;
                for (int j = 0; j < cache->sink_count[b]; ++j)
                    if (cache->sink_pos[(int64_t)b * cap + j] == p) slot = j;
                if (slot < 0) {
#pragma omp atomic write
                    bad = 1;
                    continue;
                }
                memcpy(cache->sink_k + (unit * cap + slot) * D, krow, sizeof(uint16_t) * (size_t)D);
                memcpy(cache->sink_v + (unit * cap + slot) * D, vrow, sizeof(uint16_t) * (size_t)D);
            }
            /* V: per token */
            for (int j = 0; j < ngv; ++j) {
                float sc = 0.0f, ze = 0.0f;
                for (int e = 0; e < gv; ++e) { xs[e] = half_to_float(vrow[j * gv + e]); mem[e] = (uint8_t)!sink; }
                kvo_quantize_group(xs, mem, gv, c->bits, &sc, &ze, codes);
                cache->v_scale[(unit * c->max_seq + p) * ngv + j] = sc;
                cache->v_zero[(unit * c->max_seq + p) * ngv + j] = ze;
                for (int e = 0; e < gv; ++e) v_code_put(cache->v_codes, c, b, h, p, j * gv + e, (uint32_t)codes[e]);
            }
            /* K: tail, then per channel when the group is complete */
            memcpy(tail + (int64_t)(p % G) * D, krow, sizeof(uint16_t) * (size_t)D);
            if ((p + 1) % G == 0) {
                int g = p / G;
                for (int ch = 0; ch < D; ++ch) {
                    float sc = 0.0f, ze = 0.0f;
                    for (int t = 0; t < G; ++t) {
                        xs[t] = half_to_float(tail[(int64_t)t * D + ch]);
                        mem[t] = (uint8_t)!mask_bit(cache->sink_bitmask, c, b, g * G + t);
                    }
                    kvo_quantize_group(xs, mem, G, c->bits, &sc, &ze, codes);
                    cache->k_scale[(unit * (c->max_seq / G) + g) * D + ch] = sc;
                    cache->k_zero[(unit * (c->max_seq / G) + g) * D + ch] = ze;
                    for (int t = 0; t < G; ++t) k_code_put(cache->k_codes, c, b, h, g * G + t, ch, (uint32_t)codes[t]);
                }
            }
        }
        free(xs); free(mem); free(codes);
    }
    if (bad) return KVO_ERR_BAD_ARG;
    cache->seq_len += T;
    return KVO_OK;
}

/* ---------- the K and V row that attention sees for token p (Eq. 7: sink rows exact, the rest dequantised) ---------- */
static int sink_slot(const kvo_config *c, const kvo_cache *cache, int b, int p)
{
    int cap = sink_cap_of(c);
    for (int j = 0; j < cache->sink_count[b]; ++j)
        if (cache->sink_pos[(int64_t)b * cap + j] == p) return j;
    return -1;
}

static void kv_row(const kvo_config *c, const kvo_cache *cache, int b, int h, int p, double *krow, double *vrow)
{
    const int D = c->head_dim, G = c->group, gv = v_group_of(c), ngv = D / gv, cap = sink_cap_of(c);
    int64_t unit = (int64_t)b * c->n_kv_heads + h;
    int n_body = (cache->seq_len / G) * G;
    if (mask_bit(cache->sink_bitmask, c, b, p)) {
        int slot = sink_slot(c, cache, b, p);
        for (int ch = 0; ch < D; ++ch) {
            krow[ch] = slot < 0 ? NAN : (double)half_to_float(cache->sink_k[(unit * cap + slot) * D + ch]);
            vrow[ch] = slot < 0 ? NAN : (double)half_to_float(cache->sink_v[(unit * cap + slot) * D + ch]);
        }
        return;
    }
    for (int ch = 0; ch < D; ++ch) {
        if (p >= n_body) {
            krow[ch] = (double)half_to_float(cache->k_tail[(unit * G + p % G) * D + ch]);
        } else {
            int64_t pi = (unit * (c->max_seq / G) + p / G) * D + ch;
            krow[ch] = (double)dequant(cache->k_scale[pi], cache->k_zero[pi], k_code_get(cache->k_codes, c, b, h, p, ch));
        }
        int64_t vi = (unit * c->max_seq + p) * ngv + ch / gv;
        vrow[ch] = (double)dequant(cache->v_scale[vi], cache->v_zero[vi], v_code_get(cache->v_codes, c, b, h, p, ch));
    }
}

/* Dense K', V' (binary64, [B,Hkv,seq_len,D]) exactly as attention consumes them. */
int kvo_dequant_dense(const kvo_config *c, const kvo_cache *cache, double *kd, double *vd)
{
    int rc = check_config(c);
    if (rc) return rc;
    const int D = c->head_dim, n = cache->seq_len;
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < c->n_kv_heads; ++h)
            for (int p = 0; p < n; ++p) {
                int64_t o = ((((int64_t)b * c->n_kv_heads + h) * n) + p) * D;
                kv_row(c, cache, b, h, p, kd + o, vd + o);
            }
    return KVO_OK;
}

/*
 * Eq. 3 for one query token per head, over every cached token, with Eq. 7's split: the token's K and V
 * are the fp16 side-buffer rows if it is a sink, else the dequantised codes (K from the fp16 tail while
 * its group is incomplete).  Query head hq reads KV head hq / (Hq/Hkv).  Scores are scaled by 1/sqrt(D),
 * there is no mask (a decode query sees the whole cache).  binary64 throughout.
 * out [B,Hq,D], lse [B,Hq] (natural-log sum of exp of the scaled scores) may be NULL.
 */
int kvo_decode_attention(const kvo_config *c, const kvo_cache *cache, const uint16_t *q, double *out, double *lse)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !q || !out) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, n = cache->seq_len, rep = c->n_q_heads / c->n_kv_heads;
    /* (sequence, query head) pairs are independent; the loop over them may run on several threads */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < (int64_t)c->batch * c->n_q_heads; ++bh) {
        const int b = (int)(bh / c->n_q_heads), hq = (int)(bh % c->n_q_heads);
        double *krow = (double *)malloc(sizeof(double) * (size_t)D);
        double *vrow = (double *)malloc(sizeof(double) * (size_t)D);
        double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        int h = hq / rep;
        const uint16_t *qv = q + ((int64_t)b * c->n_q_heads + hq) * D;
        double *o = out + ((int64_t)b * c->n_q_heads + hq) * D;
        double mx = -INFINITY;
        for (int p = 0; p < n; ++p) {
            kv_row(c, cache, b, h, p, krow, vrow);
            double acc = 0.0;
            for (int ch = 0; ch < D; ++ch) acc += (double)half_to_float(qv[ch]) * krow[ch];
            s[p] = acc / sqrt((double)D);
            if (s[p] > mx) mx = s[p];
        }
        double den = 0.0;
        for (int ch = 0; ch < D; ++ch) o[ch] = 0.0;
        for (int p = 0; p < n; ++p) {
            double w = exp(s[p] - mx);
            den += w;
            kv_row(c, cache, b, h, p, krow, vrow);
            for (int ch = 0; ch < D; ++ch) o[ch] += w * vrow[ch];
        }
        for (int ch = 0; ch < D; ++ch) o[ch] = n > 0 ? o[ch] / den : 0.0;
        if (lse) lse[(int64_t)b * c->n_q_heads + hq] = n > 0 ? mx + log(den) : -INFINITY;
        free(krow); free(vrow); free(s);
    }
    return KVO_OK;
}

/* =====================================================================================================
 * Analysis routines (Section 3.1 / Appendix D: where the extreme activations sit; Section 4.1, Table 1: what
 * sink tokens do to the quantization error).
 * ===================================================================================================== */

/*
 * Largest magnitude of every hidden channel over all tokens of all sequences: out[c] = max_{b,i} |H[b,i,c]|.
 * This is the scan from which the few "outlier channels" of a model (Appendix D, the table of emergence layers and
 * outlier channels) are read off: they are the channels whose maximum is orders of magnitude above the rest, and the
 * emergence layer is the first layer whose scan shows them.  A NaN never raises a maximum (|x| > best is false).
 */
int kvo_channel_absmax(const uint16_t *hidden, int32_t B, int32_t S, int32_t d, int64_t stride_b, int64_t stride_s, float *out)
{
    if (!hidden || !out || B < 0 || S < 0 || d < 1) return KVO_ERR_BAD_ARG;
    for (int c = 0; c < d; ++c) out[c] = 0.0f;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < S; ++i) {
            const uint16_t *row = hidden + b * stride_b + i * stride_s;
            for (int c = 0; c < d; ++c) {
                float a = fabsf(half_to_float(row[c]));
                if (a > out[c]) out[c] = a;
            }
        }
    return KVO_OK;
}

/*
 * Quantization error in the shape of Table 1 (Section 4.1): round-to-nearest asymmetric quantization (Eq. 8-11) of a
 * tensor x [B,Hkv,T,D], squared error (x - x')^2 with x' = scale * (Q - zero) (Eq. 9), summed separately over the
 * quantization groups that contain no sink token and over those that contain at least one.
 *   per_channel != 0 : groups of `group` consecutive tokens of one channel (keys, per channel); a last, shorter group
 *                      takes the remaining tokens
 *   per_channel == 0 : groups of min(group, D) consecutive channels of one token (per token)
 *   exclude_sinks == 0: plain RTN, every token takes part in its group's min / max (the table's dynamic rows)
 *   exclude_sinks != 0: KVSink: sink tokens take no part in the statistics and are not quantized (no error counted)
 * out[0], out[1]: sum of squared errors and number of elements over groups without a sink token;
 * out[2], out[3]: the same over groups with one.  MSE = out[0] / out[1] and out[2] / out[3].
 */
int kvo_quant_error(const kvo_config *c, const uint16_t *x, int32_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                    int per_channel, int exclude_sinks, const uint32_t *bitmask, double *out)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!x || !bitmask || !out || T < 0 || T > c->max_seq) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, G = c->group, gv = v_group_of(c);
    const int buf = G > D ? G : D;
    float *xs = (float *)malloc(sizeof(float) * (size_t)buf);
    uint8_t *mem = (uint8_t *)malloc((size_t)buf);
    int32_t *codes = (int32_t *)malloc(sizeof(int32_t) * (size_t)buf);
    out[0] = out[1] = out[2] = out[3] = 0.0;
    for (int b = 0; b < c->batch; ++b)
        for (int h = 0; h < c->n_kv_heads; ++h) {
            const uint16_t *base = x + b * stride_b + h * stride_h;
            if (per_channel) {
                for (int t0 = 0; t0 < T; t0 += G) {
                    int n = T - t0 < G ? T - t0 : G, has_sink = 0;
                    for (int t = 0; t < n; ++t) has_sink |= mask_bit(bitmask, c, b, t0 + t);
                    for (int ch = 0; ch < D; ++ch) {
                        float sc = 0.0f, ze = 0.0f;
                        for (int t = 0; t < n; ++t) {
                            xs[t] = half_to_float(base[(int64_t)(t0 + t) * stride_t + ch]);
                            mem[t] = (uint8_t)(exclude_sinks ? !mask_bit(bitmask, c, b, t0 + t) : 1);
                        }
                        kvo_quantize_group(xs, mem, n, c->bits, &sc, &ze, codes);
                        for (int t = 0; t < n; ++t) {
                            if (!mem[t]) continue;
                            double e = (double)xs[t] - (double)dequant(sc, ze, (uint32_t)codes[t]);
                            out[has_sink ? 2 : 0] += e * e;
                            out[has_sink ? 3 : 1] += 1.0;
                        }
                    }
                }
            } else {
                for (int t = 0; t < T; ++t) {
                    int has_sink = mask_bit(bitmask, c, b, t);
                    if (has_sink && exclude_sinks) continue;
                    for (int j = 0; j < D / gv; ++j) {
                        float sc = 0.0f, ze = 0.0f;
                        for (int e = 0; e < gv; ++e) { xs[e] = half_to_float(base[(int64_t)t * stride_t + j * gv + e]); mem[e] = 1; }
                        kvo_quantize_group(xs, mem, gv, c->bits, &sc, &ze, codes);
                        for (int e = 0; e < gv; ++e) {
                            double er = (double)xs[e] - (double)dequant(sc, ze, (uint32_t)codes[e]);
                            out[has_sink ? 2 : 0] += er * er;
                            out[has_sink ? 3 : 1] += 1.0;
                        }
                    }
                }
            }
        }
    free(xs); free(mem); free(codes);
    return KVO_OK;
}

/* =====================================================================================================
 * Static (calibrated) parameters: the scheme of the paper's main comparison (Section 5.1: per-channel keys with
 * per-token values, static), with sink tokens left out of the calibration as well as of the quantization
 * (Algorithm 1's remark on calibration; Section 4.1; Appendix C "Dynamic and static quantization").
 * ===================================================================================================== */

typedef struct {
    float *k_scale, *k_zero;   /* [Hkv][D]: one pair per key channel, for every token and sequence */
    float *v_scale, *v_zero;   /* [Hkv][D / v_group]: one pair per value channel group, for every token and sequence */
} kvo_static_params;

/*
 * Calibration: "global min-max" (Table 1's caption) over a calibration batch x_k, x_v [B,Hkv,T,D], per key channel
 * and per value channel group of every KV head, over all sequences and all tokens that are not sink tokens; then
 * Eq. 10-11.  A range of a single value reproduces itself (scale = |min|, or 1 for 0); no member gives scale = zero = 0.
 */
int kvo_calibrate(const kvo_config *c, const uint16_t *k_cal, const uint16_t *v_cal, int32_t T, int64_t stride_b, int64_t stride_h,
                  int64_t stride_t, const uint32_t *bitmask, kvo_static_params *sp)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!k_cal || !v_cal || !bitmask || !sp || T < 0 || T > c->max_seq) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, gv = v_group_of(c), ngv = D / gv;
    const float qmax = (float)((1 << c->bits) - 1);
    for (int h = 0; h < c->n_kv_heads; ++h)
        for (int kind = 0; kind < 2; ++kind) {
            const int ngroups = kind ? ngv : D, width = kind ? gv : 1;
            for (int j = 0; j < ngroups; ++j) {
                int any = 0;
                float mn = 0.0f, mx = 0.0f;
                for (int b = 0; b < c->batch; ++b)
                    for (int t = 0; t < T; ++t) {
                        if (mask_bit(bitmask, c, b, t)) continue;
                        const uint16_t *row = (kind ? v_cal : k_cal) + b * stride_b + h * stride_h + (int64_t)t * stride_t;
                        for (int e = 0; e < width; ++e) {
                            float v = half_to_float(row[j * width + e]);
                            if (!any) { mn = mx = v; any = 1; }
                            else { if (v < mn) mn = v; if (v > mx) mx = v; }
                        }
                    }
                float scale = 0.0f, zero = 0.0f;
                if (any) {
                    float r = mx - mn;
                    if (r == 0.0f) scale = (mn == 0.0f) ? 1.0f : fabsf(mn);
                    else scale = r / qmax;
                    zero = 0.0f - rintf(mn / scale);
                }
                if (kind) { sp->v_scale[h * ngv + j] = scale; sp->v_zero[h * ngv + j] = zero; }
                else { sp->k_scale[h * D + j] = scale; sp->k_zero[h * D + j] = zero; }
            }
        }
    return KVO_OK;
}

/* Eq. 8 with fixed parameters: values outside the calibrated range clamp to code 0 or 2^n - 1; scale 0 (a channel
 * that saw no calibration data) gives code 0. */
static uint32_t static_code(float x, float scale, float zero, int bits)
{
    if (scale == 0.0f) return 0;
    const float qmax = (float)((1 << bits) - 1);
    float q = rintf(x / scale) + zero;
    q = fminf(fmaxf(q, 0.0f), qmax);
    return (uint32_t)q;
}

/*
 * Append (Eq. 6) with static parameters: every token is coded on arrival, keys per channel and values per channel
 * group with the calibrated pairs (Eq. 8); sink tokens keep exact fp16 rows in the side buffer and code 0.  There is
 * no key tail and no per-group parameter: cache->k_scale, k_zero, v_scale, v_zero and k_tail are not touched.
 */
int kvo_quantize_append_calibrated(const kvo_config *c, kvo_cache *cache, const kvo_static_params *sp, const uint16_t *k_new,
                                   const uint16_t *v_new, int32_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !sp || !k_new || !v_new || T < 0) return KVO_ERR_BAD_ARG;
    if (cache->seq_len < 0 || (int64_t)cache->seq_len + T > c->max_seq) return KVO_ERR_SEQ_OVERFLOW;
    const int D = c->head_dim, gv = v_group_of(c), ngv = D / gv, cap = sink_cap_of(c), Hk = c->n_kv_heads;
    int bad = 0;
    for (int64_t unit = 0; unit < (int64_t)c->batch * Hk; ++unit) {
        const int b = (int)(unit / Hk), h = (int)(unit % Hk);
        for (int i = 0; i < T; ++i) {
            int p = cache->seq_len + i;
            const uint16_t *krow = k_new + b * stride_b + h * stride_h + i * stride_t;
            const uint16_t *vrow = v_new + b * stride_b + h * stride_h + i * stride_t;
            int sink = mask_bit(cache->sink_bitmask, c, b, p);
            if (sink) {
                int slot = sink_slot(c, cache, b, p);
                if (slot < 0) { bad = 1; continue; }
                memcpy(cache->sink_k + (unit * cap + slot) * D, krow, sizeof(uint16_t) * (size_t)D);
                memcpy(cache->sink_v + (unit * cap + slot) * D, vrow, sizeof(uint16_t) * (size_t)D);
            }
            for (int ch = 0; ch < D; ++ch) {
                uint32_t kc = sink ? 0 : static_code(half_to_float(krow[ch]), sp->k_scale[h * D + ch], sp->k_zero[h * D + ch], c->bits);
                uint32_t vc = sink ? 0 : static_code(half_to_float(vrow[ch]), sp->v_scale[h * ngv + ch / gv], sp->v_zero[h * ngv + ch / gv], c->bits);
                k_code_put(cache->k_codes, c, b, h, p, ch, kc);
                v_code_put(cache->v_codes, c, b, h, p, ch, vc);
            }
        }
    }
    if (bad) return KVO_ERR_BAD_ARG;
    cache->seq_len += T;
    return KVO_OK;
}

/*
 * Eq. 3 / Eq. 7 over a cache with static parameters: a sink token's K and V are its fp16 side-buffer rows, every other
 * token's are scale * (Q - zero) (Eq. 9, binary32) with the calibrated pairs.  binary64 otherwise, as kvo_decode_attention.
 */
int kvo_decode_attention_calibrated(const kvo_config *c, const kvo_cache *cache, const kvo_static_params *sp, const uint16_t *q,
                                    double *out, double *lse)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !sp || !q || !out) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, n = cache->seq_len, rep = c->n_q_heads / c->n_kv_heads, gv = v_group_of(c), ngv = D / gv;
    const int cap = sink_cap_of(c);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < (int64_t)c->batch * c->n_q_heads; ++bh) {
        const int b = (int)(bh / c->n_q_heads), hq = (int)(bh % c->n_q_heads), h = hq / rep;
        const int64_t unit = (int64_t)b * c->n_kv_heads + h;
        double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        double *vrow = (double *)malloc(sizeof(double) * (size_t)D);
        const uint16_t *qv = q + ((int64_t)b * c->n_q_heads + hq) * D;
        double *o = out + ((int64_t)b * c->n_q_heads + hq) * D;
        double mx = -INFINITY;
        for (int p = 0; p < n; ++p) {
            int slot = mask_bit(cache->sink_bitmask, c, b, p) ? sink_slot(c, cache, b, p) : -2;
            double acc = 0.0;
            for (int ch = 0; ch < D; ++ch) {
                double kv = slot == -2 ? (double)dequant(sp->k_scale[h * D + ch], sp->k_zero[h * D + ch], k_code_get(cache->k_codes, c, b, h, p, ch))
                                       : (slot < 0 ? NAN : (double)half_to_float(cache->sink_k[(unit * cap + slot) * D + ch]));
                acc += (double)half_to_float(qv[ch]) * kv;
            }
            s[p] = acc / sqrt((double)D);
            if (s[p] > mx) mx = s[p];
        }
        double den = 0.0;
        for (int ch = 0; ch < D; ++ch) o[ch] = 0.0;
        for (int p = 0; p < n; ++p) {
            int slot = mask_bit(cache->sink_bitmask, c, b, p) ? sink_slot(c, cache, b, p) : -2;
            for (int ch = 0; ch < D; ++ch)
                vrow[ch] = slot == -2 ? (double)dequant(sp->v_scale[h * ngv + ch / gv], sp->v_zero[h * ngv + ch / gv], v_code_get(cache->v_codes, c, b, h, p, ch))
                                      : (slot < 0 ? NAN : (double)half_to_float(cache->sink_v[(unit * cap + slot) * D + ch]));
            double w = exp(s[p] - mx);
            den += w;
            for (int ch = 0; ch < D; ++ch) o[ch] += w * vrow[ch];
        }
        for (int ch = 0; ch < D; ++ch) o[ch] = n > 0 ? o[ch] / den : 0.0;
        if (lse) lse[(int64_t)b * c->n_q_heads + hq] = n > 0 ? mx + log(den) : -INFINITY;
        free(s); free(vrow);
    }
    return KVO_OK;
}

/*
 * Attention of the prompt's own queries over the cache that was just quantized (Algorithm 1, the attention statement
 * after the two quantize statements; Eq. 3 with a causal mask): query token t of the chunk (t = 0 .. T-1) sits at
 * position q_pos0 + t and attends to the cached tokens 0 .. q_pos0 + t, whose K and V are what decode attention reads
 * (Eq. 7: sink tokens exact, the others dequantised; open-group keys from the fp16 tail).  binary64 throughout.
 * q: fp16 [B,Hq,T,D] with element strides; out [B,Hq,T,D]; lse [B,Hq,T] (may be NULL).
 * Requires q_pos0 >= 0 and q_pos0 + T <= seq_len.
 */
int kvo_prefill_attention(const kvo_config *c, const kvo_cache *cache, const uint16_t *q, int32_t T, int32_t q_pos0, int64_t stride_b,
                          int64_t stride_h, int64_t stride_t, double *out, double *lse)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !q || !out || T < 0 || q_pos0 < 0 || (int64_t)q_pos0 + T > cache->seq_len) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, rep = c->n_q_heads / c->n_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < (int64_t)c->batch * c->n_q_heads; ++bh) {
        const int b = (int)(bh / c->n_q_heads), hq = (int)(bh % c->n_q_heads), h = hq / rep;
        const int n_max = q_pos0 + T;
        double *kd = (double *)malloc(sizeof(double) * (size_t)(n_max > 0 ? n_max : 1) * D);
        double *vd = (double *)malloc(sizeof(double) * (size_t)(n_max > 0 ? n_max : 1) * D);
        double *s = (double *)malloc(sizeof(double) * (size_t)(n_max > 0 ? n_max : 1));
        for (int p = 0; p < n_max; ++p) kv_row(c, cache, b, h, p, kd + (int64_t)p * D, vd + (int64_t)p * D);
        for (int t = 0; t < T; ++t) {
            const int n = q_pos0 + t + 1;
            const uint16_t *qv = q + b * stride_b + hq * stride_h + t * stride_t;
            double *o = out + (((int64_t)b * c->n_q_heads + hq) * T + t) * D;
            double mx = -INFINITY;
            for (int p = 0; p < n; ++p) {
                double acc = 0.0;
                for (int ch = 0; ch < D; ++ch) acc += (double)half_to_float(qv[ch]) * kd[(int64_t)p * D + ch];
                s[p] = acc / sqrt((double)D);
                if (s[p] > mx) mx = s[p];
            }
            double den = 0.0;
            for (int ch = 0; ch < D; ++ch) o[ch] = 0.0;
            for (int p = 0; p < n; ++p) {
                double w = exp(s[p] - mx);
                den += w;
                for (int ch = 0; ch < D; ++ch) o[ch] += w * vd[(int64_t)p * D + ch];
            }
            for (int ch = 0; ch < D; ++ch) o[ch] /= den;
            if (lse) lse[((int64_t)b * c->n_q_heads + hq) * T + t] = mx + log(den);
        }
        free(kd); free(vd); free(s);
    }
    return KVO_OK;
}

/* =====================================================================================================
 * Per-token keys (Section 4.1 "Per-token quantization"; Section 5.1's "per-token Key and Value dynamic" scheme):
 * keys are quantized like values -- per token over groups of min(group, D) consecutive channels, parameters computed
 * on the fly -- so a key is coded on arrival and there is neither a token group nor a tail.  Sink tokens keep exact
 * rows in the side buffer, code 0 and parameters (0, 0) (Algorithm 1's exclusion).
 * Cache fields: k_scale, k_zero hold [B*Hkv][max_seq][D / v_group] floats (the value parameters' shape); k_tail is
 * not used.
 * ===================================================================================================== */
int kvo_quantize_append_pertoken(const kvo_config *c, kvo_cache *cache, const uint16_t *k_new, const uint16_t *v_new, int32_t T,
                                 int64_t stride_b, int64_t stride_h, int64_t stride_t)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !k_new || !v_new || T < 0) return KVO_ERR_BAD_ARG;
    if (cache->seq_len < 0 || (int64_t)cache->seq_len + T > c->max_seq) return KVO_ERR_SEQ_OVERFLOW;
    const int D = c->head_dim, gv = v_group_of(c), ngv = D / gv, cap = sink_cap_of(c), Hk = c->n_kv_heads;
    int bad = 0;
    float *xs = (float *)malloc(sizeof(float) * (size_t)gv);
    uint8_t *mem = (uint8_t *)malloc((size_t)gv);
    int32_t *codes = (int32_t *)malloc(sizeof(int32_t) * (size_t)gv);
    for (int64_t unit = 0; unit < (int64_t)c->batch * Hk; ++unit) {
        const int b = (int)(unit / Hk), h = (int)(unit % Hk);
        for (int i = 0; i < T; ++i) {
            int p = cache->seq_len + i;
            const uint16_t *krow = k_new + b * stride_b + h * stride_h + i * stride_t;
            const uint16_t *vrow = v_new + b * stride_b + h * stride_h + i * stride_t;
            int sink = mask_bit(cache->sink_bitmask, c, b, p);
            if (sink) {
                int slot = sink_slot(c, cache, b, p);
                if (slot < 0) { bad = 1; continue; }
                memcpy(cache->sink_k + (unit * cap + slot) * D, krow, sizeof(uint16_t) * (size_t)D);
                memcpy(cache->sink_v + (unit * cap + slot) * D, vrow, sizeof(uint16_t) * (size_t)D);
            }
            for (int kind = 0; kind < 2; ++kind) {
                const uint16_t *row = kind ? vrow : krow;
                float *ps = kind ? cache->v_scale : cache->k_scale, *pz = kind ? cache->v_zero : cache->k_zero;
                for (int j = 0; j < ngv; ++j) {
                    float sc = 0.0f, ze = 0.0f;
                    for (int e = 0; e < gv; ++e) { xs[e] = half_to_float(row[j * gv + e]); mem[e] = (uint8_t)!sink; }
                    kvo_quantize_group(xs, mem, gv, c->bits, &sc, &ze, codes);
                    ps[(unit * c->max_seq + p) * ngv + j] = sc;
                    pz[(unit * c->max_seq + p) * ngv + j] = ze;
                    for (int e = 0; e < gv; ++e) {
                        if (kind) v_code_put(cache->v_codes, c, b, h, p, j * gv + e, (uint32_t)codes[e]);
                        else k_code_put(cache->k_codes, c, b, h, p, j * gv + e, (uint32_t)codes[e]);
                    }
                }
            }
        }
    }
    free(xs); free(mem); free(codes);
    if (bad) return KVO_ERR_BAD_ARG;
    cache->seq_len += T;
    return KVO_OK;
}

/* Eq. 3 / Eq. 7 over a cache with per-token keys: binary64, as kvo_decode_attention. */
int kvo_decode_attention_pertoken(const kvo_config *c, const kvo_cache *cache, const uint16_t *q, double *out, double *lse)
{
    int rc = check_config(c);
    if (rc) return rc;
    if (!cache || !q || !out) return KVO_ERR_BAD_ARG;
    const int D = c->head_dim, n = cache->seq_len, rep = c->n_q_heads / c->n_kv_heads, gv = v_group_of(c), ngv = D / gv;
    const int cap = sink_cap_of(c);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < (int64_t)c->batch * c->n_q_heads; ++bh) {
        const int b = (int)(bh / c->n_q_heads), hq = (int)(bh % c->n_q_heads), h = hq / rep;
        const int64_t unit = (int64_t)b * c->n_kv_heads + h;
        double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        const uint16_t *qv = q + ((int64_t)b * c->n_q_heads + hq) * D;
        double *o = out + ((int64_t)b * c->n_q_heads + hq) * D;
        double mx = -INFINITY;
        for (int p = 0; p < n; ++p) {
            int slot = mask_bit(cache->sink_bitmask, c, b, p) ? sink_slot(c, cache, b, p) : -2;
            double acc = 0.0;
            for (int ch = 0; ch < D; ++ch) {
                int64_t pi = (unit * c->max_seq + p) * ngv + ch / gv;
                double kv = slot == -2 ? (double)dequant(cache->k_scale[pi], cache->k_zero[pi], k_code_get(cache->k_codes, c, b, h, p, ch))
                                       : (slot < 0 ? NAN : (double)half_to_float(cache->sink_k[(unit * cap + slot) * D + ch]));
                acc += (double)half_to_float(qv[ch]) * kv;
            }
            s[p] = acc / sqrt((double)D);
            if (s[p] > mx) mx = s[p];
        }
        double den = 0.0;
        for (int ch = 0; ch < D; ++ch) o[ch] = 0.0;
        for (int p = 0; p < n; ++p) {
            int slot = mask_bit(cache->sink_bitmask, c, b, p) ? sink_slot(c, cache, b, p) : -2;
            double w = exp(s[p] - mx);
            den += w;
            for (int ch = 0; ch < D; ++ch) {
                int64_t pi = (unit * c->max_seq + p) * ngv + ch / gv;
                double vv = slot == -2 ? (double)dequant(cache->v_scale[pi], cache->v_zero[pi], v_code_get(cache->v_codes, c, b, h, p, ch))
                                       : (slot < 0 ? NAN : (double)half_to_float(cache->sink_v[(unit * cap + slot) * D + ch]));
                o[ch] += w * vv;
            }
        }
        for (int ch = 0; ch < D; ++ch) o[ch] = n > 0 ? o[ch] / den : 0.0;
        if (lse) lse[(int64_t)b * c->n_q_heads + hq] = n > 0 ? mx + log(den) : -INFINITY;
        free(s);
    }
    return KVO_OK;
}
