// C-ABI entry points of libkvsink: argument validation on the host, then kernel launches on the caller's stream.
#include "common.cuh"

using namespace kvsink;

std::atomic<unsigned long long> kvsink::g_launches{0};

static int derive(const kvsink_config *cfg, Params *p)
{
    if (!cfg) return KVSINK_ERR_BAD_ARG;
    if (cfg->batch < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->hidden < 1) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->n_q_heads % cfg->n_kv_heads) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->bits < 2 || cfg->bits > 4) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->group < 16 || cfg->group % 16) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->max_seq < cfg->group || cfg->max_seq % cfg->group) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->topk < 0 || cfg->pfn_n < 0) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->n_channels < 0 || cfg->n_channels > 8) return KVSINK_ERR_BAD_CONFIG;
    for (int i = 0; i < cfg->n_channels; ++i)
        if (cfg->channels[i] < 0 || cfg->channels[i] >= cfg->hidden) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->head_dim < 16 || cfg->head_dim % 16) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return KVSINK_ERR_UNSUPPORTED;
    if (cfg->bits == 3 && cfg->head_dim != 128) return KVSINK_ERR_UNSUPPORTED;
    const int gv = cfg->group < cfg->head_dim ? cfg->group : cfg->head_dim;
    if (cfg->head_dim % gv) return KVSINK_ERR_BAD_CONFIG;
    if (cfg->head_dim / gv > 4) return KVSINK_ERR_UNSUPPORTED;
    p->B = cfg->batch; p->Hq = cfg->n_q_heads; p->Hkv = cfg->n_kv_heads; p->D = cfg->head_dim; p->hidden = cfg->hidden;
    p->bits = cfg->bits; p->G = cfg->group; p->max_seq = cfg->max_seq; p->topk = cfg->topk; p->pfn_n = cfg->pfn_n;
    p->cap = cfg->topk + cfg->pfn_n;
    p->Gv = gv; p->NGv = cfg->head_dim / gv;
    p->rep = cfg->n_q_heads / cfg->n_kv_heads;
    p->row_bytes = cfg->head_dim * cfg->bits / 8;
    p->tile_bytes = KVSINK_TILE * p->row_bytes;
    p->mask_words = (cfg->max_seq + 31) / 32;
    p->n_channels = cfg->n_channels;
    for (int i = 0; i < 8; ++i) p->channels[i] = cfg->channels[i];
    return KVSINK_OK;
}

// Whole groups: the streaming kernel where the shape has one, else the generic kernel.
static int quantize_groups(const Params &p, const kvsink_cache &c, const __half *k, const __half *v, int first_token, int n_groups,
                           int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st)
{
    int rc = KVSINK_ERR_UNSUPPORTED;
    if (do_v_and_sinks) rc = launch_quantize_groups_bulk(p, c, k, v, first_token, n_groups, sb, sh, stt, st);
    if (rc != KVSINK_ERR_UNSUPPORTED) return rc;
    rc = launch_quantize_groups_fast(p, c, k, v, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
    if (rc != KVSINK_ERR_UNSUPPORTED) return rc;
    return launch_quantize_groups(p, c, k, v, first_token, n_groups, sb, sh, stt, do_v_and_sinks, st);
}

static bool aligned16(const void *ptr) { return ptr && ((uintptr_t)ptr & 15u) == 0; }

static int check_cache(const kvsink_cache *c, const Params &p)
{
    if (!c) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(c->k_codes) || !aligned16(c->v_codes) || !aligned16(c->k_scale) || !aligned16(c->k_zero) ||
        !aligned16(c->v_scale) || !aligned16(c->v_zero) || !aligned16(c->k_tail) || !aligned16(c->sink_bitmask) || !c->sink_count ||
        !c->status)
        return KVSINK_ERR_BAD_ARG;
    if (p.cap > 0 && (!aligned16(c->sink_k) || !aligned16(c->sink_v) || !c->sink_pos)) return KVSINK_ERR_BAD_ARG;
    if (c->seq_len < 0 || c->seq_len > p.max_seq) return KVSINK_ERR_BAD_ARG;
    return KVSINK_OK;
}

extern "C" int kvsink_cache_sizes(const kvsink_config *cfg, kvsink_sizes *out)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!out) return KVSINK_ERR_BAD_ARG;
    const int64_t units = (int64_t)p.B * p.Hkv;
    out->k_codes_bytes = units * p.max_seq * p.row_bytes;
    out->v_codes_bytes = out->k_codes_bytes;
    out->k_param_floats = units * (p.max_seq / p.G) * p.D;
    out->v_param_floats = units * p.max_seq * p.NGv;
    out->k_tail_halfs = units * p.G * p.D;
    out->sink_halfs = units * p.cap * p.D;
    out->bitmask_words = (int64_t)p.B * p.mask_words;
    out->sink_pos_ints = (int64_t)p.B * p.cap;
    out->predict_workspace_bytes = (int64_t)predict_workspace_bytes(p);
    out->decode_workspace_bytes = (int64_t)decode_workspace_bytes(p);
    out->calibrate_workspace_bytes = (int64_t)calibrate_workspace_bytes(p);
    out->sink_capacity = p.cap;
    out->v_group = p.Gv;
    out->v_groups_per_row = p.NGv;
    out->tile_bytes = p.tile_bytes;
    return KVSINK_OK;
}

extern "C" int kvsink_predict_sinks(const kvsink_config *cfg, const void *hidden, int32_t S, int64_t stride_b, int64_t stride_s,
                                    uint32_t *bitmask, int32_t *sink_pos, int32_t *sink_count, void *workspace,
                                    size_t workspace_bytes, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!hidden || !bitmask || !sink_count || (p.cap > 0 && !sink_pos)) return KVSINK_ERR_BAD_ARG;
    if (S < 0 || S > p.max_seq || stride_s < p.hidden || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(workspace) || workspace_bytes < predict_workspace_bytes(p)) return KVSINK_ERR_WORKSPACE;
    return launch_predict_sinks(p, (const __half *)hidden, S, stride_b, stride_s, bitmask, sink_pos, sink_count, workspace,
                                (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_quantize_append(const kvsink_config *cfg, kvsink_cache *cache, const void *k_new, const void *v_new, int32_t T,
                                      int64_t stride_b, int64_t stride_h, int64_t stride_t, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    rc = check_cache(cache, p);
    if (rc) return rc;
    if (T < 0) return KVSINK_ERR_BAD_ARG;
    if (T == 0) return KVSINK_OK;
    if (!aligned16(k_new) || !aligned16(v_new)) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if ((int64_t)cache->seq_len + T > p.max_seq) return KVSINK_ERR_SEQ_OVERFLOW;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int S0 = cache->seq_len, G = p.G;
    const __half *k = (const __half *)k_new, *v = (const __half *)v_new;
    // A chunk that starts inside an open group first completes (or extends) that group token by token; whole groups
    // that follow take the bulk kernels; what is left goes to the tail token by token.
    int done = 0;
    if (S0 % G != 0) {
        const int head = T < G - S0 % G ? T : G - S0 % G;
        rc = launch_quantize_tokens(p, *cache, k, v, 0, S0, head, stride_b, stride_h, stride_t, st);
        if (rc) return rc;
        if ((S0 + head) % G == 0) {
            // the open group is complete: quantize its keys per channel from the fp16 tail
            rc = quantize_groups(p, *cache, (const __half *)cache->k_tail, (const __half *)cache->k_tail, S0 + head - G, 1,
                                 (int64_t)p.Hkv * G * p.D, (int64_t)G * p.D, p.D, false, st);
            if (rc) return rc;
        }
        done = head;
    }
    if (T > done) {   // position S0 + done is the start of a group
        const int n_groups = (T - done) / G;
        if (n_groups > 0) {
            rc = quantize_groups(p, *cache, k + (int64_t)done * stride_t, v + (int64_t)done * stride_t, S0 + done, n_groups, stride_b,
                                 stride_h, stride_t, true, st);
            if (rc) return rc;
        }
        rc = launch_quantize_tokens(p, *cache, k, v, done + n_groups * G, S0 + done + n_groups * G, T - done - n_groups * G, stride_b,
                                    stride_h, stride_t, st);
        if (rc) return rc;
    }
    cache->seq_len = S0 + T;
    return KVSINK_OK;
}

extern "C" int kvsink_decode_attention(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out, float *lse,
                                       void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    rc = check_cache(cache, p);
    if (rc) return rc;
    if (!aligned16(q) || !aligned16(out)) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(workspace)) return KVSINK_ERR_WORKSPACE;
    return launch_decode(p, *cache, nullptr, 0, (const __half *)q, out, lse, workspace, workspace_bytes, (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_prefill_attention(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, int32_t T, int32_t q_pos0,
                                        int64_t stride_b, int64_t stride_h, int64_t stride_t, float *out, float *lse, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    rc = check_cache(cache, p);
    if (rc) return rc;
    if (T < 0 || q_pos0 < 0 || (int64_t)q_pos0 + T > cache->seq_len) return KVSINK_ERR_BAD_ARG;
    if (T == 0) return KVSINK_OK;
    if (!aligned16(q) || !aligned16(out)) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const __half *qq = (const __half *)q;
    if (p.bits == 2) return launch_prefill_b2(p, *cache, qq, T, q_pos0, stride_b, stride_h, stride_t, out, lse, st);
    if (p.bits == 3) return launch_prefill_b3(p, *cache, qq, T, q_pos0, stride_b, stride_h, stride_t, out, lse, st);
    return launch_prefill_b4(p, *cache, qq, T, q_pos0, stride_b, stride_h, stride_t, out, lse, st);
}

extern "C" int kvsink_decode_attention_static(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out,
                                              float *lse, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (decode_workspace_bytes(p) > (size_t)KVSINK_STATIC_SCRATCH_BYTES) return KVSINK_ERR_STATIC_SCRATCH;
    rc = check_cache(cache, p);
    if (rc) return rc;
    if (!aligned16(q) || !aligned16(out)) return KVSINK_ERR_BAD_ARG;
    return launch_decode_static(p, *cache, (const __half *)q, out, lse, (cudaStream_t)cuda_stream);
}

// A cache used with static parameters: the per-group parameter arrays and the key tail are not used and may be null.
static int check_cache_calibrated(const kvsink_cache *c, const kvsink_static_params *sp, const Params &p)
{
    if (!c || !sp) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(c->k_codes) || !aligned16(c->v_codes) || !aligned16(c->sink_bitmask) || !c->sink_count || !c->status) return KVSINK_ERR_BAD_ARG;
    if (p.cap > 0 && (!aligned16(c->sink_k) || !aligned16(c->sink_v) || !c->sink_pos)) return KVSINK_ERR_BAD_ARG;
    if (!sp->k_scale || !sp->k_zero || !sp->v_scale || !sp->v_zero) return KVSINK_ERR_BAD_ARG;
    if (c->seq_len < 0 || c->seq_len > p.max_seq) return KVSINK_ERR_BAD_ARG;
    return KVSINK_OK;
}

extern "C" int kvsink_calibrate(const kvsink_config *cfg, const void *k_cal, const void *v_cal, int32_t T, int64_t stride_b, int64_t stride_h,
                                int64_t stride_t, const uint32_t *sink_bitmask, const kvsink_static_params *params, void *workspace,
                                size_t workspace_bytes, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!params || !params->k_scale || !params->k_zero || !params->v_scale || !params->v_zero || !sink_bitmask) return KVSINK_ERR_BAD_ARG;
    if (T < 0 || T > p.max_seq) return KVSINK_ERR_BAD_ARG;
    if (T > 0 && (!aligned16(k_cal) || !aligned16(v_cal))) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(workspace) || workspace_bytes < calibrate_workspace_bytes(p)) return KVSINK_ERR_WORKSPACE;
    return launch_calibrate(p, (const __half *)k_cal, (const __half *)v_cal, T, stride_b, stride_h, stride_t, sink_bitmask, *params, workspace,
                            (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_quantize_append_calibrated(const kvsink_config *cfg, kvsink_cache *cache, const kvsink_static_params *params,
                                                 const void *k_new, const void *v_new, int32_t T, int64_t stride_b, int64_t stride_h,
                                                 int64_t stride_t, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    rc = check_cache_calibrated(cache, params, p);
    if (rc) return rc;
    if (T < 0) return KVSINK_ERR_BAD_ARG;
    if (T == 0) return KVSINK_OK;
    if (!aligned16(k_new) || !aligned16(v_new)) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if ((int64_t)cache->seq_len + T > p.max_seq) return KVSINK_ERR_SEQ_OVERFLOW;
    rc = launch_quantize_calibrated(p, *cache, *params, (const __half *)k_new, (const __half *)v_new, cache->seq_len, T, stride_b, stride_h,
                                    stride_t, (cudaStream_t)cuda_stream);
    if (rc) return rc;
    cache->seq_len += T;
    return KVSINK_OK;
}

extern "C" int kvsink_decode_attention_calibrated(const kvsink_config *cfg, const kvsink_cache *cache, const kvsink_static_params *params,
                                                  const void *q, float *out, float *lse, void *workspace, size_t workspace_bytes,
                                                  void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    rc = check_cache_calibrated(cache, params, p);
    if (rc) return rc;
    if (!aligned16(q) || !aligned16(out)) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(workspace)) return KVSINK_ERR_WORKSPACE;
    return launch_decode(p, *cache, params, 1, (const __half *)q, out, lse, workspace, workspace_bytes, (cudaStream_t)cuda_stream);
}

// A cache with per-token keys: k_scale / k_zero have the value parameters' shape and there is no key tail.
static int check_cache_pertoken(const kvsink_cache *c, const Params &p)
{
    if (!c) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(c->k_codes) || !aligned16(c->v_codes) || !aligned16(c->sink_bitmask) || !c->sink_count || !c->status) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(c->k_scale) || !aligned16(c->k_zero) || !aligned16(c->v_scale) || !aligned16(c->v_zero)) return KVSINK_ERR_BAD_ARG;
    if (p.cap > 0 && (!aligned16(c->sink_k) || !aligned16(c->sink_v) || !c->sink_pos)) return KVSINK_ERR_BAD_ARG;
    if (c->seq_len < 0 || c->seq_len > p.max_seq) return KVSINK_ERR_BAD_ARG;
    return KVSINK_OK;
}

// The shapes the per-token key kernels are built for.
static bool pertoken_supported(const Params &p)
{
    if (p.D != 128 || p.NGv > 2 || p.rep > 4) return false;
    if (p.bits == 3 && (p.NGv != 1 || p.rep != 1)) return false;
    return true;
}

extern "C" int kvsink_quantize_append_pertoken(const kvsink_config *cfg, kvsink_cache *cache, const void *k_new, const void *v_new, int32_t T,
                                               int64_t stride_b, int64_t stride_h, int64_t stride_t, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!pertoken_supported(p)) return KVSINK_ERR_UNSUPPORTED;
    rc = check_cache_pertoken(cache, p);
    if (rc) return rc;
    if (T < 0) return KVSINK_ERR_BAD_ARG;
    if (T == 0) return KVSINK_OK;
    if (!aligned16(k_new) || !aligned16(v_new)) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if ((int64_t)cache->seq_len + T > p.max_seq) return KVSINK_ERR_SEQ_OVERFLOW;
    rc = launch_quantize_pertoken(p, *cache, (const __half *)k_new, (const __half *)v_new, cache->seq_len, T, stride_b, stride_h, stride_t,
                                  (cudaStream_t)cuda_stream);
    if (rc) return rc;
    cache->seq_len += T;
    return KVSINK_OK;
}

extern "C" int kvsink_decode_attention_pertoken(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out, float *lse,
                                                void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!pertoken_supported(p)) return KVSINK_ERR_UNSUPPORTED;
    rc = check_cache_pertoken(cache, p);
    if (rc) return rc;
    if (!aligned16(q) || !aligned16(out)) return KVSINK_ERR_BAD_ARG;
    if (!aligned16(workspace)) return KVSINK_ERR_WORKSPACE;
    return launch_decode(p, *cache, nullptr, 2, (const __half *)q, out, lse, workspace, workspace_bytes, (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_channel_absmax(const void *hidden, int32_t B, int32_t S, int32_t d, int64_t stride_b, int64_t stride_s, float *out,
                                     void *cuda_stream)
{
    if (!out || B < 0 || S < 0 || d < 1 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    if ((long long)B * S > 0 && (!hidden || stride_s < d)) return KVSINK_ERR_BAD_ARG;   // no tokens: nothing is read
    return launch_channel_absmax((const __half *)hidden, B, S, d, stride_b, stride_s, out, (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_quant_error(const kvsink_config *cfg, const void *x, int32_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                                  int32_t per_channel, int32_t exclude_sinks, const uint32_t *sink_bitmask, double *out, void *cuda_stream)
{
    Params p;
    int rc = derive(cfg, &p);
    if (rc) return rc;
    if (!aligned16(x) || !sink_bitmask || !out || ((uintptr_t)out & 7u) || T < 0 || T > p.max_seq) return KVSINK_ERR_BAD_ARG;
    if (stride_t < p.D || (stride_t % 8) || (stride_h % 8) || (stride_b % 8) || stride_h < 0 || stride_b < 0) return KVSINK_ERR_BAD_ARG;
    return launch_quant_error(p, (const __half *)x, T, stride_b, stride_h, stride_t, per_channel != 0, exclude_sinks != 0, sink_bitmask, out,
                              (cudaStream_t)cuda_stream);
}

extern "C" int kvsink_read_status(const kvsink_cache *cache, int32_t *host_status, void *cuda_stream)
{
    if (!cache || !cache->status || !host_status) return KVSINK_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(host_status, cache->status, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVSINK_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVSINK_ERR_CUDA;
    // the word is delivered in any case; a raised bit is also the call's result
    if (*host_status & KVSINK_STATUS_TIMEOUT) return KVSINK_ERR_TIMEOUT;
    if (*host_status & KVSINK_STATUS_BOUNDS) return KVSINK_ERR_BOUNDS;
    if (*host_status & KVSINK_STATUS_SINK_MISMATCH) return KVSINK_ERR_SINK_MISMATCH;
    return KVSINK_OK;
}

extern "C" unsigned long long kvsink_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char *kvsink_strerror(int code)
{
    switch (code) {
    case KVSINK_OK: return "ok";
    case KVSINK_ERR_BAD_ARG: return "bad argument (null or misaligned pointer, negative size, bad stride)";
    case KVSINK_ERR_BAD_CONFIG: return "configuration field out of range";
    case KVSINK_ERR_UNSUPPORTED: return "valid request without a kernel in this build";
    case KVSINK_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case KVSINK_ERR_SEQ_OVERFLOW: return "appending would exceed max_seq";
    case KVSINK_ERR_SINK_MISMATCH: return "a token whose mask bit is set is missing from the position list (status bit SINK_MISMATCH)";
    case KVSINK_ERR_BOUNDS: return "a debug build caught an index outside its array (status bit BOUNDS)";
    case KVSINK_ERR_CUDA: return "a CUDA runtime call failed";
    case KVSINK_ERR_TIMEOUT: return "a bounded device wait ran out (status bit TIMEOUT): results of that cache are invalid";
    case KVSINK_ERR_STATIC_SCRATCH:
        return "this configuration needs more split scratch than the library's built-in array holds "
               "(KVSINK_STATIC_SCRATCH_BYTES); use kvsink_decode_attention with a caller workspace";
    default: return "unknown status";
    }
}
