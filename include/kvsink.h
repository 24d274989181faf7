/*
 * libkvsink -- KVSink quantized-KV-cache hot path for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer documented "device" must point to CUDA device memory owned by the caller;
 * "host" pointers are ordinary host memory.  The library allocates no device memory, keeps no state
 * between calls (it caches two lookups: the driver's tensor-map encoder and, for kvsink_decode_attention_static,
 * the device address of its built-in scratch; and it counts its kernel launches, see kvsink_launch_count), launches all work asynchronously on the caller's stream and never
 * synchronises, except in kvsink_read_status.  Every entry point returns 0 (KVSINK_OK) or a negative KVSINK_ERR_* code; argument
 * errors are detected on the host before anything is launched.  Nothing traps or spins on the device.
 *
 * Citations are to arXiv 2508.04257 ("KVSink"): Eq. 3 / Eq. 7 (attention, split into sink and non-sink
 * sums), Eq. 6 (cache append), Eq. 8-11 (asymmetric n-bit quantization, Appendix C), Algorithm 1
 * (prefill with KVSink: sink exclusion and top-k sink prediction), Section 4.3 (the prediction rule).
 */
#ifndef KVSINK_H_
#define KVSINK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVSINK_OK 0
#define KVSINK_ERR_BAD_ARG (-1)      /* NULL / misaligned pointer, negative size, inconsistent strides */
#define KVSINK_ERR_BAD_CONFIG (-2)   /* a kvsink_config field is out of range */
#define KVSINK_ERR_UNSUPPORTED (-3)  /* a valid request this build has no kernel for */
#define KVSINK_ERR_WORKSPACE (-4)    /* workspace missing or too small */
#define KVSINK_ERR_SEQ_OVERFLOW (-5) /* seq_len + T > max_seq */
#define KVSINK_ERR_SINK_MISMATCH (-6) /* kvsink_read_status: status bit KVSINK_STATUS_SINK_MISMATCH is set */
#define KVSINK_ERR_CUDA (-7)         /* a CUDA runtime call failed (launch, attribute, copy) */
#define KVSINK_ERR_TIMEOUT (-8)       /* kvsink_read_status: status bit KVSINK_STATUS_TIMEOUT is set */
#define KVSINK_ERR_STATIC_SCRATCH (-9) /* kvsink_decode_attention_static: the built-in scratch array is too small */
#define KVSINK_ERR_BOUNDS (-10)       /* kvsink_read_status: status bit KVSINK_STATUS_BOUNDS is set (debug builds only) */

/* Size of the scratch array built into the library for kvsink_decode_attention_static (4 MiB per GPU). */
#define KVSINK_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)

/* Bits of the device status word (kvsink_cache.status, read with kvsink_read_status). */
#define KVSINK_STATUS_SINK_MISMATCH 1 /* a token whose mask bit is set was not found in sink_pos */
#define KVSINK_STATUS_TIMEOUT 2       /* a bounded wait for a shared-memory bulk copy ran out; the result is invalid */
#define KVSINK_STATUS_BOUNDS 4        /* a library built with -DKVSINK_DEBUG found an index outside its array and skipped the access */

/* Tokens per packed tile. */
#define KVSINK_TILE 16

/*
 * Problem description (Algorithm 1 "Parameters", plus the quantizer of Appendix C).
 *   batch, n_q_heads, n_kv_heads, head_dim, hidden : B, Hq, Hkv, D, d.  Hq % Hkv == 0, D in {64,128}.
 *   bits     : n of Eq. 8 (2, 3 or 4; 3 needs D == 128).
 *   group    : G.  Keys are quantized per channel over groups of G consecutive tokens; values per token
 *              over groups of min(G, D) consecutive channels.  G % 16 == 0, D % min(G,D) == 0.
 *   max_seq  : capacity of the cache in tokens, a multiple of G.
 *   topk     : k of Algorithm 1.  pfn_n: N of Preserve-First-N.  Sink capacity per sequence = topk + pfn_n.
 *   channels : the pre-identified outlier channel(s) c of Section 4.3 (indices into hidden);
 *              n_channels == 0 means "all d channels".
 */
typedef struct kvsink_config {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, hidden;
    int32_t bits, group, max_seq, topk, pfn_n;
    int32_t n_channels;
    int32_t channels[8];
} kvsink_config;

/*
 * One layer's cache.  All pointers are device pointers, 16-byte aligned, caller-allocated with the sizes
 * kvsink_cache_sizes reports and zero-filled before first use.  u = b * Hkv + h is the (sequence, KV head) unit.
 *   k_codes, v_codes : packed codes, [u][max_seq/16][tile_bytes]; one tile = 16 tokens x D channels.  A K tile
 *                      is a stack of D/16 matrices [16 tokens x 16 channels], a V tile a stack of D/16 matrices
 *                      [16 channels x 16 tokens]; element (row, col) of matrix m lives in lane
 *                      4*(row%8) + (col%8)/2, pair slot s = 4*m + row/8 + 2*(col/8), half e = col%2 (the
 *                      m16n8k16 A-operand ownership).  2 bit: lane word s/8, bits [16e+2k, +2) with k = s%8.
 *                      4 bit: lane word s/4, bits [16e+4k, +4) with k = s%4.  3 bit: low two bits as 2 bit,
 *                      high bit in a second section, word (s/8)/2, bit 16e + 4*(k/2) + 2*(1-(s/8)%2) + k%2.
 *                      A section of n words per lane is stored as planes of up to four words per lane
 *                      (plane p = words [4p, 4p+4)), lane l's words of a plane of width w at word w*l.
 *   k_scale, k_zero  : float [u][max_seq/G][D]   -- scale, zero of Eq. 10-11 per channel per token group.
 *   v_scale, v_zero  : float [u][max_seq][D/Gv]  -- per token per channel group, Gv = min(G, D).
 *   k_tail           : fp16 [u][G][D]; row p % G holds the key of token p until its group is complete.
 *   sink_k, sink_v   : fp16 [u][capacity][D]; slot j holds the exact rows of token sink_pos[b][j].
 *   sink_bitmask     : uint32 [B][ceil(max_seq/32)]; bit p%32 of word p/32 is set iff token p is a sink.
 *   sink_pos         : int32 [B][capacity] ascending, -1 beyond sink_count[b].  sink_count: int32 [B].
 *                      The three sink arrays may be shared by the caches of all layers.
 *   status           : int32 [1], OR of KVSINK_STATUS_* bits raised by kernels.
 *   seq_len          : tokens in the cache (host field, the same for every sequence); advanced by
 *                      kvsink_quantize_append.
 * Fields of tokens that were never appended are unspecified.
 */
typedef struct kvsink_cache {
    uint8_t *k_codes, *v_codes;
    float *k_scale, *k_zero, *v_scale, *v_zero;
    void *k_tail;
    void *sink_k, *sink_v;
    uint32_t *sink_bitmask;
    int32_t *sink_pos, *sink_count;
    int32_t *status;
    int32_t seq_len;
} kvsink_cache;

typedef struct kvsink_sizes {
    int64_t k_codes_bytes, v_codes_bytes;   /* each of k_codes, v_codes */
    int64_t k_param_floats, v_param_floats; /* floats in each of scale and zero */
    int64_t k_tail_halfs, sink_halfs;       /* fp16 elements; sink_halfs for each of sink_k, sink_v */
    int64_t bitmask_words, sink_pos_ints;
    int64_t predict_workspace_bytes;        /* for kvsink_predict_sinks with S == max_seq */
    int64_t decode_workspace_bytes;         /* for kvsink_decode_attention and its _calibrated and _pertoken forms */
    int64_t calibrate_workspace_bytes;      /* for kvsink_calibrate */
    int32_t sink_capacity, v_group, v_groups_per_row, tile_bytes;
} kvsink_sizes;

/*
 * Buffer sizes for a configuration (host only, no CUDA call).  With scale/zero and the position index left
 * out, k_codes_bytes + v_codes_bytes per layer and 2 * D * Hkv * 2 bytes per preserved token per layer are
 * the "KV cache memory" columns of the paper's efficiency table (Appendix F).
 */
int kvsink_cache_sizes(const kvsink_config *cfg, kvsink_sizes *out);

/*
 * Sink-token prediction (Algorithm 1, the branch taken at the emergence layer; Section 4.3 items (1)-(4)).
 * score[b][i] = max over the listed channels of |hidden[b][i][c]|; per sequence the k = topk tokens of
 * largest score are selected, ties going to the lower index; the first pfn_n tokens are OR'd in.
 *   hidden     device, fp16, element (b, i, c) at hidden + b*stride_b + i*stride_s + c (strides in elements).
 *   S          tokens per sequence, 0 <= S <= max_seq.
 *   bitmask    device out, uint32 [B][ceil(max_seq/32)], every word rewritten.
 *   sink_pos   device out, int32 [B][topk+pfn_n], ascending, -1 padded.   sink_count  device out, int32 [B].
 *   workspace  device scratch of at least kvsink_sizes.predict_workspace_bytes, 16-byte aligned.
 */
int kvsink_predict_sinks(const kvsink_config *cfg, const void *hidden, int32_t S, int64_t stride_b, int64_t stride_s,
                         uint32_t *bitmask, int32_t *sink_pos, int32_t *sink_count, void *workspace,
                         size_t workspace_bytes, void *cuda_stream);

/*
 * Append T tokens per sequence to the cache (Eq. 6) and quantize them (Eq. 8-11) with sink exclusion
 * (Algorithm 1, the two "quantize" statements): tokens whose mask bit is set keep exact fp16 K and V rows in
 * the side buffer and take no part in any group's min/max; every other value is coded as
 * clamp(rint(x/scale) + zero, 0, 2^bits - 1) with scale = (max-min)/(2^bits-1), zero = -rint(min/scale) in
 * IEEE binary32 (a constant group takes scale = |min|, or 1 when min is 0; a group of sink tokens only takes
 * scale = zero = 0).  Values are coded on arrival; a key waits in k_tail until its G-token group is complete.
 *   k_new, v_new  device, fp16, element (b, h, t, c) at base + b*stride_b + h*stride_h + t*stride_t + c;
 *                 strides in elements, multiples of 8; both tensors share the strides.
 *   T             any T >= 0 at any time (prefill, chunked prefill, one decode token): a chunk may start and end inside
 *                 a key group; the result is the same as appending its tokens one by one.
 * On success cache->seq_len (host) is advanced by T.
 */
int kvsink_quantize_append(const kvsink_config *cfg, kvsink_cache *cache, const void *k_new, const void *v_new, int32_t T,
                           int64_t stride_b, int64_t stride_h, int64_t stride_t, void *cuda_stream);

/*
 * Single-token decode attention over the whole cache (Eq. 3 with Eq. 7's split): for query head hq, KV head
 * hq / (Hq/Hkv), scores q.k/sqrt(D) over all seq_len tokens under one softmax, where a token's K and V are
 * the fp16 side-buffer rows if it is a sink, else the dequantised codes scale*(code - zero) (K from k_tail
 * while its group is incomplete).  Accumulation is fp32.
 *   q          device, fp16 [B][Hq][D] contiguous.      out  device, float [B][Hq][D].
 *   lse        device, float [B][Hq] or NULL: natural log of the sum of exp of the scaled scores.
 *   workspace  device scratch of at least kvsink_sizes.decode_workspace_bytes, 16-byte aligned.
 */
int kvsink_decode_attention(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out, float *lse,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Attention of a chunk of prompt queries over the cache that holds their own (just quantized) keys and values -- the
 * attention statement of Algorithm 1, which follows its two quantize statements; Eq. 3 with a causal mask, Eq. 7's split.
 * Query token t of the chunk (t = 0 .. T-1) sits at position q_pos0 + t and attends to the cached tokens 0 .. q_pos0 + t,
 * read exactly as kvsink_decode_attention reads them.  Call it after kvsink_quantize_append of the same chunk:
 * 0 <= q_pos0 and q_pos0 + T <= seq_len.
 *   q     device, fp16, element (b, hq, t, c) at q + b*stride_b + hq*stride_h + t*stride_t + c (strides in elements,
 *         multiples of 8).
 *   out   device out, float [B][Hq][T][D].      lse  device out, float [B][Hq][T] or NULL.
 * No workspace: every block of eight (query token, query head) rows streams its own prefix of the cache.
 */
int kvsink_prefill_attention(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, int32_t T, int32_t q_pos0, int64_t stride_b,
                             int64_t stride_h, int64_t stride_t, float *out, float *lse, void *cuda_stream);

/*
 * kvsink_decode_attention for callers that cannot allocate device memory.  (No counterpart in the paper: this is
 * a deployment convenience of this library.)
 *
 * Some hosts of this code may not call cudaMalloc at all: a plug-in that runs inside another engine's memory
 * plan, a real-time loop that forbids allocation after start-up, a process that was handed a fixed set of
 * buffers.  They can provide q, the cache and out (they own those anyway) but have nowhere to get the
 * split-partial workspace from.  This entry point computes exactly what kvsink_decode_attention computes, with
 * the same kernels, and keeps the partials in an array of KVSINK_STATIC_SCRATCH_BYTES that is part of the
 * library image: every GPU on which the library is loaded holds that memory until the process exits.  It calls
 * no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   - Arguments are those of kvsink_decode_attention without workspace / workspace_bytes.
 *   - Limit: kvsink_sizes.decode_workspace_bytes of the configuration must not exceed
 *     KVSINK_STATIC_SCRATCH_BYTES, otherwise KVSINK_ERR_STATIC_SCRATCH is returned and nothing is launched
 *     (use kvsink_decode_attention with your own workspace then).
 *   - The first call on each device looks up the array's device address (a CUDA runtime query, made with that
 *     device current, no allocation).  Make that first call outside of any stream capture.  The address is kept for
 *     the life of the device's primary context: after cudaDeviceReset (or anything else that destroys that context)
 *     the cached address is stale and this entry point must not be used again in the process.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it.  Nothing in
 *     it has to start at zero -- each call overwrites every record it later reads -- but two calls whose kernels
 *     overlap on the GPU (different streams, no ordering between them) race on it and corrupt each other's
 *     result.  Calls on one stream, or otherwise ordered, are safe.
 */
int kvsink_decode_attention_static(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out, float *lse,
                                   void *cuda_stream);

/*
 * Static (calibrated) parameters: the scheme of the paper's main comparison -- keys per channel, values per token, static
 * (Section 5.1) -- with sink tokens left out of the calibration as well as of the quantization (Algorithm 1's remark on
 * calibration; Section 4.1; Appendix C "Dynamic and static quantization").  One (scale, zero) pair per key channel and one
 * per value channel group of every KV head serves every token of every sequence.  All four arrays are device memory owned
 * by the caller: k_scale, k_zero float [Hkv][D]; v_scale, v_zero float [Hkv][D / min(G, D)].
 */
typedef struct kvsink_static_params {
    float *k_scale, *k_zero;
    float *v_scale, *v_zero;
} kvsink_static_params;

/*
 * Calibration: global min / max (the caption of the paper's error table) of every key channel and every value channel
 * group over a calibration batch, all sequences and all tokens whose mask bit is clear, then Eq. 10-11 (a single value
 * takes scale = |min|, or 1 for 0; no member at all takes scale = zero = 0).
 *   k_cal, v_cal  device, fp16 [B][Hkv][T][D] with element strides (multiples of 8), 0 <= T <= max_seq.
 *   sink_bitmask  device, uint32 [B][ceil(max_seq/32)]: the calibration batch's sink tokens (kvsink_predict_sinks).
 *   params        the four arrays of *params are rewritten.
 *   workspace     device scratch of at least kvsink_sizes.calibrate_workspace_bytes, 16-byte aligned.
 */
int kvsink_calibrate(const kvsink_config *cfg, const void *k_cal, const void *v_cal, int32_t T, int64_t stride_b, int64_t stride_h,
                     int64_t stride_t, const uint32_t *sink_bitmask, const kvsink_static_params *params, void *workspace,
                     size_t workspace_bytes, void *cuda_stream);

/*
 * kvsink_quantize_append with static parameters (Eq. 6, Eq. 8): every token is coded on arrival, keys per channel and
 * values per channel group, as clamp(rint(x/scale) + zero, 0, 2^bits - 1) -- values outside the calibrated range clamp, a
 * pair with scale 0 gives code 0; tokens whose mask bit is set keep exact fp16 rows in the side buffer and code 0.  There is
 * no key tail and there are no per-group parameters: cache->k_scale, k_zero, v_scale, v_zero and k_tail are not used and
 * may be null.  Any T >= 0 at any time.  A cache is used with one kind of parameters only.
 */
int kvsink_quantize_append_calibrated(const kvsink_config *cfg, kvsink_cache *cache, const kvsink_static_params *params, const void *k_new,
                                      const void *v_new, int32_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t, void *cuda_stream);

/*
 * kvsink_decode_attention over a cache written by kvsink_quantize_append_calibrated (Eq. 3, Eq. 7): a sink token's K and V
 * are its fp16 side-buffer rows, every other token's are scale * (code - zero) with the static pairs.  Head size 128 with
 * one or two value groups per row; other shapes return KVSINK_ERR_UNSUPPORTED.
 */
int kvsink_decode_attention_calibrated(const kvsink_config *cfg, const kvsink_cache *cache, const kvsink_static_params *params, const void *q,
                                       float *out, float *lse, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Per-token keys (Section 4.1, "Per-token quantization"; the per-token Key and Value dynamic scheme of Section 5.1's
 * evaluation with KVQuant's granularities): keys are quantized like values, one (scale, zero) of Eq. 10-11 per token and
 * channel group of min(G, D) channels.  In a cache used this way k_scale and k_zero are float [u][max_seq][D/Gv] (the
 * shape of v_scale; kvsink_sizes.v_param_floats floats each) and k_tail is not used and may be null.
 *
 * kvsink_quantize_append_pertoken: every token is coded on arrival (any T >= 0 at any time); a token whose mask bit is set
 * keeps exact fp16 rows in the side buffer, gets code 0 everywhere and scale = zero = 0.  Arguments, strides, ownership
 * and errors as kvsink_quantize_append.
 *
 * kvsink_decode_attention_pertoken: Eq. 3 / Eq. 7 over such a cache; arguments as kvsink_decode_attention.
 *
 * Both are built for head size 128, one or two channel groups per row and at most four query heads per KV head (3 bit:
 * one group and one query head); other shapes return KVSINK_ERR_UNSUPPORTED.  A cache is used with one kind of parameters
 * only.
 */
int kvsink_quantize_append_pertoken(const kvsink_config *cfg, kvsink_cache *cache, const void *k_new, const void *v_new, int32_t T,
                                    int64_t stride_b, int64_t stride_h, int64_t stride_t, void *cuda_stream);
int kvsink_decode_attention_pertoken(const kvsink_config *cfg, const kvsink_cache *cache, const void *q, float *out, float *lse,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Largest magnitude of every hidden channel over all tokens of all sequences: out[c] = max |hidden[b][i][c]| (a NaN
 * never raises a maximum).  This is the scan from which a model's outlier channels -- the `channels` of kvsink_config --
 * and the layer where they emerge are read off (Section 3.1; Appendix D, the table of emergence layers and outlier
 * channels): the few channels whose maximum stands orders of magnitude above the rest.
 *   hidden   device, fp16, element (b, i, c) at hidden + b*stride_b + i*stride_s + c (strides in elements).
 *   out      device out, float [d], every entry rewritten.
 */
int kvsink_channel_absmax(const void *hidden, int32_t B, int32_t S, int32_t d, int64_t stride_b, int64_t stride_s, float *out,
                          void *cuda_stream);

/*
 * Quantization error in the shape of the paper's error table (Section 4.1, Table 1): round-to-nearest asymmetric
 * quantization (Eq. 8-11) of x, squared error against the dequantised value (Eq. 9), summed separately over the
 * quantization groups without a sink token and over those with at least one.
 *   x              device, fp16 [B][Hkv][T][D] with element strides (multiples of 8), 0 <= T <= max_seq.
 *   per_channel    nonzero: groups of G consecutive tokens of one channel (a last shorter group takes the rest);
 *                  zero: groups of min(G, D) consecutive channels of one token.
 *   exclude_sinks  zero: plain quantization, every token takes part in its group's min / max (the table's dynamic rows);
 *                  nonzero: sink tokens take no part in the statistics and are not quantized or counted (KVSink).
 *   sink_bitmask   device, uint32 [B][ceil(max_seq/32)].
 *   out            device out, double [4]: sum of squared errors and element count over groups without a sink token,
 *                  then the same over groups with one.  Sums are accumulated in binary64 in no fixed order.
 */
int kvsink_quant_error(const kvsink_config *cfg, const void *x, int32_t T, int64_t stride_b, int64_t stride_h, int64_t stride_t,
                       int32_t per_channel, int32_t exclude_sinks, const uint32_t *sink_bitmask, double *out, void *cuda_stream);

/* Copies the device status word to *host_status and waits for the stream (the only call that synchronises).  Returns
 * KVSINK_OK for a zero word, else the error code of the most severe raised bit (TIMEOUT, BOUNDS, SINK_MISMATCH);
 * *host_status holds the word either way. */
int kvsink_read_status(const kvsink_cache *cache, int32_t *host_status, void *cuda_stream);

/* Kernel launches the library has made in this process since it was loaded (host counter; every entry point adds the
 * kernels it launched).  For accounting in benchmarks and tests; not a step of the paper's method. */
unsigned long long kvsink_launch_count(void);

/* Static text for a status code. */
const char *kvsink_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* KVSINK_H_ */
