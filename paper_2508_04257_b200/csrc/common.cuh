// Shared definitions for the libkvsink kernels (device + host).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/kvsink.h"

namespace kvsink {

// Derived, validated problem parameters passed to kernels by value.
struct Params {
    int B, Hq, Hkv, D, hidden;
    int bits, G, max_seq, topk, pfn_n, cap;
    int Gv, NGv;        // value channel-group size and groups per row
    int rep;            // query heads per KV head
    int tile_bytes;     // bytes of one packed 16-token tile
    int row_bytes;      // D * bits / 8
    int mask_words;     // bitmask words per sequence
    int n_channels;
    int channels[8];
};

// ---- physical order of codes inside a 16-token tile (see kvsink.h, kvsink_cache) ----
// Word i of lane `lane` inside a section of n words per lane stored as planes of up to four words per lane.
__host__ __device__ inline int section_word_offset(int n, int lane, int i)
{
    int off = 0, p = i >> 2;
    for (int pp = 0; pp < p; ++pp) {
        int u = n - 4 * pp;
        off += 32 * (u > 4 ? 4 : u);
    }
    int u = n - 4 * p;
    if (u > 4) u = 4;
    return off + u * lane + (i - 4 * p);
}

// Inverse: physical word offset inside a section -> (lane, i).
__host__ __device__ inline void section_word_owner(int n, int off, int *lane, int *i)
{
    int p = 0;
    for (;;) {
        int u = n - 4 * p;
        if (u > 4) u = 4;
        if (off < 32 * u) {
            *lane = off / u;
            *i = 4 * p + off % u;
            return;
        }
        off -= 32 * u;
        ++p;
    }
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Eq. 10-11 for one group from its exact fp16 extremes; all operations IEEE binary32, round to nearest even.
// any == false (no member) gives scale = zero = 0.
__device__ __forceinline__ void group_params(bool any, float mn, float mx, float qmax, float *scale, float *zero)
{
    if (!any) {
        *scale = 0.0f;
        *zero = 0.0f;
        return;
    }
    float r = __fsub_rn(mx, mn);
    float s;
    if (r == 0.0f) s = (mn == 0.0f) ? 1.0f : fabsf(mn);
    else s = __fdiv_rn(r, qmax);
    *scale = s;
    *zero = __fsub_rn(0.0f, rintf(__fdiv_rn(mn, s)));
}

// Eq. 8 for one value (exact form: IEEE division, rint, clamp).
__device__ __forceinline__ uint32_t code_exact(float x, float scale, float zero, float qmax)
{
    float q = __fadd_rn(rintf(__fdiv_rn(x, scale)), zero);
    q = fminf(fmaxf(q, 0.0f), qmax);
    return (uint32_t)(int)q;
}

// Programmatic stream serialization (dependent launch).  A kernel launched with launch_pdl may be scheduled while its
// predecessor in the stream is still draining; it must call pdl_wait() before it reads or writes anything a predecessor
// may have touched.  pdl_wait() returns once every prerequisite grid has completed and its writes are visible (at once
// when the kernel was launched the ordinary way).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Kernel launches made by the library since it was loaded (kvsink_launch_count).
extern std::atomic<unsigned long long> g_launches;
inline void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch();
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Decode attention: warps per block, the "no score yet" value of a running maximum, and 2^x.
constexpr int DEC_WARPS = 4;
constexpr float M_INIT = -1.0e30f;
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Index checks of debug builds (-DKVSINK_DEBUG): a failed check raises KVSINK_STATUS_BOUNDS in the cache's status word and
// returns false, and the caller skips the guarded work; nothing traps.  Release builds compile the condition away.
#ifdef KVSINK_DEBUG
__device__ __forceinline__ bool in_bounds(bool ok, int32_t *status)
{
    if (!ok) atomicOr(status, KVSINK_STATUS_BOUNDS);
    return ok;
}
#else
__device__ __forceinline__ bool in_bounds(bool, int32_t *) { return true; }
#endif

__device__ __forceinline__ bool mask_bit(const uint32_t *__restrict__ bm, int pos) { return (bm[pos >> 5] >> (pos & 31)) & 1u; }

// Launchers implemented in the kernel translation units; all return a KVSINK_* code.
int launch_predict_sinks(const Params &p, const __half *hidden, int S, int64_t stride_b, int64_t stride_s, uint32_t *bitmask,
                         int32_t *sink_pos, int32_t *sink_count, void *workspace, cudaStream_t st);
int launch_quantize_groups(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                           int n_groups, int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st);
int launch_quantize_groups_fast(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                                int n_groups, int64_t sb, int64_t sh, int64_t stt, bool do_v_and_sinks, cudaStream_t st);
int launch_quantize_groups_bulk(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token,
                                int n_groups, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
int launch_quantize_tokens(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int src_offset,
                           int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
int launch_decode(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, void *workspace,
                  size_t workspace_bytes, cudaStream_t st);
int launch_prefill_b2(const Params &p, const kvsink_cache &c, const __half *q, int T, int q_pos0, int64_t sb, int64_t sh, int64_t stt, float *out,
                      float *lse, cudaStream_t st);
int launch_prefill_b3(const Params &p, const kvsink_cache &c, const __half *q, int T, int q_pos0, int64_t sb, int64_t sh, int64_t stt, float *out,
                      float *lse, cudaStream_t st);
int launch_prefill_b4(const Params &p, const kvsink_cache &c, const __half *q, int T, int q_pos0, int64_t sb, int64_t sh, int64_t stt, float *out,
                      float *lse, cudaStream_t st);
int launch_calibrate(const Params &p, const __half *k, const __half *v, int T, int64_t sb, int64_t sh, int64_t stt, const uint32_t *bitmask,
                     const kvsink_static_params &sp, void *workspace, cudaStream_t st);
int launch_quantize_calibrated(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                               int first_token, int n_tokens, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
int launch_quantize_static_bulk(const Params &p, const kvsink_cache &c, const kvsink_static_params &sp, const __half *k_src, const __half *v_src,
                                int first_token, int n_groups, int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
int launch_quantize_pertoken_bulk(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_groups,
                                  int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
int launch_quantize_pertoken(const Params &p, const kvsink_cache &c, const __half *k_src, const __half *v_src, int first_token, int n_tokens,
                             int64_t sb, int64_t sh, int64_t stt, cudaStream_t st);
size_t calibrate_workspace_bytes(const Params &p);
int launch_decode_static(const Params &p, const kvsink_cache &c, const __half *q, float *out, float *lse, cudaStream_t st);
int launch_decode_b2(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st);
int launch_decode_b3(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st);
int launch_decode_b4(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st);
int launch_decode_merge(const float *ws, int nsplit, int D, int n_rows, float *out, float *lse, cudaStream_t st);
// Query heads of one KV head that one decode block serves, and the blocks per KV head that makes.  Up to four heads share a
// block.  Five to eight share one where a path with eight columns exists: the integer key side with two operand tables (2 and
// 4 bit, head size 128) or the eight-column fp16 path (head size 64); at 3 bit with head size 128 they go four at a time to
// the fp16 pair layout, whose residual columns the eight-column fp16 path lacks.
inline int decode_heads_per_block(const Params &p) { return p.rep <= 4 ? 4 : (p.D == 128 && p.bits == 3 ? 4 : 8); }
inline int decode_qchunks(const Params &p) { return (p.rep + decode_heads_per_block(p) - 1) / decode_heads_per_block(p); }
int max_splits(const Params &p);
int choose_splits(const Params &p, int n_groups);
int launch_channel_absmax(const __half *hidden, int B, int S, int d, int64_t sb, int64_t ss, float *out, cudaStream_t st);
int launch_quant_error(const Params &p, const __half *x, int T, int64_t sb, int64_t sh, int64_t stt, bool per_channel, bool exclude_sinks,
                       const uint32_t *bitmask, double *out, cudaStream_t st);
size_t decode_workspace_bytes(const Params &p);
size_t predict_workspace_bytes(const Params &p);

}  // namespace kvsink
