// Analysis kernels: the per-channel magnitude scan of a hidden state (how a model's outlier channels and the layer where
// they emerge are found: Section 3.1, Appendix D) and the quantization error split by groups with and without sink
// tokens (Section 4.1, Table 1).  Both read their input once and are bound by HBM bandwidth.
#include "common.cuh"

namespace kvsink {
namespace {

// ---- channel scan ----
// |x| of two fp16 values as their 15-bit patterns; a NaN (pattern above 0x7c00) counts as 0, as in the reference
// comparison `|x| > best`, which is false for a NaN.
__device__ __forceinline__ uint32_t magnitude2(uint32_t h2)
{
    const uint32_t a = h2 & 0x7fff7fffu;
    return a & ~__vcmpgtu2(a, 0x7c007c00u);
}
// The binary32 bit pattern of a non-negative fp16 pattern: non-negative floats order as unsigned integers.
__device__ __forceinline__ unsigned float_bits_of_half_pattern(unsigned h) { return __float_as_uint(__half2float(__ushort_as_half((unsigned short)h))); }

// grid (channel blocks, token slices); thread = eight consecutive channels, walking over the tokens of its slice.
__global__ void __launch_bounds__(256)
channel_absmax_kernel(const uint16_t *__restrict__ H, long long n_tokens, int S, int d, int64_t sb, int64_t ss, unsigned *__restrict__ out_bits)
{
    const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * 8;
    pdl_wait();
    if (c0 >= d) return;
    uint32_t best[4] = {0u, 0u, 0u, 0u};
    for (long long tok = blockIdx.y; tok < n_tokens; tok += gridDim.y) {
        const long long b = tok / S, i = tok - b * S;
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(H + b * sb + i * ss + c0));
        best[0] = __vmaxu2(best[0], magnitude2(v.x));
        best[1] = __vmaxu2(best[1], magnitude2(v.y));
        best[2] = __vmaxu2(best[2], magnitude2(v.z));
        best[3] = __vmaxu2(best[3], magnitude2(v.w));
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (best[j] & 0xffffu) atomicMax(out_bits + c0 + 2 * j, float_bits_of_half_pattern(best[j] & 0xffffu));
        if (best[j] >> 16) atomicMax(out_bits + c0 + 2 * j + 1, float_bits_of_half_pattern(best[j] >> 16));
    }
}

// Any width, any alignment: one thread per channel.
__global__ void __launch_bounds__(256)
channel_absmax_generic_kernel(const uint16_t *__restrict__ H, long long n_tokens, int S, int d, int64_t sb, int64_t ss,
                              unsigned *__restrict__ out_bits)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (c >= d) return;
    unsigned best = 0;
    for (long long tok = blockIdx.y; tok < n_tokens; tok += gridDim.y) {
        const long long b = tok / S, i = tok - b * S;
        unsigned a = __ldg(H + b * sb + i * ss + c) & 0x7fffu;
        a = a > 0x7c00u ? 0u : a;
        best = a > best ? a : best;
    }
    if (best) atomicMax(out_bits + c, float_bits_of_half_pattern(best));
}

// ---- quantization error ----
constexpr int QE_THREADS = 128;

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Squared error of one element under its group's parameters: Eq. 8, Eq. 9 in binary32, the difference in binary64.
__device__ __forceinline__ double element_error(float x, float s, float z, float qmax)
{
    const uint32_t code = code_exact(x, s, z, qmax);
    const float xq = __fmul_rn(s, __fsub_rn((float)code, z));
    const double e = (double)x - (double)xq;
    return e * e;
}

// Per channel over groups of G tokens: a block stages one (sequence, KV head, token group) tile of G x D values and
// thread c owns channel c.  The blocks walk over the items; sums stay in registers until the end.
__global__ void __launch_bounds__(QE_THREADS)
quant_error_per_channel_kernel(Params p, const __half *__restrict__ x, int T, int64_t sb, int64_t sh, int64_t stt, int exclude_sinks,
                               const uint32_t *__restrict__ bitmask, double *__restrict__ out)
{
    extern __shared__ __align__(16) unsigned char qe_smem[];
    __half *tile = reinterpret_cast<__half *>(qe_smem);                 // [G][D]
    __shared__ double red[4][QE_THREADS / 32];
    const int D = p.D, G = p.G, tid = threadIdx.x;
    const float qmax = (float)((1 << p.bits) - 1);
    const int groups = (T + G - 1) / G;
    const long long items = (long long)p.B * p.Hkv * groups;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    pdl_wait();
    for (long long it = blockIdx.x; it < items; it += gridDim.x) {
        const int grp = (int)(it % groups);
        const long long unit = it / groups;
        const int h = (int)(unit % p.Hkv), b = (int)(unit / p.Hkv);
        const int t0 = grp * G, n = min(G, T - t0);
        const uint32_t *bm = bitmask + (size_t)b * p.mask_words;
        __syncthreads();                                                // the previous item's tile is no longer read
        for (int i = tid; i < n * (D / 8); i += QE_THREADS) {
            const int r = i / (D / 8), c8 = i % (D / 8);
            *reinterpret_cast<uint4 *>(tile + r * D + c8 * 8) =
                __ldg(reinterpret_cast<const uint4 *>(x + b * sb + h * sh + (int64_t)(t0 + r) * stt + c8 * 8));
        }
        bool has_sink = false;
        for (int t = 0; t < n; ++t) has_sink |= mask_bit(bm, t0 + t);
        __syncthreads();
        for (int c = tid; c < D; c += QE_THREADS) {
            bool any = false;
            float mn = 0.f, mx = 0.f;
            for (int t = 0; t < n; ++t) {
                if (exclude_sinks && mask_bit(bm, t0 + t)) continue;
                const float v = __half2float(tile[t * D + c]);
                if (!any) { mn = mx = v; any = true; }
                else { mn = fminf(mn, v); mx = fmaxf(mx, v); }
            }
            float s, z;
            group_params(any, mn, mx, qmax, &s, &z);
            double e = 0.0;
            int cnt = 0;
            for (int t = 0; t < n; ++t) {
                if (exclude_sinks && mask_bit(bm, t0 + t)) continue;
                e += element_error(__half2float(tile[t * D + c]), s, z, qmax);
                ++cnt;
            }
            acc[has_sink ? 2 : 0] += e;
            acc[has_sink ? 3 : 1] += (double)cnt;
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const double v = warp_sum_d(acc[k]);
        if ((tid & 31) == 0) red[k][tid >> 5] = v;
    }
    __syncthreads();
    if (tid < 4) {
        double v = 0.0;
        for (int w = 0; w < QE_THREADS / 32; ++w) v += red[tid][w];
        if (v != 0.0) atomicAdd(out + tid, v);
    }
}

// Per token over groups of Gv channels: one warp per token, D / 32 channels per lane.
__global__ void __launch_bounds__(QE_THREADS)
quant_error_per_token_kernel(Params p, const __half *__restrict__ x, int T, int64_t sb, int64_t sh, int64_t stt, int exclude_sinks,
                             const uint32_t *__restrict__ bitmask, double *__restrict__ out)
{
    __shared__ double red[4][QE_THREADS / 32];
    const int D = p.D, tid = threadIdx.x, lane = tid & 31, cpl = D / 32;
    const float qmax = (float)((1 << p.bits) - 1);
    const long long tokens = (long long)p.B * p.Hkv * T;
    const long long warps = (long long)gridDim.x * (QE_THREADS / 32);
    const int lanes_per_group = p.Gv / cpl;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    pdl_wait();
    for (long long it = (long long)blockIdx.x * (QE_THREADS / 32) + (tid >> 5); it < tokens; it += warps) {
        const int t = (int)(it % T);
        const long long unit = it / T;
        const int h = (int)(unit % p.Hkv), b = (int)(unit / p.Hkv);
        const bool sink = mask_bit(bitmask + (size_t)b * p.mask_words, t);
        if (sink && exclude_sinks) continue;
        float v[4];
        const __half *row = x + b * sb + h * sh + (int64_t)t * stt + lane * cpl;
        for (int e = 0; e < cpl; ++e) v[e] = __half2float(row[e]);
        float mn = v[0], mx = v[0];
        for (int e = 1; e < cpl; ++e) { mn = fminf(mn, v[e]); mx = fmaxf(mx, v[e]); }
        for (int o = 1; o < lanes_per_group; o <<= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        float s, z;
        group_params(true, mn, mx, qmax, &s, &z);
        double e2 = 0.0;
        for (int e = 0; e < cpl; ++e) e2 += element_error(v[e], s, z, qmax);
        acc[sink ? 2 : 0] += e2;
        acc[sink ? 3 : 1] += (double)cpl;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const double v = warp_sum_d(acc[k]);
        if (lane == 0) red[k][tid >> 5] = v;
    }
    __syncthreads();
    if (tid < 4) {
        double v = 0.0;
        for (int w = 0; w < QE_THREADS / 32; ++w) v += red[tid][w];
        if (v != 0.0) atomicAdd(out + tid, v);
    }
}

}  // namespace

int launch_channel_absmax(const __half *hidden, int B, int S, int d, int64_t sb, int64_t ss, float *out, cudaStream_t st)
{
    if (cudaMemsetAsync(out, 0, sizeof(float) * (size_t)d, st) != cudaSuccess) return KVSINK_ERR_CUDA;
    const long long n_tokens = (long long)B * S;
    if (n_tokens == 0) return KVSINK_OK;
    const bool wide = d % 8 == 0 && sb % 8 == 0 && ss % 8 == 0 && ((uintptr_t)hidden & 15u) == 0;
    const int per_block = wide ? 256 * 8 : 256;
    const unsigned gx = (unsigned)((d + per_block - 1) / per_block);
    long long gy = (148 * 16 + gx - 1) / gx;          // about sixteen blocks per multiprocessor
    if (gy > n_tokens) gy = n_tokens;
    if (gy > 65535) gy = 65535;
    const dim3 grid(gx, (unsigned)gy);
    cudaError_t e = wide ? launch_pdl(channel_absmax_kernel, grid, dim3(256), 0, st, (const uint16_t *)hidden, n_tokens, S, d, sb, ss, (unsigned *)out)
                         : launch_pdl(channel_absmax_generic_kernel, grid, dim3(256), 0, st, (const uint16_t *)hidden, n_tokens, S, d, sb, ss,
                                      (unsigned *)out);
    return e == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

int launch_quant_error(const Params &p, const __half *x, int T, int64_t sb, int64_t sh, int64_t stt, bool per_channel, bool exclude_sinks,
                       const uint32_t *bitmask, double *out, cudaStream_t st)
{
    if (cudaMemsetAsync(out, 0, 4 * sizeof(double), st) != cudaSuccess) return KVSINK_ERR_CUDA;
    if (T == 0) return KVSINK_OK;
    cudaError_t e;
    if (per_channel) {
        const size_t smem = (size_t)p.G * p.D * sizeof(__half);
        if (smem > 160 * 1024) return KVSINK_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(quant_error_per_channel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return KVSINK_ERR_CUDA;
        const long long items = (long long)p.B * p.Hkv * ((T + p.G - 1) / p.G);
        const unsigned blocks = (unsigned)(items < 148 * 6 ? items : 148 * 6);
        e = launch_pdl(quant_error_per_channel_kernel, dim3(blocks), dim3(QE_THREADS), smem, st, p, x, T, sb, sh, stt, (int)exclude_sinks, bitmask, out);
    } else {
        const long long tokens = (long long)p.B * p.Hkv * T;
        const long long want = (tokens + QE_THREADS / 32 - 1) / (QE_THREADS / 32);
        const unsigned blocks = (unsigned)(want < 148 * 16 ? want : 148 * 16);
        e = launch_pdl(quant_error_per_token_kernel, dim3(blocks), dim3(QE_THREADS), 0, st, p, x, T, sb, sh, stt, (int)exclude_sinks, bitmask, out);
    }
    return e == cudaSuccess ? KVSINK_OK : KVSINK_ERR_CUDA;
}

}  // namespace kvsink
