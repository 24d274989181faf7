// Decode attention kernels for 2-bit codes (see decode_kernel.cuh).
#include "decode_kernel.cuh"

namespace kvsink {

int launch_decode_b2(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st)
{
    return launch_decode_bits<2>(p, c, cal, mode, q, out, lse, ws, st);
}

int launch_prefill_b2(const Params &p, const kvsink_cache &c, const __half *q, int T, int q_pos0, int64_t sb, int64_t sh, int64_t stt, float *out,
                      float *lse, cudaStream_t st)
{
    return launch_prefill_bits<2>(p, c, q, T, q_pos0, sb, sh, stt, out, lse, st);
}

}  // namespace kvsink
