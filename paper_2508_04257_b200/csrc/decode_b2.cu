// Decode attention kernels for 2-bit codes (see decode_kernel.cuh).
#include "decode_kernel.cuh"

namespace kvsink {

int launch_decode_b2(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st)
{
    return launch_decode_bits<2>(p, c, cal, q, out, lse, ws, st);
}

}  // namespace kvsink
