// Decode attention kernels for 4-bit codes (see decode_kernel.cuh).
#include "decode_kernel.cuh"

namespace kvsink {

int launch_decode_b4(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, const __half *q, float *out, float *lse, float *ws,
                     cudaStream_t st)
{
    return launch_decode_bits<4>(p, c, cal, q, out, lse, ws, st);
}

}  // namespace kvsink
