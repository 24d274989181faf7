// Decode attention, host side: split heuristic, merge of the sequence splits, dispatch over the code width, and the
// entry point that keeps its scratch inside the library image.  The split kernel itself is in decode_kernel.cuh.
#include <mutex>

#include "common.cuh"

namespace kvsink {

// Merge of the sequence splits (more than eight per unit): one block per (sequence, query head); thread (ch, sl) folds the
// records sl, sl + MERGE_SLICES, ... of channel ch, and the slices are combined in a fixed order (bit-reproducible).
constexpr int MERGE_SLICES = 4;

__global__ void decode_merge_kernel(const float *__restrict__ part_ws, int nsplit, int D, float *__restrict__ out, float *__restrict__ lse)
{
    __shared__ float sh_acc[MERGE_SLICES][128], sh_m[MERGE_SLICES], sh_l[MERGE_SLICES];
    const int PS = D + 2;
    const size_t oq = blockIdx.x;
    const int ch = threadIdx.x, sl = threadIdx.y;
    const float *base = part_ws + oq * nsplit * PS;
    // launched with programmatic stream serialization: the blocks may start while the split kernel drains, and wait
    // here until all of it has completed and its records are visible
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float M = M_INIT;
    for (int s = sl; s < nsplit; s += MERGE_SLICES) M = fmaxf(M, base[(size_t)s * PS + D]);
    float acc = 0.f, L = 0.f;
    for (int s = sl; s < nsplit; s += MERGE_SLICES) {
        const float f = ex2(base[(size_t)s * PS + D] - M);
        acc += base[(size_t)s * PS + ch] * f;
        L += base[(size_t)s * PS + D + 1] * f;
    }
    sh_acc[sl][ch] = acc;
    if (ch == 0) { sh_m[sl] = M; sh_l[sl] = L; }
    __syncthreads();
    if (sl != 0) return;
    float Mt = M_INIT;
#pragma unroll
    for (int i = 0; i < MERGE_SLICES; ++i) Mt = fmaxf(Mt, sh_m[i]);
    float at = 0.f, Lt = 0.f;
#pragma unroll
    for (int i = 0; i < MERGE_SLICES; ++i) {
        const float f = ex2(sh_m[i] - Mt);
        at += sh_acc[i][ch] * f;
        Lt += sh_l[i] * f;
    }
    out[oq * D + ch] = Lt > 0.f ? at / Lt : 0.f;
    if (lse && ch == 0) lse[oq] = Lt > 0.f ? (Mt + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
}

int launch_decode_merge(const float *ws, int nsplit, int D, int n_rows, float *out, float *lse, cudaStream_t st)
{
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_rows);
    cfg.blockDim = dim3(D, MERGE_SLICES);
    cfg.stream = st;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_merge_kernel, ws, nsplit, D, out, lse) != cudaSuccess) return KVSINK_ERR_CUDA;
    note_launch();
    return KVSINK_OK;
}

// ---- host side ----
constexpr int DEC_SLOTS = 148 * 4;   // resident blocks the split heuristic plans for

int max_splits(const Params &p)
{
    const int qchunks = decode_qchunks(p);
    const long units = (long)p.B * p.Hkv * qchunks;
    long ns = (2L * DEC_SLOTS + units - 1) / units;
    const long mg = p.max_seq / p.G;
    if (ns > mg) ns = mg;
    return (int)(ns < 1 ? 1 : ns);
}

int choose_splits(const Params &p, int n_groups)
{
    const int qchunks = decode_qchunks(p);
    const long units = (long)p.B * p.Hkv * qchunks;
    const int ns_max = max_splits(p) < n_groups ? max_splits(p) : (n_groups > 0 ? n_groups : 1);
    int best = 1;
    double best_cost = 1e300;
    for (int ns = 1; ns <= ns_max; ++ns) {
        const long waves = (units * ns + DEC_SLOTS - 1) / DEC_SLOTS;
        const int per_block = (n_groups + ns - 1) / ns;
        const int per_warp = (per_block + DEC_WARPS - 1) / DEC_WARPS;
        const double cost = (double)waves * (per_warp + 0.5);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = ns; }
    }
    return best;
}

size_t decode_workspace_bytes(const Params &p)
{
    return (size_t)p.B * p.Hq * max_splits(p) * (p.D + 2) * sizeof(float) + 16;
}

int launch_decode(const Params &p, const kvsink_cache &c, const kvsink_static_params *cal, int mode, const __half *q, float *out, float *lse, void *workspace,
                  size_t workspace_bytes, cudaStream_t st)
{
    if (workspace_bytes < decode_workspace_bytes(p)) return KVSINK_ERR_WORKSPACE;
    float *ws = (float *)workspace;
    if (p.bits == 2) return launch_decode_b2(p, c, cal, mode, q, out, lse, ws, st);
    if (p.bits == 3) return launch_decode_b3(p, c, cal, mode, q, out, lse, ws, st);
    if (p.bits == 4) return launch_decode_b4(p, c, cal, mode, q, out, lse, ws, st);
    return KVSINK_ERR_UNSUPPORTED;
}

// ---------------------------------------------------------------------------------------------------------
// Decode attention without caller-provided scratch: the split partials live in a fixed array inside the library
// image.  Every GPU that loads the library holds these KVSINK_STATIC_SCRATCH_BYTES until the process exits.
// ---------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_decode_scratch[KVSINK_STATIC_SCRATCH_BYTES];

// In host code `g_decode_scratch` is only a handle for the runtime, not a device address; the address is looked
// up once per device (with that device current) and cached.
static void *g_scratch_ptr[64];
static bool g_scratch_known[64];
static std::mutex g_scratch_mutex;

int launch_decode_static(const Params &p, const kvsink_cache &c, const __half *q, float *out, float *lse, cudaStream_t st)
{
    if (decode_workspace_bytes(p) > (size_t)KVSINK_STATIC_SCRATCH_BYTES) return KVSINK_ERR_STATIC_SCRATCH;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KVSINK_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_scratch_mutex);
    if (!g_scratch_known[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_decode_scratch) != cudaSuccess || ptr == nullptr) return KVSINK_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
        g_scratch_known[dev] = true;
    }
    // No clearing is needed: the split kernel writes every partial record the merge kernel reads.
    return launch_decode(p, c, nullptr, 0, q, out, lse, g_scratch_ptr[dev], (size_t)KVSINK_STATIC_SCRATCH_BYTES, st);
}

}  // namespace kvsink
