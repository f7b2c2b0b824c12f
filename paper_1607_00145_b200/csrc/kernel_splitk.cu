// Split-K reduction: the contracted index set I_k was cut into slices, each
// slice left its partial tile sums in the plan's workspace; this kernel adds the
// slices in a fixed order (so results are reproducible run to run) and performs
// the unpacking update of Eq. 11, C <- alpha * sum + beta * C, through C's own
// mode permutation.  The paper has no split-K; the nearest idea is choosing the
// GEMM variant by which of m, n, k is small (Sec. 2.1, Table I; Sec. 3.3).
#include "kernels.h"

namespace {

// ws layout: [slice][n][m] with m fastest (tile-order fused indices).
__global__ void __launch_bounds__(256) gett_splitk_reduce_kernel(const __grid_constant__ GettKernelArgs g)
{
    const uint32_t Msz = g.M.size, Nsz = g.N.size;
    const uint64_t total = (uint64_t)Msz * Nsz;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        const uint32_t n = (uint32_t)(e / Msz);
        const uint32_t m = (uint32_t)(e - (uint64_t)n * Msz);
        float s = 0.f;
        for (uint32_t z = 0; z < g.split_k; ++z)
            s += g.ws[(uint64_t)z * total + e];
        int64_t ax, cm, bx, cn;
        gett_decompose(g.M, m, ax, cm);
        gett_decompose(g.N, n, bx, cn);
        float* dst = g.C + cm + cn;
        float v = g.alpha * s;
        if (g.beta != 0.f)
            v = fmaf(g.beta, *dst, v);
        *dst = v;
    }
}

} // namespace

cudaError_t gett_launch_splitk_reduce(const GettKernelArgs& args, int sm_count, cudaStream_t stream)
{
    const uint64_t total = (uint64_t)args.M.size * args.N.size;
    uint64_t blocks = (total + 255) / 256;
    const uint64_t cap = (uint64_t)(sm_count > 0 ? sm_count : 148) * 16;
    if (blocks > cap)
        blocks = cap;
    if (blocks < 1)
        blocks = 1;
    gett_splitk_reduce_kernel<<<(unsigned)blocks, 256, 0, stream>>>(args);
    return cudaGetLastError();
}
