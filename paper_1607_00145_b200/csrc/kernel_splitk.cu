// Split-K reduction: the contracted index set I_k was cut into slices, each
// slice left its partial tile sums in the plan's workspace; this kernel adds the
// slices in a fixed order (so results are reproducible run to run) and performs
// the unpacking update of Eq. 11, C <- alpha * sum + beta * C, through C's own
// mode permutation.  The paper has no split-K; the nearest idea is choosing the
// GEMM variant by which of m, n, k is small (Sec. 2.1, Table I; Sec. 3.3).
#include "kernels.h"
#include "umma_raster.h"

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

// Stream-K: blockIdx.x = left-over tile r (tile number sk_full * grid + r), blockIdx.y = one group
// of FIX_COLS tile columns.  The tile's slab units [r S, (r + 1) S) were covered by the CTAs number
// (r S) / W ... ((r + 1) S - 1) / W (W units per CTA); CTA number first + p left piece p in
// ws[r][p][column][row].  The pieces are added in that fixed order.  A thread owns one tile row
// (its C offset is computed once) and walks the group's columns.
constexpr uint32_t FIX_COLS = 16;

__global__ void __launch_bounds__(256) gett_streamk_fixup_kernel(const __grid_constant__ GettKernelArgs g,
                                                                const uint32_t main_grid)
{
    const uint32_t r = blockIdx.x, S = g.sk_slabs, W = g.sk_units;
    const uint32_t first = (r * S) / W, last = ((r + 1) * S - 1) / W;
    const uint32_t pieces = last - first + 1;
    uint32_t tm, tn;
    gett_raster_tile(g.sk_full * main_grid + r, g.tiles_m, g.tiles_n, tm, tn);
    const uint32_t tile_m = (uint32_t)g.tile_m, tile_n = (uint32_t)g.tile_n;
    const uint32_t row = threadIdx.x % tile_m;
    const uint32_t m = tm * tile_m + row;
    const uint32_t sub = threadIdx.x / tile_m, nsub = blockDim.x / tile_m; // column sub-groups (128-row tiles: two)
    const uint32_t c_begin = blockIdx.y * FIX_COLS;
    const uint32_t c_end = min(min(c_begin + FIX_COLS, tile_n), g.N.size - tn * tile_n);
    if (m >= g.M.size || sub >= nsub)
        return;
    float* crow = g.C + gett_offset_y(g.M, m);
    const size_t piece_elems = (size_t)tile_m * tile_n;
    const float* base = g.ws + (size_t)r * g.sk_pmax * piece_elems + row;
    for (uint32_t c = c_begin + sub; c < c_end; c += nsub) {
        float s = 0.f;
        for (uint32_t p = 0; p < pieces; ++p)
            s += base[p * piece_elems + (size_t)c * tile_m];
        float* dst = crow + gett_offset_y(g.N, tn * tile_n + c);
        float v = g.alpha * s;
        if (g.beta != 0.f)
            v = fmaf(g.beta, *dst, v);
        *dst = v;
    }
}

} // namespace

cudaError_t gett_launch_streamk_fixup(const GettKernelArgs& args, int grid, cudaStream_t stream)
{
    const uint32_t left = args.tiles_m * args.tiles_n - args.sk_full * (uint32_t)grid;
    if (left == 0)
        return cudaSuccess;
    const dim3 blocks(left, ((unsigned)args.tile_n + FIX_COLS - 1) / FIX_COLS);
    gett_streamk_fixup_kernel<<<blocks, 256, 0, stream>>>(args, (uint32_t)grid);
    return cudaGetLastError();
}

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
