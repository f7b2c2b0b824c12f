// CTA-pair variant of the tensor-core kernel (kernel_umma.cu compiled with clusters of two):
// the two CTAs of a cluster take two neighbouring 256 x 256 tiles of one tile row, each
// fetches half of the shared A tile for both (a copy delivered to both CTAs' shared memory),
// so a tile pair pulls 96 KB per slab out of L2 instead of 128 KB.  Both operands must be boxes
// of tensor maps; direct epilogue; no split-K; an even number of tile columns.
//
// Built into a library of its own, which the main library loads if it is there.  This file
// and ptx_sm100_mc.cuh stay out of runs on more than one GPU; nothing else depends on them.
#define GETT_UMMA_CLUSTER 1
#include "ptx_sm100_mc.cuh"
#include "kernel_umma.cu"

namespace {

template <bool AK, bool BK>
cudaError_t launch_pair(const GettKernelArgs& args, const GettTmaMaps& maps, int smem, int sm_count,
                        cudaStream_t stream)
{
    void (*k)(GettKernelArgs, GettTmaMaps) = gett_umma_kernel<AK, BK, 256, 256>;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    const uint32_t pairs = args.tiles_m * (args.tiles_n / 2);
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(2 * (unsigned)(sm_count / 2));
    int clusters = 0; // how many pairs of SMs can hold a cluster at the same time
    e = cudaOccupancyMaxActiveClusters(&clusters, k, &cfg);
    if (e != cudaSuccess)
        return e;
    if (clusters < 1)
        return cudaErrorInvalidConfiguration;
    cfg.gridDim = dim3(2 * (unsigned)(pairs < (uint32_t)clusters ? pairs : (uint32_t)clusters));
    return cudaLaunchKernelEx(&cfg, k, args, maps);
}

} // namespace

// args.tiles_n must be even, args.tile_m == args.tile_n == 256, both maps in use, split_k == 1.
// args_bytes / maps_bytes: sizeof the two structures as the caller was compiled with; a library
// built from other headers refuses to run (the ordinary kernel then does).
extern "C" __attribute__((visibility("default"))) int
gett_launch_umma_pair(const GettKernelArgs* args, const GettTmaMaps* maps, int smem, int sm_count, void* stream,
                      size_t args_bytes, size_t maps_bytes)
{
    if (args_bytes != sizeof(GettKernelArgs) || maps_bytes != sizeof(GettTmaMaps))
        return (int)cudaErrorInvalidValue;
    if (!args || !maps || args->tile_m != 256 || args->tile_n != 256 || (args->tiles_n & 1) || args->split_k != 1 ||
        !maps->a.use || !maps->b.use || args->epilogue != GETT_EPI_DIRECT)
        return (int)cudaErrorInvalidValue;
    const bool ak = args->loader_a == GETT_LOAD_VEC_K, bk = args->loader_b == GETT_LOAD_VEC_K;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = ak && bk ? launch_pair<true, true>(*args, *maps, smem, sm_count, st)
                    : ak     ? launch_pair<true, false>(*args, *maps, smem, sm_count, st)
                    : bk     ? launch_pair<false, true>(*args, *maps, smem, sm_count, st)
                             : launch_pair<false, false>(*args, *maps, smem, sm_count, st);
    return (int)e;
}
