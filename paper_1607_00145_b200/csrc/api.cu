// C ABI of the library (declared in include/gett.h): plan life cycle, kernel
// dispatch, introspection.  Device memory is touched only here (split-K
// workspace and the status word); gett_contract itself allocates nothing.
#include <cuda.h>
#include <cuda_runtime.h>
#include <dlfcn.h>

#include <cstring>
#include <new>
#include <string>
#include <utility>

#include "kernels.h"

extern "C" GETT_API int gett_internal_pointer_is_local(int memory_type, int pointer_device, int plan_device);

namespace {

int current_device_sm_count(int* device_out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        *device_out = -1;
        return 0;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        *device_out = -1;
        return 0;
    }
    *device_out = dev;
    return sms;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup, so the library
// does not link against the driver and still loads on a machine without one.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            p = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor map of one operand for this call's base pointer.  False = use the gather loader.
bool encode_side(const GettTmaRecipe& R, int dtype, const void* base, GettTmaSide& out)
{
    memset(&out, 0, sizeof out);
    EncodeTiledFn fn = encode_tiled_fn();
    if (!R.enabled || !fn)
        return false;
    const int rank = R.co.rank;
    cuuint64_t dims[5], strides_bytes[4];
    cuuint32_t box[5], estr[5];
    for (int i = 0; i < rank; ++i) {
        dims[i] = R.dims[i];
        box[i] = R.box[i];
        estr[i] = 1;
        if (i > 0)
            strides_bytes[i - 1] = R.strides[i] * 2;
    }
    const CUtensorMapDataType dt = dtype == GETT_BF16_F32 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                          : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    CUresult rc = fn(reinterpret_cast<CUtensorMap*>(out.map), dt, (cuuint32_t)rank, const_cast<void*>(base),
                     dims, strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS)
        return false;
    out.co = R.co;
    out.hybrid = R.hybrid;
    out.use = 1;
    return true;
}

// The CTA-pair variant of the tensor-core kernel lives in a library of its own next to this
// one (it is left out of multi-GPU runs); null if it is not there.
typedef int (*LaunchPairFn)(const GettKernelArgs*, const GettTmaMaps*, int, int, void*, size_t, size_t);

LaunchPairFn launch_pair_fn()
{
    static LaunchPairFn fn = [] {
        Dl_info me;
        if (!dladdr(reinterpret_cast<const void*>(&gett_status_string), &me) || !me.dli_fname)
            return (LaunchPairFn) nullptr;
        std::string path(me.dli_fname);
        const size_t dot = path.rfind(".so");
        if (dot == std::string::npos)
            return (LaunchPairFn) nullptr;
        path.insert(dot, "_mc");
        void* h = dlopen(path.c_str(), RTLD_NOW | RTLD_LOCAL);
        return h ? reinterpret_cast<LaunchPairFn>(dlsym(h, "gett_launch_umma_pair")) : (LaunchPairFn) nullptr;
    }();
    return fn;
}

// The CTA-pair variant delivers copies to both CTAs of a cluster; its tensor maps must cover
// this GPU's own memory alone.  True if `p` is ordinary device memory of device `device`.
bool on_this_device(const void* p, int device)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return gett_internal_pointer_is_local((int)attr.type, attr.device, device) != 0;
}

int vec_kind(int loader) // the staging layout behind a loader value
{
    return loader == GETT_LOAD_TMA_FREE ? GETT_LOAD_VEC_FREE : loader == GETT_LOAD_TMA_K ? GETT_LOAD_VEC_K : loader;
}

} // namespace

extern "C" {

// (internal, exported for the host tests) the rule behind on_this_device(): memory type 2 is
// cudaMemoryTypeDevice; host, managed and unregistered memory, and another GPU's memory, are not local.
GETT_API int gett_internal_pointer_is_local(int memory_type, int pointer_device, int plan_device)
{
    return memory_type == (int)cudaMemoryTypeDevice && pointer_device == plan_device && plan_device >= 0;
}

gett_status_t gett_plan_create(gett_plan_t** out, const gett_tensor_desc_t* A,
                               const gett_tensor_desc_t* B, const gett_tensor_desc_t* C,
                               gett_dtype_t dtype, const gett_plan_opts_t* opts)
{
    if (!out || !A || !B || !C)
        return GETT_ERR_INVALID_ARG;
    gett_plan* p = new (std::nothrow) gett_plan();
    if (!p)
        return GETT_ERR_ALLOC;
    p->ws = nullptr;
    p->status = nullptr;
    int device = -1;
    const int sms = current_device_sm_count(&device);
    gett_status_t rc = gett_planner_build(p, A, B, C, dtype, opts, sms > 0 ? sms : 148);
    if (rc != GETT_OK) {
        delete p;
        return rc;
    }
    p->info.device = device;
    p->sm_count = sms > 0 ? sms : 148;
    if (device >= 0) {
        if (cudaMalloc(&p->status, sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(p->status, 0, sizeof(int32_t)) != cudaSuccess) {
            cudaGetLastError();
            gett_plan_destroy(p);
            return GETT_ERR_ALLOC;
        }
        if (p->info.workspace_bytes > 0 &&
            cudaMalloc(&p->ws, (size_t)p->info.workspace_bytes) != cudaSuccess) {
            cudaGetLastError();
            gett_plan_destroy(p);
            return GETT_ERR_ALLOC;
        }
    }
    *out = p;
    return GETT_OK;
}

gett_status_t gett_plan_destroy(gett_plan_t* plan)
{
    if (!plan)
        return GETT_OK;
    if (plan->ws)
        cudaFree(plan->ws);
    if (plan->status)
        cudaFree(plan->status);
    delete plan;
    return GETT_OK;
}

gett_status_t gett_contract(const gett_plan_t* plan, float alpha, const void* A, const void* B,
                            float beta, void* C, void* cuda_stream)
{
    if (!plan || !A || !B || !C)
        return GETT_ERR_INVALID_ARG;
    if (plan->swapped) // the kernels run with the operands exchanged
        std::swap(A, B);
    if (plan->info.device < 0)
        return GETT_ERR_CUDA;
    {
        // the plan's workspace, status word and SM count belong to the device it was created on
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) {
            cudaGetLastError();
            return GETT_ERR_CUDA;
        }
        if (dev != plan->info.device)
            return GETT_ERR_INVALID_ARG;
    }
    const uintptr_t es = plan->dtype == GETT_F32 ? 4 : 2;
    if (((uintptr_t)A % es) || ((uintptr_t)B % es) || ((uintptr_t)C % 4))
        return GETT_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    GettKernelArgs args;
    args.M = plan->M;
    args.N = plan->N;
    args.K = plan->K;
    args.A = A;
    args.B = B;
    args.C = static_cast<float*>(C);
    args.ws = plan->ws;
    args.status = plan->status;
    args.alpha = alpha;
    args.beta = beta;
    args.tiles_m = plan->tiles_m;
    args.tiles_n = plan->tiles_n;
    args.split_k = (uint32_t)plan->info.split_k;
    args.k_per_split = plan->k_per_split;
    args.dtype = plan->dtype;
    args.a_kmajor = plan->a_kmajor;
    args.b_kmajor = plan->b_kmajor;
    // (info is the caller's view: with exchanged operands its loader_a describes the kernels' B)
    args.loader_a = vec_kind(plan->swapped ? plan->info.loader_b : plan->info.loader_a);
    args.loader_b = vec_kind(plan->swapped ? plan->info.loader_a : plan->info.loader_b);
    args.tile_m = plan->info.tile_m;
    args.tile_n = plan->info.tile_n;
    args.stages = plan->info.stages;
    args.epilogue = plan->info.epilogue;
    args.debug = plan->debug;
    // a shortened wait limit applies only where a CTA that gives up has nothing in flight that
    // it cannot wait for: plans whose operands are both gathered (cp.async is drained on exit)
    const bool any_tma = plan->tma_a.enabled || plan->tma_b.enabled;
    args.wait_limit_us = (plan->wait_limit_us > 0 && !any_tma) ? (uint32_t)plan->wait_limit_us : 2000000u;
    args.c_vec = plan->c_vec;
    args.prod_groups = plan->info.path == GETT_PATH_UMMA ? gett_umma_prod_groups(plan->info.stages) : 0;
    args.epi_lean = plan->epi_lean;
#ifdef GETT_EXPERIMENT
    if (plan->debug & 2048) // probe: all producer warps as one wide group
        args.prod_groups = 1;
#endif

    int path = plan->info.path;
    // the vectorised kernels need 16-byte aligned operand bases; otherwise gather scalars
    if (path != GETT_PATH_SIMT && (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 15))
        path = GETT_PATH_SIMT;

    cudaError_t err = cudaSuccess;
    switch (path) {
    case GETT_PATH_SIMT: {
        args.tiles_m = (plan->M.size + 63) / 64;
        args.tiles_n = (plan->N.size + 63) / 64;
        const uint64_t grid = (uint64_t)args.tiles_m * args.tiles_n * args.split_k;
        if (grid >= (1ull << 31))
            return GETT_ERR_UNSUPPORTED;
        err = gett_launch_simt(args, (int)grid, stream);
        break;
    }
    case GETT_PATH_FFMA:
        err = plan->skinny ? gett_launch_ffma_skinny(args, plan->info.grid, plan->info.smem_bytes, stream)
                           : gett_launch_ffma(args, plan->info.grid, plan->info.smem_bytes, stream);
        break;
    case GETT_PATH_UMMA: {
        alignas(64) GettTmaMaps maps;
        if (plan->pair_ok && launch_pair_fn() && on_this_device(A, plan->info.device) &&
            on_this_device(B, plan->info.device)) {
            // each CTA of a pair fetches half of the A tile: a K-major A gets a half-height box
            GettTmaRecipe ra = plan->tma_a;
            if (args.loader_a == GETT_LOAD_VEC_K && ra.co.fdim[0] >= 0)
                ra.box[ra.co.fdim[0]] /= 2;
            const bool ua = encode_side(ra, plan->dtype, A, maps.a);
            const bool ub = encode_side(plan->tma_b, plan->dtype, B, maps.b);
            if (ua && ub &&
                launch_pair_fn()(&args, &maps, plan->info.smem_bytes, plan->sm_count, cuda_stream,
                                 sizeof(GettKernelArgs), sizeof(GettTmaMaps)) == 0)
                break;
            cudaGetLastError(); // the variant could not run: the ordinary kernel does
        }
        encode_side(plan->tma_a, plan->dtype, A, maps.a);
        encode_side(plan->tma_b, plan->dtype, B, maps.b);
        err = gett_launch_umma(args, maps, plan->info.grid, plan->info.smem_bytes, stream);
        break;
    }
    default: return GETT_ERR_UNSUPPORTED;
    }
    if (err == cudaSuccess && args.split_k > 1)
        err = gett_launch_splitk_reduce(args, plan->sm_count, stream);
    return err == cudaSuccess ? GETT_OK : GETT_ERR_CUDA;
}

gett_status_t gett_plan_get_info(const gett_plan_t* plan, gett_plan_info_t* info)
{
    if (!plan || !info)
        return GETT_ERR_INVALID_ARG;
    *info = plan->info;
    return GETT_OK;
}

gett_status_t gett_plan_get_table(const gett_plan_t* plan, int which, int64_t* dst, size_t capacity)
{
    if (!plan)
        return GETT_ERR_INVALID_ARG;
    return gett_planner_table(plan, which, dst, capacity);
}

gett_status_t gett_plan_last_device_status(const gett_plan_t* plan)
{
    if (!plan)
        return GETT_ERR_INVALID_ARG;
    if (!plan->status)
        return GETT_ERR_CUDA;
    int32_t host = 0;
    if (cudaMemcpy(&host, plan->status, sizeof host, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return GETT_ERR_CUDA;
    }
    return static_cast<gett_status_t>(host);
}

const char* gett_status_string(gett_status_t status)
{
    switch (status) {
    case GETT_OK: return "ok";
    case GETT_ERR_INVALID_ARG: return "invalid argument";
    case GETT_ERR_BAD_LABELS: return "bad labels";
    case GETT_ERR_EXTENT_MISMATCH: return "extent mismatch";
    case GETT_ERR_UNSUPPORTED: return "unsupported";
    case GETT_ERR_ALIGNMENT: return "misaligned operand";
    case GETT_ERR_ALLOC: return "allocation failed";
    case GETT_ERR_CUDA: return "cuda error";
    case GETT_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

} // extern "C"
