// gett_contract_noalloc: the split-K contraction for callers that must not allocate
// device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a region that
// is being captured or replayed, under a memory pool that owns the whole device, in a
// callback, or in a process whose device heap is fixed at start-up.  The ordinary flow
// (gett_plan_create) allocates a status word and, for split-K plans, a workspace for
// the partial sums.  This entry point needs neither: the partial sums go to a
// fixed-size array that is part of the library image itself.
#include <cuda_runtime.h>

#include <mutex>

#include "kernels.h"

namespace {

// Partial sums [slice][N][M] of the split-K kernel.  Lives in every device that loads
// the library until the process exits; shared by all calls, never cleared (every call
// overwrites exactly the entries it later reads).
static __device__ __align__(256) unsigned char gett_noalloc_scratch[GETT_NOALLOC_WORKSPACE_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
float* g_scratch_ptr[MAX_DEVICES]; // device address of the array, per device; null = not looked up yet

// In host code the array's name is only a handle; the device address has to be asked
// for, once per device, with that device current.
gett_status_t scratch_for_current_device(float** out, int* sm_count)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        cudaGetLastError();
        return GETT_ERR_CUDA;
    }
    if (cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return GETT_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, gett_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return GETT_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_ptr[dev];
    return GETT_OK;
}

} // namespace

extern "C" gett_status_t gett_contract_noalloc(const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                                               const gett_tensor_desc_t* C, gett_dtype_t dtype,
                                               int32_t split_k, float alpha, const void* A_data,
                                               const void* B_data, float beta, void* C_data,
                                               void* cuda_stream)
{
    if (!A || !B || !C || !A_data || !B_data || !C_data || split_k < 0)
        return GETT_ERR_INVALID_ARG;
    if (dtype == GETT_F64)
        return GETT_ERR_UNSUPPORTED; // (its partial sums are fp32)
    float* scratch = nullptr;
    int sms = 0;
    gett_status_t rc = scratch_for_current_device(&scratch, &sms);
    if (rc != GETT_OK)
        return rc;

    // Host-side planning only (no device memory): the scalar-gather kernel, which takes
    // every layout, with the requested number of K slices.
    gett_plan plan;
    plan.ws = nullptr;
    plan.status = nullptr;
    gett_plan_opts_t opts = {};
    opts.path = GETT_PATH_SIMT;
    opts.split_k = split_k;
    rc = gett_planner_build(&plan, A, B, C, dtype, &opts, sms);
    if (rc != GETT_OK)
        return rc;
    if (plan.info.workspace_bytes > (int64_t)GETT_NOALLOC_WORKSPACE_BYTES)
        return GETT_ERR_UNSUPPORTED; // split_k * M * N * 4 bytes must fit the built-in array
    const uintptr_t es = dtype == GETT_F32 ? 4 : 2;
    if (((uintptr_t)A_data % es) || ((uintptr_t)B_data % es) || ((uintptr_t)C_data % 4))
        return GETT_ERR_ALIGNMENT;

    GettKernelArgs args = {};
    args.M = plan.M;
    args.N = plan.N;
    args.K = plan.K;
    args.A = plan.swapped ? B_data : A_data; // (the plan may have exchanged the operands)
    args.B = plan.swapped ? A_data : B_data;
    args.C = static_cast<float*>(C_data);
    args.ws = scratch;
    args.status = nullptr;
    args.alpha = alpha;
    args.beta = beta;
    args.tiles_m = plan.tiles_m;
    args.tiles_n = plan.tiles_n;
    args.split_k = (uint32_t)plan.info.split_k;
    args.k_per_split = plan.k_per_split;
    args.dtype = dtype;
    args.a_kmajor = plan.a_kmajor;
    args.b_kmajor = plan.b_kmajor;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t err = gett_launch_simt(args, plan.info.grid, stream);
    if (err == cudaSuccess && args.split_k > 1)
        err = gett_launch_splitk_reduce(args, sms, stream);
    return err == cudaSuccess ? GETT_OK : GETT_ERR_CUDA;
}
