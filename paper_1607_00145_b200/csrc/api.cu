// C ABI of the library (declared in include/gett.h): plan life cycle, kernel
// dispatch, introspection.  Device memory is touched only here (split-K
// workspace and the status word); gett_contract itself allocates nothing.
#include <cuda.h>
#include <cuda_runtime.h>
#include <dlfcn.h>

#include <algorithm>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

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

// One plan from one set of overrides: host planning, then the device-side status word and workspace.
gett_status_t create_one(gett_plan_t** out, const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                         const gett_tensor_desc_t* C, gett_dtype_t dtype, const gett_plan_opts_t* opts)
{
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
    p->info.model_us = (float)gett_planner_model(p, p->sm_count, nullptr);
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

// ---- plan search (Sec. 3.3, 3.4, 7.3): candidates, model ranking, timed top-k, cache ----
std::mutex g_cache_mutex;
std::map<std::string, gett_plan_opts_t> g_plan_cache; // key: descriptors, dtype, caller's options, device

std::string cache_key(const gett_tensor_desc_t* A, const gett_tensor_desc_t* B, const gett_tensor_desc_t* C, int dtype,
                      const gett_plan_opts_t& o, int device)
{
    std::string k;
    auto put = [&](const void* p, size_t n) { k.append(static_cast<const char*>(p), n); };
    for (const gett_tensor_desc_t* t : {A, B, C}) {
        put(&t->nmodes, sizeof t->nmodes);
        for (int i = 0; i < t->nmodes; ++i) {
            put(&t->extent[i], sizeof(int64_t));
            put(&t->label[i], sizeof(int32_t));
            const int64_t st = t->stride ? t->stride[i] : -1;
            put(&st, sizeof st);
        }
    }
    put(&dtype, sizeof dtype);
    put(&o, sizeof o);
    put(&device, sizeof device);
    return k;
}

size_t span_elems(const gett_tensor_desc_t* t)
{
    size_t span = 1, packed = 1;
    for (int i = 0; i < t->nmodes; ++i) {
        const size_t st = t->stride ? (size_t)t->stride[i] : packed;
        span += (size_t)(t->extent[i] - 1) * st;
        packed *= (size_t)t->extent[i];
    }
    return span;
}

gett_status_t create_by_search(gett_plan_t** out, const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                               const gett_tensor_desc_t* C, gett_dtype_t dtype, const gett_plan_opts_t& asked)
{
    int device = -1;
    const int sms = current_device_sm_count(&device);
    if (A->nmodes < 0 || B->nmodes < 0 || C->nmodes < 0 || A->nmodes > GETT_MAX_MODES || B->nmodes > GETT_MAX_MODES ||
        C->nmodes > GETT_MAX_MODES)
        return GETT_ERR_INVALID_ARG;
    const std::string key = cache_key(A, B, C, dtype, asked, device);
    {
        std::lock_guard<std::mutex> lock(g_cache_mutex);
        auto it = g_plan_cache.find(key);
        if (it != g_plan_cache.end()) {
            gett_plan_opts_t o = it->second;
            return create_one(out, A, B, C, dtype, &o);
        }
    }
    gett_plan_opts_t base = asked;
    base.search = 0;
    const std::vector<gett_plan_opts_t> cand = gett_planner_candidates(A, B, C, dtype, base, sms > 0 ? sms : 148);
    if (cand.empty()) // not even the rule-based plan exists: report why
        return create_one(out, A, B, C, dtype, &base);
    // rank by the model
    struct Ranked {
        gett_plan_opts_t o;
        double model_us;
        float timed_us;
        bool rule_based; // the plan the planner's rules give (always timed: the search must not lose to it)
    };
    std::vector<Ranked> r;
    for (size_t i = 0; i < cand.size(); ++i) {
        gett_plan tmp;
        tmp.ws = nullptr;
        tmp.status = nullptr;
        if (gett_planner_build(&tmp, A, B, C, dtype, &cand[i], sms > 0 ? sms : 148) == GETT_OK)
            r.push_back({cand[i], gett_planner_model(&tmp, sms > 0 ? sms : 148, nullptr), 0.f, i == 0});
    }
    std::stable_sort(r.begin(), r.end(), [](const Ranked& x, const Ranked& y) { return x.model_us < y.model_us; });
    size_t best = 0;
    int timed = 0;
    if (asked.search > 1 && device >= 0) {
        // time the k best on scratch operands (zeros: finite, and the kernels do not look at values)
        const size_t es = dtype == GETT_F32 ? 4 : dtype == GETT_F64 ? 8 : 2;
        void *dA = nullptr, *dB = nullptr, *dC = nullptr, *dFlush = nullptr;
        const size_t flush_bytes = 192u << 20; // larger than L2: every timed launch starts cold
        cudaStream_t st = nullptr;
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        const size_t nA = span_elems(A) * es, nB = span_elems(B) * es, nC = span_elems(C) * (dtype == GETT_F64 ? 8 : 4);
        bool ok = cudaMalloc(&dA, nA) == cudaSuccess && cudaMalloc(&dB, nB) == cudaSuccess &&
                  cudaMalloc(&dC, nC) == cudaSuccess && cudaMalloc(&dFlush, flush_bytes) == cudaSuccess &&
                  cudaMemset(dA, 0, nA) == cudaSuccess &&
                  cudaMemset(dB, 0, nB) == cudaSuccess && cudaMemset(dC, 0, nC) == cudaSuccess &&
                  cudaStreamCreate(&st) == cudaSuccess && cudaEventCreate(&e0) == cudaSuccess &&
                  cudaEventCreate(&e1) == cudaSuccess;
        float best_ms = 0.f;
        for (size_t i = 0; ok && i < r.size(); ++i) {
            if (i >= (size_t)asked.search && !r[i].rule_based)
                continue;
            gett_plan_t* p = nullptr;
            if (create_one(&p, A, B, C, dtype, &r[i].o) != GETT_OK)
                continue;
            float ms_min = 0.f;
            bool good = gett_contract(p, 1.f, dA, dB, 0.f, dC, st) == GETT_OK; // warm-up
            for (int rep = 0; good && rep < 3; ++rep) {
                cudaMemsetAsync(dFlush, rep, flush_bytes, st);
                cudaEventRecord(e0, st);
                good = gett_contract(p, 1.f, dA, dB, 0.f, dC, st) == GETT_OK;
                cudaEventRecord(e1, st);
                if (cudaEventSynchronize(e1) != cudaSuccess)
                    good = false;
                float ms = 0.f;
                if (good && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess)
                    ms_min = rep == 0 ? ms : std::min(ms_min, ms);
            }
            good = good && gett_plan_last_device_status(p) == GETT_OK;
            gett_plan_destroy(p);
            if (!good)
                continue;
            r[i].timed_us = ms_min * 1e3f;
            ++timed;
            // (another candidate has to beat the rule-based plan by 3 % to replace it)
            const float handicap = r[i].rule_based ? 0.97f : 1.f;
            if (timed == 1 || ms_min * handicap < best_ms) {
                best_ms = ms_min * handicap;
                best = i;
            }
        }
        cudaGetLastError();
        if (e0)
            cudaEventDestroy(e0);
        if (e1)
            cudaEventDestroy(e1);
        if (st)
            cudaStreamDestroy(st);
        cudaFree(dA);
        cudaFree(dB);
        cudaFree(dC);
        cudaFree(dFlush);
        if (timed == 0)
            best = 0;
    }
    gett_status_t rc = create_one(out, A, B, C, dtype, &r[best].o);
    if (rc != GETT_OK)
        return rc;
    (*out)->info.candidates = (int32_t)r.size();
    (*out)->info.model_rank = (int32_t)best;
    (*out)->info.timed = timed;
    (*out)->info.timed_us = r[best].timed_us;
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    g_plan_cache[key] = r[best].o;
    return GETT_OK;
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
    if (opts && opts->search < 0)
        return GETT_ERR_INVALID_ARG;
    if (opts && opts->search > 0)
        return create_by_search(out, A, B, C, dtype, *opts);
    return create_one(out, A, B, C, dtype, opts);
}

gett_status_t gett_plan_model(const gett_plan_t* plan, double* total_us, double* terms_us)
{
    if (!plan || !total_us)
        return GETT_ERR_INVALID_ARG;
    *total_us = gett_planner_model(plan, plan->sm_count, terms_us);
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
    const uintptr_t es = plan->dtype == GETT_F32 ? 4 : plan->dtype == GETT_F64 ? 8 : 2;
    if (((uintptr_t)A % es) || ((uintptr_t)B % es) || ((uintptr_t)C % (plan->dtype == GETT_F64 ? 8 : 4)))
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
    args.stream_k = plan->stream_k;
    args.sk_full = plan->sk_full;
    args.sk_units = plan->sk_units;
    args.sk_slabs = plan->sk_slabs;
    args.sk_pmax = plan->sk_pmax;
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
        args.stream_k = 0; // (only reached as the fall-back for unaligned bases: the plan's slices are kept)
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
    if (err == cudaSuccess && path == GETT_PATH_UMMA && args.stream_k)
        err = gett_launch_streamk_fixup(args, plan->info.grid, stream);
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
