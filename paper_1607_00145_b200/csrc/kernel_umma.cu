// Tensor-core contraction kernel for 16-bit inputs (bf16 / fp16) with fp32
// accumulation: tcgen05.mma with the accumulator in tensor memory.
//
// Mapping of the paper's GETT loop nest (Listing 4) onto one persistent CTA per SM:
//   m-/n-loops .... the CTA's work list of 128 x TILE_N output tiles (x split-K slices)
//   k-loop ........ slabs of 64 contracted elements flowing through a ring of smem stages
//   packA / packB . producer warps gather 16-byte pieces of the A and B sub-tensors
//                   straight into the 128-byte-swizzled operand layout the tensor core
//                   reads (Eq. 9 / Eq. 10: packing is a transposition; here it is fused
//                   into the copy, so no packed copy ever exists in global memory)
//   macro-kernel .. one thread issues tcgen05.mma (128 x TILE_N x 16 per instruction)
//   unpack ........ epilogue warps read the accumulator from tensor memory, apply
//                   alpha / beta and store through C's own mode permutation (Eq. 11)
//
// Operand layouts.  If an operand's stride-1 mode is a free mode ("VEC_FREE") it is
// staged MN-major: one 128-byte smem row per k index holding 64 consecutive free
// indices.  If its stride-1 mode is contracted ("VEC_K") it is staged K-major: one
// 128-byte row per free index holding the slab's 64 k.  Either way a 16-byte piece of
// global memory lands as one 16-byte piece of shared memory, XOR-swizzled by its row.
//
// Synchronisation: full[s] (producers -> MMA), empty[s] (MMA -> producers, through
// tcgen05.commit), acc_full[b] / acc_empty[b] for the two accumulator buffers.  Every
// wait is bounded; on a timeout the CTA raises an abort flag, records
// GETT_ERR_TIMEOUT in the plan's status word, drains its copies, frees its tensor
// memory and returns.
#include "kernels.h"
#include "ptx_sm100.cuh"

namespace {

constexpr int TILE_M = 128;
constexpr int TILE_K = 64;           // 16-bit elements per slab = one 128-byte swizzle row
constexpr int A_STAGE_BYTES = TILE_M * TILE_K * 2;
constexpr int NUM_EPI_WARPS = 4;
constexpr int NUM_PROD_WARPS = 4;
constexpr int MMA_WARP = NUM_EPI_WARPS;
constexpr int PROD_WARP0 = NUM_EPI_WARPS + 1;
constexpr int NUM_THREADS = (NUM_EPI_WARPS + 1 + NUM_PROD_WARPS) * 32;
constexpr int PROD_THREADS = NUM_PROD_WARPS * 32;
constexpr int LAG = 2;               // slabs a producer keeps in flight before it signals
constexpr int MAX_STAGES = 8;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t ATOM_BYTES = 1024;      // 8 rows x 128 B
constexpr uint32_t MN_BLOCK_BYTES = 8192;  // one 64-wide block of an MN-major operand: 64 k rows

struct SmemTables {
    int64_t rowA[TILE_M];                   // A offset of each tile row (-1: beyond M)
    int64_t rowB[256];                      // B offset of each tile column (-1: beyond N)
    int64_t colC[256];                      // C offset of each tile column (epilogue)
    int64_t kTab[NUM_PROD_WARPS][2][TILE_K]; // per producer warp: A and B offsets of the slab's k
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

__host__ __device__ inline uint32_t stage_bytes(uint32_t tile_n) { return A_STAGE_BYTES + tile_n * TILE_K * 2; }

struct WorkItem {
    uint32_t m0, n0, z, kbeg, kend, nslab;
};

__device__ __forceinline__ WorkItem decode_work(const GettKernelArgs& g, uint32_t w)
{
    const uint32_t tiles = g.tiles_m * g.tiles_n;
    WorkItem it;
    it.z = w / tiles;
    const uint32_t t = w - it.z * tiles;
    const uint32_t tn = t / g.tiles_m;
    it.m0 = (t - tn * g.tiles_m) * TILE_M;
    it.n0 = tn * g.tile_n;
    it.kbeg = it.z * g.k_per_split;
    it.kend = min(g.K.size, it.kbeg + g.k_per_split);
    it.nslab = (it.kend - it.kbeg + TILE_K - 1) / TILE_K;
    return it;
}

// Gather one operand tile of `rows` free indices x 64 k into a stage buffer.
//   VEC_FREE: pieces run along the free dimension (8 consecutive free indices).
//   VEC_K   : pieces run along k (8 consecutive k).
template <bool VEC_K>
__device__ __forceinline__ void load_operand(const char* __restrict__ base, uint32_t smem_dst,
                                             const int64_t* rowTab, const int64_t* kTab,
                                             uint32_t rows, uint32_t pt)
{
    const uint32_t pieces = rows * (TILE_K / 8);
    if (VEC_K) {
        // piece q: kc = q % 8 (which 8 k of the slab), r = q / 8
        const uint32_t kc = pt & 7;
        const int64_t ko = kTab[kc * 8];
#pragma unroll 4
        for (uint32_t q = pt; q < pieces; q += PROD_THREADS) {
            const uint32_t r = q >> 3;
            const int64_t ro = rowTab[r];
            const bool ok = (ro >= 0) && (ko >= 0);
            const char* src = base + (ok ? (ro + ko) * 2 : 0);
            const uint32_t dst = smem_dst + r * 128 + ((kc ^ (r & 7)) << 4);
            ptx::cp_async_16(dst, src, ok ? 16u : 0u);
        }
    } else {
        // piece q: fc = q % (rows / 8) (which 8 free indices), k = q / (rows / 8)
        const uint32_t fpr = rows >> 3;
#pragma unroll 4
        for (uint32_t q = pt; q < pieces; q += PROD_THREADS) {
            const uint32_t k = q / fpr;
            const uint32_t fc = q - k * fpr;
            const int64_t ro = rowTab[fc * 8];
            const int64_t ko = kTab[k];
            const bool ok = (ro >= 0) && (ko >= 0);
            const char* src = base + (ok ? (ro + ko) * 2 : 0);
            const uint32_t dst = smem_dst + (fc >> 3) * MN_BLOCK_BYTES + k * 128 + (((fc & 7) ^ (k & 7)) << 4);
            ptx::cp_async_16(dst, src, ok ? 16u : 0u);
        }
    }
}

template <bool A_VEC_K, bool B_VEC_K>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gett_umma_kernel(const __grid_constant__ GettKernelArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), tables after it
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t stages = (uint32_t)g.stages;
    const uint32_t sbytes = stage_bytes(g.tile_n);
    SmemTables* T = reinterpret_cast<SmemTables*>(smem + stages * sbytes);
    const uint32_t stage0 = ptx::smem_u32(smem);

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t total_work = g.tiles_m * g.tiles_n * g.split_k;
    volatile int* abort_flag = &T->abort_flag;

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&T->full[s]), PROD_THREADS);
            ptx::mbar_init(ptx::smem_u32(&T->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&T->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&T->acc_empty[b]), NUM_EPI_WARPS * 32);
        }
        T->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_u32(&T->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = T->tmem_base;

    if (warp >= PROD_WARP0) {
        // ------------------------------ producers ------------------------------
        const uint32_t pt = threadIdx.x - PROD_WARP0 * 32;
        const uint32_t pw = warp - PROD_WARP0;
        int64_t* kA = T->kTab[pw][0];
        int64_t* kB = T->kTab[pw][1];
        uint32_t it = 0, signalled = 0;
        bool alive = true;
        for (uint32_t w = blockIdx.x; w < total_work && alive; w += gridDim.x) {
            const WorkItem wi = decode_work(g, w);
            ptx::named_barrier(1, PROD_THREADS); // previous tile's row tables no longer read
            for (uint32_t r = pt; r < TILE_M; r += PROD_THREADS) {
                int64_t x = -1, y;
                if (wi.m0 + r < g.M.size)
                    gett_decompose(g.M, wi.m0 + r, x, y);
                T->rowA[r] = x;
            }
            for (uint32_t c = pt; c < g.tile_n; c += PROD_THREADS) {
                int64_t x = -1, y;
                if (wi.n0 + c < g.N.size)
                    gett_decompose(g.N, wi.n0 + c, x, y);
                T->rowB[c] = x;
            }
            ptx::named_barrier(1, PROD_THREADS);
            for (uint32_t j = 0; j < wi.nslab; ++j, ++it) {
                const uint32_t k0 = wi.kbeg + j * TILE_K;
                __syncwarp();
#pragma unroll
                for (uint32_t h = 0; h < TILE_K / 32; ++h) {
                    const uint32_t k = k0 + h * 32 + lane;
                    int64_t x = -1, y = -1;
                    if (k < wi.kend)
                        gett_decompose(g.K, k, x, y);
                    kA[h * 32 + lane] = x;
                    kB[h * 32 + lane] = y;
                }
                __syncwarp();
                const uint32_t s = it % stages;
                if (!ptx::mbar_wait(ptx::smem_u32(&T->empty[s]), ((it / stages) & 1) ^ 1, abort_flag)) {
                    alive = false;
                    break;
                }
                const uint32_t sa = stage0 + s * sbytes;
                load_operand<A_VEC_K>(static_cast<const char*>(g.A), sa, T->rowA, kA, TILE_M, pt);
                load_operand<B_VEC_K>(static_cast<const char*>(g.B), sa + A_STAGE_BYTES, T->rowB, kB,
                                      g.tile_n, pt);
                ptx::cp_async_commit();
                if (it >= LAG) {
                    ptx::cp_async_wait<LAG>();
                    ptx::fence_proxy_async_smem();
                    ptx::mbar_arrive(ptx::smem_u32(&T->full[signalled % stages]));
                    ++signalled;
                }
            }
        }
        // drain: everything this thread issued has landed; signal the remaining slabs
        ptx::cp_async_wait<0>();
        ptx::fence_proxy_async_smem();
        if (alive)
            for (; signalled < it; ++signalled)
                ptx::mbar_arrive(ptx::smem_u32(&T->full[signalled % stages]));
    } else if (warp == MMA_WARP) {
        // ------------------------------ MMA issuer -----------------------------
        if (lane == 0) {
            const uint32_t fmt = g.dtype == GETT_BF16_F32 ? 1u : 0u;
            const uint32_t idesc = ptx::idesc_f16(fmt, A_VEC_K ? 0u : 1u, B_VEC_K ? 0u : 1u, TILE_M, g.tile_n);
            // bytes the descriptor start address advances per 16-wide k step
            const uint32_t a_step = A_VEC_K ? 32u : 2u * ATOM_BYTES;
            const uint32_t b_step = B_VEC_K ? 32u : 2u * ATOM_BYTES;
            const uint32_t lbo = (g.debug & 1) ? ATOM_BYTES : MN_BLOCK_BYTES;
            const uint32_t sbo = (g.debug & 1) ? MN_BLOCK_BYTES : ATOM_BYTES;
            uint32_t it = 0, local = 0;
            bool alive = true;
            for (uint32_t w = blockIdx.x; w < total_work && alive; w += gridDim.x, ++local) {
                const WorkItem wi = decode_work(g, w);
                const uint32_t buf = local & 1;
                if (!ptx::mbar_wait(ptx::smem_u32(&T->acc_empty[buf]), ((local >> 1) & 1) ^ 1, abort_flag))
                    break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (uint32_t j = 0; j < wi.nslab; ++j, ++it) {
                    const uint32_t s = it % stages;
                    if (!ptx::mbar_wait(ptx::smem_u32(&T->full[s]), (it / stages) & 1, abort_flag)) {
                        alive = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t sa = stage0 + s * sbytes, sb = sa + A_STAGE_BYTES;
#pragma unroll
                    for (uint32_t kk = 0; kk < TILE_K / 16; ++kk) {
                        const uint64_t ad = A_VEC_K ? ptx::smem_desc_sw128(sa + kk * a_step, 16, ATOM_BYTES)
                                                    : ptx::smem_desc_sw128(sa + kk * a_step, lbo, sbo);
                        const uint64_t bd = B_VEC_K ? ptx::smem_desc_sw128(sb + kk * b_step, 16, ATOM_BYTES)
                                                    : ptx::smem_desc_sw128(sb + kk * b_step, lbo, sbo);
                        ptx::umma_f16(d_tmem, ad, bd, idesc, (j | kk) ? 1u : 0u);
                    }
                    ptx::umma_commit(ptx::smem_u32(&T->empty[s])); // stage reusable once these MMAs retire
                }
                if (alive)
                    ptx::umma_commit(ptx::smem_u32(&T->acc_full[buf]));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------- epilogue ------------------------------
        const uint32_t et = threadIdx.x; // 0..127: tile row, = tensor-memory lane
        uint32_t local = 0;
        for (uint32_t w = blockIdx.x; w < total_work; w += gridDim.x, ++local) {
            const WorkItem wi = decode_work(g, w);
            const uint32_t buf = local & 1;
            // C offsets of this tile: my row in a register, the columns in shared memory
            int64_t rowC = -1, dummy;
            if (wi.m0 + et < g.M.size)
                gett_decompose(g.M, wi.m0 + et, dummy, rowC);
            ptx::named_barrier(2, NUM_EPI_WARPS * 32); // previous tile's column table no longer read
            for (uint32_t c = et; c < g.tile_n; c += NUM_EPI_WARPS * 32) {
                int64_t x, y = -1;
                if (wi.n0 + c < g.N.size)
                    gett_decompose(g.N, wi.n0 + c, x, y);
                T->colC[c] = y;
            }
            ptx::named_barrier(2, NUM_EPI_WARPS * 32);
            if (!ptx::mbar_wait(ptx::smem_u32(&T->acc_full[buf]), (local >> 1) & 1, abort_flag))
                break;
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + ((warp * 32u) << 16) + buf * 256;
            const bool row_ok = rowC >= 0;
            const float alpha = g.alpha, beta = g.beta;
            for (uint32_t c0 = 0; c0 < g.tile_n; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(taddr + c0, v);
                ptx::tmem_wait_ld();
                if (!row_ok)
                    continue;
                if (g.split_k > 1) {
                    float* dst = g.ws + ((size_t)wi.z * g.N.size + wi.n0 + c0) * g.M.size + wi.m0 + et;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (wi.n0 + c0 + i < g.N.size)
                            dst[(size_t)i * g.M.size] = __uint_as_float(v[i]);
                } else {
                    float* crow = g.C + rowC;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int64_t co = T->colC[c0 + i];
                        if (co >= 0) {
                            float r = alpha * __uint_as_float(v[i]);
                            if (beta != 0.f)
                                r = fmaf(beta, crow[co], r);
                            crow[co] = r;
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(ptx::smem_u32(&T->acc_empty[buf]));
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && T->abort_flag && g.status)
        *g.status = GETT_ERR_TIMEOUT;
    if (warp == MMA_WARP) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

} // namespace

int gett_umma_smem_bytes(int tile_n, int stages)
{
    return 1024 + stages * (int)stage_bytes((uint32_t)tile_n) + (int)sizeof(SmemTables);
}

int gett_umma_max_stages(int tile_n, int smem_limit)
{
    int s = (smem_limit - 1024 - (int)sizeof(SmemTables)) / (int)stage_bytes((uint32_t)tile_n);
    return s > MAX_STAGES ? MAX_STAGES : s;
}

int gett_umma_block() { return NUM_THREADS; }

cudaError_t gett_launch_umma(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    void (*k)(GettKernelArgs);
    const bool ak = args.loader_a == GETT_LOAD_VEC_K, bk = args.loader_b == GETT_LOAD_VEC_K;
    if (ak && bk)
        k = gett_umma_kernel<true, true>;
    else if (ak)
        k = gett_umma_kernel<true, false>;
    else if (bk)
        k = gett_umma_kernel<false, true>;
    else
        k = gett_umma_kernel<false, false>;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    k<<<grid, NUM_THREADS, smem, stream>>>(args);
    return cudaGetLastError();
}
