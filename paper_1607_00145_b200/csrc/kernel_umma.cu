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
    int64_t colC[256];                      // C offset of each tile column (epilogue)
    int64_t kTab[NUM_PROD_WARPS][2][TILE_K]; // per producer warp: A and B byte offsets of the slab's k
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

__host__ __device__ constexpr uint32_t stage_bytes(uint32_t tile_n) { return A_STAGE_BYTES + tile_n * TILE_K * 2; }

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
    it.n0 = tn * (uint32_t)g.tile_n;
    it.kbeg = it.z * g.k_per_split;
    it.kend = min(g.K.size, it.kbeg + g.k_per_split);
    it.nslab = (it.kend - it.kbeg + TILE_K - 1) / TILE_K;
    return it;
}

// Producer-side state for one operand tile of R free indices x 64 k.
//
// VEC_K   : 16-byte pieces run along k.  Thread pt owns k-piece kc = pt % 8 of rows
//           pt/8 + 16 p (p = 0 .. R/16-1); the byte offsets of its rows live in
//           registers for the whole tile, so a piece costs one 64-bit add.
// VEC_FREE: pieces run along the free dimension.  Thread pt owns free-piece
//           fc = pt % (R/8) of the k rows kgroup + kstep * p; its single row offset
//           lives in a register and the k offsets come from the warp's slab table.
template <bool VEC_K, int R>
struct OperandLoader {
    static constexpr int FPR = R / 8;                       // pieces per k row (VEC_FREE)
    // k rows covered per pass (VEC_FREE): the largest power of two that fits the producers
    static constexpr int KSTEP = PROD_THREADS / FPR >= 16 ? 16 : PROD_THREADS / FPR >= 8 ? 8 : 4;
    static constexpr int ACTIVE = VEC_K ? PROD_THREADS : KSTEP * FPR;
    static constexpr int NP = VEC_K ? R / 16 : TILE_K / KSTEP;
    static_assert(VEC_K || TILE_K % KSTEP == 0, "k rows must divide evenly over the passes");

    int64_t rowb[VEC_K ? R / 16 : 1]; // byte offsets of this thread's rows
    uint32_t rowmask;                 // bit p: row p is inside the tensor
    uint32_t dst_thread;              // byte offset of piece 0 inside the operand's stage buffer

    __device__ __forceinline__ void setup_tile(const GettDim& D, uint32_t origin, uint32_t pt)
    {
        rowmask = 0;
        if (VEC_K) {
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                const uint32_t r = (pt >> 3) + 16 * p;
                int64_t x = 0, y;
                if (origin + r < D.size) {
                    gett_decompose(D, origin + r, x, y);
                    rowmask |= 1u << p;
                }
                rowb[p] = x * 2;
            }
            dst_thread = (pt >> 3) * 128 + (((pt & 7) ^ ((pt >> 3) & 7)) << 4);
        } else {
            const uint32_t fc = pt % FPR, kgroup = pt / FPR;
            int64_t x = 0, y;
            if (pt < ACTIVE && origin + fc * 8 < D.size) {
                gett_decompose(D, origin + fc * 8, x, y);
                rowmask = 1;
            }
            rowb[0] = x * 2;
            dst_thread = (fc >> 3) * MN_BLOCK_BYTES + kgroup * 128;
        }
    }

    // kTab: the warp's table of byte offsets of the slab's 64 k (-1 beyond the K range).
    template <bool FAST>
    __device__ __forceinline__ void load_slab(const char* __restrict__ base, uint32_t stage_dst,
                                              const int64_t* kTab, uint32_t pt) const
    {
        if (VEC_K) {
            const int64_t kb = kTab[(pt & 7) * 8];
            const uint32_t dst = stage_dst + dst_thread;
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                if (FAST) {
                    ptx::cp_async_16(dst + p * 2048, base + rowb[p] + kb, 16u);
                } else {
                    const bool ok = kb >= 0 && ((rowmask >> p) & 1u);
                    ptx::cp_async_16(dst + p * 2048, base + (ok ? rowb[p] + kb : 0), ok ? 16u : 0u);
                }
            }
        } else {
            if (ACTIVE < PROD_THREADS && pt >= ACTIVE)
                return;
            const uint32_t fc = pt % FPR, kgroup = pt / FPR;
            const uint32_t dst = stage_dst + dst_thread;
            const char* rowp = base + rowb[0];
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                const uint32_t k = kgroup + KSTEP * p;
                const int64_t kb = kTab[k];
                const uint32_t d = dst + p * (KSTEP * 128) + (((fc & 7) ^ (k & 7)) << 4);
                if (FAST) {
                    ptx::cp_async_16(d, rowp + kb, 16u);
                } else {
                    const bool ok = kb >= 0 && rowmask;
                    ptx::cp_async_16(d, ok ? rowp + kb : base, ok ? 16u : 0u);
                }
            }
        }
    }
};

template <bool A_VEC_K, bool B_VEC_K, int TILE_N>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gett_umma_kernel(const __grid_constant__ GettKernelArgs g)
{
    extern __shared__ uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), tables after it
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t stages = (uint32_t)g.stages;
    constexpr uint32_t sbytes = stage_bytes(TILE_N);
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
        OperandLoader<A_VEC_K, TILE_M> la;
        OperandLoader<B_VEC_K, TILE_N> lb;
        const char* baseA = static_cast<const char*>(g.A);
        const char* baseB = static_cast<const char*>(g.B);
        uint32_t it = 0, signalled = 0;
        bool alive = true;
        for (uint32_t w = blockIdx.x; w < total_work && alive; w += gridDim.x) {
            const WorkItem wi = decode_work(g, w);
            la.setup_tile(g.M, wi.m0, pt);
            lb.setup_tile(g.N, wi.n0, pt);
            const bool tile_full = wi.m0 + TILE_M <= g.M.size && wi.n0 + TILE_N <= g.N.size;
            for (uint32_t j = 0; j < wi.nslab; ++j, ++it) {
                const uint32_t k0 = wi.kbeg + j * TILE_K;
                __syncwarp(); // the warp is done reading the previous slab's table
#pragma unroll
                for (uint32_t h = 0; h < TILE_K / 32; ++h) {
                    const uint32_t k = k0 + h * 32 + lane;
                    int64_t x = -1, y = -1;
                    if (k < wi.kend) {
                        gett_decompose(g.K, k, x, y);
                        x *= 2;
                        y *= 2;
                    }
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
                if (tile_full && k0 + TILE_K <= wi.kend) {
                    la.template load_slab<true>(baseA, sa, kA, pt);
                    lb.template load_slab<true>(baseB, sa + A_STAGE_BYTES, kB, pt);
                } else {
                    la.template load_slab<false>(baseA, sa, kA, pt);
                    lb.template load_slab<false>(baseB, sa + A_STAGE_BYTES, kB, pt);
                }
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
            const uint32_t idesc = ptx::idesc_f16(fmt, A_VEC_K ? 0u : 1u, B_VEC_K ? 0u : 1u, TILE_M, TILE_N);
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
            for (uint32_t c = et; c < TILE_N; c += NUM_EPI_WARPS * 32) {
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
            for (uint32_t c0 = 0; c0 < TILE_N; c0 += 32) {
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

template <bool AK, bool BK>
static cudaError_t launch_tn(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    void (*k)(GettKernelArgs);
    switch (args.tile_n) {
    case 64: k = gett_umma_kernel<AK, BK, 64>; break;
    case 128: k = gett_umma_kernel<AK, BK, 128>; break;
    case 192: k = gett_umma_kernel<AK, BK, 192>; break;
    case 256: k = gett_umma_kernel<AK, BK, 256>; break;
    default: return cudaErrorInvalidValue;
    }
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    k<<<grid, NUM_THREADS, smem, stream>>>(args);
    return cudaGetLastError();
}

cudaError_t gett_launch_umma(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    const bool ak = args.loader_a == GETT_LOAD_VEC_K, bk = args.loader_b == GETT_LOAD_VEC_K;
    if (ak && bk)
        return launch_tn<true, true>(args, grid, smem, stream);
    if (ak)
        return launch_tn<true, false>(args, grid, smem, stream);
    if (bk)
        return launch_tn<false, true>(args, grid, smem, stream);
    return launch_tn<false, false>(args, grid, smem, stream);
}
