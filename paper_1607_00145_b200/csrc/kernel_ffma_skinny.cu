// Strict-fp32 kernel for the bandwidth-bound "tensor times small matrix" regime:
// N <= 64, K <= 64, A staged K-major (its stride-1 mode is contracted).
//
// The whole of B (K x N) stays in shared memory for the life of the CTA, so the
// loop nest of Listing 4 degenerates to the m-loop alone: persistent CTAs stream
// 256-row tiles of A through a cp.async ring (packing, Eq. 9), every thread holds a
// 4-row x CPT-column register tile (micro-kernel, Sec. 3.1), and C is written once
// with 32 consecutive rows per warp store (Eq. 11).  Nothing but A is read from HBM
// and nothing but C is written, which is the compulsory traffic.
#include "kernels.h"
#include "ptx_sm100.cuh"

namespace {

constexpr int ROWS = 256, NT = 256, KMAX = 64, STAGES = 3;
constexpr int QL = NT / 4;      // threads per column group
constexpr int RPT = ROWS / QL;  // rows per thread: q, q + QL, ...
// Row tables are alive from the moment they are filled (one iteration before the tile's
// copy is issued) until the tile's epilogue: STAGES + 1 tiles at any time.
constexpr int TSLOTS = STAGES + 1;

struct SkinnyTables {
    int64_t offCM[TSLOTS][ROWS]; // C offset of each tile row (-1 beyond M)
    int64_t offCN[64];
    uint32_t kA[KMAX / 4];       // A offset of each 4-wide k piece, 16-byte units
};

// Row pitch (floats) of an A tile: a multiple of 4 whose quarter is odd, so that the
// 128-bit reads of eight consecutive rows fall into eight different bank groups.
__host__ __device__ constexpr uint32_t skinny_pitch(uint32_t K) { return K + (K % 8 == 0 ? 4 : 8); }
// ... with VR (below): a power of two >= 32, the 16-byte pieces of a row XOR-swizzled by (row / 4) % 8
__host__ __device__ constexpr uint32_t skinny_pitch_vr(uint32_t K) { return K <= 32 ? 32 : 64; }

// KCT: K / 4 when known at compile time (the k loop is then fully unrolled), 0 = run time
// VR : four consecutive tile rows are one aligned 16-byte vector of C.  A thread then owns rows
//      4 q .. 4 q + 3 (instead of q, q + 64, ...) and stores 128-bit vectors along the rows.
template <int CPT, int KCT, bool VR>
__global__ void __launch_bounds__(NT, 2) gett_ffma_skinny_kernel(const __grid_constant__ GettKernelArgs g)
{
    constexpr int NP = 4 * CPT; // padded row of B in shared memory
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t K = g.K.size, N = g.N.size, Msz = g.M.size;
    const uint32_t KC = KCT ? (uint32_t)KCT : K / 4;
    const uint32_t pitch = VR ? skinny_pitch_vr(K) : skinny_pitch(K);
    // byte offset of piece kc inside its row
    auto piece = [&](uint32_t row, uint32_t kc) { return (VR ? (kc ^ ((row >> 2) & 7)) : kc) * 16; };
    const uint32_t tile_bytes = ROWS * pitch * 4;
    float* Bs = reinterpret_cast<float*>(smem);                       // [K][NP]
    uint8_t* ring = smem + K * NP * 4;
    SkinnyTables* T = reinterpret_cast<SkinnyTables*>(ring + STAGES * tile_bytes);
    const uint32_t ring_u32 = ptx::smem_u32(ring);
    const int tid = threadIdx.x;
    const uint32_t ntiles = g.tiles_m;

    // ---- the tile-independent tables, once (B follows the first copies of A, below) ----
    auto fill_b = [&]() {
        for (uint32_t i = tid; i < K * NP; i += NT) {
            const uint32_t k = i / NP, n = i - k * NP;
            float v = 0.f;
            if (n < N) {
                int64_t bn, cn, ak, bk;
                gett_decompose(g.N, n, bn, cn);
                gett_decompose(g.K, k, ak, bk);
                v = __ldg(static_cast<const float*>(g.B) + bn + bk);
            }
            Bs[i] = v;
        }
    };
    if (tid < 64) {
        int64_t bn, cn = -1;
        if ((uint32_t)tid < N)
            gett_decompose(g.N, tid, bn, cn);
        T->offCN[tid] = cn;
    }
    if ((uint32_t)tid < KC) {
        int64_t ak, bk;
        gett_decompose(g.K, tid * 4, ak, bk);
        T->kA[tid] = (uint32_t)(ak >> 2);
    }
    // Thread `tid` owns rows tid and tid + NT of every tile: it computes their offsets,
    // copies their K/4 pieces, and publishes their C offsets for whoever accumulates them.
    // Each CTA takes a contiguous run of row tiles, so that per column of C it writes one
    // sequential stream (better DRAM page locality than tiles strided by the grid size).
    const uint32_t chunk = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t t_begin = blockIdx.x * chunk;
    const uint32_t t_end = min(ntiles, t_begin + chunk);
    const bool affine_rows = g.M.ndig == 1 && ROWS == NT;
    auto issue = [&](uint32_t it) {
        const uint32_t t = t_begin + it;
        if (t < t_end) {
#pragma unroll
            for (int h = 0; h < ROWS / NT; ++h) {
                const uint32_t row = tid + h * NT;
                const uint32_t m = t * ROWS + row;
                int64_t x = 0, y = -1;
                const bool ok = m < Msz;
                if (ok)
                    gett_decompose(g.M, m, x, y);
                T->offCM[it % TSLOTS][row] = y;
                const char* src = static_cast<const char*>(g.A) + (ok ? x * 4 : 0);
                const uint32_t dst = ring_u32 + (it % STAGES) * tile_bytes + row * pitch * 4;
                if (!affine_rows) {
#pragma unroll 2
                    for (uint32_t kc = 0; kc < KC; ++kc)
                        ptx::cp_async_16(dst + piece(row, kc), src + (ok ? ((uint64_t)T->kA[kc] << 4) : 0),
                                         ok ? 16u : 0u);
                }
            }
            if (affine_rows) {
                // M is a single digit: a row's offset is m * stride, so consecutive threads can
                // take consecutive 16-byte pieces of the tile (full 128-byte lines per warp)
                const uint32_t dst0 = ring_u32 + (it % STAGES) * tile_bytes;
#pragma unroll(KCT ? KCT : 2)
                for (uint32_t p = 0; p < KC; ++p) {
                    const uint32_t q = tid + NT * p;
                    const uint32_t row = q / KC, kc = q - row * KC;
                    const uint32_t m = t * ROWS + row;
                    const bool ok = m < Msz;
                    ptx::cp_async_16(dst0 + row * pitch * 4 + piece(row, kc),
                                     static_cast<const char*>(g.A) +
                                         (ok ? ((uint64_t)m * (uint64_t)g.M.sX[0] * 4 + ((uint64_t)T->kA[kc] << 4)) : 0),
                                     ok ? 16u : 0u);
                }
            }
        }
        ptx::cp_async_commit();
    };

    __syncthreads(); // kA, offCN ready
    for (uint32_t s = 0; s < STAGES - 1; ++s)
        issue(s);
    fill_b(); // while the first tiles are on their way; visible after the loop's first barrier

    const uint32_t q = tid % QL, cg = tid / QL; // rows q + QL i; a warp shares one column group
    const float alpha = g.alpha, beta = g.beta;
    int64_t cn[CPT]; // C offsets of my columns (the same for every tile)
#pragma unroll
    for (int j = 0; j < CPT; ++j)
        cn[j] = T->offCN[cg * CPT + j];
    for (uint32_t it = 0; t_begin + it < t_end; ++it) {
        ptx::cp_async_wait<STAGES - 2>();
        __syncthreads(); // tile `it` and its row table visible; the stage of tile it-1 is free
        issue(it + STAGES - 1);
        const float* As = reinterpret_cast<const float*>(ring + (it % STAGES) * tile_bytes);
        // accumulators are kept as column pairs: one packed instruction performs two
        // independent round-to-nearest fp32 FMAs (same results as two scalar fmaf)
        float2 acc[RPT][CPT / 2];
#pragma unroll
        for (int i = 0; i < RPT; ++i)
#pragma unroll
            for (int j = 0; j < CPT / 2; ++j)
                acc[i][j] = make_float2(0.f, 0.f);
#pragma unroll(KCT ? KCT : 2)
        for (uint32_t kc = 0; kc < KC && !GETT_DBG(g, 64); ++kc) { // (debug & 64: experiment, no math)
            float4 a[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const uint32_t row = VR ? 4 * q + i : q + QL * i;
                a[i] = *reinterpret_cast<const float4*>(reinterpret_cast<const char*>(As) + row * pitch * 4 +
                                                        piece(row, kc));
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                float2 b[CPT / 2];
                const float* brow = Bs + (kc * 4 + kk) * NP + cg * CPT;
                // cg * CPT * 4 bytes is 16-byte aligned when CPT % 4 == 0, else 8-byte aligned
#pragma unroll
                for (int j = 0; j < CPT; j += 2) {
                    if (CPT % 4 == 0 && j % 4 == 0) {
                        const float4 v = *reinterpret_cast<const float4*>(brow + j);
                        b[j / 2] = make_float2(v.x, v.y);
                        b[j / 2 + 1] = make_float2(v.z, v.w);
                    } else if (CPT % 4 != 0) {
                        b[j / 2] = *reinterpret_cast<const float2*>(brow + j);
                    }
                }
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const float av = kk == 0 ? a[i].x : kk == 1 ? a[i].y : kk == 2 ? a[i].z : a[i].w;
                    const float2 a2 = make_float2(av, av);
#pragma unroll
                    for (int j = 0; j < CPT / 2; ++j)
                        acc[i][j] = __ffma2_rn(a2, b[j], acc[i][j]);
                }
            }
        }
        const int64_t* offCM = T->offCM[it % TSLOTS];
        if constexpr (VR) {
            const int64_t cm = offCM[4 * q];
            if (cm < 0 || GETT_DBG(g, 2)) // (debug & 2: experiment, no stores)
                continue;
#pragma unroll
            for (int j = 0; j < CPT; ++j) {
                if (cn[j] < 0)
                    continue;
                float4* dst = reinterpret_cast<float4*>(g.C + cm + cn[j]);
                float4 v;
                v.x = alpha * ((j & 1) ? acc[0][j / 2].y : acc[0][j / 2].x);
                v.y = alpha * ((j & 1) ? acc[1][j / 2].y : acc[1][j / 2].x);
                v.z = alpha * ((j & 1) ? acc[2][j / 2].y : acc[2][j / 2].x);
                v.w = alpha * ((j & 1) ? acc[3][j / 2].y : acc[3][j / 2].x);
                if (beta != 0.f) {
                    const float4 o = __ldcg(dst);
                    v.x = fmaf(beta, o.x, v.x);
                    v.y = fmaf(beta, o.y, v.y);
                    v.z = fmaf(beta, o.z, v.z);
                    v.w = fmaf(beta, o.w, v.w);
                }
                *dst = v;
            }
        } else {
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int64_t cm = offCM[q + QL * i];
                if (cm < 0 || GETT_DBG(g, 2)) // (debug & 2: experiment, no stores)
                    continue;
                float* crow = g.C + cm;
                float old[CPT];
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    old[j] = (beta != 0.f && cn[j] >= 0) ? __ldcg(crow + cn[j]) : 0.f;
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    if (cn[j] >= 0)
                        crow[cn[j]] = fmaf(beta, old[j], alpha * ((j & 1) ? acc[i][j / 2].y : acc[i][j / 2].x));
            }
        }
    }
    ptx::cp_async_wait_all();
}

// ---- the same regime with A staged MN-major (A's stride-1 mode is a free mode) ----
// A tile is [k][256 rows] in shared memory, filled with 16-byte pieces of four consecutive
// rows; a thread owns the four rows 4 q .. 4 q + 3 (one 128-bit read per k delivers all four)
// and CPT columns, and writes C with 128-bit stores along the rows when four consecutive rows
// are one aligned vector of C.
struct SkinnyMnTables {
    int64_t offCM[TSLOTS][ROWS]; // C offset of each tile row (-1 beyond M)
    int64_t offCN[64];
    uint32_t kA[KMAX];           // A offset of each k, 16-byte units
};

// KT: K when known at compile time (the k loop is then fully unrolled), 0 = run time
template <int CPT, int KT>
__global__ void __launch_bounds__(NT, 2) gett_ffma_skinny_mn_kernel(const __grid_constant__ GettKernelArgs g)
{
    constexpr int NP = 4 * CPT; // padded row of B in shared memory
    constexpr uint32_t NONE = 0xFFFFFFFFu;
    extern __shared__ __align__(16) uint8_t smem[];
    const uint32_t K = KT ? (uint32_t)KT : g.K.size, N = g.N.size, Msz = g.M.size;
    const uint32_t tile_bytes = K * ROWS * 4;
    float* Bs = reinterpret_cast<float*>(smem);                       // [K][NP]
    uint8_t* ring = smem + K * NP * 4;
    SkinnyMnTables* T = reinterpret_cast<SkinnyMnTables*>(ring + STAGES * tile_bytes);
    const uint32_t ring_u32 = ptx::smem_u32(ring);
    const int tid = threadIdx.x;
    const uint32_t ntiles = g.tiles_m;

    auto fill_b = [&]() {
        for (uint32_t i = tid; i < K * NP; i += NT) {
            const uint32_t k = i / NP, n = i - k * NP;
            float v = 0.f;
            if (n < N) {
                int64_t bn, cn, ak, bk;
                gett_decompose(g.N, n, bn, cn);
                gett_decompose(g.K, k, ak, bk);
                v = __ldg(static_cast<const float*>(g.B) + bn + bk);
            }
            Bs[i] = v;
        }
    };
    if (tid < 64) {
        int64_t bn, cn = -1;
        if ((uint32_t)tid < N)
            gett_decompose(g.N, tid, bn, cn);
        T->offCN[tid] = cn;
    }
    if ((uint32_t)tid < K) {
        int64_t ak, bk;
        gett_decompose(g.K, tid, ak, bk);
        T->kA[tid] = (uint32_t)(ak >> 2);
    }
    const uint32_t chunk = (ntiles + gridDim.x - 1) / gridDim.x;
    const uint32_t t_begin = blockIdx.x * chunk;
    const uint32_t t_end = min(ntiles, t_begin + chunk);
    // Thread tid publishes the C offset of tile row tid, and copies the pieces (k, quad) with
    // quad = tid % 64 (rows 4 quad ..), k = tid / 64 + 4 p: lanes run along the rows.
    const uint32_t quad = tid & 63, kq = tid >> 6;
    auto issue = [&](uint32_t it) {
        const uint32_t t = t_begin + it;
        if (t < t_end) {
            const uint32_t m = t * ROWS + tid;
            T->offCM[it % TSLOTS][tid] = m < Msz ? gett_offset_y(g.M, m) : -1;
            const uint32_t mq = t * ROWS + 4 * quad;
            uint32_t x4 = NONE; // (M's leading extent is a multiple of 4: a quad is inside M or outside)
            if (mq < Msz) {
                int64_t x, y;
                gett_decompose(g.M, mq, x, y);
                x4 = (uint32_t)(x >> 2);
            }
            const uint32_t dst = ring_u32 + (it % STAGES) * tile_bytes + quad * 16;
            const char* base = static_cast<const char*>(g.A);
#pragma unroll(KT ? KT / 4 : 2)
            for (uint32_t k = kq; k < K; k += NT / 64) {
                const bool ok = x4 != NONE;
                ptx::cp_async_16(dst + k * (ROWS * 4), base + (ok ? ((uint64_t)(x4 + T->kA[k]) << 4) : 0),
                                 ok ? 16u : 0u);
            }
        }
        ptx::cp_async_commit();
    };

    __syncthreads(); // kA, offCN ready
    for (uint32_t s = 0; s < STAGES - 1; ++s)
        issue(s);
    fill_b(); // while the first tiles are on their way; visible after the loop's first barrier

    const uint32_t q = tid % QL, cg = tid / QL; // rows 4 q ..; a warp shares one column group
    const float alpha = g.alpha, beta = g.beta;
    const bool vec_rows = g.c_vec == 1;
    int64_t cn[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j)
        cn[j] = T->offCN[cg * CPT + j];
    for (uint32_t it = 0; t_begin + it < t_end; ++it) {
        ptx::cp_async_wait<STAGES - 2>();
        __syncthreads(); // tile `it` and its row table visible; the stage of tile it-1 is free
        issue(it + STAGES - 1);
        const float* As = reinterpret_cast<const float*>(ring + (it % STAGES) * tile_bytes) + 4 * q;
        float2 acc[4][CPT / 2]; // column pairs: one packed instruction = two independent fp32 FMAs
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < CPT / 2; ++j)
                acc[i][j] = make_float2(0.f, 0.f);
#pragma unroll(KT ? KT : 4)
        for (uint32_t k = 0; k < K && !GETT_DBG(g, 64); ++k) { // (debug & 64: experiment, no math)
            const float4 a = *reinterpret_cast<const float4*>(As + k * ROWS);
            float2 b[CPT / 2];
            const float* brow = Bs + k * NP + cg * CPT;
#pragma unroll
            for (int j = 0; j < CPT; j += 2) {
                if (CPT % 4 == 0 && j % 4 == 0) {
                    const float4 v = *reinterpret_cast<const float4*>(brow + j);
                    b[j / 2] = make_float2(v.x, v.y);
                    b[j / 2 + 1] = make_float2(v.z, v.w);
                } else if (CPT % 4 != 0) {
                    b[j / 2] = *reinterpret_cast<const float2*>(brow + j);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float av = i == 0 ? a.x : i == 1 ? a.y : i == 2 ? a.z : a.w;
                const float2 a2 = make_float2(av, av);
#pragma unroll
                for (int j = 0; j < CPT / 2; ++j)
                    acc[i][j] = __ffma2_rn(a2, b[j], acc[i][j]);
            }
        }
        if (GETT_DBG(g, 2)) // (experiment: no stores)
            continue;
        const int64_t* offCM = T->offCM[it % TSLOTS] + 4 * q;
        if (vec_rows) {
            const int64_t cm = offCM[0];
            if (cm < 0)
                continue;
#pragma unroll
            for (int j = 0; j < CPT; ++j) {
                if (cn[j] < 0)
                    continue;
                float4* dst = reinterpret_cast<float4*>(g.C + cm + cn[j]);
                float4 v;
                v.x = alpha * ((j & 1) ? acc[0][j / 2].y : acc[0][j / 2].x);
                v.y = alpha * ((j & 1) ? acc[1][j / 2].y : acc[1][j / 2].x);
                v.z = alpha * ((j & 1) ? acc[2][j / 2].y : acc[2][j / 2].x);
                v.w = alpha * ((j & 1) ? acc[3][j / 2].y : acc[3][j / 2].x);
                if (beta != 0.f) {
                    const float4 o = __ldcg(dst);
                    v.x = fmaf(beta, o.x, v.x);
                    v.y = fmaf(beta, o.y, v.y);
                    v.z = fmaf(beta, o.z, v.z);
                    v.w = fmaf(beta, o.w, v.w);
                }
                *dst = v;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t cm = offCM[i];
                if (cm < 0)
                    continue;
                float* crow = g.C + cm;
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    if (cn[j] >= 0) {
                        const float v = alpha * ((j & 1) ? acc[i][j / 2].y : acc[i][j / 2].x);
                        crow[cn[j]] = beta != 0.f ? fmaf(beta, __ldcg(crow + cn[j]), v) : v;
                    }
            }
        }
    }
    ptx::cp_async_wait_all();
}

} // namespace

static int skinny_cpt(uint32_t N) { return (int)((N + 3) / 4 + 1) & ~1; } // even, 4 * cpt >= N

int gett_ffma_skinny_mn_smem_bytes(int N, int K)
{
    return K * 4 * skinny_cpt((uint32_t)N) * 4 + STAGES * K * ROWS * 4 + (int)sizeof(SkinnyMnTables);
}

int gett_ffma_skinny_smem_bytes(int N, int K, int vec_rows)
{
    const int pitch = vec_rows ? (int)skinny_pitch_vr((uint32_t)K) : (int)skinny_pitch((uint32_t)K);
    return K * 4 * skinny_cpt((uint32_t)N) * 4 + STAGES * ROWS * pitch * 4 + (int)sizeof(SkinnyTables);
}

int gett_ffma_skinny_max_k() { return KMAX; }

int gett_ffma_skinny_rows() { return ROWS; }

cudaError_t gett_launch_ffma_skinny(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    const int cpt = skinny_cpt(args.N.size);
    void (*k)(GettKernelArgs);
    const uint32_t K = args.K.size;
    if (args.loader_a == GETT_LOAD_VEC_FREE) { // A staged MN-major
#define SKINNY_MN_PICK(CPT) k = K == 24 ? gett_ffma_skinny_mn_kernel<CPT, 24> : K == 32 ? gett_ffma_skinny_mn_kernel<CPT, 32> \
                                : K == 48 ? gett_ffma_skinny_mn_kernel<CPT, 48> : gett_ffma_skinny_mn_kernel<CPT, 0>
        switch (cpt) {
        case 2: SKINNY_MN_PICK(2); break;
        case 4: SKINNY_MN_PICK(4); break;
        case 6: SKINNY_MN_PICK(6); break;
        case 8: SKINNY_MN_PICK(8); break;
        case 10: SKINNY_MN_PICK(10); break;
        case 12: SKINNY_MN_PICK(12); break;
        case 14: SKINNY_MN_PICK(14); break;
        case 16: SKINNY_MN_PICK(16); break;
        default: return cudaErrorInvalidValue;
        }
#undef SKINNY_MN_PICK
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess)
            return e;
        k<<<grid, NT, smem, stream>>>(args);
        return cudaGetLastError();
    }
#define SKINNY_PICK(CPT)                                                                                   \
    k = vr ? (K == 24   ? gett_ffma_skinny_kernel<CPT, 6, true>                                                \
              : K == 32 ? gett_ffma_skinny_kernel<CPT, 8, true>                                                \
                        : gett_ffma_skinny_kernel<CPT, 0, true>)                                               \
           : (K == 24   ? gett_ffma_skinny_kernel<CPT, 6, false>                                               \
              : K == 32 ? gett_ffma_skinny_kernel<CPT, 8, false>                                               \
                        : gett_ffma_skinny_kernel<CPT, 0, false>)
    const bool vr = args.c_vec == 1; // four consecutive rows are one aligned vector of C
    switch (cpt) {
    case 2: SKINNY_PICK(2); break;
    case 4: SKINNY_PICK(4); break;
    case 6: SKINNY_PICK(6); break;
    case 8: SKINNY_PICK(8); break;
    case 10: SKINNY_PICK(10); break;
    case 12: SKINNY_PICK(12); break;
    case 14: SKINNY_PICK(14); break;
    case 16: SKINNY_PICK(16); break;
    default: return cudaErrorInvalidValue;
    }
#undef SKINNY_PICK
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    k<<<grid, NT, smem, stream>>>(args);
    return cudaGetLastError();
}
