// Strict-fp32 contraction kernel: 16-byte cp.async gathers, register-blocked FFMA.
//
// One CTA of 2 TM threads owns a TM x TN tile (TM = 128 or 64) of the fused (M, N) output
// and walks its K range in slabs of 32 through a ring of shared-memory stages (Listing 4 with the
// m-/n-loops spread over the grid).  Packing (Eq. 9 / Eq. 10) is the gather of
// 16-byte pieces of the A and B sub-tensors into one of two shared layouts:
//   stride-1 mode free  ("VEC_FREE") -> [k][row]  rows contiguous, as the FMA loop reads it
//   stride-1 mode in K  ("VEC_K")    -> [row][k]  32 k = 128 B per row, 16-byte pieces
//                                       XOR-swizzled by (row / 4) % 8 so that both the
//                                       copy and the 128-bit fragment reads are
//                                       bank-conflict free
//   no usable stride-1 mode ("SCALAR") -> [k][row], gathered element by element with
//                                       4-byte cp.async (also chosen on purpose when the
//                                       vector-friendly order would scatter the stores to C)
// The macro-kernel is an 8 x (TN/16) register tile per thread fed by 128-bit shared
// loads (Sec. 3.1: outer products into a register-resident tile); unpacking
// (Eq. 11) writes alpha*acc + beta*C through C's permutation: as 128-bit stores
// along M when C's stride-1 mode leads the M order, through a shared-memory transpose
// (whole tile rows per warp, 128-bit accesses along C) when it runs along the columns.
#include "kernels.h"
#include "ptx_sm100.cuh"

namespace {

constexpr int TK = 32;
constexpr uint32_t INVALID16 = 0xFFFFFFFFu;

template <int TM, int TN>
struct FfmaSmem {
    int64_t offCM[TM];
    int64_t offCN[TN];
    uint32_t rowA[TM];       // A row offsets in elements (INVALID16 beyond M)
    uint32_t rowB[TN];
    uint32_t kTab[2][2][TK]; // [parity][A/B][k] offsets of a slab's k, in elements
};

template <int TM, int TN>
__host__ __device__ constexpr int ffma_stage_bytes() { return (TM + TN) * TK * 4; }

// Gather one operand slab: R rows x 32 k, by NT threads.  L is the operand's gett_loader_t.
template <int L, int R, int NT>
__device__ __forceinline__ void load_operand(const char* __restrict__ base, uint32_t dst,
                                             const uint32_t* rowTab, const uint32_t* kTab, int tid,
                                             bool k_fastest)
{
    if (L == GETT_LOAD_SCALAR) {
        constexpr int NP = R * TK / NT;
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const uint32_t q = tid + NT * p;
            // consecutive threads follow the direction in which the operand is denser in memory
            const uint32_t k = k_fastest ? q % TK : q / R;
            const uint32_t r = k_fastest ? q / TK : q % R;
            const uint32_t r1 = rowTab[r], k1 = kTab[k];
            const bool ok = r1 != INVALID16 && k1 != INVALID16;
            ptx::cp_async_4(dst + (k * R + r) * 4, base + (ok ? ((uint64_t)(r1 + k1) << 2) : 0), ok ? 4u : 0u);
        }
        return;
    }
    constexpr int PIECES = R * TK / 4;
    constexpr int NP = (PIECES + NT - 1) / NT;
    if (L == GETT_LOAD_VEC_K || L == GETT_LOAD_VEC_KT) {
        const uint32_t kc = tid & 7;
        // VEC_KT: the 16-byte pieces run along K's SECOND digit (the slab is 4 indices of the
        // first digit x 8 of the second, first fastest): piece kc = 4 j + c starts at k = c + 16 j
        // and holds second-digit indices 4 j .. 4 j + 3 of first-digit index c, i.e. the
        // transpose of what slots 4 j .. 4 j + 3 must hold; transpose_kt() puts that right.
        const uint32_t k1 = kTab[L == GETT_LOAD_VEC_KT ? (kc & 3) + 16 * (kc >> 2) : kc * 4];
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const uint32_t m = (tid >> 3) + (NT / 8) * p;
            if (PIECES % NT != 0 && m >= (uint32_t)R)
                break;
            const uint32_t r1 = rowTab[m];
            const bool ok = r1 != INVALID16 && k1 != INVALID16;
            ptx::cp_async_16(dst + m * 128 + ((kc ^ ((m >> 2) & 7)) << 4),
                             base + (ok ? ((uint64_t)(r1 + k1) << 2) : 0), ok ? 16u : 0u);
        }
    } else {
        constexpr int PPR = R / 4; // pieces per k row
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const uint32_t q = tid + NT * p;
            if (PIECES % NT != 0 && q >= (uint32_t)PIECES)
                break;
            const uint32_t k = q / PPR, mc = q % PPR;
            const uint32_t r1 = rowTab[mc * 4], k1 = kTab[k];
            const bool ok = r1 != INVALID16 && k1 != INVALID16;
            ptx::cp_async_16(dst + (k * R + mc * 4) * 4, base + (ok ? ((uint64_t)(r1 + k1) << 2) : 0),
                             ok ? 16u : 0u);
        }
    }
}

// In-place transposition of the 4 x 4 blocks of a [row][k] tile loaded with VEC_KT (packing
// as a transposition, Sec. 3.2.2, at the granularity of one 16-byte vector): block j of a row
// occupies slots 4 j .. 4 j + 3; before, slot 4 j + c holds (c; d = 4 j .. 4 j + 3), after,
// slot 4 j + dd holds (c = 0 .. 3; d = 4 j + dd) = k 4 (4 j + dd) .. + 3.
template <int R, int NT>
__device__ __forceinline__ void transpose_kt(char* tile, int tid)
{
    for (int b = tid; b < 2 * R; b += NT) {
        const uint32_t row = (uint32_t)b >> 1, j = (uint32_t)b & 1, sw = (row >> 2) & 7;
        float4 v[4];
#pragma unroll
        for (uint32_t c = 0; c < 4; ++c)
            v[c] = *reinterpret_cast<const float4*>(tile + row * 128 + (((4 * j + c) ^ sw) << 4));
        *reinterpret_cast<float4*>(tile + row * 128 + (((4 * j + 0) ^ sw) << 4)) = make_float4(v[0].x, v[1].x, v[2].x, v[3].x);
        *reinterpret_cast<float4*>(tile + row * 128 + (((4 * j + 1) ^ sw) << 4)) = make_float4(v[0].y, v[1].y, v[2].y, v[3].y);
        *reinterpret_cast<float4*>(tile + row * 128 + (((4 * j + 2) ^ sw) << 4)) = make_float4(v[0].z, v[1].z, v[2].z, v[3].z);
        *reinterpret_cast<float4*>(tile + row * 128 + (((4 * j + 3) ^ sw) << 4)) = make_float4(v[0].w, v[1].w, v[2].w, v[3].w);
    }
}

// Fragment of F (4 or 8, or 2) rows for 4 consecutive k from a [row][k] swizzled tile.
template <int F>
__device__ __forceinline__ void frag_kmajor(const char* tile, const uint32_t (&rows)[F], uint32_t sw,
                                            int k4, float (&out)[F][4])
{
#pragma unroll
    for (int i = 0; i < F; ++i) {
        const float4 v = *reinterpret_cast<const float4*>(tile + rows[i] * 128 + (((uint32_t)k4 ^ sw) << 4));
        out[i][0] = v.x;
        out[i][1] = v.y;
        out[i][2] = v.z;
        out[i][3] = v.w;
    }
}

template <int LA, int LB, int TN, int TM>
__global__ void __launch_bounds__(2 * TM, 256 / TM) gett_ffma_kernel(const __grid_constant__ GettKernelArgs g)
{
    constexpr int NT = 2 * TM;
    constexpr bool B_KT = LB == GETT_LOAD_VEC_KT;
    constexpr bool A_K = LA == GETT_LOAD_VEC_K, B_K = LB == GETT_LOAD_VEC_K || B_KT; // staged [row][k]
    constexpr int FN = TN / 16;                 // columns per thread (8 or 2)
    constexpr int STAGE = ffma_stage_bytes<TM, TN>();
    extern __shared__ __align__(128) uint8_t smem[];
    const int stages = g.stages;
    FfmaSmem<TM, TN>* T = reinterpret_cast<FfmaSmem<TM, TN>*>(smem + stages * STAGE);
    const uint32_t smem0 = ptx::smem_u32(smem);

    const uint32_t tiles = g.tiles_m * g.tiles_n;
    const uint32_t z = blockIdx.x / tiles;
    const uint32_t tile = blockIdx.x - z * tiles;
    const uint32_t tn = tile / g.tiles_m, tm = tile - tn * g.tiles_m;
    const uint32_t m0 = tm * TM, n0 = tn * TN;
    const uint32_t Msz = g.M.size, Nsz = g.N.size;
    const uint32_t kbeg = z * g.k_per_split;
    const uint32_t kend = min(g.K.size, kbeg + g.k_per_split);
    const int nslab = (int)((kend - kbeg + TK - 1) / TK);
    const int tid = threadIdx.x;
    // TM/8 x 16 threads with 8 x FN outputs each.  A warp is 8 (along M) x 4 (along N) of
    // them: its fragment reads touch 128 + 64 distinct bytes per k (one wavefront each).
    const int tx = ((tid >> 5) % (TM / 64)) * 8 + (tid & 7), ty = ((tid >> 5) / (TM / 64)) * 4 + ((tid >> 3) & 3);

    // ---- per-tile tables ----
    for (int r = tid; r < TM + TN; r += NT) {
        const bool isA = r < TM;
        const uint32_t idx = isA ? m0 + r : n0 + (r - TM);
        int64_t x = 0, y = 0;
        const bool ok = idx < (isA ? Msz : Nsz);
        if (ok)
            gett_decompose(isA ? g.M : g.N, idx, x, y);
        if (isA) {
            T->rowA[r] = ok ? (uint32_t)x : INVALID16;
            T->offCM[r] = ok ? y : -1;
        } else {
            T->rowB[r - TM] = ok ? (uint32_t)x : INVALID16;
            T->offCN[r - TM] = ok ? y : -1;
        }
    }
    auto fill_ktab = [&](int slab) {
        if (tid < TK) {
            const uint32_t k = kbeg + slab * TK + tid;
            uint32_t xa = INVALID16, xb = INVALID16;
            if (slab < nslab && k < kend) {
                int64_t x, y;
                gett_decompose(g.K, k, x, y);
                xa = (uint32_t)x;
                xb = (uint32_t)y;
            }
            T->kTab[slab & 1][0][tid] = xa;
            T->kTab[slab & 1][1][tid] = xb;
        }
    };
    auto issue = [&](int slab) {
        if (slab < nslab) {
            const uint32_t dst = smem0 + (slab % stages) * STAGE;
            load_operand<LA, TM, NT>(static_cast<const char*>(g.A), dst, T->rowA, T->kTab[slab & 1][0], tid,
                                 g.a_kmajor != 0);
            load_operand<LB, TN, NT>(static_cast<const char*>(g.B), dst + TM * TK * 4, T->rowB,
                                 T->kTab[slab & 1][1], tid, g.b_kmajor != 0);
        }
        ptx::cp_async_commit();
    };

    // ---- prologue: fill stages - 1 slabs ----
    for (int s = 0; s < stages - 1; ++s) {
        fill_ktab(s);
        __syncthreads();
        issue(s);
    }
    fill_ktab(stages - 1);

    // rows / columns this thread accumulates
    uint32_t rows[8], cols[FN];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        rows[i] = (i < 4 ? 0 : TM / 2) + tx * 4 + (i & 3);
#pragma unroll
    for (int j = 0; j < FN; ++j)
        cols[j] = FN == 8 ? (j < 4 ? 0 : 64) + ty * 4 + (j & 3) : ty * FN + j;
    const uint32_t swA = tx & 7;
    const uint32_t swB = FN == 8 ? (ty & 7) : ((ty * FN) >> 2) & 7;

    // beta != 0: ask L2 for the old values of this thread's part of C now, so that the
    // read-modify-write at the end finds them on chip (the request holds no register).
    // The offset tables were completed before the prologue's first barrier.
    if (g.beta != 0.f && g.split_k == 1 && stages >= 2) {
        if (FN == 8 && (g.c_vec == 2 || g.c_vec == 4)) {
            // the same (row, 16-byte group) assignment as the unpacking below
            const int warp = tid >> 5, lane = tid & 31;
            const int64_t cn = T->offCN[g.c_vec == 4 ? (lane >> 3) + 16 * (lane & 7) : lane * 4];
#pragma unroll 4
            for (int r = 0; r < 16; ++r) {
                const int64_t cm = T->offCM[warp * 16 + r];
                if (cm >= 0 && cn >= 0)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(g.C + cm + cn));
            }
        } else if (g.c_vec == 1) {
#pragma unroll
            for (int j = 0; j < FN; ++j) {
                const int64_t cn = T->offCN[cols[j]];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int64_t cm = T->offCM[rows[4 * h]];
                    if (cm >= 0 && cn >= 0)
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(g.C + cm + cn));
                }
            }
        }
    }

    // Accumulators are held in pairs so that one packed instruction (two independent
    // round-to-nearest fp32 FMAs, results identical to two scalar fmaf) updates two of
    // them.  Pairs run along rows when A's fragment delivers neighbouring rows together
    // ([k][row] staging), else along columns.
    constexpr bool PAIR_ROWS = !A_K || B_K;
    constexpr int PI = PAIR_ROWS ? 4 : 8, PJ = PAIR_ROWS ? FN : FN / 2;
    float2 accp[PI][PJ];
#pragma unroll
    for (int i = 0; i < PI; ++i)
#pragma unroll
        for (int j = 0; j < PJ; ++j)
            accp[i][j] = make_float2(0.f, 0.f);
#define ACC(i, j)                                                                       \
    (PAIR_ROWS ? (((i) & 1) ? accp[(i) / 2 % PI][(j) % PJ].y : accp[(i) / 2 % PI][(j) % PJ].x) \
               : (((j) & 1) ? accp[(i) % PI][(j) / 2 % PJ].y : accp[(i) % PI][(j) / 2 % PJ].x))

    for (int slab = 0; slab < nslab; ++slab) {
        // all but the newest (stages - 2) copy groups have landed => this slab is complete
        if (stages == 2)
            ptx::cp_async_wait<0>();
        else if (stages == 3)
            ptx::cp_async_wait<1>();
        else
            ptx::cp_async_wait<2>();
        __syncthreads(); // slab's data visible; previous slab's stage free; kTab ready
        issue(slab + stages - 1);
        fill_ktab(slab + stages); // for the issue of the next iteration
        const char* As = reinterpret_cast<const char*>(smem) + (slab % stages) * STAGE;
        const char* Bs = As + TM * TK * 4;
        if (B_KT) { // B's rows have landed transposed block by block
            transpose_kt<TN, NT>(reinterpret_cast<char*>(smem) + (slab % stages) * STAGE + TM * TK * 4, tid);
            __syncthreads();
        }
#pragma unroll
        for (int k4 = 0; k4 < TK / 4 && !GETT_DBG(g, 64); ++k4) { // (debug & 64: experiment, no math)
            float a[8][4], b[FN][4];
            if (A_K) {
                frag_kmajor<8>(As, rows, swA, k4, a);
            } else {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const float* row = reinterpret_cast<const float*>(As) + (k4 * 4 + kk) * TM;
                    const float4 lo = *reinterpret_cast<const float4*>(row + tx * 4);
                    const float4 hi = *reinterpret_cast<const float4*>(row + TM / 2 + tx * 4);
                    a[0][kk] = lo.x; a[1][kk] = lo.y; a[2][kk] = lo.z; a[3][kk] = lo.w;
                    a[4][kk] = hi.x; a[5][kk] = hi.y; a[6][kk] = hi.z; a[7][kk] = hi.w;
                }
            }
            if (B_K) {
                frag_kmajor<FN>(Bs, cols, swB, k4, b);
            } else {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const float* row = reinterpret_cast<const float*>(Bs) + (k4 * 4 + kk) * TN;
                    if constexpr (FN == 8) {
                        const float4 lo = *reinterpret_cast<const float4*>(row + ty * 4);
                        const float4 hi = *reinterpret_cast<const float4*>(row + 64 + ty * 4);
                        b[0][kk] = lo.x; b[1][kk] = lo.y; b[2][kk] = lo.z; b[3][kk] = lo.w;
                        b[4][kk] = hi.x; b[5][kk] = hi.y; b[6][kk] = hi.z; b[7][kk] = hi.w;
                    } else {
                        const float2 v = *reinterpret_cast<const float2*>(row + ty * 2);
                        b[0][kk] = v.x;
                        b[1][kk] = v.y;
                    }
                }
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                if constexpr (A_K && B_K) {
                    // both fragments deliver 4 k of ONE row / column per load: neither operand
                    // has neighbours in adjacent registers, and building the pairs costs more
                    // issue slots than the packed instruction saves -> plain FMAs
#pragma unroll
                    for (int i = 0; i < 8; ++i)
#pragma unroll
                        for (int j = 0; j < FN; ++j)
                            ACC(i, j) = fmaf(a[i][kk], b[j][kk], ACC(i, j));
                } else if constexpr (PAIR_ROWS) {
                    float2 b2[FN];
#pragma unroll
                    for (int j = 0; j < FN; ++j)
                        b2[j] = make_float2(b[j][kk], b[j][kk]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 a2 = make_float2(a[2 * i][kk], a[2 * i + 1][kk]);
#pragma unroll
                        for (int j = 0; j < FN; ++j)
                            accp[i][j] = __ffma2_rn(a2, b2[j], accp[i][j]);
                    }
                } else {
                    float2 b2[FN / 2];
#pragma unroll
                    for (int j = 0; j < FN / 2; ++j)
                        b2[j] = make_float2(b[2 * j][kk], b[2 * j + 1][kk]);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float2 a2 = make_float2(a[i][kk], a[i][kk]);
#pragma unroll
                        for (int j = 0; j < FN / 2; ++j)
                            accp[i][j] = __ffma2_rn(a2, b2[j], accp[i][j]);
                    }
                }
            }
        }
    }
    ptx::cp_async_wait_all();
    __syncthreads();

    // ---- unpack: C <- alpha * acc + beta * C (or the raw slice sums under split-K) ----
    const float alpha = g.alpha, beta = g.beta;
    const bool vec_m = g.c_vec == 1;
    if (GETT_DBG(g, 2)) // experiment: no stores
        return;
    if (FN == 8 && (g.c_vec == 2 || g.c_vec == 4) && g.split_k == 1) {
        // C's stride-1 mode runs along the tile's columns.  The scaled accumulators pass
        // through shared memory (the stage ring is free now) so that a warp owns whole tile
        // rows and its 32 lanes cover the row's 128 "slots", four consecutive slots being
        // one 16-byte vector of C: the read-modify-write of C then moves whole runs of C
        // per instruction instead of 16-byte pieces (Eq. 11 as a transposition).
        //   c_vec == 2: slot = column
        //   c_vec == 4: column = a + 4 p (a: piece of B's stride-1 mode, p along C's)
        //               -> slot = 32 a + p
        // 16-byte groups are XOR-swizzled by (row / 4) % 8: conflict-free for the 128-bit
        // writes (lanes = rows) and reads (lanes = groups), two-way for the scalar writes.
        float* S = reinterpret_cast<float*>(smem);
        if (g.c_vec == 2) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t row = rows[i];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t c4 = cols[(4 * h) % FN] >> 2;
                    *reinterpret_cast<float4*>(S + row * TN + ((c4 ^ ((row >> 2) & 7)) << 2)) =
                        make_float4(alpha * ACC(i, (4 * h) % FN), alpha * ACC(i, (4 * h + 1) % FN),
                                    alpha * ACC(i, (4 * h + 2) % FN), alpha * ACC(i, (4 * h + 3) % FN));
                }
            }
        } else {
            // cols[j] = (j < 4 ? 0 : 64) + 4 ty + j % 4  ->  a = j % 4, p = ty + (j < 4 ? 0 : 16)
            const uint32_t sw = (uint32_t)(tx & 7) << 2; // (row / 4) % 8 of all my rows
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float* Srow = S + ((i < 4 ? 0 : TM / 2) + tx * 4 + (i & 3)) * TN;
#pragma unroll
                for (int j = 0; j < FN; ++j)
                    Srow[((j & 3) * (TN / 4) + (j < 4 ? 0 : 16) + ty) ^ sw] = alpha * ACC(i, j);
            }
        }
        __syncthreads();
        const int warp = tid >> 5, lane = tid & 31;
        const int64_t cn = T->offCN[g.c_vec == 4 ? (lane >> 3) + 16 * (lane & 7) : lane * 4];
#pragma unroll
        for (int r0 = 0; r0 < 16; r0 += 8) {
            float4 old[8];
            float4* dst[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const int64_t cm = T->offCM[warp * 16 + r0 + r];
                dst[r] = (cm >= 0 && cn >= 0) ? reinterpret_cast<float4*>(g.C + cm + cn) : nullptr;
                old[r] = (beta != 0.f && dst[r]) ? __ldcg(dst[r]) : make_float4(0, 0, 0, 0);
            }
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const uint32_t row = warp * 16 + r0 + r;
                const float4 v = *reinterpret_cast<const float4*>(S + row * TN + ((lane ^ ((row >> 2) & 7)) << 2));
                if (dst[r])
                    *dst[r] = make_float4(fmaf(beta, old[r].x, v.x), fmaf(beta, old[r].y, v.y),
                                          fmaf(beta, old[r].z, v.z), fmaf(beta, old[r].w, v.w));
            }
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < FN; ++j) {
        const int64_t cn = T->offCN[cols[j]];
        if (cn < 0)
            continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t r0 = rows[4 * h];
            if (g.split_k > 1) {
                float* dst = g.ws + ((size_t)z * Nsz + n0 + cols[j]) * Msz + m0 + r0;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (m0 + r0 + i < Msz)
                        dst[i] = ACC(4 * h + i, j);
            } else if (vec_m) {
                const int64_t cm = T->offCM[r0];
                if (cm < 0)
                    continue;
                float4* dst = reinterpret_cast<float4*>(g.C + cm + cn);
                float4 v = make_float4(alpha * ACC(4 * h, j), alpha * ACC(4 * h + 1, j),
                                       alpha * ACC(4 * h + 2, j), alpha * ACC(4 * h + 3, j));
                if (beta != 0.f) {
                    const float4 o = *dst;
                    v.x = fmaf(beta, o.x, v.x);
                    v.y = fmaf(beta, o.y, v.y);
                    v.z = fmaf(beta, o.z, v.z);
                    v.w = fmaf(beta, o.w, v.w);
                }
                *dst = v;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int64_t cm = T->offCM[r0 + i];
                    if (cm < 0)
                        continue;
                    float* dst = g.C + cm + cn;
                    float v = alpha * ACC(4 * h + i, j);
                    if (beta != 0.f)
                        v = fmaf(beta, *dst, v);
                    *dst = v;
                }
            }
        }
    }
}

template <int LA, int LB>
cudaError_t launch_tn(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    void (*k)(GettKernelArgs);
    if (args.tile_n == 128 && args.tile_m == 128)
        k = gett_ffma_kernel<LA, LB, 128, 128>;
    else if (args.tile_n == 128 && args.tile_m == 64)
        k = gett_ffma_kernel<LA, LB, 128, 64>;
    else if (args.tile_n == 32 && args.tile_m == 128)
        k = gett_ffma_kernel<LA, LB, 32, 128>;
    else
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    k<<<grid, 2 * args.tile_m, smem, stream>>>(args);
    return cudaGetLastError();
}

template <int LA>
cudaError_t launch_b(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    if (args.loader_b == GETT_LOAD_VEC_KT) { // (planned only together with a K-major A)
        if constexpr (LA == GETT_LOAD_VEC_K)
            return launch_tn<LA, GETT_LOAD_VEC_KT>(args, grid, smem, stream);
        else
            return cudaErrorInvalidValue;
    }
    switch (args.loader_b) {
    case GETT_LOAD_VEC_K: return launch_tn<LA, GETT_LOAD_VEC_K>(args, grid, smem, stream);
    case GETT_LOAD_VEC_FREE: return launch_tn<LA, GETT_LOAD_VEC_FREE>(args, grid, smem, stream);
    default: return launch_tn<LA, GETT_LOAD_SCALAR>(args, grid, smem, stream);
    }
}

#undef ACC

} // namespace

int gett_ffma_smem_bytes(int tile_m, int tile_n, int stages)
{
    if (tile_m == 64)
        return stages * ffma_stage_bytes<64, 128>() + (int)sizeof(FfmaSmem<64, 128>);
    return tile_n == 128 ? stages * ffma_stage_bytes<128, 128>() + (int)sizeof(FfmaSmem<128, 128>)
                         : stages * ffma_stage_bytes<128, 32>() + (int)sizeof(FfmaSmem<128, 32>);
}

cudaError_t gett_launch_ffma(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream)
{
    switch (args.loader_a) {
    case GETT_LOAD_VEC_K: return launch_b<GETT_LOAD_VEC_K>(args, grid, smem, stream);
    case GETT_LOAD_VEC_FREE: return launch_b<GETT_LOAD_VEC_FREE>(args, grid, smem, stream);
    default: return launch_b<GETT_LOAD_SCALAR>(args, grid, smem, stream);
    }
}
