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
#include "umma_raster.h"

// The file is compiled a second time, with GETT_UMMA_CLUSTER defined, by the source that adds
// the CTA-pair variant (two CTAs of a cluster work on two neighbouring tile columns of one
// tile row and share the A tile: each fetches half of it for both).  Work distribution then
// runs over tile pairs and clusters instead of tiles and CTAs.
#ifdef GETT_UMMA_CLUSTER
#define GETT_WB (blockIdx.x >> 1)  // this CTA's position in the work list ...
#define GETT_WG (gridDim.x >> 1)   // ... and the list's stride
#define GETT_WRANK (blockIdx.x & 1u) // which tile of the pair is mine
#else
#define GETT_WB blockIdx.x
#define GETT_WG gridDim.x
#define GETT_WRANK 0u
#endif

namespace {

constexpr int MMA_M = 128;            // rows of one tcgen05.mma and of one accumulator buffer
constexpr int TILE_K = 64;           // 16-bit elements per slab = one 128-byte swizzle row
constexpr int NUM_EPI_WARPS = 8;           // two sets of four: set s takes the CTA's tiles number s, s+2, ...
constexpr int EPI_SET_THREADS = 128;
#ifndef GETT_PROD_GROUPS
#define GETT_PROD_GROUPS 4
#endif
#ifndef GETT_WARPS_PER_GROUP
#define GETT_WARPS_PER_GROUP 2
#endif
constexpr int PROD_GROUPS = GETT_PROD_GROUPS; // slab number it belongs to producer group it % PROD_GROUPS
constexpr int WARPS_PER_GROUP = GETT_WARPS_PER_GROUP;
constexpr int GROUP_LANES = WARPS_PER_GROUP * 32;
constexpr int NUM_PROD_WARPS = PROD_GROUPS * WARPS_PER_GROUP;
constexpr int MMA_WARP = NUM_EPI_WARPS;
constexpr int PROD_WARP0 = NUM_EPI_WARPS + 1;
constexpr int NUM_THREADS = (NUM_EPI_WARPS + 1 + NUM_PROD_WARPS) * 32;
constexpr int PROD_THREADS = NUM_PROD_WARPS * 32;
constexpr int MAX_STAGES = 8;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t ATOM_BYTES = 1024;      // 8 rows x 128 B
constexpr uint32_t MN_BLOCK_BYTES = 8192;  // one 64-wide block of an MN-major operand: 64 k rows
constexpr int EPI_PITCH = 68;              // floats per staged row: 64 + 4 keeps 128-bit accesses conflict-free
constexpr int EPI_GROUPS = 256 / 4;          // 16-byte groups per tile row, at most
constexpr int EPI_DEPTH = 2;                 // staging buffers per warp: old C is fetched EPI_DEPTH-1 chunks ahead
// staging bytes of one epilogue warp: chunk buffers + group tables (cv, lean as in StagedShape)
__host__ __device__ constexpr int epi_pitch(int tile_n, int cv, int lean)
{
    return cv == 8 ? tile_n / 4 + 4 : lean ? 32 + 4 : EPI_PITCH;
}
__host__ __device__ constexpr int epi_warp_bytes(int tile_n, int cv, int lean)
{
    return (lean ? 1 : EPI_DEPTH) * 32 * epi_pitch(tile_n, cv, lean) * 4 + EPI_DEPTH * EPI_GROUPS * 8;
}

constexpr uint32_t INVALID16 = 0xFFFFFFFFu; // "outside the tensor" in the 16-byte-unit offset tables
constexpr uint32_t SKIP16 = 0xFFFFFFFEu;    // "not mine": the piece belongs to an atom that arrives by TMA

// Offsets in the producer tables are in units of 16 bytes (every vector a producer
// copies starts on a 16-byte boundary), which keeps them in 32 bits.
struct alignas(16) SmemTables { // the staging rows that follow it hold 128-bit vectors
    int64_t colC[2][256];                     // per epilogue set: C offset of each tile column
    uint32_t kTab[PROD_GROUPS][2][TILE_K];    // per producer group: A / B offsets of the slab's k
    uint32_t rowTab[PROD_GROUPS][256 + 256];  // per producer group: row offsets (K-major operands)
    int32_t atomc[PROD_GROUPS][2][4][8];      // per producer group and operand: TMA coordinates (5) and
                                              // segment of each 64-wide atom of the current tile
    int32_t slabc[PROD_GROUPS][2][8];         // ... and the current slab's part of the coordinates
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
    uint64_t drain; // after a give-up: the tensor core has finished what had been issued
    uint32_t tmem_base;
    int abort_flag;
};

static_assert(sizeof(SmemTables) % 16 == 0, "staging area must stay 16-byte aligned");

// Time stamps of CTA 0's roles (experiment builds only, opts.experiment & 4096): role = producer
// group 0 .. 3, 6 = MMA issuer, 4 / 5 = first warp of epilogue set 0 / 1; one thread per role writes.
#ifdef GETT_EXPERIMENT
__device__ unsigned long long gett_trace_buf[8][4096];
__device__ unsigned int gett_trace_n[8];
#define GETT_TRACE(role, tag)                                                                          \
    do {                                                                                               \
        if (blockIdx.x == 0 && (g.debug & 4096)) {                                                     \
            const unsigned n_ = gett_trace_n[role];                                                    \
            if (n_ < 4096) {                                                                           \
                gett_trace_buf[role][n_] = ((unsigned long long)(tag) << 56) | (clock64() & 0xFFFFFFFFFFFFFFull); \
                gett_trace_n[role] = n_ + 1;                                                           \
            }                                                                                          \
        }                                                                                              \
    } while (0)
#else
#define GETT_TRACE(role, tag)                                                                          \
    do {                                                                                               \
    } while (0)
#endif

__host__ __device__ constexpr uint32_t stage_bytes(uint32_t tile_m, uint32_t tile_n)
{
    return (tile_m + tile_n) * TILE_K * 2;
}

struct WorkItem {
    uint32_t m0, n0, z, kbeg, kend, nslab;
    uint32_t r;   // stream-K: number of the left-over tile the item is a piece of
    bool partial; // the item's sums go to the workspace (a K slice, or a piece of a tile), not to C
};

// Origin of output tile (or, in the CTA-pair build, tile pair) number t.
__device__ __forceinline__ void tile_origin(const GettKernelArgs& g, uint32_t t, uint32_t tile_m, uint32_t& m0,
                                            uint32_t& n0)
{
    uint32_t tm, tn;
#ifdef GETT_UMMA_CLUSTER
    gett_raster_tile(t, g.tiles_m, g.tiles_n >> 1, tm, tn); // columns of tile pairs
    n0 = (2 * tn + GETT_WRANK) * (uint32_t)g.tile_n;
#else
    gett_raster_tile(t, g.tiles_m, g.tiles_n, tm, tn);
    n0 = tn * (uint32_t)g.tile_n;
#endif
    m0 = tm * tile_m;
}

__device__ __forceinline__ WorkItem decode_work(const GettKernelArgs& g, uint32_t w, uint32_t tile_m)
{
#ifdef GETT_UMMA_CLUSTER
    const uint32_t tiles = g.tiles_m * (g.tiles_n >> 1);
#else
    const uint32_t tiles = g.tiles_m * g.tiles_n;
#endif
    WorkItem it;
    it.z = w / tiles;
    tile_origin(g, w - it.z * tiles, tile_m, it.m0, it.n0);
    it.kbeg = it.z * g.k_per_split;
    it.kend = min(g.K.size, it.kbeg + g.k_per_split);
    it.nslab = (it.kend - it.kbeg + TILE_K - 1) / TILE_K;
    it.partial = g.split_k > 1;
    return it;
}

// The CTA's work list.  Ordinarily the (tile, K slice) pairs number WB, WB + WG, ... of
// `total_work`.  With stream-K (Sec. 2.1 / Sec. 3.3: choosing how the three loops are cut; here
// the cut that leaves no SM idle in a last partial wave) the first sk_full rounds of tiles are
// dealt out the same way, and the tiles that are left (fewer than there are CTAs) are cut along
// K: their tiles x slabs space is one sequence of slab units of which every CTA takes
// sk_units consecutive ones.  Such an item is a piece of one tile; its sums go to the
// workspace as piece number z of that tile, and a second kernel adds the pieces.
__device__ __forceinline__ uint32_t item_count(const GettKernelArgs& g, uint32_t total_work)
{
    if (g.stream_k) {
        const uint32_t tiles = g.tiles_m * g.tiles_n;
        const uint32_t total = (tiles - g.sk_full * GETT_WG) * g.sk_slabs; // slab units of the left-over tiles
        const uint32_t beg = GETT_WB * g.sk_units;
        if (beg >= total)
            return g.sk_full;
        const uint32_t end = min(total, beg + g.sk_units);
        return g.sk_full + (end - 1) / g.sk_slabs - beg / g.sk_slabs + 1;
    }
    return total_work > GETT_WB ? (total_work - GETT_WB + GETT_WG - 1) / GETT_WG : 0;
}

__device__ __forceinline__ WorkItem decode_item(const GettKernelArgs& g, uint32_t i, uint32_t tile_m)
{
    if (!g.stream_k || i < g.sk_full) {
        WorkItem it = decode_work(g, GETT_WB + i * GETT_WG, tile_m);
        it.r = 0;
        return it;
    }
    const uint32_t S = g.sk_slabs, W = g.sk_units;
    const uint32_t tiles = g.tiles_m * g.tiles_n, done = g.sk_full * GETT_WG;
    const uint32_t total = (tiles - done) * S;
    const uint32_t beg = GETT_WB * W, end = min(total, beg + W);
    const uint32_t r = beg / S + (i - g.sk_full); // which of the left-over tiles
    const uint32_t ub = max(beg, r * S), ue = min(end, (r + 1) * S);
    WorkItem it;
    tile_origin(g, done + r, tile_m, it.m0, it.n0);
    it.r = r;
    it.z = GETT_WB - (r * S) / W; // pieces of a tile are numbered from the first CTA that touches it
    it.kbeg = (ub - r * S) * TILE_K;
    it.kend = min(g.K.size, (ue - r * S) * TILE_K);
    it.nslab = ue - ub;
    it.partial = true; // (even a whole left-over tile goes through the workspace: the fix-up treats all alike)
    return it;
}

// One producer group (GROUP_LANES threads) gathers a whole operand slab of R free
// indices x 64 k.  gl = the thread's index inside its group.
//
// VEC_K   : 16-byte pieces run along k (K-major staging).  Thread gl owns k-piece
//           kc = gl % 8 of rows gl/8 + RP p; the rows' offsets come from the group's row
//           table (filled once per tile), the k offset is one register per slab.
// VEC_FREE: pieces run along the free dimension (MN-major staging).  Thread gl owns
//           free-piece fc = gl % FPR of the k rows gl/FPR + KSTEP p; its row offset is
//           one register per tile, the k offsets come from the group's slab table.
template <bool VEC_K, int R, int LANES>
struct OperandLoader {
    static constexpr int FPR = R / 8;                 // pieces per k row (VEC_FREE)
    static constexpr int pow2_floor(int x) { return x >= 64 ? 64 : x >= 32 ? 32 : x >= 16 ? 16 : x >= 8 ? 8 : x >= 4 ? 4 : x >= 2 ? 2 : 1; }
    static constexpr int KSTEP = pow2_floor(LANES / FPR); // k rows per pass (VEC_FREE)
    static constexpr int RP = LANES / 8;                  // rows per pass (VEC_K)
    static constexpr int ACTIVE = VEC_K ? LANES : KSTEP * FPR;
    static constexpr int NP = VEC_K ? (R + RP - 1) / RP : TILE_K / KSTEP;
    static_assert(ACTIVE <= LANES, "tile too wide for one producer group");

    uint32_t row16;    // VEC_FREE: this thread's row offset (16-byte units), INVALID16 if outside
    uint32_t dst_lane; // byte offset of this thread's piece 0 inside the operand's stage buffer

    // Hybrid tiles (VEC_FREE only): the 64-wide atoms that lie in segment 0 of the dimension
    // arrive by TMA; only the atoms of segment 1 are gathered, eight 16-byte pieces per k row.
    // Thread gl owns piece gl % 8 of the k rows gl / 8 + (LANES / 8) p of every such atom.
    static constexpr int HY_ATOMS = R / 64 > 0 ? R / 64 : 1;
    static constexpr int HY_KROWS = LANES / 8;
    uint32_t hy_row16[HY_ATOMS]; // offset of my piece of atom b, SKIP16 if the atom is not gathered

    __device__ __forceinline__ void setup_hybrid(const GettDim& D, uint32_t origin, uint32_t gl)
    {
#pragma unroll
        for (int b = 0; b < HY_ATOMS; ++b) {
            const uint32_t f = origin + 64u * b + 8u * (gl & 7);
            hy_row16[b] = SKIP16;
            if (f < D.size) {
                int64_t x, y;
                if (gett_decompose(D, f, x, y) == 1)
                    hy_row16[b] = (uint32_t)(x >> 3);
            }
        }
    }

    // The slab is a box of I_k (that is how plans with such tiles order I_k): k row number k of the
    // slab lies k % 2^kshift steps of K's first digit and k >> kshift steps of its second digit
    // from the slab's first row, so its offset needs no table.  k16_0: offset of the slab's first
    // row, s0_16 / s1_16: the two digit strides (all in 16-byte units); nvalid: rows inside K.
    __device__ __forceinline__ void load_hybrid(const char* __restrict__ base, uint32_t stage_dst, uint32_t gl,
                                                uint32_t k16_0, uint32_t s0_16, uint32_t s1_16, uint32_t kshift,
                                                uint32_t nvalid) const
    {
        const uint32_t pc = gl & 7, krow = gl >> 3;
#pragma unroll
        for (int b = 0; b < HY_ATOMS; ++b) {
            if (hy_row16[b] == SKIP16)
                continue;
            const char* src = base + ((uint64_t)(hy_row16[b] + k16_0) << 4);
#pragma unroll
            for (int p = 0; p < TILE_K / HY_KROWS; ++p) {
                const uint32_t k = krow + HY_KROWS * p;
                const uint32_t off16 = (k & ((1u << kshift) - 1u)) * s0_16 + (k >> kshift) * s1_16;
                const bool ok = k < nvalid;
                ptx::cp_async_16(stage_dst + b * MN_BLOCK_BYTES + k * 128 + ((pc ^ (k & 7)) << 4),
                                 ok ? src + ((uint64_t)off16 << 4) : base, ok ? 16u : 0u);
            }
        }
    }

    // rowTab: the group's table for this operand (used by VEC_K only; the caller
    // synchronises the group before and after).
    __device__ __forceinline__ void setup_tile(const GettDim& D, uint32_t origin, uint32_t gl,
                                               uint32_t* rowTab)
    {
        if (VEC_K) {
            for (uint32_t r = gl; r < (uint32_t)R; r += LANES) {
                uint32_t v = INVALID16;
                if (origin + r < D.size) {
                    int64_t x, y;
                    gett_decompose(D, origin + r, x, y);
                    v = (uint32_t)(x >> 3);
                }
                rowTab[r] = v;
            }
            // rows gl/8 + RP p all share r % 8, so the swizzle term is a per-thread constant
            dst_lane = (gl >> 3) * 128 + (((gl & 7) ^ ((gl >> 3) & 7)) << 4);
            row16 = 0;
        } else {
            const uint32_t fc = gl % FPR, kgroup = gl / FPR;
            row16 = INVALID16;
            if (gl < ACTIVE && origin + fc * 8 < D.size) {
                int64_t x, y;
                gett_decompose(D, origin + fc * 8, x, y);
                row16 = (uint32_t)(x >> 3);
            }
            dst_lane = (fc >> 3) * MN_BLOCK_BYTES + kgroup * 128;
        }
    }

    // KT (K-major staging only): the operand's 16-byte pieces run along K's SECOND digit while the
    // slab's k order is first digit (extent 8) fastest.  Piece number i of a row is then read
    // from first-digit index i (table entry i, not 8 i) and holds eight consecutive indices of
    // the second digit: the row arrives as the transpose of what the tensor core needs, and
    // transpose_rows() below puts it right.
    template <bool FAST, bool KT = false>
    __device__ __forceinline__ void load_slab(const char* __restrict__ base, uint32_t stage_dst,
                                              const uint32_t* kTab, const uint32_t* rowTab,
                                              uint32_t gl) const
    {
        if (VEC_K) {
            const uint32_t k16 = kTab[KT ? (gl & 7) : (gl & 7) * 8];
            const uint32_t dst = stage_dst + dst_lane;
            const uint32_t* rows = rowTab + (gl >> 3);
#pragma unroll 8
            for (int p = 0; p < NP; ++p) {
                if (R % RP != 0 && (gl >> 3) + RP * p >= (uint32_t)R)
                    break;
                const uint32_t r16 = rows[RP * p];
                if (FAST) {
                    ptx::cp_async_16(dst + p * (RP * 128), base + ((uint64_t)(r16 + k16) << 4), 16u);
                } else {
                    const bool ok = r16 != INVALID16 && k16 != INVALID16;
                    ptx::cp_async_16(dst + p * (RP * 128), base + (ok ? ((uint64_t)(r16 + k16) << 4) : 0),
                                     ok ? 16u : 0u);
                }
            }
        } else {
            if (ACTIVE < LANES && gl >= ACTIVE)
                return;
            const uint32_t fc = gl % FPR, kgroup = gl / FPR;
            const uint32_t dst = stage_dst + dst_lane;
#pragma unroll 8
            for (int p = 0; p < NP; ++p) {
                const uint32_t k = kgroup + KSTEP * p;
                const uint32_t k16 = kTab[k];
                const uint32_t d = dst + p * (KSTEP * 128) + (((fc & 7) ^ (k & 7)) << 4);
                if (FAST) {
                    ptx::cp_async_16(d, base + ((uint64_t)(row16 + k16) << 4), 16u);
                } else {
                    const bool ok = row16 != INVALID16 && k16 != INVALID16;
                    ptx::cp_async_16(d, base + (ok ? ((uint64_t)(row16 + k16) << 4) : 0), ok ? 16u : 0u);
                }
            }
        }
    }
};

// In-place transposition of the rows a warp has just copied with load_slab<.., KT = true>
// (packing as a transposition, Sec. 3.2.2 / Eq. 10, at the granularity of 8 x 8 blocks).
// A row of the K-major stage (one free index, 128 bytes, pieces XOR-swizzled by row % 8) holds
// an 8 x 8 block of 16-bit elements: piece i = first-digit index i, eight second-digit indices.
// The tensor core needs piece j = second-digit index j, eight first-digit indices.  A warp
// owns rows r0 .. r0 + 3 of every pass (the rows its own lanes copied), reads four blocks
// transposed (ldmatrix.trans: lanes 8 q .. 8 q + 7 give the piece addresses of block q) and
// writes them back to the same rows (stmatrix).
template <int R, int LANES>
__device__ __forceinline__ void transpose_rows(uint32_t stage_dst, uint32_t gl)
{
    constexpr int RP = LANES / 8; // rows per pass of the K-major gather
    const uint32_t lane = gl & 31;
    const uint32_t row0 = ((gl >> 5) << 2) + (lane >> 3); // my block's row in pass 0
    const uint32_t i = lane & 7;                          // the piece whose address I supply
#pragma unroll 4
    for (uint32_t r = row0; r < (uint32_t)R; r += RP) {
        // (rows of a pass beyond R do not exist; R and RP are multiples of 4, so a warp's four
        //  blocks are either all inside or all outside)
        const uint32_t addr = stage_dst + r * 128 + ((i ^ (r & 7)) << 4);
        uint32_t v0, v1, v2, v3;
        ptx::ldmatrix_x4_trans(addr, v0, v1, v2, v3);
        __syncwarp(); // all four blocks are in registers before any of them is overwritten
        ptx::stmatrix_x4(addr, v0, v1, v2, v3);
    }
}

// ---- staged epilogue (Eq. 11 as a transposition through shared memory) ----
// The accumulator is walked in chunks of up to 64 columns, and inside a chunk the columns
// are re-ordered into "slots" so that four consecutive slots are four consecutive floats of C:
//   CV == 1: the tile's columns already run along C's stride-1 mode; a chunk is 64
//            consecutive columns and slot = column.
//   CV == 8: the first N digit a (extent 8) is the 8-wide piece of B's stride-1 mode and the
//            second digit is C's stride-1 mode, i.e. column = a + 8 p with p running along
//            C.  A chunk is a pair of a values over ALL p of the tile (TILE_N / 4 columns,
//            read from tensor memory two at a time with a stride of 8 columns), slot =
//            (a & 1) * TILE_N/8 + p: each row of the chunk is two runs of TILE_N/8
//            consecutive floats of C, so the reads and writes of C cover whole runs of its
//            stride-1 mode instead of 32-byte pieces of them.
// LEAN: one staging buffer per warp instead of two (the old C of a chunk is requested when
// the previous chunk is done, not one chunk ahead) and 32-column chunks for CV == 1: a third
// of the shared memory, for long contractions, where the operand ring needs the space and
// the unpacking hides behind the next tile's main loop anyway.
template <int TILE_N, int CV, int LEAN>
struct StagedShape {
    static constexpr uint32_t NP = TILE_N / 8;                      // CV == 8: pieces (values of p) per tile
    static constexpr uint32_t SLOTS = CV == 8 ? TILE_N / 4 : LEAN ? 32 : 64; // slots per row of a chunk
    static constexpr uint32_t NCH = CV == 8 ? 4 : TILE_N / SLOTS;   // chunks per tile
    static constexpr uint32_t DEPTH = LEAN ? 1 : EPI_DEPTH;         // staging buffers
    static constexpr uint32_t PITCH = epi_pitch(TILE_N, CV, LEAN);  // SLOTS + 4 keeps 128-bit accesses conflict-free
    static constexpr uint32_t GPR = SLOTS / 4;                      // 16-byte groups per row of a chunk
    static_assert(PITCH == SLOTS + 4, "staging pitch");
    // first tile column of the 16-byte group number e (e = chunk * GPR + group in the row)
    static __device__ __forceinline__ uint32_t col_of_group(uint32_t e)
    {
        return CV == 8 ? e / (NP / 4) + 32 * (e % (NP / 4)) : 4 * e;
    }
};

// Staged epilogue, run by each epilogue warp on its own 32 tile rows, one chunk at a
// time, software-pipelined one chunk ahead (across tile boundaries):
//   prepare(c+1): (first chunk of a tile) C offsets of my row and of the tile's 16-byte
//                 groups; if beta != 0, cp.async the old C values of chunk c+1 into the
//                 other staging buffer -- the reads of C never wait for the accumulator
//   process(c)  : accumulator -> registers, alpha*acc + beta*old (old read from staging,
//                 one row per lane), result written back to staging with 128-bit stores;
//                 then the warp re-reads staging with lanes running along C and issues
//                 128-bit global stores
template <int TILE_N, int CV, int LEAN>
__device__ __forceinline__ void epilogue_staged(const GettKernelArgs& g, SmemTables* T, uint8_t* epi_smem,
                                                uint32_t tmem_base, uint32_t warp, uint32_t lane,
                                                uint32_t total_work, volatile int* abort_flag)
{
    using Sh = StagedShape<TILE_N, CV, LEAN>;
    const uint64_t wait_ns = (uint64_t)g.wait_limit_us * 1000ull;
    constexpr uint32_t NCH = Sh::NCH, PITCH = Sh::PITCH, GPR = Sh::GPR, NP = Sh::NP, DEPTH = Sh::DEPTH;
    float* S = reinterpret_cast<float*>(epi_smem + warp * epi_warp_bytes(TILE_N, CV, LEAN));
    // C offsets, in units of 16 bytes (every group of four slots is one aligned vector of C; the
    // planner keeps C's largest offset below 2^36 bytes for this epilogue), for tiles j even / odd:
    uint32_t* grp16 = reinterpret_cast<uint32_t*>(S + DEPTH * 32 * PITCH); // ... of the tile's 16-byte column groups
    uint32_t* row16 = grp16 + 2 * EPI_GROUPS;                              // ... of this warp's 32 rows
    static_assert(2 * EPI_GROUPS * 4 + 2 * 32 * 4 <= EPI_DEPTH * EPI_GROUPS * 8, "offset tables fit their space");
    const uint32_t s_u32 = ptx::smem_u32(S);
    const float alpha = g.alpha, beta = g.beta;
    const bool rmw = beta != 0.f && !GETT_DBG(g, 128); // (debug & 128: experiment, old C not read)
    // this warp's set handles the CTA's tiles with local number es, es + 2, ...; `j` counts them
    const uint32_t es = warp >> 2, eq = warp & 3;
    const uint32_t ncta = total_work > GETT_WB ? (total_work - GETT_WB + GETT_WG - 1) / GETT_WG : 0;
    const uint32_t ntile = ncta > es ? (ncta - es + 1) / 2 : 0;
    const uint32_t nchunk = ntile * NCH;
    // Moving a chunk (32 rows x GPR groups of 16 bytes) between C and the staging buffer, lanes
    // running along C: copy number t of a lane is item lane + 32 t, item q = group q % GPR of row
    // q / GPR.  32 t % GPR has period GCYC in t, so a lane meets only GCYC different groups --
    // whose C offsets it reads once per chunk -- and its rows advance by RSTEP per period:
    // what is left per copy is one table read (the row's offset), one add and the copy.
    constexpr uint32_t GCYC = 32 % GPR == 0 ? 1 : 3;
    static_assert((32 * GCYC) % GPR == 0 && GPR % GCYC == 0, "GPR is 4, 8, 12 or 16");
    constexpr uint32_t RSTEP = 32 * GCYC / GPR, NU = GPR / GCYC;
    uint32_t it_row[GCYC], it_grp[GCYC];
#pragma unroll
    for (uint32_t v = 0; v < GCYC; ++v) {
        it_row[v] = (lane + 32 * v) / GPR;
        it_grp[v] = (lane + 32 * v) % GPR;
    }

    // C offsets of the warp's rows and of the 16-byte groups of tile j's columns
    auto tile_offsets = [&](uint32_t j) {
        const WorkItem wi = decode_work(g, GETT_WB + (es + 2 * j) * GETT_WG, MMA_M);
        const uint32_t m = wi.m0 + eq * 32 + lane;
        row16[(j & 1) * 32 + lane] = m < g.M.size ? (uint32_t)(gett_offset_y(g.M, m) >> 2) : INVALID16;
        for (uint32_t e = lane; e < TILE_N / 4; e += 32) {
            const uint32_t col = Sh::col_of_group(e);
            grp16[(j & 1) * EPI_GROUPS + e] =
                wi.n0 + col < g.N.size ? (uint32_t)(gett_offset_y(g.N, wi.n0 + col) >> 2) : INVALID16;
        }
        __syncwarp();
    };

    // (elements outside C are not fetched: what the staging slots then hold is combined but never stored)
    auto prepare = [&](uint32_t cj) {
        if (cj < nchunk) {
            const uint32_t j = cj / NCH, ch = cj - j * NCH;
            if (ch == 0)
                tile_offsets(j);
            if (rmw) {
                const uint32_t dst = s_u32 + (cj & (DEPTH - 1)) * (32 * PITCH * 4);
                const uint32_t* gt = grp16 + (j & 1) * EPI_GROUPS + ch * GPR;
                const uint32_t* rt = row16 + (j & 1) * 32;
#pragma unroll
                for (uint32_t v = 0; v < GCYC; ++v) {
                    const uint32_t g16 = gt[it_grp[v]];
                    const uint32_t d0 = dst + (it_row[v] * PITCH + 4 * it_grp[v]) * 4;
#pragma unroll
                    for (uint32_t u = 0; u < NU; ++u) {
                        const uint32_t r16 = rt[it_row[v] + u * RSTEP];
                        if (g16 != INVALID16 && r16 != INVALID16)
                            ptx::cp_async_16(d0 + u * (RSTEP * PITCH * 4),
                                             reinterpret_cast<const float4*>(g.C) + ((uint64_t)r16 + g16), 16u);
                    }
                }
            }
        }
        ptx::cp_async_commit();
    };

    // alpha * acc (+ beta * old, read from the same staging slots) -> staging.  Four
    // 16-byte groups at a time: the old values are read first, then the results written,
    // so that the loads do not queue up behind the stores to the same buffer.
    auto combine4 = [&](float* const (&p)[4], float4 (&q)[4]) {
        float4 o[4];
        if (rmw) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                o[k] = *reinterpret_cast<const float4*>(p[k]);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            q[k].x *= alpha;
            q[k].y *= alpha;
            q[k].z *= alpha;
            q[k].w *= alpha;
            if (rmw) {
                q[k].x = fmaf(beta, o[k].x, q[k].x);
                q[k].y = fmaf(beta, o[k].y, q[k].y);
                q[k].z = fmaf(beta, o[k].z, q[k].z);
                q[k].w = fmaf(beta, o[k].w, q[k].w);
            }
            if (!GETT_DBG(g, 512)) // (debug & 512: experiment, no staging writes)
                *reinterpret_cast<float4*>(p[k]) = q[k];
        }
    };

    if (DEPTH == 2)
        prepare(0);
    const bool tracer = eq == 0 && lane == 0;
    for (uint32_t ci = 0; ci < nchunk; ++ci) {
        if (tracer)
            GETT_TRACE(4 + es, 0);
        if (DEPTH == 2) {
            prepare(ci + 1);
            if (tracer)
                GETT_TRACE(4 + es, 5);
            ptx::cp_async_wait<1>(); // chunk ci's old C has landed (my copies) ...
        } else {
            prepare(ci);
            ptx::cp_async_wait<0>();
        }
        __syncwarp(); // ... and everybody else's
        if (tracer)
            GETT_TRACE(4 + es, 1);
        const uint32_t j = ci / NCH, ch = ci - j * NCH, buf = es; // tile es + 2j uses accumulator es
        if (ch == 0) {
            if (!ptx::mbar_wait(ptx::smem_u32(&T->acc_full[buf]), j & 1, abort_flag, wait_ns))
                break;
            ptx::tc_fence_after();
        }
        if (tracer)
            GETT_TRACE(4 + es, 2);
        float* Sb = S + (ci & (DEPTH - 1)) * (32 * PITCH);
        float* Srow = Sb + lane * PITCH;
        const uint32_t tacc = tmem_base + ((eq * 32u) << 16) + buf * 256;
        if constexpr (CV == 1) {
#pragma unroll
            for (uint32_t h = 0; h < Sh::SLOTS / 32; ++h) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tacc + ch * Sh::SLOTS + h * 32, v);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int u0 = 0; u0 < 8; u0 += 4) {
                    float* p[4];
                    float4 q[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int u = u0 + k;
                        p[k] = Srow + h * 32 + 4 * u;
                        q[k] = make_float4(__uint_as_float(v[4 * u]), __uint_as_float(v[4 * u + 1]),
                                           __uint_as_float(v[4 * u + 2]), __uint_as_float(v[4 * u + 3]));
                    }
                    combine4(p, q);
                }
            }
        } else {
            // columns 2 ch + aa + 8 p: half of the tile's p values at a time
            constexpr uint32_t HP = NP / 2;
            static_assert(HP % 4 == 0 && HP <= 16, "tile widths 64, 128, 192, 256");
#pragma unroll
            for (uint32_t h = 0; h < 2; ++h) {
                uint32_t v[2 * HP];
#pragma unroll
                for (uint32_t i = 0; i < HP; ++i)
                    ptx::tmem_ld_32x2(tacc + 2 * ch + 8 * (h * HP + i), v[2 * i], v[2 * i + 1]);
                ptx::tmem_wait_ld();
                // 2 * HP / 4 groups: group u covers a = 2 ch + u / (HP / 4), p = h HP + 4 (u % (HP / 4)) ...
                constexpr uint32_t NG = HP / 2, Q = HP / 4;
                static_assert(NG % 2 == 0, "groups are combined two or four at a time");
#pragma unroll
                for (uint32_t u0 = 0; u0 < NG; u0 += 4) {
                    float* p[4];
                    float4 q[4];
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k) {
                        const uint32_t u = u0 + k < NG ? u0 + k : NG - 1; // (NG = 2 or 6: the tail repeats the last group)
                        const uint32_t aa = u / Q, i4 = u % Q;
                        p[k] = Srow + aa * NP + h * HP + 4 * i4;
                        q[k] = make_float4(__uint_as_float(v[8 * i4 + aa]), __uint_as_float(v[8 * i4 + 2 + aa]),
                                           __uint_as_float(v[8 * i4 + 4 + aa]), __uint_as_float(v[8 * i4 + 6 + aa]));
                    }
                    combine4(p, q);
                }
            }
        }
        if (ch == NCH - 1) { // the accumulator buffer can be overwritten by the set's next tile
            ptx::tc_fence_before();
            ptx::mbar_arrive(ptx::smem_u32(&T->acc_empty[buf]));
        }
        __syncwarp();
        if (tracer)
            GETT_TRACE(4 + es, 3);
        if (!GETT_DBG(g, 256)) { // (debug & 256: experiment, no store phase)
            const uint32_t* gt = grp16 + (j & 1) * EPI_GROUPS + ch * GPR;
            const uint32_t* rt = row16 + (j & 1) * 32;
#pragma unroll
            for (uint32_t v = 0; v < GCYC; ++v) {
                const uint32_t g16 = gt[it_grp[v]];
                const float* src = Sb + it_row[v] * PITCH + 4 * it_grp[v];
                // four groups at a time: staging reads first, then the global stores
#pragma unroll
                for (uint32_t u0 = 0; u0 < NU; u0 += 4) {
                    float4 val[4];
                    uint32_t r16[4];
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k) {
                        r16[k] = rt[it_row[v] + (u0 + k) * RSTEP];
                        val[k] = *reinterpret_cast<const float4*>(src + (u0 + k) * (RSTEP * PITCH));
                    }
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k)
                        if (g16 != INVALID16 && r16[k] != INVALID16 && !GETT_DBG(g, 2)) // (debug & 2: no stores)
                            reinterpret_cast<float4*>(g.C)[(uint64_t)r16[k] + g16] = val[k];
                }
            }
        }
        __syncwarp(); // this staging buffer is free for the next prefetch into it
        if (tracer)
            GETT_TRACE(4 + es, 4);
    }
    ptx::cp_async_wait_all();
}

// The producer role.  A group of LANES threads (index gl inside the group, named barrier
// gbar) owns the slabs with number it % ng == pg and fills their ring stage.
template <bool A_VEC_K, bool B_VEC_K, int TILE_N, int TILE_M, int LANES, bool HYBRID, bool B_TRANS>
__device__ __forceinline__ void producer_role(const GettKernelArgs& g, const GettTmaMaps& tm, SmemTables* T,
                                              uint32_t stage0, uint32_t stages, uint32_t total_work,
                                              volatile int* abort_flag, uint32_t pg, uint32_t ng, uint32_t gl,
                                              uint32_t gbar)
{
    constexpr uint32_t sbytes = stage_bytes(TILE_M, TILE_N);
    constexpr uint32_t A_STAGE_BYTES = TILE_M * TILE_K * 2;
    const uint64_t wait_ns = (uint64_t)g.wait_limit_us * 1000ull;
    // ------------------------------ producers ------------------------------
    // Slab number `it` (counted over the CTA's whole work list) belongs to producer
    // group it % PROD_GROUPS, so PROD_GROUPS slabs are gathered concurrently.  The
    // ring depth is a multiple of PROD_GROUPS, hence a stage's barriers are always
    // used by the same group, which therefore observes every one of their phases.
    uint32_t* kA = T->kTab[pg][0];
    uint32_t* kB = T->kTab[pg][1];
    uint32_t* rowA = T->rowTab[pg];
    uint32_t* rowB = T->rowTab[pg] + 256;
    OperandLoader<A_VEC_K, TILE_M, LANES> la;
    OperandLoader<B_VEC_K, TILE_N, LANES> lb;
    const char* baseA = static_cast<const char*>(g.A);
    const char* baseB = static_cast<const char*>(g.B);
    // An operand whose tile is a box -- or a list of 64-wide atoms that are boxes -- of a
    // <= 5-D tensor map is fetched by TMA: thread 0 of the group issues the copies and the
    // stage's barrier counts their bytes.
    const bool tmaA = tm.a.use != 0, tmaB = tm.b.use != 0;
    // hybrid: the atoms of segment 1 of the operand's free dimension are gathered
    // (HYBRID is the compile-time form of "some operand is hybrid": the common case carries no state for it)
    const bool hybridA = HYBRID && tmaA && !A_VEC_K && tm.a.hybrid, hybridB = HYBRID && tmaB && !B_VEC_K && tm.b.hybrid;
    const bool all_tma = tmaA && tmaB; // no offset tables (and no barriers of the group) are needed
    constexpr uint32_t ATOM_STAGE_BYTES = 64 * TILE_K * 2; // one atom: 64 free indices x 64 k
    constexpr int NATOM_A = A_VEC_K ? 1 : TILE_M / 64, NATOM_B = B_VEC_K ? 1 : TILE_N / 64;
    int32_t (*atomA)[8] = T->atomc[pg][0];
    int32_t (*atomB)[8] = T->atomc[pg][1];
    uint32_t tma_bytes = 0; // what the current tile's TMA copies deliver per stage
    int natomA = 0, natomB = 0;
    // coordinates of the atoms of a tile (the free-dimension part, kept for all slabs of the
    // tile) and their segment; returns the bytes per stage of those that come by TMA
    auto atom_coords = [&](const GettDim& D, const GettTmaCoords& co, uint32_t origin, int natom_max,
                           int32_t (*out)[8], int& natom) {
        uint32_t bytes = 0;
        natom = 0;
        for (int b = 0; b < natom_max; ++b) {
            const uint32_t f = origin + 64u * (uint32_t)b;
            if (b > 0 && f >= D.size)
                break; // atoms past the end of the dimension are not fetched (their rows are never stored)
#pragma unroll
            for (int i = 0; i < 5; ++i)
                out[b][i] = 0;
            const int seg = gett_add_coords(D, f, co.fdim, co.fmul, out[b]);
            out[b][5] = seg;
            bytes += seg == 0 ? ATOM_STAGE_BYTES : 0u;
            ++natom;
        }
        return bytes;
    };
    uint32_t first = 0; // slab number of the current work item's first slab
    bool alive = true;
    const uint32_t nitems = item_count(g, total_work);
    for (uint32_t wn = 0; wn < nitems && pg < ng; ++wn) {
        const WorkItem wi = decode_item(g, wn, TILE_M);
        // my group's first slab in this item: smallest j with (first + j) % ng == pg
        uint32_t j = (pg + ng - first % ng) % ng;
        if (j < wi.nslab) {
            if (!all_tma)
                ptx::named_barrier(gbar, LANES); // the group is done with the previous tables
            tma_bytes = 0;
            if (!tmaA)
                la.setup_tile(g.M, wi.m0, gl, rowA);
            else if (hybridA)
                la.setup_hybrid(g.M, wi.m0, gl);
            if (tmaA && gl == 0) {
                const uint32_t bytes = atom_coords(g.M, tm.a.co, wi.m0, NATOM_A, atomA, natomA);
                tma_bytes += A_VEC_K ? A_STAGE_BYTES : bytes;
            }
            if (!tmaB)
                lb.setup_tile(g.N, wi.n0, gl, rowB);
            else if (hybridB)
                lb.setup_hybrid(g.N, wi.n0, gl);
            if (tmaB && gl == 0) {
                const uint32_t bytes = atom_coords(g.N, tm.b.co, wi.n0, NATOM_B, atomB, natomB);
                tma_bytes += B_VEC_K ? TILE_N * TILE_K * 2 : bytes;
            }
        }
        const bool tile_full = wi.m0 + TILE_M <= g.M.size && wi.n0 + TILE_N <= g.N.size;
        for (; j < wi.nslab; j += ng) {
            const uint32_t it = first + j;
            const uint32_t k0 = wi.kbeg + j * TILE_K;
            if (gl == 0)
                GETT_TRACE(pg, 0);
            if (!all_tma) {
                ptx::named_barrier(gbar, LANES); // previous slab's k table no longer read
                if (gl < TILE_K) {
                    const uint32_t k = k0 + gl;
                    uint32_t xa = INVALID16, xb = INVALID16;
                    if (k < wi.kend) {
                        int64_t x, y;
                        gett_decompose(g.K, k, x, y);
                        xa = (uint32_t)(x >> 3);
                        xb = (uint32_t)(y >> 3);
                    }
                    kA[gl] = xa;
                    kB[gl] = xb;
                }
                ptx::named_barrier(gbar, LANES); // tables (rows and k) complete
            }
            if (gl == 0)
                GETT_TRACE(pg, 1);
            const uint32_t s = it % stages;
            // the slab's part of the TMA coordinates, before the wait for the stage
            int32_t* ckA = T->slabc[pg][0]; // (written and read by thread 0 of the group only)
            int32_t* ckB = T->slabc[pg][1];
            if (gl == 0 && alive && (tmaA || tmaB)) {
#pragma unroll
                for (int i = 0; i < 5; ++i)
                    ckA[i] = ckB[i] = 0;
                if (tmaA)
                    gett_add_coords(g.K, k0, tm.a.co.kdim, tm.a.co.kmul, ckA);
                if (tmaB)
                    gett_add_coords(g.K, k0, tm.b.co.kdim, tm.b.co.kmul, ckB);
            }
            // After a timeout a thread keeps walking the loop (so its group's named
            // barriers stay matched) but neither waits nor copies any more.
            if (alive && !ptx::mbar_wait(ptx::smem_u32(&T->empty[s]), ((it / stages) & 1) ^ 1, abort_flag, wait_ns))
                alive = false;
            if (!alive)
                continue;
            if (gl == 0)
                GETT_TRACE(pg, 2);
            const uint32_t sa = stage0 + s * sbytes;
            const uint32_t fullbar = ptx::smem_u32(&T->full[s]);
            if (gl == 0 && tma_bytes && !GETT_DBG(g, 4)) {
                ptx::mbar_expect_tx(fullbar, tma_bytes);
                if (tmaA) {
                    const int32_t* ck = ckA;
                    int32_t c[5];
#ifdef GETT_UMMA_CLUSTER
                    // my half of the A tile, delivered to both CTAs of the pair (the partner
                    // fetches the other half); each CTA's barrier counts the whole stage
                    const uint32_t half = GETT_WRANK;
                    if (A_VEC_K) { // the map's box is TILE_M / 2 rows high
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            c[i] = atomA[0][i] + ck[i];
                        const int fd0 = tm.a.co.fdim[0];
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            c[i] += i == fd0 ? (int32_t)(half * (TILE_M / 2)) : 0;
                        ptx_mc::tma_load_pair(sa + half * (A_STAGE_BYTES / 2), tm.a.map, fullbar, tm.a.co.rank, c);
                    } else {
                        for (int b = (int)half * (NATOM_A / 2); b < (int)(half + 1) * (NATOM_A / 2) && b < natomA; ++b) {
#pragma unroll
                            for (int i = 0; i < 5; ++i)
                                c[i] = atomA[b][i] + ck[i];
                            ptx_mc::tma_load_pair(sa + b * MN_BLOCK_BYTES, tm.a.map, fullbar, tm.a.co.rank, c);
                        }
                    }
#else
                    for (int b = 0; b < natomA; ++b) {
                        if (atomA[b][5])
                            continue; // an atom of segment 1: gathered below
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            c[i] = atomA[b][i] + ck[i];
                        ptx::tma_load(sa + b * MN_BLOCK_BYTES, tm.a.map, fullbar, tm.a.co.rank, c);
                    }
#endif
                }
                if (tmaB) {
                    const int32_t* ck = ckB;
                    int32_t c[5];
                    for (int b = 0; b < natomB; ++b) {
                        if (atomB[b][5])
                            continue;
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            c[i] = atomB[b][i] + ck[i];
                        ptx::tma_load(sa + A_STAGE_BYTES + b * MN_BLOCK_BYTES, tm.b.map, fullbar, tm.b.co.rank, c);
                    }
                }
            }
            if (GETT_DBG(g, 4)) {
                // experiment switch: no copies at all (measures the rest of the pipeline)
            } else if (tile_full && k0 + TILE_K <= wi.kend) {
                if (!tmaA)
                    la.template load_slab<true>(baseA, sa, kA, rowA, gl);
                if (!tmaB && !B_TRANS)
                    lb.template load_slab<true>(baseB, sa + A_STAGE_BYTES, kB, rowB, gl);
                if (B_TRANS) { // B first, as a copy group of its own (waited for below)
                    lb.template load_slab<true, true>(baseB, sa + A_STAGE_BYTES, kB, rowB, gl);
                    ptx::cp_async_commit();
                }
            } else {
                if (!tmaA)
                    la.template load_slab<false>(baseA, sa, kA, rowA, gl);
                if (!tmaB && !B_TRANS)
                    lb.template load_slab<false>(baseB, sa + A_STAGE_BYTES, kB, rowB, gl);
                if (B_TRANS) {
                    lb.template load_slab<false, true>(baseB, sa + A_STAGE_BYTES, kB, rowB, gl);
                    ptx::cp_async_commit();
                }
            }
            if (B_TRANS) {
                // B's rows have arrived transposed: once this warp's own copies of them have landed,
                // it transposes its rows in place.  Those are ordinary stores, so the thread also
                // arrives on the barrier in the ordinary way (A's copies are tracked separately).
                ptx::cp_async_wait<0>();
                __syncwarp();
                transpose_rows<TILE_N, LANES>(sa + A_STAGE_BYTES, gl);
                ptx::mbar_arrive(fullbar);
            }
            if ((hybridA || hybridB) && !GETT_DBG(g, 4 | 1024)) { // (probe 1024: the gathered atoms are skipped)
                int64_t xa, xb;
                gett_decompose(g.K, k0, xa, xb);
                // (a slab spans the first digit -- a power of two -- and part of the second, or lies in the first)
                const uint32_t e0 = (g.K.ndig <= 1 || g.K.ext[0] >= (uint32_t)TILE_K) ? (uint32_t)TILE_K : g.K.ext[0];
                const uint32_t kbox0 = 31u - (uint32_t)__clz((int)e0), nvalid = wi.kend - k0;
                if (hybridA)
                    la.load_hybrid(baseA, sa, gl, (uint32_t)(xa >> 3), (uint32_t)(g.K.sX[0] >> 3),
                                   (uint32_t)(g.K.sX[1] >> 3), kbox0, nvalid);
                if (hybridB)
                    lb.load_hybrid(baseB, sa + A_STAGE_BYTES, gl, (uint32_t)(xb >> 3), (uint32_t)(g.K.sY[0] >> 3),
                                   (uint32_t)(g.K.sY[1] >> 3), kbox0, nvalid);
            }
            // full[s] hears from this thread when its copies for the slab have landed
            ptx::cp_async_mbar_arrive_noinc(fullbar);
            if (gl == 0)
                GETT_TRACE(pg, 3);
        }
        first += wi.nslab;
    }
    ptx::cp_async_wait_all();
}

template <bool A_VEC_K, bool B_VEC_K, int TILE_N, int TILE_M, bool B_TRANS = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gett_umma_kernel(const __grid_constant__ GettKernelArgs g, const __grid_constant__ GettTmaMaps tm)
{
    extern __shared__ uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), tables after it
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t stages = (uint32_t)g.stages;
    constexpr uint32_t sbytes = stage_bytes(TILE_M, TILE_N);
    constexpr uint32_t A_STAGE_BYTES = TILE_M * TILE_K * 2;
    constexpr bool TWO_HALVES = TILE_M == 2 * MMA_M; // one tile fills both accumulator buffers
    SmemTables* T = reinterpret_cast<SmemTables*>(smem + stages * sbytes);
    const uint32_t stage0 = ptx::smem_u32(smem);

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef GETT_UMMA_CLUSTER
    const uint32_t total_work = g.tiles_m * (g.tiles_n >> 1) * g.split_k; // tile pairs
#else
    const uint32_t total_work = g.tiles_m * g.tiles_n * g.split_k;
#endif
    volatile int* abort_flag = &T->abort_flag;
    const uint64_t wait_ns = (uint64_t)g.wait_limit_us * 1000ull; // bound of every wait on a barrier

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < stages; ++s) {
            // the slab's producers (twice each with the transposing loader: once for their asynchronous
            // copies, once for their ordinary stores)
            ptx::mbar_init(ptx::smem_u32(&T->full[s]),
                           (g.prod_groups == 1                        ? PROD_THREADS
                            : g.prod_groups == 2 && PROD_GROUPS == 4 ? 2 * GROUP_LANES
                                                                     : GROUP_LANES) *
                               (B_TRANS ? 2 : 1));
#ifdef GETT_UMMA_CLUSTER
            ptx::mbar_init(ptx::smem_u32(&T->empty[s]), 2); // both CTAs of the pair are done with the stage
#else
            ptx::mbar_init(ptx::smem_u32(&T->empty[s]), 1);
#endif
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&T->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&T->acc_empty[b]), EPI_SET_THREADS);
        }
        ptx::mbar_init(ptx::smem_u32(&T->drain), 1);
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
#ifdef GETT_UMMA_CLUSTER
    ptx_mc::cluster_sync(); // the partner's barriers exist before anything is sent to them
#endif

    if (warp >= PROD_WARP0) {
        // Producers.  With a ring of one stage (tiles of a single slab) all producer warps
        // form one wide group and share every slab; otherwise groups of WARPS_PER_GROUP
        // warps own whole slabs round-robin.  The ring depth is a multiple of the group
        // count, so a stage's barriers are always used by the same group.
        const uint32_t ng = (uint32_t)g.prod_groups;
        const bool hybrid = (tm.a.use && tm.a.hybrid) || (tm.b.use && tm.b.hybrid);
        if (ng == 1) {
            if (hybrid)
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, PROD_THREADS, true, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, 0, 1, threadIdx.x - PROD_WARP0 * 32, 3);
            else
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, PROD_THREADS, false, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, 0, 1, threadIdx.x - PROD_WARP0 * 32, 3);
        } else if (ng == 2 && PROD_GROUPS == 4) {
            // a ring of two stages: two groups of twice the width, so that no producer warp idles
            constexpr uint32_t WPG = 2 * WARPS_PER_GROUP;
            const uint32_t pg = (warp - PROD_WARP0) / WPG;
            const uint32_t gl = threadIdx.x - (PROD_WARP0 + pg * WPG) * 32;
            if (hybrid)
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, 2 * GROUP_LANES, true, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, pg, ng, gl, 3 + pg);
            else
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, 2 * GROUP_LANES, false, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, pg, ng, gl, 3 + pg);
        } else {
            const uint32_t pg = (warp - PROD_WARP0) / WARPS_PER_GROUP;
            const uint32_t gl = threadIdx.x - (PROD_WARP0 + pg * WARPS_PER_GROUP) * 32;
            if (hybrid)
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, GROUP_LANES, true, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, pg, ng, gl, 3 + pg);
            else
                producer_role<A_VEC_K, B_VEC_K, TILE_N, TILE_M, GROUP_LANES, false, B_TRANS>(
                    g, tm, T, stage0, stages, total_work, abort_flag, pg, ng, gl, 3 + pg);
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------ MMA issuer -----------------------------
        if (lane == 0) {
            const uint32_t fmt = g.dtype == GETT_BF16_F32 ? 1u : 0u;
            const uint32_t idesc = ptx::idesc_f16(fmt, A_VEC_K ? 0u : 1u, B_VEC_K ? 0u : 1u, MMA_M, TILE_N);
            // bytes the descriptor start address advances per 16-wide k step
            const uint32_t a_step = A_VEC_K ? 32u : 2u * ATOM_BYTES;
            const uint32_t b_step = B_VEC_K ? 32u : 2u * ATOM_BYTES;
            const uint32_t lbo = MN_BLOCK_BYTES, sbo = ATOM_BYTES;
            uint32_t it = 0, local = 0;
            bool alive = true;
            const uint32_t nitems = item_count(g, total_work);
            for (; local < nitems && alive; ++local) {
                const WorkItem wi = decode_item(g, local, TILE_M);
                // 128-row tiles alternate between the two accumulator buffers; a 256-row tile
                // uses both (rows 0-127 in buffer 0, rows 128-255 in buffer 1)
                const uint32_t buf = TWO_HALVES ? 0u : (local & 1);
                const uint32_t par = TWO_HALVES ? (local & 1) : ((local >> 1) & 1);
                GETT_TRACE(6, 0);
                if (!ptx::mbar_wait(ptx::smem_u32(&T->acc_empty[buf]), par ^ 1, abort_flag, wait_ns))
                    break;
                GETT_TRACE(6, 1);
                if (TWO_HALVES && !ptx::mbar_wait(ptx::smem_u32(&T->acc_empty[1]), par ^ 1, abort_flag, wait_ns))
                    break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (uint32_t j = 0; j < wi.nslab; ++j, ++it) {
                    const uint32_t s = it % stages;
                    if (!ptx::mbar_wait(ptx::smem_u32(&T->full[s]), (it / stages) & 1, abort_flag, wait_ns)) {
                        alive = false;
                        break;
                    }
                    GETT_TRACE(6, 2);
                    // the copies were generic-proxy writes; the tensor core reads through the
                    // async proxy, so order the two before issuing
                    ptx::fence_proxy_async_smem();
                    ptx::tc_fence_after();
                    const uint32_t sa = stage0 + s * sbytes, sb = sa + A_STAGE_BYTES;
#pragma unroll
                    for (uint32_t h = 0; h < (TWO_HALVES ? 2u : 1u); ++h) {
                        // rows 128 h .. of the A tile start 16 KB further in either staging layout
                        const uint32_t sah = sa + h * (MMA_M * TILE_K * 2);
#pragma unroll
                        for (uint32_t kk = 0; kk < TILE_K / 16; ++kk) {
                            const uint64_t ad = A_VEC_K ? ptx::smem_desc_sw128(sah + kk * a_step, 16, ATOM_BYTES)
                                                        : ptx::smem_desc_sw128(sah + kk * a_step, lbo, sbo);
                            const uint64_t bd = B_VEC_K ? ptx::smem_desc_sw128(sb + kk * b_step, 16, ATOM_BYTES)
                                                        : ptx::smem_desc_sw128(sb + kk * b_step, lbo, sbo);
                            ptx::umma_f16(d_tmem + h * 256, ad, bd, idesc, (j | kk) ? 1u : 0u);
                        }
                    }
#ifdef GETT_UMMA_CLUSTER
                    // ... in both CTAs: the partner's copies land in this stage too
                    ptx_mc::umma_commit_pair(ptx::smem_u32(&T->empty[s]));
#else
                    ptx::umma_commit(ptx::smem_u32(&T->empty[s])); // stage reusable once these MMAs retire
#endif
                }
                GETT_TRACE(6, 3);
                if (alive) {
                    ptx::umma_commit(ptx::smem_u32(&T->acc_full[buf]));
                    if (TWO_HALVES)
                        ptx::umma_commit(ptx::smem_u32(&T->acc_full[1]));
                }
            }
            if (*abort_flag) {
                // somebody gave up: let the tensor core finish what was issued (it still reads the
                // stages and writes tensor memory) before the CTA frees both; bounded like every wait
                int never = 0;
                ptx::umma_commit(ptx::smem_u32(&T->drain));
                ptx::mbar_wait(ptx::smem_u32(&T->drain), 0, &never, 2000000000ull);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------- epilogue ------------------------------
        // Epilogue set es = warp / 4 takes the CTA's tiles number es, es + 2, ... (exactly
        // the tiles whose accumulator lives in buffer es); warp % 4 selects the 32
        // tensor-memory lanes (= tile rows) a warp may read.
        const uint32_t es = warp >> 2, eq = warp & 3;
        const uint32_t et = eq * 32 + lane; // tile row
        bool alive = true;
        const bool staged = g.epilogue == GETT_EPI_STAGED && g.split_k == 1;
        if (staged) {
            uint8_t* epi_smem = smem + stages * sbytes + sizeof(SmemTables);
            if (g.c_vec == 8 && g.epi_lean)
                epilogue_staged<TILE_N, 8, 1>(g, T, epi_smem, tmem_base, warp, lane, total_work, abort_flag);
            else if (g.c_vec == 8)
                epilogue_staged<TILE_N, 8, 0>(g, T, epi_smem, tmem_base, warp, lane, total_work, abort_flag);
            else if (g.epi_lean)
                epilogue_staged<TILE_N, 1, 1>(g, T, epi_smem, tmem_base, warp, lane, total_work, abort_flag);
            else
                epilogue_staged<TILE_N, 1, 0>(g, T, epi_smem, tmem_base, warp, lane, total_work, abort_flag);
        }
        int64_t* colC = T->colC[es];
        uint32_t j = 0; // counts this set's tiles
        // 128-row tiles: set es takes every other tile.  256-row tiles: both sets work on
        // every tile, set es on its rows 128 es .. 128 es + 127.
        const uint32_t nitems = item_count(g, total_work);
        for (uint32_t wn = TWO_HALVES ? 0u : es; wn < nitems && !staged; wn += TWO_HALVES ? 1u : 2u, ++j) {
            WorkItem wi = decode_item(g, wn, TILE_M);
            if (TWO_HALVES)
                wi.m0 += es * MMA_M;
            const uint32_t buf = es;
            // C offsets of this tile: my row in a register, the columns in shared memory
            int64_t rowC = -1;
            if (wi.m0 + et < g.M.size)
                rowC = gett_offset_y(g.M, wi.m0 + et);
            ptx::named_barrier(1 + es, EPI_SET_THREADS); // previous tile's column table no longer read
            for (uint32_t c = et; c < TILE_N; c += EPI_SET_THREADS) {
                int64_t y = -1;
                if (wi.n0 + c < g.N.size)
                    y = gett_offset_y(g.N, wi.n0 + c);
                colC[c] = y;
            }
            ptx::named_barrier(1 + es, EPI_SET_THREADS);
            const bool row_ok = rowC >= 0;
            const float alpha = g.alpha, beta = g.beta;
            // beta != 0: the old values of C do not depend on the accumulator, so those of the
            // first 16 columns are asked for before the wait for it, and those of every later
            // group of 16 one group ahead of their use (two register buffers, A and B)
            // (the same for every lane of the warp: the tensor-memory loads below are warp-wide
            //  instructions and must not sit in branches that lanes take differently; a lane
            //  whose row lies outside C fetches and stores nothing)
            const bool rmw = beta != 0.f && !wi.partial && !GETT_DBG(g, 2);
            float oldA[16], oldB[16];
            auto fetch = [&](uint32_t c0, float (&old)[16]) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int64_t co = colC[c0 + i];
                    old[i] = (row_ok && co >= 0) ? __ldcg(g.C + rowC + co) : 0.f;
                }
            };
            if (rmw)
                fetch(0, oldA);
            if (et == 0)
                GETT_TRACE(4 + es, 0);
            if (alive && !ptx::mbar_wait(ptx::smem_u32(&T->acc_full[buf]), j & 1, abort_flag, wait_ns))
                alive = false;
            if (!alive)
                continue; // keep the named barriers above matched, do nothing else
            ptx::tc_fence_after();
            if (et == 0)
                GETT_TRACE(4 + es, 1);
            const uint32_t taddr = tmem_base + ((eq * 32u) << 16) + buf * 256;
            if (rmw) {
                auto step = [&](uint32_t c0, float (&old)[16], float (&nxt)[16]) {
                    if (c0 + 16 < (uint32_t)TILE_N)
                        fetch(c0 + 16, nxt);
                    uint32_t v[16];
                    ptx::tmem_ld_32x16(taddr + c0, v);
                    ptx::tmem_wait_ld();
                    if (!row_ok)
                        return;
                    float* crow = g.C + rowC;
#pragma unroll
                    for (int h = 0; h < 2; ++h) { // eight columns at a time: their offsets, then the stores
                        int64_t co[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            co[i] = colC[c0 + 8 * h + i];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (co[i] >= 0)
                                crow[co[i]] = fmaf(beta, old[8 * h + i], alpha * __uint_as_float(v[8 * h + i]));
                    }
                };
                static_assert(TILE_N % 32 == 0, "two groups of 16 columns per turn");
                for (uint32_t c0 = 0; c0 < TILE_N; c0 += 32) {
                    step(c0, oldA, oldB);
                    step(c0 + 16, oldB, oldA);
                }
            } else {
                for (uint32_t c0 = 0; c0 < TILE_N; c0 += 16) {
                    uint32_t v[16];
                    ptx::tmem_ld_32x16(taddr + c0, v);
                    ptx::tmem_wait_ld();
                    if (!row_ok || GETT_DBG(g, 2)) // (debug & 2: experiment switch, no stores)
                        continue;
                    if (wi.partial && g.stream_k) {
                        // piece z of left-over tile r: a whole tile_m x TILE_N buffer [column][row]
                        float* dst = g.ws + (((size_t)wi.r * g.sk_pmax + wi.z) * TILE_N + c0) * (size_t)g.tile_m +
                                     (TWO_HALVES ? es * MMA_M : 0u) + et;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            dst[(size_t)i * g.tile_m] = __uint_as_float(v[i]);
                    } else if (wi.partial) {
                        float* dst = g.ws + ((size_t)wi.z * g.N.size + wi.n0 + c0) * g.M.size + wi.m0 + et;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (wi.n0 + c0 + i < g.N.size)
                                dst[(size_t)i * g.M.size] = __uint_as_float(v[i]);
                    } else {
                        float* crow = g.C + rowC;
                        int64_t co[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            co[i] = colC[c0 + i];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (co[i] >= 0)
                                crow[co[i]] = alpha * __uint_as_float(v[i]);
                    }
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(ptx::smem_u32(&T->acc_empty[buf]));
            if (et == 0)
                GETT_TRACE(4 + es, 2);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
#ifdef GETT_UMMA_CLUSTER
    ptx_mc::cluster_sync(); // the partner no longer writes to this CTA's shared memory or barriers
#endif
    if (threadIdx.x == 0 && T->abort_flag && g.status)
        *g.status = GETT_ERR_TIMEOUT;
    if (warp == MMA_WARP) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

} // namespace

#ifndef GETT_UMMA_CLUSTER
int gett_umma_smem_bytes(int tile_m, int tile_n, int stages, int staged_cv, int lean)
{
    return 1024 + stages * (int)stage_bytes((uint32_t)tile_m, (uint32_t)tile_n) + (int)sizeof(SmemTables) +
           (staged_cv ? NUM_EPI_WARPS * epi_warp_bytes(tile_n, staged_cv, lean) : 0);
}

int gett_umma_max_stages(int tile_m, int tile_n, int smem_limit, int staged_cv, int lean)
{
    int s = (smem_limit - 1024 - (int)sizeof(SmemTables) -
             (staged_cv ? NUM_EPI_WARPS * epi_warp_bytes(tile_n, staged_cv, lean) : 0)) /
            (int)stage_bytes((uint32_t)tile_m, (uint32_t)tile_n);
    s = s > MAX_STAGES ? MAX_STAGES : s;
    return s >= PROD_GROUPS ? s - s % PROD_GROUPS : s; // a stage is always served by the same group
}

int gett_umma_block() { return NUM_THREADS; }

int gett_umma_prod_groups(int stages) { return stages >= PROD_GROUPS ? PROD_GROUPS : stages; }

template <bool AK, bool BK, bool BT = false>
static cudaError_t launch_tn(const GettKernelArgs& args, const GettTmaMaps& maps, int grid, int smem,
                             cudaStream_t stream)
{
    void (*k)(GettKernelArgs, GettTmaMaps);
    if (args.tile_m == 256) {
        if (args.tile_n != 256)
            return cudaErrorInvalidValue;
        k = gett_umma_kernel<AK, BK, 256, 256, BT>;
    } else {
        switch (args.tile_n) {
        case 64: k = gett_umma_kernel<AK, BK, 64, 128, BT>; break;
        case 128: k = gett_umma_kernel<AK, BK, 128, 128, BT>; break;
        case 192: k = gett_umma_kernel<AK, BK, 192, 128, BT>; break;
        case 256: k = gett_umma_kernel<AK, BK, 256, 128, BT>; break;
        default: return cudaErrorInvalidValue;
        }
    }
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess)
        return e;
    k<<<grid, NUM_THREADS, smem, stream>>>(args, maps);
    return cudaGetLastError();
}

cudaError_t gett_launch_umma(const GettKernelArgs& args, const GettTmaMaps& maps, int grid, int smem,
                             cudaStream_t stream)
{
    const bool ak = args.loader_a == GETT_LOAD_VEC_K, bk = args.loader_b == GETT_LOAD_VEC_K;
    if (args.loader_b == GETT_LOAD_VEC_KT) // B staged K-major through the transposing loader; A K-major
        return ak ? launch_tn<true, true, true>(args, maps, grid, smem, stream) : cudaErrorInvalidValue;
    if (ak && bk)
        return launch_tn<true, true>(args, maps, grid, smem, stream);
    if (ak)
        return launch_tn<true, false>(args, maps, grid, smem, stream);
    if (bk)
        return launch_tn<false, true>(args, maps, grid, smem, stream);
    return launch_tn<false, false>(args, maps, grid, smem, stream);
}
#endif // !GETT_UMMA_CLUSTER

#if defined(GETT_EXPERIMENT) && !defined(GETT_UMMA_CLUSTER)
// experiment builds: fetch (and reset) the time stamps; out holds 8 x 4096 values, n 8 counts
extern "C" __attribute__((visibility("default"))) int gett_debug_trace(unsigned long long* out, unsigned int* n)
{
    if (cudaDeviceSynchronize() != cudaSuccess)
        return -1;
    if (cudaMemcpyFromSymbol(out, gett_trace_buf, sizeof(gett_trace_buf)) != cudaSuccess ||
        cudaMemcpyFromSymbol(n, gett_trace_n, sizeof(gett_trace_n)) != cudaSuccess)
        return -1;
    const unsigned int zero[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    return cudaMemcpyToSymbol(gett_trace_n, zero, sizeof(zero)) == cudaSuccess ? 0 : -1;
}
#endif
