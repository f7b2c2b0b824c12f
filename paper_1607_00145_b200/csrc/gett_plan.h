// Internal plan object: what the host planner decides and what every kernel
// launch receives.  Nothing in this header is part of the public ABI.
#pragma once
#include <stdint.h>

#include <vector>

#include "../../include/gett.h"
#include "gett_dims.h"

// One mode of the contraction after classification (Sec. 2.2).
struct GettMode {
    int32_t label;
    int64_t ext;
    int64_t sA, sB, sC; // element strides; 0 where the tensor does not carry the mode
};

// One digit of a tile-order fused index: value v of the digit stands for index
// off + v * mult of mode `mode` (an index into the canonical list of that set).
// mult > 1 or ext < mode extent means the mode was split by factors of its extent
// (Sec. 3.2.1, Examples 1-2); off > 0 (or a range shorter than the extent) means the
// digit covers a sub-range of the mode, which happens only in two-segment dimensions.
struct GettDigit {
    int32_t mode;
    int64_t ext;
    int64_t mult;
    int64_t off;
};

// Timing probes ("skip the stores", "skip the math", ...) that give wrong results on purpose
// exist only in builds made with -DGETT_EXPERIMENT; in the library as shipped GETT_DBG()
// is the constant 0 and the code behind it is compiled out.
#ifdef GETT_EXPERIMENT
#define GETT_DBG(g, bits) (((g).debug & (bits)) != 0)
#else
#define GETT_DBG(g, bits) false
#endif

// Arguments common to every contraction kernel (passed by value).
struct GettKernelArgs {
    GettDim M, N, K; // tile-order digits, merged where contiguous
    const void* A;
    const void* B;
    float* C;
    float* ws;      // split-K partial sums [split][N][M] (tile-order fused indices), or null
    int32_t* status; // device status word, written only on failure
    float alpha, beta;
    uint32_t tiles_m, tiles_n;
    uint32_t split_k;     // >= 1
    uint32_t k_per_split; // K elements per slice, a multiple of tile_k
    int32_t dtype;        // gett_dtype_t
    int32_t a_kmajor;     // A's fastest-varying direction in memory is K (else M)
    int32_t b_kmajor;
    int32_t loader_a, loader_b; // gett_loader_t of the vectorised kernels
    int32_t tile_m;       // tile height of the tensor-core kernel (128 or 256)
    int32_t tile_n;       // tile width of the tensor-core / FFMA kernels
    int32_t stages;       // depth of the shared-memory ring
    int32_t epilogue;     // gett_epilogue_t
    int32_t c_vec;        // four consecutive tile rows (1) or columns (2) are one aligned 16-byte
                          // vector of C; column-to-slot pattern of the staged epilogues: 1 or 8
                          // (tensor-core kernel), 4 (fp32 kernel: column = a + 4 p, p along C)
    int32_t debug;        // opts.experiment: timing probes, read only by GETT_EXPERIMENT builds
    uint32_t wait_limit_us; // bound of every device-side wait on a barrier
    int32_t prod_groups;  // producer groups the tensor-core kernel uses (divides stages)
    int32_t epi_lean;     // staged epilogue of the tensor-core kernel with one narrow staging buffer per warp
    uint32_t stream_k;    // tensor-core kernel: the tiles left over after whole rounds are cut along K (see item_count())
    uint32_t sk_full;     // ... whole rounds of tiles (one tile per CTA and round)
    uint32_t sk_units;    // ... slab units of the left-over tiles per CTA
    uint32_t sk_slabs;    // ... slabs per tile
    uint32_t sk_pmax;     // ... pieces per left-over tile, at most (workspace: [tile][piece][tile_n][tile_m])
};

// How the coordinates of a TMA box follow from fused indices: digit d of the operand's free
// dimension adds (digit value) * fmul[d] to coordinate fdim[d], digit d of K adds
// (digit value) * kmul[d] to coordinate kdim[d] (a negative dimension: none).
struct GettTmaCoords {
    int32_t rank;
    int8_t fdim[GETT_MAX_DIGITS], kdim[GETT_MAX_DIGITS];
    int32_t fmul[GETT_MAX_DIGITS], kmul[GETT_MAX_DIGITS];
};

// Recipe for one operand's TMA tensor map (the map itself is encoded per call, since it
// embeds the operand's base address).  Dimension 0 is the operand's stride-1 mode.
// K-major staging: the whole tile (rows x 64 k) is one box.  MN-major staging: the tile is
// fetched in "atoms" of 64 free indices x 64 k, one box each; when the free dimension has
// two segments (gett_dims.h), only the atoms of segment 0 are boxes and those of segment 1
// are gathered (`hybrid`).
struct GettTmaRecipe {
    int32_t enabled;
    int32_t hybrid;
    uint64_t dims[5];
    uint64_t strides[5]; // elements; strides[0] == 1
    uint32_t box[5];
    GettTmaCoords co;
};

// What the tensor-core kernel receives besides GettKernelArgs when an operand is
// loaded through TMA.  `map` is an opaque CUtensorMap (128 bytes, 64-byte aligned).
struct alignas(64) GettTmaSide {
    uint64_t map[16];
    int32_t use;    // 0: the operand is gathered
    int32_t hybrid; // 1: atoms of segment 1 of the free dimension are gathered, the others come by TMA
    GettTmaCoords co;
};
struct alignas(64) GettTmaMaps {
    GettTmaSide a, b;
};

struct gett_plan {
    int32_t dtype;
    std::vector<GettMode> im, in, ik; // canonical order (what get_info reports)
    std::vector<GettDigit> tm, tn, tk; // tile order, before merging
    int32_t tm_seg1, tn_seg1;          // position in tm / tn where segment 1 starts, -1: a plain order
    int32_t tm_hi, tn_hi;              // ... and where the high part starts (see gett_dims.h)
    GettDim M, N, K;                   // tile order, merged: what the kernels get
    gett_plan_info_t info;
    // geometry
    uint32_t tiles_m, tiles_n, k_per_split;
    int32_t a_kmajor, b_kmajor;
    int32_t c_vec;
    int32_t skinny; // fp32: B resident in shared memory, A streamed (small N and K)
    int32_t epi_lean; // see GettKernelArgs
    int32_t pair_ok;  // the CTA-pair variant of the tensor-core kernel applies (used if its library is there)
    uint32_t stream_k, sk_full, sk_units, sk_slabs, sk_pmax; // see GettKernelArgs
    int32_t swapped;  // the kernels get the caller's B as their A and vice versa (im / in / ik, tm / tn / tk,
                      // M / N / K and the loaders below are the kernels' view; info is the caller's)
    GettTmaRecipe tma_a, tma_b;
    // device side
    float* ws;
    int32_t* status;
    int32_t sm_count;
    int32_t debug;     // opts.experiment
    int32_t flags;     // opts.flags
    int32_t wait_limit_us;
};

// Host planner (planner.cpp): everything except device allocation.
gett_status_t gett_planner_build(gett_plan* p, const gett_tensor_desc_t* A,
                                 const gett_tensor_desc_t* B, const gett_tensor_desc_t* C,
                                 gett_dtype_t dtype, const gett_plan_opts_t* opts, int sm_count);
gett_status_t gett_planner_table(const gett_plan* p, int which, int64_t* dst, size_t capacity);

// Candidate enumeration and the performance model (search.cpp).
double gett_planner_model(const gett_plan* p, int sm_count, double terms[4]);
std::vector<gett_plan_opts_t> gett_planner_candidates(const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                                                     const gett_tensor_desc_t* C, gett_dtype_t dtype,
                                                     const gett_plan_opts_t& base, int sm_count);

// Geometry of the tensor-core kernel (kernel_umma.cu), needed by the planner.
int gett_umma_smem_bytes(int tile_m, int tile_n, int stages, int staged_cv, int lean); // staged_cv: 0, 1 or 8
int gett_umma_max_stages(int tile_m, int tile_n, int smem_limit, int staged_cv, int lean);
int gett_umma_block();
int gett_umma_prod_groups(int stages); // producer groups in use; must divide the ring depth

// Geometry of the fp32 kernel (kernel_ffma.cu).
int gett_ffma_smem_bytes(int tile_m, int tile_n, int stages);

// fp32 kernel for N <= 64, K <= gett_ffma_skinny_max_k(), A K-major (kernel_ffma_skinny.cu).
int gett_ffma_skinny_smem_bytes(int N, int K, int vec_rows); // vec_rows: c_vec == 1
int gett_ffma_skinny_mn_smem_bytes(int N, int K); // ... A staged MN-major (its stride-1 mode is free)
int gett_ffma_skinny_rows();
int gett_ffma_skinny_max_k();
