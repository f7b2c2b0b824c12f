/*
 * gett.h -- C ABI of the B200 (sm_100a) GEMM-like tensor-tensor multiplication.
 *
 * The operation (Sec. 2.2, Eq. 2 / Eq. 3 of "Design of a High-Performance
 * GEMM-like Tensor-Tensor Multiplication"):
 *
 *     C[Pi_C(I_m u I_n)] <- alpha * sum_{I_k} A[Pi_A(I_m u I_k)] * B[Pi_B(I_k u I_n)]
 *                           + beta * C[Pi_C(I_m u I_n)]
 *
 * I_m = labels carried by A and C (free in A), I_n = labels carried by B and C
 * (free in B), I_k = labels carried by A and B (contracted).  The contraction is
 * computed GEMM-like (Sec. 3, Listing 4): the three index sets are fused into
 * logical M, N, K dimensions, sub-tensors of A and B are packed into on-chip
 * memory tile by tile, multiplied by a macro-kernel, and C is updated in place
 * through its own mode permutation.  No transposed copy of A, B or C is ever
 * written to global memory.
 *
 * Everything here is plain C: sizes, host/device pointers, no C++ or torch types.
 * The library never prints, throws or aborts; every call returns a status.
 */
#ifndef GETT_H
#define GETT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GETT_MAX_MODES 12 /* modes per tensor */

#if defined(__GNUC__)
#define GETT_API __attribute__((visibility("default")))
#else
#define GETT_API
#endif

typedef struct gett_plan gett_plan_t; /* opaque, library-owned */

typedef enum {
    GETT_OK = 0,
    GETT_ERR_INVALID_ARG = 1,     /* NULL, mode count, extent < 1, stride < 1, overlapping C */
    GETT_ERR_BAD_LABELS = 2,      /* label twice in a tensor, in all three, or in one only  */
    GETT_ERR_EXTENT_MISMATCH = 3, /* the two carriers of a label disagree on its extent     */
    GETT_ERR_UNSUPPORTED = 4,     /* dtype / size outside what the kernels cover            */
    GETT_ERR_ALIGNMENT = 5,       /* operand base not aligned to its element size           */
    GETT_ERR_ALLOC = 6,           /* workspace allocation failed                            */
    GETT_ERR_CUDA = 7,            /* no device, launch failure                              */
    GETT_ERR_TIMEOUT = 8          /* a bounded device-side wait gave up (see gett_plan_last_device_status) */
} gett_status_t;

typedef enum {
    GETT_F32 = 0,      /* A, B, C fp32; strict fp32 FMA accumulation          */
    GETT_BF16_F32 = 1, /* A, B bf16; fp32 accumulation; C fp32                */
    GETT_F16_F32 = 2,  /* A, B fp16; fp32 accumulation; C fp32                */
    GETT_F64 = 3       /* A, B, C fp64; fp64 FMA accumulation (the precision of the paper's
                          Table IV); scalar-gather kernel only, no K slices       */
} gett_dtype_t;

/*
 * One tensor: mode i has extent[i] >= 1, stride[i] >= 1 (in elements) and an
 * integer label.  stride == NULL means packed with the FIRST mode stride-1
 * (the paper's Fortran-order convention, Sec. 2.2).  The arrays are copied by
 * gett_plan_create; the caller keeps ownership.
 */
typedef struct {
    int32_t nmodes; /* 0 .. GETT_MAX_MODES */
    const int64_t* extent;
    const int64_t* stride;
    const int32_t* label;
} gett_tensor_desc_t;

typedef enum {
    GETT_PATH_AUTO = 0,
    GETT_PATH_SIMT = 1, /* scalar gathers, any layout, any dtype (always available)        */
    GETT_PATH_FFMA = 2, /* fp32: 16-byte cp.async gathers, register-blocked FFMA           */
    GETT_PATH_UMMA = 3  /* bf16/fp16: 16-byte gathers into swizzled smem, tcgen05 + TMEM   */
} gett_path_t;

typedef enum {
    GETT_LOAD_SCALAR = 0, /* element-wise gather                                           */
    GETT_LOAD_VEC_FREE = 1, /* 16-byte vectors along the operand's free (M or N) dimension */
    GETT_LOAD_VEC_K = 2,    /* 16-byte vectors along the contracted dimension              */
    GETT_LOAD_TMA_FREE = 3, /* tensor-map (TMA) boxes, operand's stride-1 mode is free      */
    GETT_LOAD_TMA_K = 4,    /* tensor-map (TMA) boxes, operand's stride-1 mode is contracted */
    GETT_LOAD_VEC_KT = 5    /* 16-bit operand whose stride-1 mode is a contracted mode other than the one
                               the other operand runs along: 16-byte pieces are read along its own
                               stride-1 mode and 8 x 8 blocks are transposed in registers on their way
                               to shared memory (Sec. 3.2.2: packing is a transposition)             */
} gett_loader_t;

typedef enum {
    GETT_EPI_AUTO = 0,
    GETT_EPI_DIRECT = 1, /* each thread stores its accumulators straight to C              */
    GETT_EPI_STAGED = 2  /* accumulators pass through a shared-memory transpose so that
                            stores run along C's stride-1 mode (Eq. 11 as a transposition);
                            available when that mode is a mode of I_n and four consecutive
                            tile columns -- or, after B's stride-1 mode has been split into
                            16-byte pieces around it (Sec. 3.2.1), four consecutive values of
                            it -- are one aligned 16-byte vector of C.  GETT_EPI_DIRECT also
                            switches that split off.                                        */
} gett_epilogue_t;

/* Bits of gett_plan_opts_t.flags: each switches one automatic choice of the planner off.
 * Results are the same with or without them; they exist so that every loader / launch
 * variant can be run on the same problem (tests, comparisons). */
typedef enum {
    GETT_OPT_NO_TMA = 1,      /* gather with 16-byte copies even where tensor-map (TMA) boxes apply  */
    GETT_OPT_NO_PAIR = 2,     /* never launch the CTA-pair variant of the tensor-core kernel         */
    GETT_OPT_NO_EXCHANGE = 4, /* never exchange the roles of A and B                                 */
    GETT_OPT_NO_ATOMS = 8,    /* no re-ordering of I_m, I_n, I_k into 64 x 64 atoms that are boxes   */
    GETT_OPT_STREAMK = 16,    /* tensor-core kernel: cut the tiles that are left over after whole rounds
                                 (one tile per SM) along K wherever that is possible (more tiles than
                                 SMs, direct epilogue, no K slices), not only when the last round of
                                 tiles would be mostly empty                                          */
    GETT_OPT_NO_STREAMK = 32  /* ... never                                                           */
} gett_opt_flags_t;

/* Planner overrides; zero-initialise for "auto".  Unsupported combinations make
 * gett_plan_create return GETT_ERR_UNSUPPORTED rather than being silently changed. */
typedef struct {
    int32_t path;     /* gett_path_t                                     */
    int32_t tile_m;   /* 0 = auto; UMMA 128 | 256, FFMA 128 | 64 (256: small-N kernel), SIMT 64 */
    int32_t tile_n;   /* 0 = auto; UMMA 64 | 128 | 192 | 256, FFMA 128 | 32, SIMT 64            */
    int32_t tile_k;   /* 0 = auto (K elements per pipeline stage)        */
    int32_t stages;   /* 0 = auto                                        */
    int32_t split_k;  /* 0 = auto, 1 = never, s > 1 = exactly s slices   */
    int32_t epilogue; /* gett_epilogue_t                                 */
    int32_t flags;    /* gett_opt_flags_t bits                           */
    int32_t wait_limit_us; /* 0 = default (2 s): how long a device-side wait on a barrier may last
                              before the kernel gives up and records GETT_ERR_TIMEOUT.  Honoured by
                              the tensor-core kernel when both operands are gathered (its TMA
                              loaders keep the default); meant for tests of the give-up path.   */
    int32_t experiment; /* ignored, except by builds made with -DGETT_EXPERIMENT (timing probes) */
    int32_t search;   /* 0 = the planner's rules decide (default).  k >= 1: enumerate the candidate
                         plans (tile height and width, epilogue, loaders, operand exchange, split-K:
                         Sec. 3.3), rank them with the performance model (Sec. 3.4, Eq. 12-14,
                         re-parameterised for this GPU) and take the model's best (k == 1) or time
                         the k best and the rule-based plan on the device (cold L2, scratch operands
                         allocated for the purpose) and take the fastest (Sec. 7.3).  The choice is remembered per process
                         for equal descriptors, dtype, options and device.                      */
    int32_t reserved[5];
} gett_plan_opts_t;

/* What the planner decided (Sec. 3.2.1: index sets, fused sizes, blocking). */
typedef struct {
    int64_t M, N, K;                  /* S_{I_m}, S_{I_n}, S_{I_k}                         */
    int32_t n_m, n_n, n_k;            /* sizes of I_m, I_n, I_k after dropping extent-1    */
    int32_t labels_m[GETT_MAX_MODES]; /* canonical order: ascending stride in C            */
    int32_t labels_n[GETT_MAX_MODES]; /* canonical order: ascending stride in C            */
    int32_t labels_k[GETT_MAX_MODES]; /* canonical order: ascending stride in A            */
    int32_t merged_m, merged_n, merged_k; /* super-indices left after merging (Sec. 6)     */
    int32_t path;                     /* gett_path_t actually chosen                       */
    int32_t loader_a, loader_b;       /* gett_loader_t                                     */
    int32_t epilogue;                 /* gett_epilogue_t                                   */
    int32_t tile_m, tile_n, tile_k, stages, split_k;
    int32_t grid, block, smem_bytes;
    int32_t digits_m, digits_n, digits_k; /* digits of the tile-order fused indices        */
    int64_t workspace_bytes;          /* split-K partial sums owned by the plan            */
    int64_t tiles;                    /* output tiles (M tiles x N tiles)                  */
    int32_t device;                   /* CUDA device the plan is bound to, -1 = none       */
    int32_t swapped;                  /* 1: the kernel runs with the operands exchanged (its rows
                                         run over I_n, its columns over I_m; tile_m and tile_n are
                                         the kernel's).  Everything else here is the caller's view. */
    int32_t candidates;               /* opts.search > 0: candidate plans enumerated (0 when the choice
                                         was remembered from an earlier search), else 0             */
    int32_t model_rank;               /* position of this plan in the model's ranking (0 = its best) */
    int32_t timed;                    /* candidates that were timed on the device                  */
    float model_us;                   /* the performance model's estimate for this plan            */
    float timed_us;                   /* measured time of this plan during the search, else 0      */
    int32_t stream_k;                 /* 1: the tiles left over after whole rounds are cut along K and shared
                                         by all SMs (stream-K); workspace_bytes holds their pieces    */
} gett_plan_info_t;

typedef enum {
    GETT_TABLE_A_M = 0, /* offset in A of fused free-in-A index m   (length M) */
    GETT_TABLE_A_K = 1, /* offset in A of fused contracted index k  (length K) */
    GETT_TABLE_B_N = 2,
    GETT_TABLE_B_K = 3,
    GETT_TABLE_C_M = 4,
    GETT_TABLE_C_N = 5
} gett_table_t;

/*
 * gett_plan_create -- classify the labels into I_m, I_n, I_k (Sec. 2.2), drop
 * extent-1 modes, merge adjacent modes into super-indices (Sec. 6, stage 1),
 * choose the order in which each set is fused so that the stride-1 modes of A,
 * B and C stay inside a tile (Sec. 3.2.1), and pick kernel, blocking and split-K.
 *   out    : receives the plan (host pointer to host pointer).  Untouched on error.
 *   A,B,C  : host descriptors; copied.  C's modes must not overlap in memory, and the
 *            library recognises that only for NESTED layouts: sorted by stride, every mode of
 *            extent > 1 must step over the whole extent of the previous one (stride_j >=
 *            stride_i * extent_i).  Packed and padded layouts are nested; an interleaved
 *            layout that is overlap-free without being nested is rejected (INVALID_ARG).
 *   dtype  : gett_dtype_t.
 *   opts   : host pointer or NULL for automatic choices.
 * The plan is bound to the CUDA device current at the call; its split-K
 * workspace (device memory, info.workspace_bytes) is allocated here.  Without
 * any CUDA device the plan is still created (device = -1) and can be
 * inspected, but gett_contract returns GETT_ERR_CUDA.
 * Errors: INVALID_ARG, BAD_LABELS, EXTENT_MISMATCH, UNSUPPORTED (fused M, N or
 * K >= 2^31, dtype, impossible opts), ALLOC.
 */
GETT_API gett_status_t gett_plan_create(gett_plan_t** out, const gett_tensor_desc_t* A,
                               const gett_tensor_desc_t* B, const gett_tensor_desc_t* C,
                               gett_dtype_t dtype, const gett_plan_opts_t* opts);

/*
 * gett_contract -- run C <- alpha * A*B + beta * C (Eq. 2) on `cuda_stream`
 * (a cudaStream_t passed as void*; NULL = the default stream).
 *   A, B, C : DEVICE pointers, caller-owned, covering 1 + sum (extent-1)*stride
 *             elements each; A/B of the plan's input type, C fp32 (fp64 for GETT_F64).  Bases must be
 *             aligned to the element size; 16-byte aligned bases enable the
 *             vectorised kernels, otherwise the scalar path is used.
 *   alpha, beta : host scalars.  beta == 0 means C is not read (NaN/Inf in the
 *             old C do not propagate).  alpha == 0 takes no shortcut.
 * The device current at the call must be the one the plan was created on
 * (info.device), otherwise GETT_ERR_INVALID_ARG.  (Where the optional CTA-pair variant
 * of the tensor-core kernel is installed, it is used only when A and B are ordinary
 * device memory of that same GPU: its copies are delivered to two CTAs at once and its
 * tensor maps must cover this GPU's memory alone; only single-GPU processes use it.)
 * Asynchronous; allocates nothing; returns launch-time errors only.  C must not
 * alias A or B.  A plan may be reused; calls that use the same plan concurrently
 * on different streams race on its workspace when info.split_k > 1.
 * Every element of C that its descriptor addresses is written exactly once per
 * call; gaps left by padded strides are not touched.
 */
GETT_API gett_status_t gett_contract(const gett_plan_t* plan, float alpha, const void* A, const void* B,
                            float beta, void* C, void* cuda_stream);

/* gett_plan_destroy -- free the plan and its workspace.  NULL is a no-op. */
GETT_API gett_status_t gett_plan_destroy(gett_plan_t* plan);

/* gett_plan_get_info -- copy the planner's decisions into *info (host). */
GETT_API gett_status_t gett_plan_get_info(const gett_plan_t* plan, gett_plan_info_t* info);

/*
 * gett_plan_get_table -- one of the six offset tables of Sec. 3.2 ("identify
 * sub-tensor"): entry i is the storage offset (elements) contributed by fused
 * index i, fused in the canonical order reported by gett_plan_get_info with the
 * first mode fastest.  The element addressed by (m, n) of C is
 * C_M[m] + C_N[n]; likewise A_M[m] + A_K[k] and B_N[n] + B_K[k].
 * The entries are produced by the same index-decomposition routine and digit
 * data that the kernels use on the device (evaluated here on the host, through
 * the tile-order digits the kernels receive).
 *   dst : host array of `capacity` int64; needs capacity >= table length,
 *         else INVALID_ARG.
 */
GETT_API gett_status_t gett_plan_get_table(const gett_plan_t* plan, int which, int64_t* dst,
                                  size_t capacity);

/*
 * gett_plan_last_device_status -- 0 if no kernel launched from this plan has
 * reported a problem, else the gett_status_t a kernel recorded (GETT_ERR_TIMEOUT
 * when a bounded wait on a barrier ran out).  Synchronises with the device.
 */
GETT_API gett_status_t gett_plan_last_device_status(const gett_plan_t* plan);

/*
 * gett_contract_noalloc -- the same contraction for callers that cannot allocate
 * device memory.  (The paper has no counterpart: it is an addition of this library.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are not allowed or not
 * wanted -- while a stream is being captured, under an allocator that has claimed
 * the whole device, inside a latency-critical loop, or in a host callback.  The
 * plan-based calls above allocate a status word and, for split-K plans, a workspace
 * when the plan is created.  This call creates no plan object on the device and
 * calls no allocating routine at all: the contraction runs through the scalar-gather
 * kernel with the contracted range cut into `split_k` slices, and the slices'
 * partial sums are kept in an array of GETT_NOALLOC_WORKSPACE_BYTES that is built
 * into the library image (each GPU that loads the library holds that array until
 * the process exits).
 *
 *   A, B, C   : host descriptors, as for gett_plan_create (read during the call only).
 *   split_k   : 0 = let the planner choose, 1 = no slicing, s > 1 = s slices.
 *   A_data, B_data, C_data : device pointers, as for gett_contract.
 *   cuda_stream : cudaStream_t as void*, NULL = default stream.  Asynchronous.
 *
 * Limit: split_k * M * N * 4 bytes must not exceed GETT_NOALLOC_WORKSPACE_BYTES,
 * otherwise GETT_ERR_UNSUPPORTED is returned and nothing is launched.  Other errors
 * as for gett_plan_create / gett_contract.
 *
 * The first call on each device looks up the device address of the built-in array
 * (with that device current); make that first call outside any stream capture.
 * All calls share the one array, and it keeps the previous call's partial sums:
 * every call overwrites exactly the entries it later reads, so nothing has to be
 * cleared, but two calls whose kernels overlap on the GPU (different streams) race
 * on it -- order them on one stream or with events.
 */
#define GETT_NOALLOC_WORKSPACE_BYTES (16u << 20)
GETT_API gett_status_t gett_contract_noalloc(const gett_tensor_desc_t* A, const gett_tensor_desc_t* B,
                                    const gett_tensor_desc_t* C, gett_dtype_t dtype,
                                    int32_t split_k, float alpha, const void* A_data,
                                    const void* B_data, float beta, void* C_data,
                                    void* cuda_stream);

/*
 * gett_plan_model -- the performance model's estimate for a plan (Sec. 3.4: Time = Time_macro +
 * Time_A + Time_B + Time_C, Eq. 12-14, with this GPU's rates and with the loads overlapping the
 * macro-kernel).  terms_us: host array of 4 doubles or NULL; receives the four terms in
 * microseconds for the whole job.  total_us: host pointer, receives the estimate.
 */
GETT_API gett_status_t gett_plan_model(const gett_plan_t* plan, double* total_us, double* terms_us);

/* Human-readable name of a status; never NULL. */
GETT_API const char* gett_status_string(gett_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* GETT_H */
