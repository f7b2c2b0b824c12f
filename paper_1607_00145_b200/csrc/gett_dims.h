// Fused-dimension descriptors shared by the host planner and the device kernels.
//
// Each of the three logical GEMM dimensions (M = I_m, N = I_n, K = I_k fused;
// Sec. 2.2 / Sec. 3 of the paper) is a mixed-radix number: digit d has extent
// ext[d] and contributes idx_d * sX[d] to the offset in one carrier tensor and
// idx_d * sY[d] in the other (M: X = A, Y = C;  N: X = B, Y = C;  K: X = A, Y = B).
// Splitting a mode into two digits or merging two contiguous modes into one
// (Sec. 3.2.1, Sec. 6) changes only this list, never the data.
//
// decompose() below is the single routine that turns a fused index into storage
// offsets ("identify_subtensor" of Listing 4, done arithmetically); the kernels
// call it on the device and the planner calls it on the host to produce the
// tables that gett_plan_get_table returns.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define GETT_HD __host__ __device__ __forceinline__
#else
#define GETT_HD inline
#endif

#define GETT_MAX_DIGITS 12

struct GettDim {
    int32_t ndig;                  // 0 => fused size 1
    uint32_t size;                 // product of ext[], < 2^31
    uint32_t ext[GETT_MAX_DIGITS]; // first digit fastest
    uint32_t mul[GETT_MAX_DIGITS]; // magic multiplier for division by ext[d]
    uint32_t sh[GETT_MAX_DIGITS];  // shift after the high multiply
    int64_t sX[GETT_MAX_DIGITS];
    int64_t sY[GETT_MAX_DIGITS];
};

GETT_HD uint32_t gett_mulhi(uint32_t a, uint32_t b)
{
#if defined(__CUDA_ARCH__)
    return __umulhi(a, b);
#else
    return (uint32_t)(((uint64_t)a * (uint64_t)b) >> 32);
#endif
}

// n / d for n < 2^31 with (mul, sh) from gett_magic(); d == 1 is encoded as mul == 0.
GETT_HD uint32_t gett_fastdiv(uint32_t n, uint32_t mul, uint32_t sh)
{
    return mul ? (gett_mulhi(n, mul) >> sh) : n;
}

// Offsets of fused index `idx` in the two carrier tensors.
GETT_HD void gett_decompose(const GettDim& D, uint32_t idx, int64_t& oX, int64_t& oY)
{
    int64_t x = 0, y = 0;
    uint32_t rem = idx;
#pragma unroll 1
    for (int d = 0; d < D.ndig; ++d) {
        uint32_t q = gett_fastdiv(rem, D.mul[d], D.sh[d]);
        uint32_t r = rem - q * D.ext[d];
        x += (int64_t)r * D.sX[d];
        y += (int64_t)r * D.sY[d];
        rem = q;
    }
    oX = x;
    oY = y;
}

// The offset in the second carrier alone (M, N: the offset in C), for the unpacking code.
GETT_HD int64_t gett_offset_y(const GettDim& D, uint32_t idx)
{
    int64_t y = 0;
    uint32_t rem = idx;
#pragma unroll 1
    for (int d = 0; d < D.ndig; ++d) {
        uint32_t q = gett_fastdiv(rem, D.mul[d], D.sh[d]);
        y += (int64_t)(rem - q * D.ext[d]) * D.sY[d];
        rem = q;
    }
    return y;
}

// Per-digit indices of fused index `idx` (first `n` digits are written).
GETT_HD void gett_digit_indices(const GettDim& D, uint32_t idx, int32_t* out, int n)
{
    uint32_t rem = idx;
#pragma unroll 1
    for (int d = 0; d < D.ndig && d < n; ++d) {
        uint32_t q = gett_fastdiv(rem, D.mul[d], D.sh[d]);
        out[d] = (int32_t)(rem - q * D.ext[d]);
        rem = q;
    }
}

#if !defined(__CUDA_ARCH__)
// Host only: magic numbers such that floor(n / d) == mulhi(n, mul) >> sh for all n < 2^31.
inline void gett_magic(uint32_t d, uint32_t& mul, uint32_t& sh)
{
    if (d <= 1) {
        mul = 0;
        sh = 0;
        return;
    }
    uint32_t l = 0;
    while ((1ull << l) < d)
        ++l; // l = ceil(log2 d) >= 1
    uint64_t p = 1ull << (31 + l);
    mul = (uint32_t)((p + d - 1) / d); // ceil(2^(31+l) / d) <= 2^32 - 1 for d >= 2
    sh = l - 1;
}
#endif
