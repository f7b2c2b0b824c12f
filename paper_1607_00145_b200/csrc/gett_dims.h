// Fused-dimension descriptors shared by the host planner and the device kernels.
//
// Each of the three logical GEMM dimensions (M = I_m, N = I_n, K = I_k fused;
// Sec. 2.2 / Sec. 3 of the paper) is a mixed-radix number: digit d has extent
// ext[d] and contributes idx_d * sX[d] to the offset in one carrier tensor and
// idx_d * sY[d] in the other (M: X = A, Y = C;  N: X = B, Y = C;  K: X = A, Y = B).
// Splitting a mode into two digits or merging two contiguous modes into one
// (Sec. 3.2.1, Sec. 6) changes only this list, never the data.
//
// A dimension may have a two-shaped low part.  Its fused index is then
//     idx = hi * period + lo,   lo in [0, period),
// where lo < seg1_start is taken apart by the digits [0, seg1_dig) ("segment 0"), lo >=
// seg1_start by the digits [seg1_dig, hi_dig) on top of the offsets seg1_bX / seg1_bY
// ("segment 1"), and hi by the digits [hi_dig, ndig).  This is how a stride-1 mode whose
// extent e = 64 q + r is not a multiple of the 64-wide operand rows is cut into rows of 64
// of its first 64 q indices (segment 0) and rows made of its last r indices times 64 / r
// indices of a second mode (segment 1): the sub-tensor choice of Sec. 3.2.1 with two shapes
// of sub-tensor, interleaved with period e * 64 / r so that every tile holds both kinds in
// the same proportion.  A dimension without such a low part has seg1_dig == hi_dig == ndig.
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
    uint32_t size;                 // number of fused indices, < 2^31
    uint32_t ext[GETT_MAX_DIGITS]; // first digit of a range fastest
    uint32_t mul[GETT_MAX_DIGITS]; // magic multiplier for division by ext[d]
    uint32_t sh[GETT_MAX_DIGITS];  // shift after the high multiply
    int64_t sX[GETT_MAX_DIGITS];
    int64_t sY[GETT_MAX_DIGITS];
    int32_t seg1_dig, hi_dig;      // digit ranges of segment 0, segment 1 and the high part (see above)
    uint32_t seg1_start;           // first low index of segment 1
    uint32_t period, period_mul, period_sh; // size of the low part and the magic numbers to divide by it
    int64_t seg1_bX, seg1_bY;      // offsets of segment 1's origin
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

// Walks the digits of a fused index: first the low part (one of the two segments; for a
// plain dimension, all digits), then the high part, if there is one.
//     GettWalk w(D, idx);
//     do { for (d = w.d; d < w.dend; ++d) <take digit d out of w.rem>; } while (w.next(D));
struct GettWalk {
    uint32_t rem, hi;
    int d, dend, seg;
    bool more;
    GETT_HD GettWalk(const GettDim& D, uint32_t idx)
    {
        rem = idx;
        hi = 0;
        d = 0;
        dend = D.ndig;
        seg = 0;
        more = false;
        if (D.seg1_dig < D.hi_dig) {
            hi = gett_fastdiv(idx, D.period_mul, D.period_sh);
            rem = idx - hi * D.period;
            dend = D.seg1_dig;
            if (rem >= D.seg1_start) {
                rem -= D.seg1_start;
                d = D.seg1_dig;
                dend = D.hi_dig;
                seg = 1;
            }
            more = true;
        }
    }
    GETT_HD bool next(const GettDim& D)
    {
        if (!more)
            return false;
        more = false;
        rem = hi;
        d = D.hi_dig;
        dend = D.ndig;
        return true;
    }
};

// Offsets of fused index `idx` in the two carrier tensors; returns the segment (0 or 1).
// (A plain dimension takes the first loop, which is all the arithmetic it needs.)
GETT_HD int gett_decompose(const GettDim& D, uint32_t idx, int64_t& oX, int64_t& oY)
{
    int64_t x = 0, y = 0;
    if (D.seg1_dig == D.hi_dig) {
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
        return 0;
    }
    GettWalk w(D, idx);
    if (w.seg) {
        x = D.seg1_bX;
        y = D.seg1_bY;
    }
    do {
#pragma unroll 1
        for (int d = w.d; d < w.dend; ++d) {
            uint32_t q = gett_fastdiv(w.rem, D.mul[d], D.sh[d]);
            uint32_t r = w.rem - q * D.ext[d];
            x += (int64_t)r * D.sX[d];
            y += (int64_t)r * D.sY[d];
            w.rem = q;
        }
    } while (w.next(D));
    oX = x;
    oY = y;
    return w.seg;
}

// The offset in the second carrier alone (M, N: the offset in C), for the unpacking code.
GETT_HD int64_t gett_offset_y(const GettDim& D, uint32_t idx)
{
    int64_t y = 0;
    if (D.seg1_dig == D.hi_dig) {
        uint32_t rem = idx;
#pragma unroll 1
        for (int d = 0; d < D.ndig; ++d) {
            uint32_t q = gett_fastdiv(rem, D.mul[d], D.sh[d]);
            y += (int64_t)(rem - q * D.ext[d]) * D.sY[d];
            rem = q;
        }
        return y;
    }
    GettWalk w(D, idx);
    if (w.seg)
        y = D.seg1_bY;
    do {
#pragma unroll 1
        for (int d = w.d; d < w.dend; ++d) {
            uint32_t q = gett_fastdiv(w.rem, D.mul[d], D.sh[d]);
            y += (int64_t)(w.rem - q * D.ext[d]) * D.sY[d];
            w.rem = q;
        }
    } while (w.next(D));
    return y;
}

// Tensor-map coordinates of fused index `idx`: digit d adds (its value) * cmul[d] to
// coordinate cdim[d] (cdim[d] < 0: none).  Returns the segment (0 or 1) the index lies in.
GETT_HD int gett_add_coords(const GettDim& D, uint32_t idx, const int8_t* cdim, const int32_t* cmul, int32_t* c)
{
    GettWalk w(D, idx);
    do {
#pragma unroll 1
        for (int d = w.d; d < w.dend; ++d) {
            uint32_t q = gett_fastdiv(w.rem, D.mul[d], D.sh[d]);
            if (cdim[d] >= 0)
                c[cdim[d]] += (int32_t)(w.rem - q * D.ext[d]) * cmul[d];
            w.rem = q;
        }
    } while (w.next(D));
    return w.seg;
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
