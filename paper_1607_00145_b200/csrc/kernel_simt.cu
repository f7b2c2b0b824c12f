// Scalar-gather contraction kernel: correct for every layout and input type.
//
// One CTA owns a 64 x 64 tile of the fused (M, N) output and walks its K range in
// slabs of 16 (the loop nest of Listing 4 with the m- and n-loops spread over the
// grid).  "Packing" (Sec. 3.2.2) is the element-wise gather of the A and B
// sub-tensors into shared memory; the macro-kernel is a 4 x 4 register tile per
// thread; "unpacking" (Eq. 11) is the alpha/beta update written straight to C's
// own permutation.  This is the fallback for shapes the vectorised kernels
// cannot take (odd extents, unaligned bases, padded strides).
#include <cuda_fp16.h>

#include "kernels.h"

namespace {

constexpr int TM = 64, TN = 64, TK = 16, NT = 256;

// The type the sums are kept in (and C is stored as): double for GETT_F64, else float.
template <int DT>
struct Acc {
    typedef float type;
};
template <>
struct Acc<GETT_F64> {
    typedef double type;
};

template <int DT>
__device__ __forceinline__ typename Acc<DT>::type load_elem(const void* base, int64_t off)
{
    if (DT == GETT_F64)
        return __ldg(reinterpret_cast<const double*>(base) + off);
    if (DT == GETT_F32)
        return __ldg(reinterpret_cast<const float*>(base) + off);
    unsigned short h = __ldg(reinterpret_cast<const unsigned short*>(base) + off);
    if (DT == GETT_BF16_F32)
        return __uint_as_float(static_cast<unsigned int>(h) << 16);
    return __half2float(__ushort_as_half(h));
}

template <int DT>
__global__ void __launch_bounds__(NT) gett_simt_kernel(const __grid_constant__ GettKernelArgs g)
{
    __shared__ int64_t offAM[TM], offCM[TM], offBN[TN], offCN[TN], offAK[TK], offBK[TK];
    typedef typename Acc<DT>::type T; // fp32, or fp64 for GETT_F64 (round-to-nearest FMAs either way)
    __shared__ T As[TK][TM + 1], Bs[TK][TN + 1];

    const uint32_t tiles = g.tiles_m * g.tiles_n;
    const uint32_t z = blockIdx.x / tiles;
    const uint32_t tile = blockIdx.x - z * tiles;
    const uint32_t tn = tile / g.tiles_m, tm = tile - tn * g.tiles_m;
    const uint32_t m0 = tm * TM, n0 = tn * TN;
    const uint32_t Msz = g.M.size, Nsz = g.N.size, Ksz = g.K.size;
    const uint32_t kbeg = z * g.k_per_split;
    const uint32_t kend = min(Ksz, kbeg + g.k_per_split);
    const int tid = threadIdx.x;

    if (tid < TM) {
        int64_t x = 0, y = 0;
        if (m0 + tid < Msz)
            gett_decompose(g.M, m0 + tid, x, y);
        offAM[tid] = x;
        offCM[tid] = y;
    } else if (tid < TM + TN) {
        int c = tid - TM;
        int64_t x = 0, y = 0;
        if (n0 + c < Nsz)
            gett_decompose(g.N, n0 + c, x, y);
        offBN[c] = x;
        offCN[c] = y;
    }

    T acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            acc[i][j] = 0;
    const int tx = tid & 15, ty = tid >> 4;

    for (uint32_t k0 = kbeg; k0 < kend; k0 += TK) {
        __syncthreads(); // previous slab consumed; also orders the offset tables above
        if (tid < TK) {
            int64_t x = 0, y = 0;
            if (k0 + tid < kend)
                gett_decompose(g.K, k0 + tid, x, y);
            offAK[tid] = x;
            offBK[tid] = y;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < TM * TK / NT; ++i) {
            int e = tid + i * NT;
            int r, k;
            if (g.a_kmajor) {
                k = e % TK;
                r = e / TK;
            } else {
                r = e % TM;
                k = e / TM;
            }
            T v = 0;
            if (m0 + r < Msz && k0 + k < kend)
                v = load_elem<DT>(g.A, offAM[r] + offAK[k]);
            As[k][r] = v;
        }
#pragma unroll
        for (int i = 0; i < TN * TK / NT; ++i) {
            int e = tid + i * NT;
            int c, k;
            if (g.b_kmajor) {
                k = e % TK;
                c = e / TK;
            } else {
                c = e % TN;
                k = e / TN;
            }
            T v = 0;
            if (n0 + c < Nsz && k0 + k < kend)
                v = load_elem<DT>(g.B, offBN[c] + offBK[k]);
            Bs[k][c] = v;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            T a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                a[i] = As[k][tx + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                b[j] = Bs[k][ty + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    acc[i][j] = fma(a[i], b[j], acc[i][j]);
        }
    }
    __syncthreads(); // offset tables visible even when the K range was empty

#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = ty + 16 * j;
        if (n0 + c >= Nsz)
            continue;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = tx + 16 * i;
            if (m0 + r >= Msz)
                continue;
            if (g.split_k > 1) {
                g.ws[((size_t)z * Nsz + (n0 + c)) * Msz + (m0 + r)] = (float)acc[i][j]; // (never GETT_F64)
            } else {
                T* dst = reinterpret_cast<T*>(g.C) + offCM[r] + offCN[c];
                T v = (T)g.alpha * acc[i][j];
                if (g.beta != 0.f)
                    v = fma((T)g.beta, *dst, v);
                *dst = v;
            }
        }
    }
}

} // namespace

cudaError_t gett_launch_simt(const GettKernelArgs& args, int grid, cudaStream_t stream)
{
    switch (args.dtype) {
    case GETT_F32: gett_simt_kernel<GETT_F32><<<grid, NT, 0, stream>>>(args); break;
    case GETT_BF16_F32: gett_simt_kernel<GETT_BF16_F32><<<grid, NT, 0, stream>>>(args); break;
    case GETT_F64: gett_simt_kernel<GETT_F64><<<grid, NT, 0, stream>>>(args); break;
    default: gett_simt_kernel<GETT_F16_F32><<<grid, NT, 0, stream>>>(args); break;
    }
    return cudaGetLastError();
}
