// Measurement helper, not part of the contraction path: a register-only fp32 FMA loop whose
// rate the benchmark uses as the measured peak of the FMA pipe (the denominator of the
// strict-fp32 roofline fractions).  Built into a small library of its own.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int CHAINS = 32; // independent accumulators per thread

// PACKED = 0: one fmaf per chain and step.  PACKED = 1: the two-wide packed FMA the fp32
// kernels use (two independent round-to-nearest FMAs per instruction).
template <int PACKED>
__global__ void __launch_bounds__(1024, 1) ffma_peak_kernel(float* out, float a, float b, int iters)
{
    float acc[CHAINS];
#pragma unroll
    for (int i = 0; i < CHAINS; ++i)
        acc[i] = (float)threadIdx.x * 1e-6f + (float)i;
    for (int it = 0; it < iters; ++it) {
        if (PACKED) {
            const float2 a2 = make_float2(a, a), b2 = make_float2(b, b);
#pragma unroll
            for (int i = 0; i < CHAINS; i += 2) {
                float2 v = __ffma2_rn(make_float2(acc[i], acc[i + 1]), a2, b2);
                acc[i] = v.x;
                acc[i + 1] = v.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < CHAINS; ++i)
                acc[i] = fmaf(acc[i], a, b);
        }
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < CHAINS; ++i)
        s += acc[i];
    if (s == 12345.678f) // keeps the loop alive; practically never true
        out[0] = s;
}

// The same loop in double precision (the denominator for GETT_F64 rows).
__global__ void __launch_bounds__(1024, 1) dfma_peak_kernel(double* out, double a, double b, int iters)
{
    double acc[CHAINS / 2];
#pragma unroll
    for (int i = 0; i < CHAINS / 2; ++i)
        acc[i] = (double)threadIdx.x * 1e-6 + (double)i;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < CHAINS / 2; ++i)
            acc[i] = fma(acc[i], a, b);
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < CHAINS / 2; ++i)
        s += acc[i];
    if (s == 12345.678)
        out[0] = s;
}

} // namespace

// Launches the loop on `stream`; returns the FMA count (one FMA = 2 flop) or -1 on a launch
// failure.  out: device pointer to at least one float.  The caller times it with CUDA events.
extern "C" __attribute__((visibility("default"))) long long gett_bench_ffma_peak(int packed, int iters,
                                                                                 int blocks, float* out,
                                                                                 void* stream)
{
    if (iters < 1 || blocks < 1 || !out)
        return -1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (packed == 2) { // double precision; out must then hold at least one double
        dfma_peak_kernel<<<blocks, 1024, 0, s>>>(reinterpret_cast<double*>(out), 1.0000001, 1e-9, iters);
        if (cudaGetLastError() != cudaSuccess)
            return -1;
        return (long long)blocks * 1024 * (CHAINS / 2) * (long long)iters;
    }
    if (packed)
        ffma_peak_kernel<1><<<blocks, 1024, 0, s>>>(out, 1.0000001f, 1e-9f, iters);
    else
        ffma_peak_kernel<0><<<blocks, 1024, 0, s>>>(out, 1.0000001f, 1e-9f, iters);
    if (cudaGetLastError() != cudaSuccess)
        return -1;
    return (long long)blocks * 1024 * CHAINS * (long long)iters;
}
