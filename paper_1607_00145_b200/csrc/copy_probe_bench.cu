// Measurement helper, not part of the contraction path: how the memory system merges the 16-byte
// asynchronous copies of a warp.  One launch per access pattern; read the bytes that cross from L2
// to the SMs per launch with a profiler (l1tex__m_xbar2l1tex_read_bytes).  Built into the
// measurement library beside the FMA-rate loop.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ void copy16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// Lane l of a warp copies 16 bytes from base + off(l); every warp and iteration has a 1 KB region.
// pattern 0: 512 contiguous bytes, 128-byte aligned      1: the same shifted by 16 bytes
//         2: shifted by 32                               3: shifted by 64
//         4: neighbouring lanes swapped                  5: even pieces by lanes 0-15, odd by 16-31
//         6: shifted by 16, lanes rotated by one (lane pairs cover whole 32-byte sectors again)
//         7: four 128-byte runs 256 bytes apart          8: those runs shifted by 16
//         9: those runs shifted by 64                   10: every lane in a sector of its own
//        11: pattern 0 with the DESTINATIONS rotated by one lane: every aligned pair of lanes
//            reads the two halves of one sector but writes to two different 32-byte units
//            of shared memory
__global__ void copy_probe_kernel(const char* __restrict__ g, int pattern, int iters, size_t span)
{
    extern __shared__ __align__(1024) uint8_t sm[];
    const uint32_t s0 = (uint32_t)__cvta_generic_to_shared(sm);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t wid = (size_t)blockIdx.x * (blockDim.x >> 5) + warp;
    for (int it = 0; it < iters; ++it) {
        const size_t base = ((wid * iters + it) * 1024) % span;
        size_t off;
        switch (pattern) {
        case 1: off = 16 + lane * 16; break;
        case 2: off = 32 + lane * 16; break;
        case 3: off = 64 + lane * 16; break;
        case 4: off = (lane ^ 1) * 16; break;
        case 5: off = ((lane & 15) * 2 + (lane >> 4)) * 16; break;
        case 6: off = 16 + ((lane + 31) & 31) * 16; break;
        case 7: off = (lane >> 3) * 256 + (lane & 7) * 16; break;
        case 8: off = (lane >> 3) * 256 + 16 + (lane & 7) * 16; break;
        case 9: off = (lane >> 3) * 256 + 64 + (lane & 7) * 16; break;
        case 10: off = lane * 32; break;
        default: off = lane * 16; break;
        }
        const int dlane = pattern == 11 ? ((lane + 1) & 31) : lane;
        copy16(s0 + warp * 1024 + (it & 1) * 512 + dlane * 16, g + base + off);
        // two copies per thread in flight, each to a destination of its own: a copy whose
        // destination is overwritten by a later one while it is still in flight need not be
        // carried out, which would make the byte counts depend on timing
        if (it & 1)
            asm volatile("cp.async.wait_all;" ::: "memory");
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
}

} // namespace

// src: device buffer of span + 4096 bytes (span a multiple of 1024).  Returns the bytes the copies ask for.
extern "C" __attribute__((visibility("default"))) long long gett_bench_copy_probe(int pattern, int iters, int blocks,
                                                                                  const void* src, size_t span,
                                                                                  void* stream)
{
    if (pattern < 0 || pattern > 11 || iters < 1 || blocks < 1 || !src || span < 1024 || span % 1024)
        return -1;
    copy_probe_kernel<<<blocks, 256, 8 * 1024, static_cast<cudaStream_t>(stream)>>>(static_cast<const char*>(src),
                                                                                   pattern, iters, span);
    if (cudaGetLastError() != cudaSuccess)
        return -1;
    return (long long)blocks * 8 * iters * 512;
}
