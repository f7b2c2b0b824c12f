// Launch entry points of the device kernels (internal).
#pragma once
#include <cuda_runtime.h>

#include "gett_plan.h"

// Scalar-gather kernel, any layout / dtype.  grid = tiles * split_k.
cudaError_t gett_launch_simt(const GettKernelArgs& args, int grid, cudaStream_t stream);

// Sum the split-K slices in `ws` and apply C <- alpha * sum + beta * C (Eq. 11).
cudaError_t gett_launch_splitk_reduce(const GettKernelArgs& args, int sm_count,
                                      cudaStream_t stream);

// Stream-K: add the pieces of the left-over tiles (workspace [tile][piece][tile_n][tile_m]) and apply
// C <- alpha * sum + beta * C.  grid: CTAs of the contraction kernel's launch.
cudaError_t gett_launch_streamk_fixup(const GettKernelArgs& args, int grid, cudaStream_t stream);

// Tensor-core kernel (16-bit inputs, tcgen05 + tensor memory), persistent grid.
cudaError_t gett_launch_umma(const GettKernelArgs& args, const GettTmaMaps& maps, int grid, int smem,
                             cudaStream_t stream);

// Strict-fp32 kernel: 16-byte gathers, register-blocked FFMA.  grid = tiles * split_k.
cudaError_t gett_launch_ffma(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream);

// fp32, small N and K: B resident in shared memory, persistent CTAs stream A.
cudaError_t gett_launch_ffma_skinny(const GettKernelArgs& args, int grid, int smem, cudaStream_t stream);
