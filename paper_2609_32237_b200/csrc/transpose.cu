// Out-of-place matrix transpose through shared memory, for the "transpose, then transform the
// rows" form of a column FFT (the four-pass pipeline of the paper's Section "End to End", which
// its direct column kernel replaces). Kept as a measured comparison against the direct kernel.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "registry.h"

namespace b200fft {

// out[c * ld_out + r] = in[r * ld_in + c], 0 <= r < rows, 0 <= c < cols. One CTA moves a 32 x 32
// tile: rows of the tile are read and written as contiguous runs (256 bytes for 8-byte elements),
// and the odd pitch keeps the transposed shared-memory reads free of bank conflicts.
template <class T>
__global__ void __launch_bounds__(256) transpose_kernel(const T* __restrict__ in, T* __restrict__ out, int rows, int cols,
                                                        int64_t ld_in, int64_t ld_out) {
    __shared__ T tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty + 8 * i, c = c0 + tx;
        if (r < rows && c < cols) tile[ty + 8 * i][tx] = in[(int64_t)r * ld_in + c];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i, r = r0 + tx;
        if (r < rows && c < cols) out[(int64_t)c * ld_out + r] = tile[tx][ty + 8 * i];
    }
}

cudaError_t transpose_launch(const void* in, void* out, int rows, int cols, int64_t ld_in, int64_t ld_out, int elem_bytes,
                             cudaStream_t st) {
    const dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32));
    if (elem_bytes == 8)
        transpose_kernel<float2><<<grid, 256, 0, st>>>(reinterpret_cast<const float2*>(in), reinterpret_cast<float2*>(out),
                                                       rows, cols, ld_in, ld_out);
    else
        transpose_kernel<__half2><<<grid, 256, 0, st>>>(reinterpret_cast<const __half2*>(in),
                                                        reinterpret_cast<__half2*>(out), rows, cols, ld_in, ld_out);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace b200fft
