// Host-side table of compiled kernel variants.
#pragma once
#include <cuda_runtime.h>
#include <atomic>
#include <cstdint>
#include "fft_core.cuh"

namespace b200fft {

extern std::atomic<int64_t> g_launch_count;

struct KernelEntry {
    int n, w, g, threads, smem_bytes, tw_total;
    bool inverse;
    int in_dtype, out_dtype;                 // 0 = c64, 1 = c32h
    cudaError_t (*launch)(const FftArgs&, cudaStream_t);
    cudaError_t (*build_tw)(float2*, cudaStream_t);
};

// Raise the dynamic shared-memory limit of a kernel once per device.
template <class K>
inline cudaError_t ensure_smem(K kernel, int bytes, bool* done_per_device) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!done_per_device[dev]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
        done_per_device[dev] = true;
    }
    return cudaSuccess;
}

template <class C, bool INV, class TI, class TO>
cudaError_t launch_fft(const FftArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(fft_kernel<C, INV, TI, TO>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    const int64_t grid = (a.tiles + C::G - 1) / C::G;
    fft_kernel<C, INV, TI, TO><<<(unsigned)grid, C::THREADS, C::SMEM_BYTES, st>>>(a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <class C>
cudaError_t launch_build_tw(float2* tw, cudaStream_t st) {
    build_twiddles_kernel<C><<<(C::TW_TOTAL + 255) / 256, 256, 0, st>>>(tw);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <class C, bool INV, class TI, class TO>
constexpr KernelEntry make_entry() {
    return KernelEntry{C::N, C::W, C::G, C::THREADS, C::SMEM_BYTES, C::TW_TOTAL, INV,
                       TI::ELEM_BYTES == 8 ? 0 : 1, TO::ELEM_BYTES == 8 ? 0 : 1,
                       &launch_fft<C, INV, TI, TO>, &launch_build_tw<C>};
}

// four storage/direction variants of one configuration
#define B200FFT_ENTRIES_STD(C)                              \
    make_entry<C, false, StoreC64, StoreC64>(),             \
    make_entry<C, true, StoreC64, StoreC64>(),              \
    make_entry<C, false, StoreC32H, StoreC32H>(),           \
    make_entry<C, true, StoreC32H, StoreC32H>()

const KernelEntry* find_rows_kernel(int n, bool inverse, int in_dtype, int out_dtype);
const KernelEntry* find_cols_kernel(int n, bool inverse, int in_dtype, int out_dtype);

}  // namespace b200fft
