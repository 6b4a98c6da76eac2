// Host-side table of compiled kernel variants.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <atomic>
#include <cstdint>
#include "fft_core.cuh"

namespace b200fft {

extern std::atomic<int64_t> g_launch_count;

// Which kernel family an entry belongs to. The default family is the plain kernel for its size and
// cluster width; the others are alternatives that a plan option or a default rule selects.
enum Variant : int {
    VAR_PLAIN = 0,
    VAR_TW_TABLE,        // rows, n = 4096: every first-stage twiddle row loaded from the table (test knob)
    VAR_FOUR_STAGE,      // rows, n = 16384 as 16 x 4 x 16 x 16 (test knob)
    VAR_STAGED,          // rows: persistent kernel, next transform staged by untiled bulk copies
    VAR_STREAM,          // columns: persistent kernel, tiles staged in and out by the tensor memory accelerator
    VAR_WIDE,            // columns: tiles wider than four columns on one CTA
    VAR_WIDE_CLUSTER,    // columns: tiles of 32768 / n columns shared by a cluster of two CTAs
    VAR_TINY,            // rows, n <= 32, contiguous batch: one thread per transform, chunk staged through shared memory
};

struct KernelEntry {
    int n, w, g, cl, threads, smem_bytes, tw_total;
    int variant;
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

// Launch `kernel` over `tiles` tiles of configuration C: G tiles per CTA, or a
// cluster of CL CTAs per tile.
template <class C, class K, class A>
cudaError_t launch_tiles(K kernel, const A& a, int64_t tiles, cudaStream_t st) {
    const int64_t grid = (C::CL > 1) ? tiles * C::CL : (tiles + C::G - 1) / C::G;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(C::THREADS, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C::CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (C::CL > 1) ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <class C, bool INV, class TI, class TO>
cudaError_t launch_fft(const FftArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(fft_kernel<C, INV, TI, TO>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    return launch_tiles<C>(fft_kernel<C, INV, TI, TO>, a, a.tiles, st);
}

template <class C>
cudaError_t launch_build_tw(float2* tw, cudaStream_t st) {
    build_twiddles_kernel<C><<<(C::TW_TOTAL + 255) / 256, 256, 0, st>>>(tw);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <class C, bool INV, class TI, class TO>
constexpr KernelEntry make_entry() {
    return KernelEntry{C::N, C::W, C::G, C::CL, C::THREADS, C::SMEM_BYTES, C::TW_TOTAL, VAR_PLAIN, INV,
                       TI::ELEM_BYTES == 8 ? 0 : 1, TO::ELEM_BYTES == 8 ? 0 : 1,
                       &launch_fft<C, INV, TI, TO>, &launch_build_tw<C>};
}

// four storage/direction variants of one configuration
#define B200FFT_ENTRIES_STD(C)                              \
    make_entry<C, false, StoreC64, StoreC64>(),             \
    make_entry<C, true, StoreC64, StoreC64>(),              \
    make_entry<C, false, StoreC32H, StoreC32H>(),           \
    make_entry<C, true, StoreC32H, StoreC32H>()

// block-floating-point row transforms (fp16 storage, one exponent per transform)
struct BfpEntry {
    int n;
    bool inverse;
    int tw_total;
    cudaError_t (*launch)(const FftArgs&, const int* in_exp, int* out_exp, cudaStream_t);
    cudaError_t (*build_tw)(float2*, cudaStream_t);
};
const BfpEntry* find_bfp_kernel(int n, bool inverse);

// The kernel tables are spread over several translation units so that they compile in parallel.
struct EntryList {
    const KernelEntry* first;
    int count;
};
EntryList rows_entries_small();     // N = 8 .. 2048
EntryList rows_entries_tiny();      // N = 8 .. 32, contiguous batches
EntryList rows_entries_large();     // N = 4096 .. 16384 and the alternative factorisations
EntryList rows_entries_cluster();   // transforms shared by a cluster of CTAs
EntryList cols_entries_more();      // column tiles on clusters, wide column tiles
// a rows x ld matrix of elem_bytes-sized complex elements as a 2-D tensor map of 4-byte words, boxes of
// box_rows rows x w elements (cuTensorMapEncodeTiled through the runtime's driver entry point)
bool make_column_map(CUtensorMap* m, const void* base, int64_t rows, int64_t ld, int w, int box_rows, int elem_bytes);

// cl: CTAs per tile (cluster size); 0 picks the default for that size and batch (plain kernels only)
const KernelEntry* find_rows_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl = 0,
                                    int64_t batch = (int64_t)1 << 40, int variant = VAR_PLAIN);
const KernelEntry* find_cols_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl = 0, int variant = VAR_PLAIN);
// column tiles of the SAR chain on the slab layout: w = 2 or 4 columns, any pair of storage types
const KernelEntry* find_sar_cols_kernel(int n, int w, bool inverse, int in_dtype, int out_dtype);
// out[c * ld_out + r] = in[r * ld_in + c]; elem_bytes 8 (complex64) or 4 (complex half)
cudaError_t transpose_launch(const void* in, void* out, int rows, int cols, int64_t ld_in, int64_t ld_out, int elem_bytes,
                             cudaStream_t st);
int tma_timeouts();   // CTAs of the streaming column kernel whose wait for a copy ran out of polls since load
int rows_stage_timeouts();   // the same for the staged persistent row kernels

}  // namespace b200fft
