// Single-pass FFT along the columns of a row-major matrix: one tile = W adjacent
// columns, so every row of the tile is one contiguous W*8-byte segment in memory.
#include <cuda.h>
#include "bulk_copy.cuh"
#include "configs.h"
#include "registry.h"

namespace b200fft {

// Column tile staged through the tensor memory accelerator on both ends: the tile arrives
// as 2-D boxes (256 rows x W columns) in a dense [row][column] image in shared memory,
// counted on an mbarrier; the first stage reads its registers from that image; after the
// last stage the results are written back as the dense image and leave as TMA stores. No
// warp-level load or store touches 16 different lines. Measured on B200 it runs exactly as
// fast as the plain-load kernel (94 us for 4096 x 4096): the strided 32-byte access pattern
// itself, not the way the SM issues it, sets the time (a copy-only kernel with the same
// pattern takes 72 us). It stays selectable with the plan option "tma".
__device__ int g_tma_timeouts = 0;   // counts mbarrier waits that ran out of polls (never expected)

template <class C, bool INV, class TIn, class TOut>
__global__ void __launch_bounds__(C::THREADS, C::MINB)
    fft_cols_bulk_kernel(const FftArgs a, const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out) {
    extern __shared__ __align__(128) float2 smem_tma[];   // TMA destinations are 128-byte aligned
    constexpr int W = C::W, N = C::N, S = C::S;
    static_assert(C::CL == 1 && C::G == 1 && W >= 2, "single-CTA column tiles");
    static_assert(TIn::ELEM_BYTES == 8 && TOut::ELEM_BYTES == 8, "complex64 tiles");
    __shared__ __align__(8) uint64_t bar;
    const int t = threadIdx.x;
    const int64_t tile = blockIdx.x;
    float2* sm = smem_tma;
    if (t == 0) mbar_init(&bar, 1);
    __syncthreads();
    if (t == 0) mbar_expect_tx(&bar, (unsigned)(N * W * 8));
    constexpr int BOX_ROWS = 256;
    if (t < N / BOX_ROWS) tma_load_2d(sm + t * BOX_ROWS * W, &tm_in, (int)(tile * W * 2), t * BOX_ROWS, &bar);
    if (!mbar_wait(&bar, 0)) atomicAdd(&g_tma_timeouts, 1);   // bounded wait: record and carry on
    Engine<C> e;
    e.setup(t);
    {
        using G = Geo<C, 1>;
        constexpr int V = G::V, r = G::r;
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            const int c = C::template cidx<V>(t, v, 0);
            const int q = c % W, lo = c / W;
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const float4 u = *reinterpret_cast<const float4*>(sm + (j * G::Ls + lo) * W + q);
                e.x[j * V + v] = make_float2(u.x, INV ? -u.y : u.y);
                e.x[j * V + v + 1] = make_float2(u.z, INV ? -u.w : u.w);
            });
        });
    }
    __syncthreads();                 // the dense image is consumed; the exchanges may overwrite it
    e.dif(sm, a.tw);
    __syncthreads();                 // the last exchange is consumed
    {
        using G = Geo<C, S>;
        constexpr int V = G::V, r = G::r, KS = N / r;
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            int b0, q;
            e.last_index(v, b0, q);
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const float2 p = e.x[j * V + v], w = e.x[j * V + v + 1];
                *reinterpret_cast<float4*>(sm + (j * KS + b0) * W + q) =
                    make_float4(p.x * a.scale, (INV ? -p.y : p.y) * a.scale, w.x * a.scale, (INV ? -w.y : w.y) * a.scale);
            });
        });
    }
    fence_async_smem();
    __syncthreads();
    if (t < N / BOX_ROWS) {
        tma_store_2d(&tm_out, (int)(tile * W * 2), t * BOX_ROWS, sm + t * BOX_ROWS * W);
        bulk_commit();
        bulk_wait_all();
    }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}
// rows x (ld complex64) matrix seen as fp32, boxes of box_rows rows x W complex
static bool make_column_map(CUtensorMap* m, const void* base, int64_t rows, int64_t ld, int w, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)ld * 2, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 8};
    const cuuint32_t box[2] = {(cuuint32_t)w * 2, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <class C, bool INV>
cudaError_t launch_cols_bulk(const FftArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(fft_cols_bulk_kernel<C, INV, StoreC64, StoreC64>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    CUtensorMap tin, tout;
    if (!make_column_map(&tin, a.in, C::N, a.dist, C::W, 256) || !make_column_map(&tout, a.out, C::N, a.dist, C::W, 256))
        return cudaErrorNotSupported;
    fft_cols_bulk_kernel<C, INV, StoreC64, StoreC64><<<(unsigned)a.tiles, C::THREADS, C::SMEM_BYTES, st>>>(a, tin, tout);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}
template <class C, bool INV>
constexpr KernelEntry make_bulk_entry() {
    return KernelEntry{C::N, C::W, C::G, 77, C::THREADS, C::SMEM_BYTES, C::TW_TOTAL, INV, 0, 0,
                       &launch_cols_bulk<C, INV>, &launch_build_tw<C>};
}
static const KernelEntry k_cols_bulk[] = {make_bulk_entry<T1024, false>(), make_bulk_entry<T1024, true>(),
                                         make_bulk_entry<T2048, false>(), make_bulk_entry<T2048, true>(),
                                         make_bulk_entry<T4096, false>(), make_bulk_entry<T4096, true>()};

int tma_timeouts() {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_tma_timeouts, sizeof(int));
    return v;
}

static const KernelEntry k_cols[] = {
    B200FFT_ENTRIES_STD(T64),   B200FFT_ENTRIES_STD(T128),
    B200FFT_ENTRIES_STD(T256),  B200FFT_ENTRIES_STD(T512),  B200FFT_ENTRIES_STD(T1024),
    B200FFT_ENTRIES_STD(T2048), B200FFT_ENTRIES_STD(T4096), B200FFT_ENTRIES_STD(T8192),
};

static int default_cluster(int n) { return 1; }

const KernelEntry* find_cols_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl) {
    if (cl == 77) {                                   // TMA-staged tiles (plan option "tma")
        for (const KernelEntry& e : k_cols_bulk)
            if (e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
        return nullptr;
    }
    const EntryList more = cols_entries_more();
    if (cl == 1023) {                                 // wider tiles on a cluster of two CTAs
        for (int i = 0; i < more.count; ++i) {
            const KernelEntry& e = more.first[i];
            if (e.cl == 2 && e.w * e.n == 32768 && e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype)
                return &e;
        }
        return nullptr;
    }
    if (cl == 1019) {                                 // wide tiles (their entries carry w > 4)
        for (int i = 0; i < more.count; ++i) {
            const KernelEntry& e = more.first[i];
            if (e.w > 4 && e.cl == 1 && e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
        }
        return nullptr;
    }
    if (cl == 0) cl = default_cluster(n);
    for (const KernelEntry& e : k_cols)
        if (e.n == n && e.cl == cl && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
    for (int i = 0; i < more.count; ++i) {
        const KernelEntry& e = more.first[i];
        if (e.w <= 4 && e.w * e.n != 32768 && e.n == n && e.cl == cl && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype)
            return &e;
    }
    return nullptr;
}

}  // namespace b200fft
