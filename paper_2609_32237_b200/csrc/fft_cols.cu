// Single-pass FFT along the columns of a row-major matrix: one tile = W adjacent
// columns, so every row of the tile is one contiguous W*8-byte segment in memory.
#include <cuda.h>
#include "bulk_copy.cuh"
#include "configs.h"
#include "registry.h"

namespace b200fft {

// Persistent streaming variant for the tiles that fill a multiprocessor (n = 4096 x 4 columns). With one
// CTA per SM the plain kernel's phases run one after the other: load (10.5 K of its 25 K cycles per tile:
// 4096 row segments of 32 bytes, sixteen cache lines per warp-level access), transform, store (another
// 8 K). Here each CTA loops over tiles and the tensor memory accelerator moves the rows instead of the
// load/store unit: while tile i is transformed, the boxes of tile i+1 (256 rows x W columns each) land in
// a staging buffer beside the exchange buffer, counted on an mbarrier; the first stage reads its registers
// from that dense image. The staging buffer holds the part of the tile that fits (12 of 16 boxes of
// complex64, all of an fp16 tile); the remaining rows are asked into L2 at the same time and read with
// plain loads. After the last stage the results go back to shared memory as a dense image (the exchange
// buffer is free by then) and leave as TMA stores, which the next tile's first stage overlaps; the stores
// must have read shared memory before the next exchange overwrites it (wait_group.read). Tensor maps cover
// this GPU's own memory and every copy is addressed to the issuing CTA alone. Measured on 4096 x 4096 complex64: 74 us against 92 us for the plain
// kernel. Variants that were built, tested and measured without gain, and dropped: two-column tiles at two CTAs
// per multiprocessor, i.e. boxes with 16-byte rows (144 us); two warp groups of two columns each that take
// turns on one 64 KiB exchange buffer, so that one group computes while the other exchanges, with the whole
// next tile staged (76 us, the same with the 32-byte swizzle against the bank conflicts of its half-row
// accesses, and 74 us on contiguous tiles moved as 64 KiB boxes: the access pattern in main memory is not what
// sets the time; a second form of it that spends the freed 64 KiB on half of the output image, so that the
// stores need not be read out before the next exchange, took 89 us: its plain-load quarter touches 32 cache
// lines per warp-level load). Every wait is bounded: a CTA whose wait runs out raises
// g_tma_timeouts once, stops taking tiles, waits (bounded again) for the copies it still has in flight
// and returns; the output of that call is then incomplete.
__device__ int g_tma_timeouts = 0;   // CTAs whose wait for a copy ran out of polls (never expected)

template <class C, class TIn, int CPS = 1>     // CPS: CTAs per multiprocessor the shared memory is divided among
struct Stream {
    static constexpr int BOX_ROWS = 256, NBOX = C::N / BOX_ROWS;
    static constexpr int X_BYTES = C::N * C::W * 8;                         // exchange buffer = output image
    static constexpr int BOX_BYTES = BOX_ROWS * C::W * TIn::ELEM_BYTES;
    static constexpr int ROOM = 232448 / CPS - 2048 - X_BYTES;
    static constexpr int SBOX = (ROOM / BOX_BYTES) < NBOX ? (ROOM / BOX_BYTES) : NBOX;   // boxes staged by TMA
    static constexpr int SMEM_BYTES = X_BYTES + SBOX * BOX_BYTES;
    static_assert(C::N % BOX_ROWS == 0 && SBOX >= 1, "whole boxes");
    static_assert(C::CL == 1 && C::G == 1 && C::W >= 2 && C::THREADS >= NBOX, "single-CTA column tiles");
};

template <class C, bool INV, class TIn, class TOut, int CPS>
__global__ void __launch_bounds__(C::THREADS, CPS)
    fft_cols_stream_kernel(const FftArgs a, const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out) {
    using L = Stream<C, TIn, CPS>;
    extern __shared__ __align__(128) float2 smem_stream[];   // TMA destinations and sources are 128-byte aligned
    constexpr int W = C::W, N = C::N, S = C::S;
    constexpr int XW_IN = W * TIn::ELEM_BYTES / 4, XW_OUT = W * TOut::ELEM_BYTES / 4;   // tile width in 4-byte map elements
    using G1 = Geo<C, 1>;
    using GS = Geo<C, S>;
    constexpr int V = G1::V, r = G1::r, rs = GS::r, KS = N / rs;
    static_assert(V == 2 && GS::V == 2 && (rs == 8 || rs == 16 || rs == 32), "one register pair per slot at both ends");
    // When the staging buffer cannot hold the whole tile, the rows left to plain loads are the first-stage
    // slots j = 3 mod 4: the composite butterfly consumes its inputs subset by subset (j = a + 4 b, a = 0..3),
    // so these are needed last and their latency hides behind the arithmetic on the other three subsets.
    constexpr bool ALL_STAGED = L::SBOX == L::NBOX;
    constexpr bool SPLIT4 = !ALL_STAGED && G1::Ls == L::BOX_ROWS && r == 16 && L::SBOX >= 12;
    static_assert(ALL_STAGED || SPLIT4, "a partly staged tile keeps three of every four first-stage slots");
    constexpr int STAGED_BOXES = ALL_STAGED ? L::NBOX : 12;
    // With fp16 storage the results leave in four batches (output rows k * KS + b0 with k = c mod 4, as soon as
    // the last stage has emitted them), so that the copy engine reads the image while the rest is still being
    // computed, and the first stage's arithmetic runs before the wait for the previous tile's stores (measured
    // 62 -> 60 us on 4096 x 4096; with complex64 the same order measured slower, 74 -> 77 us, and is not used).
    constexpr bool PROGRESSIVE = KS == L::BOX_ROWS && rs == 16 && TOut::ELEM_BYTES == 4;
    constexpr int STORE_THREADS = PROGRESSIVE ? 4 : L::NBOX;
    __shared__ __align__(8) uint64_t bar[2];                  // [0] counts the copies; [1] is never completed
    const int t = threadIdx.x;
    float2* X = smem_stream;
    char* Sb = reinterpret_cast<char*>(smem_stream) + L::X_BYTES;
    const int polls = a.wait_polls > 0 ? a.wait_polls : kDefaultWaitPolls;

    auto issue = [&](int64_t tile) {                          // thread 0: boxes of `tile` into the staging buffer
        mbar_expect_tx(&bar[0], (unsigned)(STAGED_BOXES * L::BOX_BYTES));
        if constexpr (ALL_STAGED) {
            for (int b = 0; b < L::NBOX; ++b)
                tma_load_2d(Sb + b * L::BOX_BYTES, &tm_in, (int)(tile * XW_IN), b * L::BOX_ROWS, &bar[0]);
        } else {
            for (int b = 0; b < L::NBOX; ++b) {
                if ((b & 3) != 3)
                    tma_load_2d(Sb + (b - (b >> 2)) * L::BOX_BYTES, &tm_in, (int)(tile * XW_IN), b * L::BOX_ROWS, &bar[0]);
                else
                    tma_prefetch_2d(&tm_in, (int)(tile * XW_IN), b * L::BOX_ROWS);
            }
        }
    };
    if (t == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
    }
    __syncthreads();
    int64_t tile = blockIdx.x;
    int in_flight = 0;                                        // thread 0: loads issued and not yet waited for
    if (t == 0 && tile < a.tiles) {
        issue(tile);
        in_flight = 1;
    }
    Engine<C> e;
    e.setup(t);
    unsigned phase = 0;
    bool gave_up = false;
    for (; tile < a.tiles; tile += gridDim.x) {
        const int64_t next = tile + gridDim.x;
        asm volatile("" : "+r"(e.t));                         // keep the thread index opaque per tile (register pressure)
        const int c = C::template cidx<V>(e.t, 0, 0);
        const int q = c % W, lo = c / W;
        const int64_t gbase = tile * W;
        auto fix = [&](int j) {
            if constexpr (INV) {
                e.x[j * V].y = -e.x[j * V].y;
                e.x[j * V + 1].y = -e.x[j * V + 1].y;
            }
        };
        // rows that did not fit the staging buffer: plain loads (L2 was asked for them a tile ago)
        static_for<0, r>([&](auto j_) {
            constexpr int j = decltype(j_)::value;
            if constexpr (!ALL_STAGED && (j & 3) == 3) {
                TIn::load2(a.in, gbase + (int64_t)(j * G1::Ls + lo) * a.dist + q, e.x[j * V], e.x[j * V + 1]);
                fix(j);
            }
        });
        if (!mbar_wait(a.starve_wait ? &bar[1] : &bar[0], a.starve_wait ? 0u : phase, polls)) gave_up = true;
        gave_up = __syncthreads_or(gave_up);                  // one decision per CTA
        if (gave_up) break;
        if (t == 0) in_flight = 0;
        static_for<0, r>([&](auto j_) {
            constexpr int j = decltype(j_)::value;
            if constexpr (ALL_STAGED) {
                TIn::load2(Sb, (j * G1::Ls + lo) * W + q, e.x[j * V], e.x[j * V + 1]);
                fix(j);
            } else if constexpr ((j & 3) != 3) {
                TIn::load2(Sb, ((j - (j >> 2)) * G1::Ls + lo) * W + q, e.x[j * V], e.x[j * V + 1]);
                fix(j);
            }
        });
        phase ^= 1;
        if constexpr (!PROGRESSIVE) {
            if (t < STORE_THREADS) bulk_wait_read_all();      // the previous tile's stores have read the output image
        }
        __syncthreads();                                      // staging buffer consumed (and the exchange buffer free)
        if (t == 0 && next < a.tiles) {
            issue(next);
            in_flight = 1;
        }
        if constexpr (PROGRESSIVE) {
            e.template compute<1, false>(a.tw);
            if (t < STORE_THREADS) bulk_wait_read_all();
            __syncthreads();                                  // exchange buffer free
            e.template smem_rw<1, true>(X);
            __syncthreads();
            e.template smem_rw<2, false>(X);
            static_for<2, S>([&](auto s_) {
                constexpr int s = decltype(s_)::value;
                if constexpr (Engine<C>::template fused_write_ok<s>()) {
                    e.template compute_and_write<s>(X, a.tw);
                } else {
                    e.template compute<s, false>(a.tw);
                    e.template smem_rw<s, true>(X);
                }
                __syncthreads();
                e.template smem_rw<s + 1, false>(X);
            });
        } else {
            e.template dif<false>(X, a.tw);
        }
        __syncthreads();                                      // the last exchange is consumed: X becomes the output image
        {
            int b0, qq;
            e.last_index(0, b0, qq);
            const bool scaled = a.scale != 1.0f;
            e.template compute<S, false>(nullptr, [&](auto, auto k_, float2 pa, float2 pb) {
                constexpr int k = decltype(k_)::value;
                if constexpr (INV) {
                    pa.y = -pa.y;
                    pb.y = -pb.y;
                }
                if (scaled) {
                    pa = make_float2(pa.x * a.scale, pa.y * a.scale);
                    pb = make_float2(pb.x * a.scale, pb.y * a.scale);
                }
                TOut::store2(X, (k * KS + b0) * W + qq, pa, pb);
                if constexpr (PROGRESSIVE && k >= 12) {       // outputs arrive as k = c, c + 4, c + 8, c + 12 for c = 0..3
                    fence_async_smem();
                    __syncthreads();
                    if (t < 4) {
                        const int box = (k - 12) + 4 * t;
                        tma_store_2d(&tm_out, (int)(tile * XW_OUT), box * L::BOX_ROWS,
                                     reinterpret_cast<const char*>(X) + box * (L::BOX_ROWS * W * TOut::ELEM_BYTES));
                        bulk_commit();
                    }
                }
            });
        }
        if constexpr (!PROGRESSIVE) {
            fence_async_smem();
            __syncthreads();
            if (t < L::NBOX) {
                tma_store_2d(&tm_out, (int)(tile * XW_OUT), t * L::BOX_ROWS,
                             reinterpret_cast<const char*>(X) + t * (L::BOX_ROWS * W * TOut::ELEM_BYTES));
                bulk_commit();
            }
        }
    }
    if (gave_up) {
        if (t == 0) {
            atomicAdd(&g_tma_timeouts, 1);
            // copies still in flight must land before the shared memory goes away
            if (in_flight) mbar_wait(&bar[0], phase, kDefaultWaitPolls);
        }
    }
    if (t < STORE_THREADS) bulk_wait_all();
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
bool make_column_map(CUtensorMap* m, const void* base, int64_t rows, int64_t ld, int w, int box_rows, int elem_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const int words = elem_bytes / 4;
    const cuuint64_t dims[2] = {(cuuint64_t)ld * words, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(w * words), (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <class C, bool INV, class TI, class TO, int CPS>
cudaError_t launch_cols_stream(const FftArgs& a, cudaStream_t st) {
    using L = Stream<C, TI, CPS>;
    static bool done[64] = {};
    static int sms[64] = {};
    cudaError_t e = ensure_smem(fft_cols_stream_kernel<C, INV, TI, TO, CPS>, L::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    // the copy engine wants 16-byte aligned bases and row pitches, and tile columns that start on 16 bytes
    if ((reinterpret_cast<uintptr_t>(a.in) & 15) || (reinterpret_cast<uintptr_t>(a.out) & 15) ||
        ((a.dist * TI::ELEM_BYTES) & 15) || ((a.dist * TO::ELEM_BYTES) & 15) || a.tpg != 0 || a.out_dist != 0)
        return cudaErrorMisalignedAddress;
    CUtensorMap tin, tout;
    if (!make_column_map(&tin, a.in, C::N, a.dist, C::W, L::BOX_ROWS, TI::ELEM_BYTES) ||
        !make_column_map(&tout, a.out, C::N, a.dist, C::W, L::BOX_ROWS, TO::ELEM_BYTES))
        return cudaErrorNotSupported;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!sms[dev]) cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
    const int64_t slots = (int64_t)sms[dev] * CPS;
    const unsigned grid = (unsigned)(a.tiles < slots ? a.tiles : slots);
    fft_cols_stream_kernel<C, INV, TI, TO, CPS><<<grid, C::THREADS, L::SMEM_BYTES, st>>>(a, tin, tout);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}
template <class C, bool INV, class TS, class TO = TS, int CPS = 1>
constexpr KernelEntry make_stream_entry() {
    return KernelEntry{C::N, C::W, C::G, 1, C::THREADS, Stream<C, TS, CPS>::SMEM_BYTES, C::TW_TOTAL,
                       VAR_STREAM, INV,
                       TS::ELEM_BYTES == 8 ? 0 : 1, TO::ELEM_BYTES == 8 ? 0 : 1,
                       &launch_cols_stream<C, INV, TS, TO, CPS>, &launch_build_tw<C>};
}
static const KernelEntry k_cols_stream[] = {
    make_stream_entry<T4096, false, StoreC64>(), make_stream_entry<T4096, true, StoreC64>(),
    make_stream_entry<T4096, false, StoreC32H>(), make_stream_entry<T4096, true, StoreC32H>(),
    make_stream_entry<T2048, false, StoreC64>(), make_stream_entry<T2048, true, StoreC64>(),
    make_stream_entry<T4096, true, StoreC32H, StoreC64>(),    // SAR with fp16 intermediates: the last pass writes the complex64 image
};

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

const KernelEntry* find_cols_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl, int variant) {
    auto match = [&](const KernelEntry& e) {
        return e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype && e.variant == variant;
    };
    if (variant == VAR_STREAM) {
        for (const KernelEntry& e : k_cols_stream)
            if (match(e)) return &e;
        return nullptr;
    }
    if (cl == 0) cl = 1;
    for (const KernelEntry& e : k_cols)
        if (match(e) && e.cl == cl) return &e;
    const EntryList more = cols_entries_more();
    for (int i = 0; i < more.count; ++i) {
        const KernelEntry& e = more.first[i];
        if (match(e) && (variant != VAR_PLAIN || e.cl == cl)) return &e;
    }
    return nullptr;
}

}  // namespace b200fft
