// Single-pass batched FFT over contiguous rows: one tile = one transform.
#include "bulk_copy.cuh"
#include "configs.h"
#include "registry.h"

namespace b200fft {

// ------------------------------------------------------------------------------------------
// Persistent, staged variant for the largest tiles. A tile that fills the register file and
// most of shared memory leaves one CTA per SM, whose phases (load, arithmetic, exchange, store)
// run in lock step, so the memory system idles while the CTA computes. Here each CTA loops
// over tiles and the copy engine brings the NEXT tile into shared memory while this one is
// being transformed: the part of it that fits beside the exchange buffer right after the
// current tile has been read into registers, the rest into the head of the exchange buffer
// once the last exchange has been read. The loads then cost no load instructions and overlap
// all of the arithmetic; the stores leave from registers as before.
__device__ int g_rows_stage_timeouts = 0;

template <class C, class TIn, int CTAS_PER_SM>
struct Staged {
    static constexpr int EB = TIn::ELEM_BYTES;
    static constexpr int TILE_BYTES = C::N * EB;
    static constexpr int X_BYTES = C::N * 8;                        // exchange buffer (fp32 complex)
    static constexpr int SLICE = C::L(1) * EB;                      // one first-stage register index j
    static constexpr int BUDGET = 232448 / CTAS_PER_SM - 1024 - 64; // per-CTA dynamic shared memory
    static constexpr int ROOM0 = ((BUDGET - X_BYTES) / SLICE) * SLICE;
    // a tile that does not fit whole is staged by halves: filling shared memory to the brim (3/4 of an
    // fp32 tile) leaves the L1 cache 30 KiB for the twiddle rows and measured slower (478 against 455 us)
    static constexpr int ROOM = (ROOM0 >= TILE_BYTES) ? ROOM0 : TILE_BYTES / 2;
    static constexpr int S_BYTES = ROOM >= TILE_BYTES ? TILE_BYTES : ROOM;   // staged beside the exchange buffer
    static constexpr int Q_BYTES = TILE_BYTES - S_BYTES;                     // staged in its head
    static constexpr int SMEM_BYTES = X_BYTES + S_BYTES;
    static_assert(S_BYTES > 0 && Q_BYTES <= X_BYTES, "tile does not fit");
    static_assert(C::W == 1 && C::CL == 1 && C::G == 1, "one contiguous transform per CTA");
};

template <class C, bool INV, class TIn, class TOut, int CTAS_PER_SM>
__global__ void __launch_bounds__(C::THREADS, CTAS_PER_SM) fft_rows_staged_kernel(const FftArgs a) {
    using L = Staged<C, TIn, CTAS_PER_SM>;
    extern __shared__ __align__(128) float2 smem_staged[];
    __shared__ __align__(8) uint64_t bar[2];
    float2* X = smem_staged;
    char* Sb = reinterpret_cast<char*>(smem_staged) + L::X_BYTES;
    const int tid = threadIdx.x;
    const char* in = reinterpret_cast<const char*>(a.in);
    const int64_t tile_pitch = a.dist * L::EB;
    constexpr unsigned CHUNK = 16384;

    auto issue = [&](char* dst, const char* src, unsigned bytes, uint64_t* b) {
        mbar_expect_tx(b, bytes);
        for (unsigned off = 0; off < bytes; off += CHUNK)
            bulk_load_1d(dst + off, src + off, (bytes - off < CHUNK) ? bytes - off : CHUNK, b);
    };
    if (tid == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
    }
    __syncthreads();
    int64_t tile = blockIdx.x;
    if (tid == 0 && tile < a.tiles) {
        issue(Sb, in + tile * tile_pitch, L::S_BYTES, &bar[0]);
        if constexpr (L::Q_BYTES > 0) issue(reinterpret_cast<char*>(X), in + tile * tile_pitch + L::S_BYTES, L::Q_BYTES, &bar[1]);
    }
    Engine<C> e;
    e.setup(tid);
    unsigned phase = 0;
    bool gave_up = false;
    for (; tile < a.tiles; tile += gridDim.x) {
        const int64_t next = tile + gridDim.x;
        // keep the thread index opaque per tile: addresses hoisted out of the loop would stay live
        // through the whole network, which already uses every register
        asm volatile("" : "+r"(e.t));
        auto wait_for = [&](uint64_t* b) {   // bounded wait: record, carry on, never spin for ever
            if (!gave_up && !mbar_wait(b, phase)) {
                gave_up = true;
                if (tid == 0) atomicAdd(&g_rows_stage_timeouts, 1);
            }
        };
        wait_for(&bar[0]);
        {   // first-stage registers from the staged tile (natural order: position j * L1 + lo)
            using G = Geo<C, 1>;
            constexpr int V = G::V, r = G::r;
            auto src = [&](auto j_) -> const void* {
                constexpr int j = decltype(j_)::value;
                if constexpr (j * L::SLICE < L::S_BYTES) return Sb + j * L::SLICE;
                else return reinterpret_cast<const char*>(X) + (j * L::SLICE - L::S_BYTES);
            };
            if constexpr (V == 1) {
                static_for<0, r>([&](auto j_) {
                    constexpr int j = decltype(j_)::value;
                    if constexpr (L::Q_BYTES > 0 && j * L::SLICE == L::S_BYTES) wait_for(&bar[1]);
                    e.x[j] = TIn::load1(src(j_), e.t);
                    if constexpr (INV) e.x[j].y = -e.x[j].y;
                });
            } else {
                static_for<0, V / 2>([&](auto h_) {
                    constexpr int v = 2 * decltype(h_)::value;
                    const int lo = C::template cidx<V>(e.t, v, 0);
                    static_for<0, r>([&](auto j_) {
                        constexpr int j = decltype(j_)::value;
                        if constexpr (L::Q_BYTES > 0 && v == 0 && j * L::SLICE == L::S_BYTES) wait_for(&bar[1]);
                        TIn::load2(src(j_), lo, e.x[j * V + v], e.x[j * V + v + 1]);
                        if constexpr (INV) {
                            e.x[j * V + v].y = -e.x[j * V + v].y;
                            e.x[j * V + v + 1].y = -e.x[j * V + v + 1].y;
                        }
                    });
                });
            }
        }
        phase ^= 1;
        __syncthreads();                     // the staged tile is in registers
        if (tid == 0 && next < a.tiles) {
            issue(Sb, in + next * tile_pitch, L::S_BYTES, &bar[0]);
            // the rest of that tile can only land after the last exchange: have L2 fetch it now
            if constexpr (L::Q_BYTES > 0) prefetch_l2_bulk(in + next * tile_pitch + L::S_BYTES, L::Q_BYTES);
        }
        static_for<1, C::S + 1>([&](auto s_) {
            constexpr int s = decltype(s_)::value;
            if constexpr (s == C::S && L::Q_BYTES > 0) {
                fence_async_smem();
                __syncthreads();             // the last exchange is in registers: its buffer's head is free
                if (tid == 0 && next < a.tiles)
                    issue(reinterpret_cast<char*>(X), in + next * tile_pitch + L::S_BYTES, L::Q_BYTES, &bar[1]);
            }
            e.template compute<s, false>(a.tw);
            if constexpr (s < C::S) {
                e.template smem_rw<s, true>(X);
                __syncthreads();
                e.template smem_rw<s + 1, false>(X);
            }
        });
        e.template store_last<TOut, INV>(a.out, tile * a.dist, a.dist, a.scale);
    }
}

template <class C, bool INV, class TI, class TO, int CPS>
cudaError_t launch_staged(const FftArgs& a, cudaStream_t st) {
    using L = Staged<C, TI, CPS>;
    // the copy engine wants 16-byte aligned sources; the plan has checked that already
    if ((reinterpret_cast<uintptr_t>(a.in) & 15) || ((a.dist * L::EB) & 15)) return cudaErrorMisalignedAddress;
    static bool done[64] = {};
    static int sms[64] = {};
    cudaError_t e = ensure_smem(fft_rows_staged_kernel<C, INV, TI, TO, CPS>, L::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!sms[dev]) cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
    const int64_t slots = (int64_t)sms[dev] * CPS;
    const unsigned grid = (unsigned)(a.tiles < slots ? a.tiles : slots);
    fft_rows_staged_kernel<C, INV, TI, TO, CPS><<<grid, C::THREADS, L::SMEM_BYTES, st>>>(a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}
template <class C, bool INV, class TI, class TO, int CPS>
constexpr KernelEntry make_staged_entry() {
    return KernelEntry{C::N, C::W, C::G, 1, C::THREADS, Staged<C, TI, CPS>::SMEM_BYTES, C::TW_TOTAL, VAR_STAGED, INV,
                       TI::ELEM_BYTES == 8 ? 0 : 1, TO::ELEM_BYTES == 8 ? 0 : 1,
                       &launch_staged<C, INV, TI, TO, CPS>, &launch_build_tw<C>};
}
#define B200FFT_ENTRIES_STAGED(C, CPS)                                   \
    make_staged_entry<C, false, StoreC64, StoreC64, CPS>(),           \
    make_staged_entry<C, true, StoreC64, StoreC64, CPS>(),            \
    make_staged_entry<C, false, StoreC32H, StoreC32H, CPS>(),         \
    make_staged_entry<C, true, StoreC32H, StoreC32H, CPS>()

static const KernelEntry k_rows_staged[] = {B200FFT_ENTRIES_STAGED(R16384, 1)};

int rows_stage_timeouts() {
    int v = 0;
    cudaMemcpyFromSymbol(&v, g_rows_stage_timeouts, sizeof(int));
    return v;
}

// Small batches leave most SMs idle with one CTA per transform (the paper's "when not to
// use it"): there a transform is split over a cluster of CTAs through distributed shared
// memory. Measured on B200, device time per launch (replayed from a CUDA graph, data in L2):
// n = 16384, batch <= 32: 8.2 us with one CTA per transform, 6.8 with 2, 5.1-5.6 with 4; batch 64: 8.5 / 7.2 / 7.6;
// n = 8192, batch <= 32: 5.2 / 5.1 / 4.3-4.5; batch 64: 5.4 / 5.3 / 5.6. From a batch of 148 on one CTA wins.
static int default_cluster(int n, int64_t batch) {
    if (n == 32768) return 2;
    if (n == 16384 && batch <= 32) return 4;
    if (n == 16384 && batch <= 64) return 2;
    if (n == 8192 && batch <= 32) return 4;
    return 1;
}

const KernelEntry* find_rows_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl, int64_t batch, int variant) {
    auto match = [&](const KernelEntry& e) {
        return e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype && e.variant == variant;
    };
    if (variant == VAR_STAGED) {
        for (const KernelEntry& e : k_rows_staged)
            if (match(e)) return &e;
        return nullptr;
    }
    if (variant == VAR_PLAIN && cl == 0) cl = default_cluster(n, batch);
    const EntryList lists[4] = {rows_entries_small(), rows_entries_large(), rows_entries_cluster(), rows_entries_tiny()};
    for (const EntryList& l : lists)
        for (int i = 0; i < l.count; ++i) {
            const KernelEntry& e = l.first[i];
            if (match(e) && (variant != VAR_PLAIN || e.cl == cl)) return &e;
        }
    return nullptr;
}

}  // namespace b200fft
