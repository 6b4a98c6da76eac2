// Row transforms of 8, 16 and 32 points on contiguous batches (dist == n): one thread per transform, the
// CTA's 128 transforms staged through shared memory so that every global access is one contiguous run.
//
// With one thread per transform a direct load has each lane read 16 bytes at a pitch of one transform (64 to
// 256 bytes): every request touches 32 lines and uses an eighth to a half of each sector it pulls in. Here
// the CTA copies its chunk (128 transforms, 4 to 32 KiB) with lane i reading the i-th 16-byte piece, parks
// the pieces in shared memory, and each thread then picks up its own transform from there; results go back
// the same way. Pieces are placed at (piece index) XOR (a few bits of the transform index), which makes both
// the contiguous copy and the one-transform-per-lane access free of bank conflicts.
#include "configs.h"
#include "registry.h"

namespace b200fft {

template <int N, bool INV, class TS>
__global__ void __launch_bounds__(128) fft_rows_tiny_kernel(const FftArgs a) {
    constexpr int EB = TS::ELEM_BYTES;
    constexpr int CH = N * EB / 16;            // 16-byte pieces per transform: 2 .. 16
    constexpr int PER = 16 / EB;               // complex values per piece
    constexpr int TPB = 128;
    static_assert(CH >= 2 && CH <= 16, "transform of 32 to 256 bytes");
    __shared__ uint4 sm[TPB * CH];
    const int t = threadIdx.x;
    const int64_t first = (int64_t)blockIdx.x * TPB;
    const int64_t left = a.tiles - first;
    const int count = left < TPB ? (int)left : TPB;
    const int total = count * CH;
    const uint4* in = reinterpret_cast<const uint4*>(a.in) + first * CH;
    uint4* out = reinterpret_cast<uint4*>(a.out) + first * CH;
    // piece c of transform tt; eight consecutive lanes hit eight different 16-byte bank groups both when
    // they walk along one transform and when they hold one transform each
    auto place = [](int tt, int c) {
        const int s = (CH >= 8) ? (tt & 7) : ((tt / (8 / CH)) % CH);
        return tt * CH + (c ^ s);
    };
#pragma unroll
    for (int k = 0; k < CH; ++k) {
        const int i = k * TPB + t;
        if (i < total) sm[place(i / CH, i % CH)] = in[i];
    }
    __syncthreads();
    if (t < count) {
        float2 v[N];
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const uint4 q = sm[place(t, c)];
            if constexpr (EB == 8) {
                v[2 * c] = make_float2(__uint_as_float(q.x), __uint_as_float(q.y));
                v[2 * c + 1] = make_float2(__uint_as_float(q.z), __uint_as_float(q.w));
            } else {
                const unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) v[4 * c + i] = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            }
        }
        if constexpr (INV) {
#pragma unroll
            for (int i = 0; i < N; ++i) v[i].y = -v[i].y;
        }
        Dft<N>::run(v);
        if constexpr (INV) {
#pragma unroll
            for (int i = 0; i < N; ++i) v[i] = make_float2(v[i].x * a.scale, -v[i].y * a.scale);
        }
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            uint4 q;
            if constexpr (EB == 8) {
                q = make_uint4(__float_as_uint(v[2 * c].x), __float_as_uint(v[2 * c].y), __float_as_uint(v[2 * c + 1].x),
                               __float_as_uint(v[2 * c + 1].y));
            } else {
                unsigned w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const __half2 h = __float22half2_rn(v[PER * c + i]);
                    w[i] = *reinterpret_cast<const unsigned*>(&h);
                }
                q = make_uint4(w[0], w[1], w[2], w[3]);
            }
            sm[place(t, c)] = q;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < CH; ++k) {
        const int i = k * TPB + t;
        if (i < total) out[i] = sm[place(i / CH, i % CH)];
    }
}

template <int N, bool INV, class TS>
static cudaError_t launch_tiny(const FftArgs& a, cudaStream_t st) {
    const int64_t grid = (a.tiles + 127) / 128;
    fft_rows_tiny_kernel<N, INV, TS><<<(unsigned)grid, 128, 0, st>>>(a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

static cudaError_t no_table(float2*, cudaStream_t) { return cudaSuccess; }

template <int N, bool INV, class TS>
constexpr KernelEntry make_tiny_entry() {
    return KernelEntry{N, 1, 128, 1, 128, 128 * N * TS::ELEM_BYTES, 1, VAR_TINY, INV,
                       TS::ELEM_BYTES == 8 ? 0 : 1, TS::ELEM_BYTES == 8 ? 0 : 1, &launch_tiny<N, INV, TS>, &no_table};
}
#define B200FFT_TINY(N)                                                                  \
    make_tiny_entry<N, false, StoreC64>(), make_tiny_entry<N, true, StoreC64>(),          \
    make_tiny_entry<N, false, StoreC32H>(), make_tiny_entry<N, true, StoreC32H>()

static const KernelEntry k_rows_tiny[] = {B200FFT_TINY(8), B200FFT_TINY(16), B200FFT_TINY(32)};

EntryList rows_entries_tiny() { return EntryList{k_rows_tiny, (int)(sizeof(k_rows_tiny) / sizeof(k_rows_tiny[0]))}; }

}  // namespace b200fft
