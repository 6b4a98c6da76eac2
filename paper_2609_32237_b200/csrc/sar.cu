// Range-Doppler SAR image formation in three passes over memory (paper, Section
// "End to End: Range-Doppler SAR"):
//   step 0  fused range compression per pulse: FFT, multiply by the conjugate
//           chirp spectrum (1/n_range folded in), inverse FFT; the forward
//           transform leaves digit-reversed positions and the inverse runs the
//           network backwards from them, so nothing is reordered in between
//   step 1  azimuth FFT along every range bin, read as columns in place,
//           output scaled by 1/n_azimuth (the paper's fixed-shift schedule)
//   step 2  fused range cell migration correction (8-tap sinc), azimuth filter
//           exp(+j 4 pi R0 (D - 1) / lambda) and inverse azimuth FFT on column tiles
// Between the steps the image lives in the caller's workspace, row-major by default (the azimuth transforms
// read it as column tiles in place; step 2 runs as a row pass, RCMC + filter, followed by the inverse column
// transform). Two other organisations are selectable (option "layout"): the slab layout of fft_core.cuh with
// 32-byte granules, and azimuth transforms by transposition (the paper's four-pass form).
// The azimuth steps also run on a strip of range bins cut from a larger image (sar_rda_shard_*): the strip is
// then a frame of its own whose first range bin sits `first_bin` bins into the whole swath.
// The filter and the migration are affine in the range index with per-Doppler-bin
// coefficients, built once in float64. The paper's four numerical fixes are kept:
// baseband filter (D - 1); phase in cycles with a split that makes the fp32
// product exact; a continuous interpolator (evaluated directly, no table);
// the fractional shift taken from the migration alone.
#include <cuda_runtime.h>
#include <cstring>
#include <new>
#include "../../include/b200fft.h"
#include "configs.h"
#include "registry.h"

namespace b200fft {

constexpr double kLight = 299792458.0;

struct SarTables {
    const float2* H;     // conj chirp spectrum / n_range, natural order, n_range entries
    const float4* mig;   // per Doppler bin: (g_hi, g_lo, a_frac, a_int as bits)
    const float4* phs;   // per Doppler bin: (A mod 1, B_hi, B_lo, 0)  [cycles]
    const float2* stp;   // per Doppler bin: exp(j 2 pi B), the filter's step from one range bin to the next
};

struct SarArgs {
    const void* in;
    void* out;
    const float2* tw;
    SarTables tab;
    int64_t tiles;
    int64_t ld;          // row pitch in elements (n_range)
    int nr;
    float scale;
    int na;              // rows of the image (n_azimuth)
    // Row pass of step 2: output column j (0 .. out_cols - 1) is range bin j + col0 of the input frame and is
    // stored at a row pitch of out_ld elements. Whole image: col0 = 0, out_cols = nr, out_ld = ld.
    int col0, out_cols;
    int64_t out_ld;
    // Range compression that scatters its rows over the strips of a column-strip decomposition: strip g covers
    // range bins [g * strip_cols - halo_l, (g + 1) * strip_cols + halo_r) of the whole frame, stored as
    // n_azimuth rows of sw = halo_l + strip_cols + halo_r elements at strip[g] (an address this device can
    // store to: its own memory or a peer's). Bins outside the frame are written as zeros.
    struct {
        unsigned long long strip[8];
        int world, strip_cols, strip_shift, halo_l, halo_r, sw;   // strip_cols = 1 << strip_shift
        int64_t row0;    // first pulse of this launch within the whole frame
    } sh;
};

// ---------------------------------------------------------------- step 0
// MODE 0: row-major output; 1: the slab layout (granules of 32 bytes); 2: scattered over the strips of a
// column-strip decomposition (SarArgs::sh), every pair stored to the strip that owns it and to the neighbour
// whose halo it falls into.
template <class C, class TOut, int MODE>
__global__ void __launch_bounds__(C::THREADS, C::MINB) sar_range_compress_kernel(const SarArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    static_assert(C::W == 1, "range compression works on contiguous rows");
    static_assert(C::P / C::radix(1) >= 2 && C::P / C::radix(C::S) >= 2,
                  "the filter multiply and the final store work on register pairs: two butterflies per thread at both ends");
    const int g = threadIdx.x / C::T, t = threadIdx.x % C::T;
    int64_t tile = (C::CL > 1) ? (int64_t)(blockIdx.x / C::CL) : (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    const int64_t base = tile * a.ld;
    Engine<C> e;
    e.setup(t);
    e.template load_first<StoreC64, false>(a.in, base, a.ld);
    e.dif(sm, a.tw);
    {
        // registers hold X[b0 + KS j]; multiply by H at the same index, conjugate for the inverse
        using G = Geo<C, C::S>;
        constexpr int V = G::V, r = G::r, KS = C::N / r;
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            int b0, qq;
            e.last_index(v, b0, qq);
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const float4 h = __ldg(reinterpret_cast<const float4*>(a.tab.H + j * KS + b0));
                float2 p = cmul(e.x[j * V + v], make_float2(h.x, h.y));
                float2 q = cmul(e.x[j * V + v + 1], make_float2(h.z, h.w));
                e.x[j * V + v] = make_float2(p.x, -p.y);
                e.x[j * V + v + 1] = make_float2(q.x, -q.y);
            });
        });
    }
    e.template dit<false>(sm, a.tw);
    if (!active) return;
    if constexpr (MODE == 1) {
        constexpr int GS = 32 / TOut::ELEM_BYTES;
        const int64_t na = a.na;
        e.template first_stage_dit_and_store_at<TOut, true>(a.tw, a.out, 1.0f, [&](int p, int) -> int64_t {
            return ((int64_t)(p / GS) * na + tile) * GS + (p % GS);
        });
    } else if constexpr (MODE == 2) {
        const int sc = a.sh.strip_cols, hl = a.sh.halo_l, hr = a.sh.halo_r, last = a.sh.world - 1;
        const int64_t rowoff = (a.sh.row0 + tile) * (int64_t)a.sh.sw;      // this pulse's row in every strip
        auto strip = [&](int g) { return reinterpret_cast<void*>(a.sh.strip[g]); };
        e.template first_stage_dit_emit<true>(a.tw, 1.0f, [&](int p, int, float2 pa, float2 pb) {
            const int g = p >> a.sh.strip_shift, lc = p & (sc - 1);     // sc, hl, hr are even: a pair stays together
            TOut::store2(strip(g), rowoff + hl + lc, pa, pb);
            if (lc < hr && g > 0) TOut::store2(strip(g - 1), rowoff + hl + sc + lc, pa, pb);
            if (lc >= sc - hl && g < last) TOut::store2(strip(g + 1), rowoff + lc - (sc - hl), pa, pb);
        });
        const float2 z = make_float2(0.f, 0.f);
        for (int i = 2 * t; i < hl; i += 2 * C::T) TOut::store2(strip(0), rowoff + i, z, z);
        for (int i = 2 * t; i < hr; i += 2 * C::T) TOut::store2(strip(last), rowoff + hl + sc + i, z, z);
    } else {
        e.template first_stage_dit_and_store<TOut, true>(a.tw, a.out, base, a.ld, 1.0f);
    }
}

// ---------------------------------------------------------------- step 2
// Migration of (Doppler bin, range bin n): integer part and fraction, from the
// per-bin slope split so that n * g_hi is exact in fp32.
__device__ __forceinline__ void migration(const float4 m, int n, int& i0, float& mu) {
    const float fn = (float)n;
    const float t = fn * m.x;                       // exact: g_hi has 10 significant bits, n < 2^14
    const float ti = floorf(t);
    const float f = (t - ti) + fmaf(fn, m.y, m.z);  // fractions only: small numbers, small error
    const float fi = floorf(f);
    i0 = __float_as_int(m.w) + (int)ti + (int)fi;
    mu = f - fi;
}

// exp(+j 2 pi (A + n B)) with n * B_hi exact and reduced before the sum
__device__ __forceinline__ float2 filter_phase(const float4 p, int n) {
    const float fn = (float)n;
    const float t = fn * p.y;
    const float f = (t - floorf(t)) + fmaf(fn, p.z, p.x);
    // fraction of a cycle in [-0.5, 0.5): the hardware sine/cosine are accurate to about
    // 4e-7 absolute on [-pi, pi], well inside the error budget of the fp32 chain
    float fr = f - floorf(f);
    fr = (fr >= 0.5f) ? fr - 1.0f : fr;
    float s, c;
    __sincosf(6.283185307179586f * fr, &s, &c);
    return make_float2(c, s);
}

// 16-byte asynchronous copy global -> shared, bypassing L1; `valid` false writes zeros
// (samples outside the row read as zero).
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src, bool valid) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int src = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "r"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// weights of the 8-tap sinc interpolator, taps j = -3..4, unit sum:
// sinc(mu - j) = (-1)^j sin(pi mu) / (pi (mu - j)); after normalisation the common factor
// drops out: w_j = [(-1)^j / (mu - j)] / sum_j' [(-1)^j' / (mu - j')]. This returns the
// magnitudes m_i = |1 / (mu - j)| * inv with the sign (-1)^j left to the caller (tap i = j + 3
// is negative for even i). mu = 0 is nudged to 1e-30, which gives w_0 = 1 and the others
// 1e-30: the exact limit to fp32 precision.
__device__ __forceinline__ void sinc8_weights_rcp(float mu, float (&w)[8]) {
    mu = fmaxf(mu, 1e-30f);
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w[i] = rcp_approx(mu - (float)(i - 3));     // sign (-1)^(i-3) applied below and by the caller
        s = ((i - 3) & 1) ? s - w[i] : s + w[i];
    }
    float inv = rcp_approx(s);
    inv = inv * (2.0f - s * inv);                    // one Newton step: full fp32 accuracy
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] *= inv;
}

// The staged row windows share the transform tile's shared memory, which is idle until
// the first exchange: 4 buffers of ROWS rows, 16 elements of the intermediate type each
// at a pitch of 16 + 16 bytes' worth (an odd number of 16-byte granules, so rows read
// in parallel start in different banks).
template <class C, class TIn>
__host__ __device__ constexpr int rcmc_pitch() { return 16 + 16 / TIn::ELEM_BYTES; }
template <class C, class TIn>
__host__ __device__ constexpr int rcmc_stage_bytes() { return 4 * (C::N / 16) * rcmc_pitch<C, TIn>() * TIn::ELEM_BYTES; }
template <class C, class TIn>
__host__ __device__ constexpr int rcmc_smem_bytes() {
    constexpr int st = rcmc_stage_bytes<C, TIn>();
    return (st > C::SMEM_BYTES ? st : C::SMEM_BYTES) + C::N * 4;   // + one window start per row
}

template <class C, class TIn, bool SLAB>
__global__ void __launch_bounds__(C::THREADS, 1) sar_rcmc_filter_ifft_kernel(const SarArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    constexpr int W = C::W;
    static_assert(W == 4 && C::CL == 1 && C::G == 1 && C::radix(1) == 16, "column tiles of four range bins");
    using G1 = Geo<C, 1>;
    constexpr int V = G1::V, r = G1::r, ROWS = G1::Ls;          // ROWS Doppler bins per chunk, r chunks
    static_assert(V == 2, "two adjacent range bins per thread");
    constexpr int EB = TIn::ELEM_BYTES;
    constexpr int WIN = 16;                                     // staged samples per row
    constexpr int GRAN = 16 / EB;                               // samples per 16-byte copy
    constexpr int NG = WIN / GRAN;                              // copies per row
    constexpr int COPIES = ROWS * NG / C::THREADS;              // copies per thread per chunk
    static_assert(ROWS * NG % C::THREADS == 0 && COPIES >= 1, "staging copies divide among threads");
    constexpr int PITCH = rcmc_pitch<C, TIn>();
    constexpr int REGION = (rcmc_stage_bytes<C, TIn>() > C::SMEM_BYTES ? rcmc_stage_bytes<C, TIn>() : C::SMEM_BYTES);
    using elem_t = typename std::conditional<EB == 8, float2, __half2>::type;

    const int t = threadIdx.x;
    const int64_t tile = blockIdx.x;
    float2* sm = smem_dyn;
    elem_t* stg = reinterpret_cast<elem_t*>(smem_dyn);
    int* wstart = reinterpret_cast<int*>(reinterpret_cast<char*>(smem_dyn) + REGION);
    const int n0 = (int)(tile * W);                              // first range bin of the tile
    const elem_t* in = reinterpret_cast<const elem_t*>(a.in);

    // window start of every Doppler bin of this tile: n0 + floor(migration at n0) - 3,
    // rounded down to a 16-byte boundary
    for (int k = t; k < C::N; k += C::THREADS) {
        int i0;
        float mu;
        migration(__ldg(a.tab.mig + k), n0, i0, mu);
        wstart[k] = (n0 + i0 - 3) & ~(GRAN - 1);
    }
    __syncthreads();

    auto stg_index = [&](int buf, int row, int smp) { return (buf * ROWS + row) * PITCH + smp; };
    auto stage_chunk = [&](int j) {
#pragma unroll
        for (int i = 0; i < COPIES; ++i) {
            const int idx = i * C::THREADS + t;
            const int row = idx / NG, gr = idx % NG;
            const int k = j * ROWS + row;
            const int col = wstart[k] + gr * GRAN;
            const bool valid = col >= 0 && col + GRAN <= a.nr;
            const int cc = valid ? col : 0;                  // a 16-byte piece never straddles a 32-byte granule
            const int64_t src = SLAB ? slab_index(k, cc, a.na, 32 / EB) : (int64_t)k * a.ld + cc;
            cp_async_16(stg + stg_index(j & 3, row, gr * GRAN), in + src, valid);
        }
    };

    Engine<C> e;
    e.setup(t);
    const int c0 = C::template cidx<V>(t, 0, 0);
    const int q = c0 % W, lo = c0 / W;                           // range bins n0+q, n0+q+1; row lo of each chunk

    auto interp_chunk = [&](auto j_) {
        constexpr int j = decltype(j_)::value;
        const int k = j * ROWS + lo;                             // Doppler bin
        const float4 mg = __ldg(a.tab.mig + k);
        const float4 ph = __ldg(a.tab.phs + k);
        int ia, ib;
        float mua, mub;
        migration(mg, n0 + q, ia, mua);
        // one range bin on: the migration grows by the slope g = g_hi + g_lo
        mub = mua + (mg.x + mg.y);
        ib = ia;
        if (mub >= 1.0f) {
            mub -= 1.0f;
            ib += 1;
        }
        float wa[8], wb[8];
        sinc8_weights_rcp(mua, wa);
        sinc8_weights_rcp(mub, wb);
        const int ws = wstart[k];
        // first tap (j = -3) of each bin, relative to the staged window
        const int oa = min(max(n0 + q + ia - 3 - ws, 0), WIN - 8);
        const int ob = min(max(n0 + q + 1 + ib - 3 - ws, 0), WIN - 8);
        float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
        const elem_t* pa = stg + stg_index(j & 3, lo, oa);
        const elem_t* pb = stg + stg_index(j & 3, lo, ob);
#pragma unroll
        for (int tap = 0; tap < 8; ++tap) {
            float2 u, w2;
            if constexpr (EB == 8) {
                u = pa[tap];
                w2 = pb[tap];
            } else {
                u = __half22float2(pa[tap]);
                w2 = __half22float2(pb[tap]);
            }
            if ((tap - 3) & 1) {                                  // odd tap: weight is -|w|
                sa.x = fmaf(-wa[tap], u.x, sa.x);
                sa.y = fmaf(-wa[tap], u.y, sa.y);
                sb.x = fmaf(-wb[tap], w2.x, sb.x);
                sb.y = fmaf(-wb[tap], w2.y, sb.y);
            } else {
                sa.x = fmaf(wa[tap], u.x, sa.x);
                sa.y = fmaf(wa[tap], u.y, sa.y);
                sb.x = fmaf(wb[tap], w2.x, sb.x);
                sb.y = fmaf(wb[tap], w2.y, sb.y);
            }
        }
        const float2 fa = filter_phase(ph, n0 + q);
        const float2 fb = cmul(fa, __ldg(a.tab.stp + k));        // one more range bin: times exp(j 2 pi B)
        const float2 ya = cmul(sa, fa), yb = cmul(sb, fb);
        // conjugate: the inverse transform is conj(FFT(conj(.)))
        e.x[j * V] = make_float2(ya.x, -ya.y);
        e.x[j * V + 1] = make_float2(yb.x, -yb.y);
    };

    // two chunks per step; the pair two steps back has been consumed when its buffers are refilled
    stage_chunk(0);
    stage_chunk(1);
    cp_async_commit();
    stage_chunk(2);
    stage_chunk(3);
    cp_async_commit();
    static_for<0, r / 2>([&](auto p_) {
        constexpr int p = decltype(p_)::value;
        if constexpr (p == 0) cp_async_wait<1>();
        else cp_async_wait<0>();
        __syncthreads();                       // pair p has landed for everyone; pair p-1 is consumed
        if constexpr (p >= 1 && p + 1 < r / 2) {
            stage_chunk(2 * p + 2);
            stage_chunk(2 * p + 3);
            cp_async_commit();
        }
        interp_chunk(IntC<2 * p>{});
        interp_chunk(IntC<2 * p + 1>{});
    });
    __syncthreads();                           // staging is done with the tile buffer
    e.dif(sm, a.tw);
    e.template store_last<StoreC64, true>(a.out, (int64_t)n0, a.ld, a.scale);
}

// ---------------------------------------------------------------- step 2, unfused variant
// Range cell migration correction and azimuth filter along the rows (range is the
// contiguous axis, so the 8-tap windows are plain neighbouring samples), written as
// complex64 into the output image; the inverse azimuth FFT then runs in place on the
// output with the plain column kernel. One more trip through memory than the fused
// kernel, but every thread is independent here (no tile-wide barriers), which on this
// machine is faster than doing the interpolation inside the lock-stepped column tile.
__device__ __forceinline__ void sinc8_weights_pair(float mua, float mub, float2 (&w)[8]);

struct RcmcRows {
    static constexpr int COLS = 2048;   // range bins per CTA (8 per thread: measured 1024 / 2048 / 4096 -> step 2 of a
                                        // 4096 x 4096 frame 160 / 159 / 161 us with fp32, 144 / 136 / 138 us with fp16 input)
    static constexpr int HALO = 128;    // extra staged samples: taps, alignment, growth of the shift over COLS bins
    static constexpr int TPB = 256;
};

// Measured on B200, 4096 x 4096: with the window in one interleaved array half of the 18.4 M shared-memory
// wavefronts were bank-conflict replays and the L1/shared pipe was 92 % busy; split by parity the kernel
// issues 9.9 M wavefronts (L1 53 %) and takes the same time, so that pipe was not what bound it: issue slots
// (64 % active, 123 thread instructions per pixel) and the special-function pipe (60 %) are. Taking the eight
// reciprocals of a pixel from four (1/a = b / (ab)) and asking for six (fp32 input) or five (fp16 input)
// resident CTAs gave 163 -> 159 us for step 2; other register bounds measured 1-3 % slower.
template <class TIn, class TOut = StoreC64>
__global__ void __launch_bounds__(RcmcRows::TPB, TIn::ELEM_BYTES == 8 ? 6 : 5) sar_rcmc_filter_rows_kernel(const SarArgs a, int chunks) {
    constexpr int COLS = RcmcRows::COLS, HALO = RcmcRows::HALO, TPB = RcmcRows::TPB;
    constexpr int EB = TIn::ELEM_BYTES, GRAN = 16 / EB;
    using elem_t = typename std::conditional<EB == 8, float2, __half2>::type;
    // The staged window is kept de-interleaved: even samples in the first half, odd samples in the second.
    // A thread works on two adjacent range bins, so the lanes of a warp read every other sample; in one
    // interleaved array that is a 16-byte stride (two wavefronts where one would do), in the split arrays the
    // lanes read neighbouring words.
    constexpr int HALF = (COLS + HALO) / 2;
    __shared__ __align__(16) elem_t srow[2 * HALF];
    const int k = blockIdx.x / chunks;                 // Doppler bin
    const int j0 = (blockIdx.x % chunks) * COLS;       // first output column of this CTA
    const int c0 = j0 + a.col0;                        // its range bin in the input frame
    const float4 mg = __ldg(a.tab.mig + k);
    const float4 ph = __ldg(a.tab.phs + k);
    const float2 step = __ldg(a.tab.stp + k);
    int i0;
    float mu0;
    migration(mg, c0, i0, mu0);
    const int start = (c0 + i0 - 3) & ~(GRAN - 1);     // staged window starts on a 16-byte boundary
    const elem_t* in = reinterpret_cast<const elem_t*>(a.in) + (int64_t)k * a.ld;
    for (int i = threadIdx.x; i < (COLS + HALO) / GRAN; i += TPB) {
        const int col = start + i * GRAN;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (col >= 0 && col + GRAN <= a.nr) v = *reinterpret_cast<const uint4*>(in + col);
        if constexpr (EB == 8) {           // samples 2i, 2i + 1
            *reinterpret_cast<uint2*>(srow + i) = make_uint2(v.x, v.y);
            *reinterpret_cast<uint2*>(srow + HALF + i) = make_uint2(v.z, v.w);
        } else {                           // samples 4i .. 4i + 3
            *reinterpret_cast<uint2*>(srow + 2 * i) = make_uint2(v.x, v.z);
            *reinterpret_cast<uint2*>(srow + HALF + 2 * i) = make_uint2(v.y, v.w);
        }
    }
    __syncthreads();
    const int64_t orow = (int64_t)k * a.out_ld;
    const float g = mg.x + mg.y;
#pragma unroll
    for (int h = 0; h < COLS / (2 * TPB); ++h) {
        const int j = j0 + h * 2 * TPB + 2 * threadIdx.x;          // output columns j, j + 1
        if (j >= a.out_cols) break;                                // a narrow strip ends inside the CTA's columns
        const int n = j + a.col0;                                  // range bins n, n + 1
        int ia, ib;
        float mua, mub;
        migration(mg, n, ia, mua);
        mub = mua + g;
        ib = ia;
        if (mub >= 1.0f) {
            mub -= 1.0f;
            ib += 1;
        }
        float2 wt[8];                                  // .x: bin n, .y: bin n + 1
        sinc8_weights_pair(mua, mub, wt);
        const int oa = min(max(n + ia - 3 - start, 0), COLS + HALO - 8);
        const int ob = min(max(n + 1 + ib - 3 - start, 0), COLS + HALO - 8);
        float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
        // sample o + tap lives at (o + tap) / 2 in the half that matches its parity
        const elem_t* ea = srow + (oa >> 1) + ((oa & 1) ? HALF : 0);      // even taps: ea[tap / 2]
        const elem_t* da = srow + (oa >> 1) + ((oa & 1) ? 1 : HALF);      // odd taps: da[(tap - 1) / 2]
        const elem_t* eb = srow + (ob >> 1) + ((ob & 1) ? HALF : 0);
        const elem_t* db = srow + (ob >> 1) + ((ob & 1) ? 1 : HALF);
#pragma unroll
        for (int tap = 0; tap < 8; ++tap) {
            float2 u, w2;
            const elem_t ua = (tap & 1) ? da[tap / 2] : ea[tap / 2];
            const elem_t ub = (tap & 1) ? db[tap / 2] : eb[tap / 2];
            if constexpr (EB == 8) {
                u = ua;
                w2 = ub;
            } else {
                u = __half22float2(ua);
                w2 = __half22float2(ub);
            }
            if ((tap - 3) & 1) {
                sa.x = fmaf(-wt[tap].x, u.x, sa.x);
                sa.y = fmaf(-wt[tap].x, u.y, sa.y);
                sb.x = fmaf(-wt[tap].y, w2.x, sb.x);
                sb.y = fmaf(-wt[tap].y, w2.y, sb.y);
            } else {
                sa.x = fmaf(wt[tap].x, u.x, sa.x);
                sa.y = fmaf(wt[tap].x, u.y, sa.y);
                sb.x = fmaf(wt[tap].y, w2.x, sb.x);
                sb.y = fmaf(wt[tap].y, w2.y, sb.y);
            }
        }
        const float2 fa = filter_phase(ph, n);
        const float2 fb = cmul(fa, step);
        const float2 ya = cmul(sa, fa), yb = cmul(sb, fb);
        TOut::store2(a.out, orow + j, ya, yb);
    }
}

// ---------------------------------------------------------------- step 2a on the slab layout
// The same row pass for the slab layout, organised the other way round. A CTA works on 32 consecutive
// Doppler bins (the lanes of every warp) by NC consecutive range bins (four per thread). The window of samples it needs is staged in shared memory as [sample][row] with an
// odd pitch, so a lane's eight taps come from its own column: conflict-free whatever the row's shift is.
// The four pixels of a thread share one window of 11 samples when their integer shifts agree (else each
// fetches its own eight). The window of a CTA starts at its smallest integer shift; how far the shift may
// spread inside a CTA is checked when the parameters are created. In the slab layout 32 rows of a granule
// column are one contiguous kilobyte, so the window arrives and the results leave as whole lines. (The same
// organisation on row-major images, with the results turned around in shared memory before they are
// stored, measured 140 us against 89 us for the row-wise kernel above: its loads are exposed with two CTAs
// per multiprocessor; it was dropped.)
template <class TIn, class TOut>
struct RcmcPass {
    static constexpr int ROWS = 32, NC = 64, HALO = 32, NS = NC + HALO, PITCH = ROWS + 1;
    static constexpr int THREADS = NC / 4 * 32;
    static constexpr int GI = 32 / TIn::ELEM_BYTES, GO = 32 / TOut::ELEM_BYTES;
    static constexpr int MAX_SPREAD = HALO - 8 - 6;     // allowed (largest - smallest) integer shift in a CTA
};

// interpolator weights of two pixels at once (lane x: first pixel, lane y: second), as magnitudes with the
// sign (-1)^j left to the caller like sinc8_weights_rcp. The eight reciprocals 1 / (mu - j) come two at a
// time from one hardware reciprocal of their product (1/a = b / (ab)), and the sums and products run as
// packed fp32 pairs: about 22 issue slots and 5 special-function operations per pixel.
__device__ __forceinline__ void sinc8_weights_pair(float mua, float mub, float2 (&w)[8]) {
    const float2 mu = make_float2(fmaxf(mua, 1e-30f), fmaxf(mub, 1e-30f));
    float2 x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = (i == 3) ? mu : __fadd2_rn(mu, make_float2((float)(3 - i), (float)(3 - i)));
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const float2 pr = __fmul2_rn(x[2 * h], x[2 * h + 1]);
        const float2 r = make_float2(rcp_approx(pr.x), rcp_approx(pr.y));
        w[2 * h] = __fmul2_rn(x[2 * h + 1], r);
        w[2 * h + 1] = __fmul2_rn(x[2 * h], r);
    }
    float2 s = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 8; ++i) s = ((i - 3) & 1) ? s - w[i] : s + w[i];
    const float2 inv = make_float2(rcp_approx(s.x), rcp_approx(s.y));
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = __fmul2_rn(w[i], inv);
}

template <class TIn, class TOut>
__global__ void __launch_bounds__(RcmcPass<TIn, TOut>::THREADS) sar_rcmc_filter_slab_kernel(const SarArgs a) {
    using L = RcmcPass<TIn, TOut>;
    constexpr int NS = L::NS, GI = L::GI, GO = L::GO, PITCH = L::PITCH, EBI = TIn::ELEM_BYTES;
    __shared__ __align__(16) float2 win[NS * PITCH];     // [sample][row]
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int kblocks = a.na / 32;
    const int k0 = (blockIdx.x % kblocks) * 32, n0 = (blockIdx.x / kblocks) * L::NC;
    const int k = k0 + lane;
    const float4 mg = __ldg(a.tab.mig + k);
    int s0;
    {   // |f| is monotonic over the 32 rows (a block never straddles n_azimuth / 2) and the shift grows
        // with the range bin: the smallest shift is at the first range bin of the first or last row
        int ia, ib;
        float mu;
        migration(__ldg(a.tab.mig + k0), n0, ia, mu);
        migration(__ldg(a.tab.mig + k0 + 31), n0, ib, mu);
        s0 = (n0 + min(ia, ib) - 3) & ~(GI - 1);        // floors for negative values too
    }
    auto put = [&](float2* dst, const uint4 v) {         // 16 bytes = GRAN samples, converted to fp32
        if constexpr (EBI == 8) {
            dst[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
            dst[PITCH] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
        } else {
            dst[0] = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
            dst[PITCH] = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
            dst[2 * PITCH] = __half22float2(*reinterpret_cast<const __half2*>(&v.z));
            dst[3 * PITCH] = __half22float2(*reinterpret_cast<const __half2*>(&v.w));
        }
    };
    const char* in = reinterpret_cast<const char*>(a.in);
    {   // a warp takes one half of the granules of 32 rows at a time: lanes = rows
        const int slab0 = s0 / GI;                       // exact: s0 is a multiple of GI
        const int nslabs = a.nr / GI;
        const char* src = in + ((int64_t)slab0 * a.na + k0 + lane) * 32;
        const int64_t slab_bytes = (int64_t)a.na * 32;
#pragma unroll
        for (int id = 0; id < (NS / GI) * 2; id += L::THREADS / 32) {
            const int piece = id + w;                    // (slab, half)
            if ((NS / GI) * 2 % (L::THREADS / 32) == 0 || piece < (NS / GI) * 2) {
                const int rel = piece >> 1, half = piece & 1;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);   // samples outside the row read as zero
                if ((unsigned)(slab0 + rel) < (unsigned)nslabs)
                    v = __ldg(reinterpret_cast<const uint4*>(src + rel * slab_bytes + half * 16));
                put(win + (rel * GI + half * (GI / 2)) * PITCH + lane, v);
            }
        }
    }
    __syncthreads();
    const int n = n0 + 4 * w;
    int i0[4];
    float mu[4];
    migration(mg, n, i0[0], mu[0]);
    const float g = mg.x + mg.y;
#pragma unroll
    for (int p = 1; p < 4; ++p) {                        // one range bin on: the migration grows by the slope
        mu[p] = mu[p - 1] + g;
        i0[p] = i0[p - 1];
        if (mu[p] >= 1.0f) {
            mu[p] -= 1.0f;
            i0[p] += 1;
        }
    }
    float2 wt[2][8];                                     // [pixel pair][tap], lanes x / y = the two pixels
    sinc8_weights_pair(mu[0], mu[1], wt[0]);
    sinc8_weights_pair(mu[2], mu[3], wt[1]);
    const float2* col = win + lane;
    float2 acc[4];
    auto taps = [&](int p, const float2* u) {            // u[0..7]: the eight samples of pixel p, tap j = -3 first
        float2 sum = make_float2(0.f, 0.f);
#pragma unroll
        for (int tap = 0; tap < 8; ++tap) {
            const float m = (p & 1) ? wt[p >> 1][tap].y : wt[p >> 1][tap].x;
            const float ww = ((tap - 3) & 1) ? -m : m;
            sum.x = fmaf(ww, u[tap].x, sum.x);
            sum.y = fmaf(ww, u[tap].y, sum.y);
        }
        acc[p] = sum;
    };
    if (i0[3] == i0[0]) {                                // the usual case: one window of 11 samples serves all four
        const int o = min(max(n + i0[0] - 3 - s0, 0), NS - 11);
        float2 u[11];
#pragma unroll
        for (int i = 0; i < 11; ++i) u[i] = col[(o + i) * PITCH];
#pragma unroll
        for (int p = 0; p < 4; ++p) taps(p, u + p);
    } else {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const int o = min(max(n + p + i0[p] - 3 - s0, 0), NS - 8);
            float2 u[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) u[i] = col[(o + i) * PITCH];
            taps(p, u);
        }
    }
    float2 f = filter_phase(__ldg(a.tab.phs + k), n);
    const float2 step = __ldg(a.tab.stp + k);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        acc[p] = cmul(acc[p], f);
        if (p < 3) f = cmul(f, step);                    // one more range bin: times exp(j 2 pi B)
    }
    {
        if constexpr (TOut::ELEM_BYTES == 8) {
            float4* o = reinterpret_cast<float4*>(reinterpret_cast<float2*>(a.out) + slab_index(k, n, a.na, GO));
            o[0] = make_float4(acc[0].x, acc[0].y, acc[1].x, acc[1].y);
            o[1] = make_float4(acc[2].x, acc[2].y, acc[3].x, acc[3].y);
        } else {
            __half2 h[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) h[p] = __float22half2_rn(acc[p]);
            *reinterpret_cast<uint4*>(reinterpret_cast<__half2*>(a.out) + slab_index(k, n, a.na, GO)) =
                *reinterpret_cast<const uint4*>(h);
        }
    }
}

// ---------------------------------------------------------------- tables (float64, built once)
// H[k] = conj( sum_i h[i] exp(-2 pi i k i / nr) ) / nr,  h[i] = exp(j pi K (i/fs)^2), i = -P/2 .. P-P/2-1
__global__ void sar_build_matched_filter(float2* H, int nr, int pulse_samples, double kappa) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= nr) return;
    double sr = 0.0, si = 0.0;
    for (int i = -(pulse_samples / 2); i < pulse_samples - pulse_samples / 2; ++i) {
        const double chirp_turns = 0.5 * kappa * (double)i * (double)i;
        long long m = ((long long)k * (long long)i) % nr;       // may be negative
        if (m < 0) m += nr;
        double turns = chirp_turns - (double)m / (double)nr;
        turns -= floor(turns);
        double s, c;
        sincospi(2.0 * turns, &s, &c);
        sr += c;
        si += s;
    }
    H[k] = make_float2((float)(sr / nr), (float)(-si / nr));
}

__device__ double round_to_bits(double v, int bits) {
    if (v == 0.0) return 0.0;
    int ex;
    const double m = frexp(v, &ex);
    return ldexp(rint(ldexp(m, bits)), ex - bits);
}

// nr: range bins of the whole frame, whose centre bin nr / 2 is at r_center; first_bin: range bin of the whole
// frame that the tables call n = 0 (0 for the whole frame, a strip's first bin otherwise).
__global__ void sar_build_doppler_tables(float4* mig, float4* phs, float2* stp, int na, int nr, double wavelength,
                                         double prf, double velocity, double r_center, double dr, double first_bin) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= na) return;
    const int kk = (k < na / 2) ? k : k - na;
    const double f = (double)kk * prf / (double)na;
    const double aa = wavelength * f / (2.0 * velocity);
    const double u = aa * aa;
    const double sq = sqrt(1.0 - u);
    const double inv_d_minus_1 = u / ((1.0 + sq) * sq);    // 1/D - 1, no cancellation
    const double d_minus_1 = -u / (1.0 + sq);              // D - 1
    // migration in bins: dn(n) = (r_center/dr - nr/2 + n) * (1/D - 1) = a0 + n g
    const double gslope = inv_d_minus_1;
    const double a0 = (r_center / dr - (double)(nr / 2) + first_bin) * gslope;
    const double g_hi = round_to_bits(gslope, 10);
    const double a_int = floor(a0);
    mig[k] = make_float4((float)g_hi, (float)(gslope - g_hi), (float)(a0 - a_int), __int_as_float((int)a_int));
    // filter phase in cycles: (2/lambda) R0(n) (D - 1) = A + n B
    const double A = (2.0 / wavelength) * (r_center + (first_bin - (double)(nr / 2)) * dr) * d_minus_1;
    const double B = (2.0 * dr / wavelength) * d_minus_1;
    const double b_hi = round_to_bits(B, 10);
    phs[k] = make_float4((float)(A - floor(A)), (float)b_hi, (float)(B - b_hi), 0.0f);
    double sn, cs;
    sincospi(2.0 * (B - floor(B)), &sn, &cs);
    stp[k] = make_float2((float)cs, (float)sn);
}

// ---------------------------------------------------------------- host side
template <class C, class TOut, int MODE>
cudaError_t launch_range(const SarArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(sar_range_compress_kernel<C, TOut, MODE>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    return launch_tiles<C>(sar_range_compress_kernel<C, TOut, MODE>, a, a.tiles, st);
}
template <class C, class TIn, bool SLAB>
cudaError_t launch_rcmc(const SarArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    constexpr int smem = rcmc_smem_bytes<C, TIn>();
    static_assert(smem <= 227 * 1024, "tile + staging must fit one CTA's shared memory");
    cudaError_t e = ensure_smem(sar_rcmc_filter_ifft_kernel<C, TIn, SLAB>, smem, done);
    if (e != cudaSuccess) return e;
    sar_rcmc_filter_ifft_kernel<C, TIn, SLAB><<<(unsigned)a.tiles, C::THREADS, smem, st>>>(a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}
template <class TI, class TO>
cudaError_t launch_rcmc_pass(const SarArgs& a, cudaStream_t st) {
    using L = RcmcPass<TI, TO>;
    const unsigned grid = (unsigned)((a.na / L::ROWS) * (a.nr / L::NC));
    sar_rcmc_filter_slab_kernel<TI, TO><<<grid, L::THREADS, 0, st>>>(a);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

struct SarEntry {
    int n, dtype, w, tw_total;
    int mode;            // 0 row-major, 1 slab layout, 2 (range compression only) scattered over column strips
    cudaError_t (*launch)(const SarArgs&, cudaStream_t);
    cudaError_t (*build_tw)(float2*, cudaStream_t);
};
template <class C, class T, bool RANGE, int MODE>
constexpr SarEntry sar_entry() {
    if constexpr (RANGE)
        return SarEntry{C::N, T::ELEM_BYTES == 8 ? 0 : 1, C::W, C::TW_TOTAL, MODE, &launch_range<C, T, MODE>, &launch_build_tw<C>};
    else
        return SarEntry{C::N, T::ELEM_BYTES == 8 ? 0 : 1, C::W, C::TW_TOTAL, MODE, &launch_rcmc<C, T, MODE == 1>, &launch_build_tw<C>};
}
#define SAR_QUAD(C, RANGE)                                                                \
    sar_entry<C, StoreC64, RANGE, 0>(), sar_entry<C, StoreC32H, RANGE, 0>(),             \
    sar_entry<C, StoreC64, RANGE, 1>(), sar_entry<C, StoreC32H, RANGE, 1>()
#define SAR_SHARD(C) sar_entry<C, StoreC64, true, 2>(), sar_entry<C, StoreC32H, true, 2>()
static const SarEntry k_range[] = {SAR_QUAD(R1024p, true), SAR_QUAD(R2048, true), SAR_QUAD(R4096, true), SAR_QUAD(R8192, true),
                                   SAR_SHARD(R1024p),      SAR_SHARD(R2048),      SAR_SHARD(R4096),      SAR_SHARD(R8192)};
static const SarEntry k_rcmc[] = {SAR_QUAD(T1024, false), SAR_QUAD(T2048, false), SAR_QUAD(T4096, false)};

template <size_t K>
static const SarEntry* find(const SarEntry (&tab)[K], int n, int dtype, int mode) {
    for (const SarEntry& e : tab)
        if (e.n == n && e.dtype == dtype && e.mode == mode) return &e;
    return nullptr;
}

// largest spread of the integer shift inside one CTA of the row pass (32 Doppler bins x NC range bins),
// over the whole image, in float64
static double slab_shift_spread(const sar_rda_desc* d, int nc) {
    const double wavelength = kLight / d->carrier_hz, dr = kLight / (2.0 * d->fs_hz);
    const int na = (int)d->n_azimuth, nr = (int)d->n_range;
    auto mig = [&](int k, int n) {
        const int kk = (k < na / 2) ? k : k - na;
        const double f = (double)kk * d->prf_hz / (double)na;
        const double aa = wavelength * f / (2.0 * d->velocity_mps), u = aa * aa, sq = sqrt(1.0 - u);
        return (d->r_center_m / dr - (double)(nr / 2) + (double)n) * (u / ((1.0 + sq) * sq));
    };
    double worst = 0.0;
    for (int k0 = 0; k0 + 31 < na; k0 += 32) {
        // the spread is largest at the far end of the swath
        const double lo = fmin(mig(k0, nr - nc), mig(k0 + 31, nr - nc));
        const double hi = fmax(mig(k0, nr - 1), mig(k0 + 31, nr - 1));
        worst = fmax(worst, hi - lo);
    }
    return worst;
}

}  // namespace b200fft

using namespace b200fft;

struct b200fft_sar_s {
    sar_rda_desc d;
    // row-major intermediate ("layout" 0)
    const SarEntry* range;
    const KernelEntry* azfft;
    const SarEntry* rcmc;
    const KernelEntry* azifft;   // in-place inverse column transform of the unfused variant
    const KernelEntry* azifft_h; // fp16 intermediates: inverse column transform from an fp16 image to the complex64 output
    bool can_unfuse;
    // slab intermediate ("layout" 1)
    const SarEntry* range_slab;
    const SarEntry* rcmc_slab;
    const KernelEntry* azfft_slab[2];    // forward column tiles of 2 and of 4 range bins, intermediate type both ways
    const KernelEntry* azifft_slab[2];   // inverse column tiles, intermediate type in, complex64 out
    bool can_slab;
    // azimuth transforms by transposition ("layout" 2): the paper's four-pass form, as a measured comparison
    const KernelEntry* rows_fwd;         // n_azimuth-point row transforms of the transposed image, intermediate type
    const KernelEntry* rows_inv;         // the same, inverse, complex64
    float2* tw_rows;
    bool can_transpose;
    int layout;                  // 0 row-major (direct column kernels), 1 slab, 2 row-major with transposes
    int tile_columns;            // slab layout: range bins per column tile, 2 or 4
    bool fused;                  // step 2 as one kernel (true) or as row pass + column pass (false)
    float2 *tw_range, *tw_az, *H;
    float4 *mig, *phs;
    float2* stp;
    void* workspace;
    size_t workspace_bytes;
    // A strip of range bins cut from a larger frame (sar_rda_shard_*): steps 1 and 2 only. The frame described
    // by `d` is the strip with its halos; step 2 keeps out_cols columns starting at column col0.
    bool strip;
    int col0;
    int64_t out_cols;
};

// how a strip sits in the whole frame
struct SarStrip {
    int64_t nr_whole;    // range bins of the whole frame
    int64_t first_bin;   // range bin of the whole frame at which column 0 of the strip's frame sits (may be negative)
    int col0;            // first kept column
    int64_t out_cols;    // kept columns
};

static void sar_release(b200fft_sar_s* p) {
    if (p->tw_range) cudaFree(p->tw_range);
    if (p->tw_az) cudaFree(p->tw_az);
    if (p->tw_rows) cudaFree(p->tw_rows);
    if (p->H) cudaFree(p->H);
    if (p->mig) cudaFree(p->mig);
    if (p->phs) cudaFree(p->phs);
    if (p->stp) cudaFree(p->stp);
}

static size_t image_bytes(const b200fft_sar_s* p) {
    return (size_t)p->d.n_azimuth * (size_t)p->d.n_range * (p->d.intermediate_dtype == B200FFT_C64 ? 8 : 4);
}

static int sar_create(sar_rda_params_t* params, const sar_rda_desc* d, const SarStrip* strip);

extern "C" int sar_rda_params_create(sar_rda_params_t* params, const sar_rda_desc* d) { return sar_create(params, d, nullptr); }

// strip == nullptr: the whole chain on the frame `d`. Otherwise `d` describes the strip's own frame (n_range =
// its columns with halos; r_center_m still that of the whole frame) and only the azimuth steps are prepared.
static int sar_create(sar_rda_params_t* params, const sar_rda_desc* d, const SarStrip* strip) {
    if (!params || !d) return B200FFT_ERR_INVALID_ARG;
    *params = nullptr;
    if (d->n_azimuth <= 0 || d->n_range <= 0 || d->carrier_hz <= 0 || d->bandwidth_hz <= 0 || d->fs_hz <= 0 ||
        d->pulse_s <= 0 || d->prf_hz <= 0 || d->velocity_mps <= 0 || d->r_center_m <= 0)
        return B200FFT_ERR_INVALID_ARG;
    if (d->intermediate_dtype != B200FFT_C64 && d->intermediate_dtype != B200FFT_C32H) return B200FFT_ERR_INVALID_ARG;
    if (d->rcmc_taps != 8) return B200FFT_ERR_UNSUPPORTED;
    const double wavelength = kLight / d->carrier_hz;
    if (wavelength * d->prf_hz / (4.0 * d->velocity_mps) >= 0.5) return B200FFT_ERR_INVALID_ARG;  // D must stay real
    {   // the staged window assumes the migration grows by less than one bin across four range bins
        const double aa = wavelength * d->prf_hz / (4.0 * d->velocity_mps), u = aa * aa, sq = sqrt(1.0 - u);
        if (4.0 * u / ((1.0 + sq) * sq) >= 1.0) return B200FFT_ERR_UNSUPPORTED;
    }
    const long long pulse_samples = llround(d->pulse_s * d->fs_hz);
    if (!strip && (pulse_samples < 1 || pulse_samples > d->n_range)) return B200FFT_ERR_INVALID_ARG;

    b200fft_sar_s* p = new (std::nothrow) b200fft_sar_s();
    if (!p) return B200FFT_ERR_ALLOC;
    p->d = *d;
    const int na = (int)d->n_azimuth, nr = (int)d->n_range, dt = d->intermediate_dtype;
    p->strip = strip != nullptr;
    p->col0 = strip ? strip->col0 : 0;
    p->out_cols = strip ? strip->out_cols : nr;
    const int ocols = (int)p->out_cols;        // columns the inverse azimuth transform runs on
    p->range = strip ? nullptr : find(k_range, nr, dt, 0);
    p->range_slab = strip ? nullptr : find(k_range, nr, dt, 1);
    // Column tiles of the row-major layout: the persistent streaming kernel where it is compiled (4096 rows) and
    // the image gives every multiprocessor several tiles; else, with fp16 intermediates, the wider tile on a
    // cluster of two CTAs (32-byte instead of 16-byte row segments); else the plain 4-column tile.
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    auto cols_kernel = [&](bool inverse, int dtype, int cols) {
        if (cols / 4 > sms) {
            const KernelEntry* k = find_cols_kernel(na, inverse, dtype, dtype, 0, VAR_STREAM);
            if (k && k->n >= 4096 && cols % k->w == 0) return k;
        }
        if (dtype == B200FFT_C32H) {
            const KernelEntry* k = find_cols_kernel(na, inverse, dtype, dtype, 0, VAR_WIDE_CLUSTER);
            if (k && cols % k->w == 0) return k;
        }
        return find_cols_kernel(na, inverse, dtype, dtype, 1);
    };
    p->azfft = cols_kernel(false, dt, nr);
    p->rcmc = find(k_rcmc, na, dt, 0);
    p->rcmc_slab = find(k_rcmc, na, dt, 1);
    p->azifft = cols_kernel(true, B200FFT_C64, ocols);
    p->azifft_h = nullptr;
    if (dt == B200FFT_C32H && ocols / 4 > sms && p->rcmc) {
        const KernelEntry* k = find_cols_kernel(na, true, B200FFT_C32H, B200FFT_C64, 0, VAR_STREAM);
        if (k && ocols % k->w == 0 && k->tw_total == p->rcmc->tw_total) p->azifft_h = k;
    }
    for (int i = 0; i < 2; ++i) {
        p->azfft_slab[i] = find_sar_cols_kernel(na, 2 << i, false, dt, dt);
        p->azifft_slab[i] = find_sar_cols_kernel(na, 2 << i, true, dt, B200FFT_C64);
    }
    using RS = RcmcPass<StoreC64, StoreC64>;
    // the slab row pass stages NC + HALO samples per row: the integer shift may spread by MAX_SPREAD inside a CTA
    const bool row_pass_ok = na % 64 == 0 && nr % RS::NC == 0 && slab_shift_spread(d, RS::NC) + 2.0 <= (double)RS::MAX_SPREAD;
    {   // the row-major row pass stages COLS + HALO samples: the shift may grow by at most HALO - 16 bins over COLS bins
        const double aa = wavelength * d->prf_hz / (4.0 * d->velocity_mps), u = aa * aa, sq = sqrt(1.0 - u);
        const double gmax = u / ((1.0 + sq) * sq);
        // (a strip's row pass may end inside a CTA's 1024 columns: the kernel checks the column before it stores)
        p->can_unfuse = p->azifft != nullptr && ocols % p->azifft->w == 0 && ocols % 2 == 0 &&
                        gmax * RcmcRows::COLS + 16.0 <= (double)RcmcRows::HALO;
    }
    p->can_slab = !strip && p->range_slab && p->rcmc_slab && p->azfft_slab[0] && p->azfft_slab[1] && p->azifft_slab[0] &&
                  p->azifft_slab[1] && row_pass_ok;
    p->rows_fwd = find_rows_kernel(na, false, dt, dt, 1, nr);
    p->rows_inv = find_rows_kernel(na, true, B200FFT_C64, B200FFT_C64, 1, nr);
    p->can_transpose = !strip && p->rows_fwd && p->rows_inv && p->rows_fwd->tw_total == p->rows_inv->tw_total && p->can_unfuse;
    p->layout = 0;
    p->tile_columns = 4;
    p->fused = p->layout == 0 && !p->can_unfuse;
    if ((!strip && !p->range) || !p->azfft || !p->rcmc || d->n_azimuth > 16384 || d->n_range > 16384 || nr % p->rcmc->w ||
        nr % p->azfft->w || (strip && p->fused)) {
        delete p;
        return B200FFT_ERR_UNSUPPORTED;
    }
    static_assert(T1024::TW_TOTAL == S1024::TW_TOTAL && T2048::TW_TOTAL == S2048::TW_TOTAL && T4096::TW_TOTAL == S4096::TW_TOTAL &&
                      T4096::radix(1) == S4096::radix(1) && T4096::radix(2) == S4096::radix(2) &&
                      T2048::radix(1) == S2048::radix(1) && T2048::radix(2) == S2048::radix(2) &&
                      T1024::radix(1) == S1024::radix(1) && T1024::radix(2) == S1024::radix(2),
                  "the 2- and 4-column tiles share one twiddle table: same factorisation");
    if (p->azfft->tw_total != p->rcmc->tw_total || (p->azifft && p->azifft->tw_total != p->rcmc->tw_total)) {
        delete p;                  // every azimuth kernel reads the one table built below
        return B200FFT_ERR_UNSUPPORTED;
    }
    bool ok = (strip || (cudaMalloc(&p->tw_range, sizeof(float2) * (size_t)p->range->tw_total) == cudaSuccess &&
                         cudaMalloc(&p->H, sizeof(float2) * (size_t)nr) == cudaSuccess)) &&
              cudaMalloc(&p->tw_az, sizeof(float2) * (size_t)p->rcmc->tw_total) == cudaSuccess &&
              cudaMalloc(&p->mig, sizeof(float4) * (size_t)na) == cudaSuccess &&
              cudaMalloc(&p->phs, sizeof(float4) * (size_t)na) == cudaSuccess &&
              cudaMalloc(&p->stp, sizeof(float2) * (size_t)na) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        sar_release(p);
        delete p;
        return B200FFT_ERR_ALLOC;
    }
    const double dr = kLight / (2.0 * d->fs_hz);
    const double kappa = (d->bandwidth_hz / d->pulse_s) / (d->fs_hz * d->fs_hz);
    ok = (strip || p->range->build_tw(p->tw_range, 0) == cudaSuccess) && p->rcmc->build_tw(p->tw_az, 0) == cudaSuccess;
    if (ok && p->can_transpose)
        ok = cudaMalloc(&p->tw_rows, sizeof(float2) * (size_t)p->rows_fwd->tw_total) == cudaSuccess &&
             p->rows_fwd->build_tw(p->tw_rows, 0) == cudaSuccess;
    if (!strip) sar_build_matched_filter<<<(nr + 127) / 128, 128>>>(p->H, nr, (int)pulse_samples, kappa);
    sar_build_doppler_tables<<<(na + 127) / 128, 128>>>(p->mig, p->phs, p->stp, na, strip ? (int)strip->nr_whole : nr, wavelength,
                                                       d->prf_hz, d->velocity_mps, d->r_center_m, dr,
                                                       strip ? (double)strip->first_bin : 0.0);
    g_launch_count.fetch_add(strip ? 1 : 2, std::memory_order_relaxed);
    ok = ok && cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(0) == cudaSuccess;
    if (!ok) {
        sar_release(p);
        delete p;
        return B200FFT_ERR_CUDA;
    }
    *params = p;
    return B200FFT_OK;
}

extern "C" int sar_rda_workspace_bytes(sar_rda_params_t p, size_t* bytes) {
    if (!p || !bytes) return B200FFT_ERR_INVALID_ARG;
    *bytes = 2 * image_bytes(p);       // two intermediate images (the slab layout's step 2 goes from one to the other)
    return B200FFT_OK;
}

extern "C" int sar_rda_set_workspace(sar_rda_params_t p, void* ptr, size_t bytes) {
    if (!p || !ptr) return B200FFT_ERR_INVALID_ARG;
    size_t need = 0;
    sar_rda_workspace_bytes(p, &need);
    if (reinterpret_cast<uintptr_t>(ptr) % 16) return B200FFT_ERR_ALIGNMENT;
    if (bytes < need) return B200FFT_ERR_WORKSPACE;
    p->workspace = ptr;
    p->workspace_bytes = bytes;
    return B200FFT_OK;
}

extern "C" int sar_rda_run_step(const void* raw, sar_rda_params_t p, void* out, int step, void* stream) {
    if (!p || step < 0 || step > 2) return B200FFT_ERR_INVALID_ARG;
    if (!p->workspace) return B200FFT_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int64_t na = p->d.n_azimuth, nr = p->d.n_range;
    const bool slab = p->layout == 1;
    const int dt = p->d.intermediate_dtype;
    const int gcols = dt == B200FFT_C64 ? 4 : 8;                 // range bins per 32-byte granule
    void* buf0 = p->workspace;
    void* buf1 = static_cast<char*>(p->workspace) + image_bytes(p);
    auto ok = [](cudaError_t e) { return e == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA; };
    auto slab_geometry = [&](FftArgs& f, int w) {
        f.tpg = gcols / w;
        f.slab_stride = na * gcols;
        f.dist = gcols;
    };
    if (p->strip && step == 0) return B200FFT_ERR_INVALID_ARG;     // a strip is filled by sar_rda_shard_range_compress
    if (step == 0) {
        if (!raw) return B200FFT_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(raw) % 16) return B200FFT_ERR_ALIGNMENT;
        SarArgs a{};
        a.in = raw; a.out = buf0; a.tw = p->tw_range;
        a.tab = SarTables{p->H, p->mig, p->phs, p->stp};
        a.tiles = na; a.ld = nr; a.nr = (int)nr; a.na = (int)na; a.scale = 1.0f;
        return ok((slab ? p->range_slab : p->range)->launch(a, st));
    }
    if (p->layout == 2 && step >= 1) {
        // The paper's four-pass form: an azimuth transform is a transpose, transforms along the (now contiguous)
        // rows, and a transpose back. Step 1 goes workspace -> second half -> workspace; step 2 runs the row pass
        // into `out`, then takes the whole workspace as one complex64 image for the inverse transform.
        const int eb = dt == B200FFT_C64 ? 8 : 4;
        FftArgs f{};
        f.tw = p->tw_rows;
        f.tiles = nr; f.dist = na;
        f.prefetch_ahead = 0;
        if (step == 1) {
            if (transpose_launch(buf0, buf1, (int)na, (int)nr, nr, na, eb, st) != cudaSuccess) return B200FFT_ERR_CUDA;
            f.in = buf1; f.out = buf1;
            f.scale = (float)(1.0 / (double)na);
            if (p->rows_fwd->launch(f, st) != cudaSuccess) return B200FFT_ERR_CUDA;
            return ok(transpose_launch(buf1, buf0, (int)nr, (int)na, na, nr, eb, st));
        }
        if (!out) return B200FFT_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
        SarArgs a{};
        a.in = buf0; a.out = out; a.tw = p->tw_az;
        a.tab = SarTables{p->H, p->mig, p->phs, p->stp};
        a.ld = nr; a.nr = (int)nr; a.na = (int)na; a.scale = 1.0f;
        a.col0 = 0; a.out_cols = (int)nr; a.out_ld = nr;
        const int chunks = (int)((nr + RcmcRows::COLS - 1) / RcmcRows::COLS);
        if (dt == B200FFT_C64)
            sar_rcmc_filter_rows_kernel<StoreC64><<<(unsigned)(na * chunks), RcmcRows::TPB, 0, st>>>(a, chunks);
        else
            sar_rcmc_filter_rows_kernel<StoreC32H><<<(unsigned)(na * chunks), RcmcRows::TPB, 0, st>>>(a, chunks);
        g_launch_count.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return B200FFT_ERR_CUDA;
        if (2 * image_bytes(p) < (size_t)na * (size_t)nr * 8) return B200FFT_ERR_WORKSPACE;
        if (transpose_launch(out, buf0, (int)na, (int)nr, nr, na, 8, st) != cudaSuccess) return B200FFT_ERR_CUDA;
        f.in = buf0; f.out = buf0;
        f.scale = 1.0f;                     // 1/n_azimuth was applied after the forward azimuth FFT
        if (p->rows_inv->launch(f, st) != cudaSuccess) return B200FFT_ERR_CUDA;
        return ok(transpose_launch(buf0, out, (int)nr, (int)na, na, nr, 8, st));
    }
    if (step == 1) {
        FftArgs a{};
        a.in = buf0; a.out = buf0; a.tw = p->tw_az;
        a.scale = (float)(1.0 / (double)na);
        a.prefetch_ahead = 0;
        const KernelEntry* k = slab ? p->azfft_slab[p->tile_columns == 4] : p->azfft;
        a.tiles = nr / k->w; a.dist = nr;
        if (slab) slab_geometry(a, k->w);
        return ok(k->launch(a, st));
    }
    if (!out) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
    SarArgs a{};
    a.in = buf0; a.out = out; a.tw = p->tw_az;
    a.tab = SarTables{p->H, p->mig, p->phs, p->stp};
    a.tiles = nr / p->rcmc->w; a.ld = nr; a.nr = (int)nr; a.na = (int)na; a.scale = 1.0f;
    if (p->fused) return ok((slab ? p->rcmc_slab : p->rcmc)->launch(a, st));
    FftArgs f{};
    f.tw = p->tw_az;
    f.scale = 1.0f;                         // 1/n_azimuth was applied after the forward azimuth FFT
    f.prefetch_ahead = 0;
    if (slab) {
        a.out = buf1;
        cudaError_t e = dt == B200FFT_C64 ? launch_rcmc_pass<StoreC64, StoreC64>(a, st)
                                          : launch_rcmc_pass<StoreC32H, StoreC32H>(a, st);
        if (e != cudaSuccess) return B200FFT_ERR_CUDA;
        const KernelEntry* k = p->azifft_slab[p->tile_columns == 4];
        f.in = buf1; f.out = out;
        f.tiles = nr / k->w;
        slab_geometry(f, k->w);
        f.out_dist = nr;                    // the image leaves row-major
        return ok(k->launch(f, st));
    }
    const int64_t oc = p->out_cols;          // columns kept (all of them unless this is a strip with halos)
    const int chunks = (int)((oc + RcmcRows::COLS - 1) / RcmcRows::COLS);
    a.col0 = p->col0; a.out_cols = (int)oc; a.out_ld = oc;
    // With fp16 intermediates the row pass writes a second fp16 image (one more rounding, as in the paper's
    // four-pass accounting of 40 bytes per pixel) where the inverse column kernel for it is compiled; else the
    // complex64 output image, on which the inverse column pass then runs in place.
    const bool half_image = dt == B200FFT_C32H && p->azifft_h != nullptr;
    if (dt == B200FFT_C64) {
        sar_rcmc_filter_rows_kernel<StoreC64><<<(unsigned)(na * chunks), RcmcRows::TPB, 0, st>>>(a, chunks);
    } else if (half_image) {
        a.out = buf1;
        sar_rcmc_filter_rows_kernel<StoreC32H, StoreC32H><<<(unsigned)(na * chunks), RcmcRows::TPB, 0, st>>>(a, chunks);
    } else {
        sar_rcmc_filter_rows_kernel<StoreC32H><<<(unsigned)(na * chunks), RcmcRows::TPB, 0, st>>>(a, chunks);
    }
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return B200FFT_ERR_CUDA;
    const KernelEntry* inv = half_image ? p->azifft_h : p->azifft;
    f.in = half_image ? buf1 : out; f.out = out;
    f.tiles = oc / inv->w; f.dist = oc;
    return ok(inv->launch(f, st));
}

extern "C" int sar_rda_set_option(sar_rda_params_t p, const char* key, int64_t value) {
    if (!p || !key) return B200FFT_ERR_INVALID_ARG;
    if (p->strip) return B200FFT_ERR_UNSUPPORTED;
    if (std::strcmp(key, "fused_rcmc") == 0) {
        if (!value && p->layout == 0 && !p->can_unfuse) return B200FFT_ERR_UNSUPPORTED;
        if (value && p->layout == 2) return B200FFT_ERR_UNSUPPORTED;
        p->fused = value != 0;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "layout") == 0) {
        if (value < 0 || value > 2) return B200FFT_ERR_INVALID_ARG;
        if ((value == 1 && !p->can_slab) || (value == 2 && !p->can_transpose)) return B200FFT_ERR_UNSUPPORTED;
        p->layout = (int)value;
        if (value == 0 && !p->can_unfuse) p->fused = true;
        if (value == 2) p->fused = false;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "tile_columns") == 0) {
        if (value != 2 && value != 4) return B200FFT_ERR_INVALID_ARG;
        p->tile_columns = (int)value;
        return B200FFT_OK;
    }
    return B200FFT_ERR_INVALID_ARG;
}

extern "C" int sar_rda_form_image(const void* raw, sar_rda_params_t p, void* out, void* stream) {
    if (!p || !raw || !out) return B200FFT_ERR_INVALID_ARG;
    if (raw == out || out == p->workspace || raw == p->workspace) return B200FFT_ERR_INVALID_ARG;
    for (int step = 0; step < 3; ++step) {
        int rc = sar_rda_run_step(raw, p, out, step, stream);
        if (rc != B200FFT_OK) return rc;
    }
    return B200FFT_OK;
}

extern "C" int sar_rda_form_image_host(const void* host_raw, sar_rda_params_t p, void* host_out,
                                       void* dev_raw, void* dev_out, void* stream) {
    if (!p || !host_raw || !host_out || !dev_raw || !dev_out) return B200FFT_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)p->d.n_azimuth * (size_t)p->d.n_range * 8;
    if (cudaMemcpyAsync(dev_raw, host_raw, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    int rc = sar_rda_form_image(dev_raw, p, dev_out, stream);
    if (rc != B200FFT_OK) return rc;
    if (cudaMemcpyAsync(host_out, dev_out, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    return B200FFT_OK;
}

extern "C" int sar_rda_params_destroy(sar_rda_params_t p) {
    if (!p) return B200FFT_ERR_INVALID_ARG;
    sar_release(p);
    delete p;
    return B200FFT_OK;
}

// ---------------------------------------------------------------- column-strip decomposition over several devices
struct b200fft_sar_shard_s {
    b200fft_sar_s* whole;      // tables and kernel of the range compression (whole range lines)
    b200fft_sar_s* strip;      // azimuth steps on this rank's strip
    const SarEntry* scatter;   // range compression that stores into every rank's strip
    sar_rda_shard_geometry g;
    int rank, world;
};

extern "C" int sar_rda_shard_geometry_of(const sar_rda_desc* d, int32_t rank, int32_t world, sar_rda_shard_geometry* g) {
    if (!d || !g) return B200FFT_ERR_INVALID_ARG;
    if (world != 1 && world != 2 && world != 4 && world != 8) return B200FFT_ERR_INVALID_ARG;
    if (rank < 0 || rank >= world) return B200FFT_ERR_INVALID_ARG;
    if (d->n_azimuth <= 0 || d->n_range <= 0 || d->carrier_hz <= 0 || d->fs_hz <= 0 || d->prf_hz <= 0 || d->velocity_mps <= 0 ||
        d->r_center_m <= 0)
        return B200FFT_ERR_INVALID_ARG;
    if (d->intermediate_dtype != B200FFT_C64 && d->intermediate_dtype != B200FFT_C32H) return B200FFT_ERR_INVALID_ARG;
    if (d->n_azimuth % world || d->n_range % (8 * world)) return B200FFT_ERR_UNSUPPORTED;
    if ((d->n_range / world) & (d->n_range / world - 1)) return B200FFT_ERR_UNSUPPORTED;     // strips of 2^k bins
    const double wavelength = kLight / d->carrier_hz, dr = kLight / (2.0 * d->fs_hz);
    const double aa = wavelength * d->prf_hz / (4.0 * d->velocity_mps);
    if (aa >= 0.5) return B200FFT_ERR_INVALID_ARG;
    const double u = aa * aa, sq = sqrt(1.0 - u);
    // largest migration in the frame: far edge of the swath at the Doppler edge
    const double far_bin = d->r_center_m / dr - (double)(d->n_range / 2) + (double)(d->n_range - 1);
    const double smax = far_bin * (u / ((1.0 + sq) * sq));
    if (smax < 0.0 || smax > 4096.0) return B200FFT_ERR_UNSUPPORTED;
    const int64_t bins = d->n_range / world;
    g->first_pulse = (int64_t)rank * (d->n_azimuth / world);
    g->pulses = d->n_azimuth / world;
    g->first_bin = (int64_t)rank * bins;
    g->bins = bins;
    g->halo_left = 8;                                               // taps reach 3 bins back; 8 keeps every row 32-byte aligned
    g->halo_right = (((int64_t)ceil(smax) + 5) + 7) / 8 * 8;        // largest integer shift + 4 taps ahead
    if (world > 1 && g->halo_left + g->halo_right > bins) return B200FFT_ERR_UNSUPPORTED;
    g->strip_width = g->halo_left + bins + g->halo_right;
    const int64_t eb = d->intermediate_dtype == B200FFT_C64 ? 8 : 4;
    g->strip_bytes = d->n_azimuth * g->strip_width * eb;
    g->workspace_bytes = 2 * g->strip_bytes;
    return B200FFT_OK;
}

extern "C" int sar_rda_shard_create(sar_rda_shard_t* out, const sar_rda_desc* d, int32_t rank, int32_t world) {
    if (!out || !d) return B200FFT_ERR_INVALID_ARG;
    *out = nullptr;
    sar_rda_shard_geometry g;
    int rc = sar_rda_shard_geometry_of(d, rank, world, &g);
    if (rc != B200FFT_OK) return rc;
    b200fft_sar_shard_s* s = new (std::nothrow) b200fft_sar_shard_s();
    if (!s) return B200FFT_ERR_ALLOC;
    s->g = g;
    s->rank = rank;
    s->world = world;
    s->scatter = find(k_range, (int)d->n_range, d->intermediate_dtype, 2);
    rc = s->scatter ? sar_create(&s->whole, d, nullptr) : B200FFT_ERR_UNSUPPORTED;
    if (rc == B200FFT_OK) {
        sar_rda_desc sd = *d;
        sd.n_range = g.strip_width;
        const SarStrip geo{d->n_range, g.first_bin - g.halo_left, (int)g.halo_left, g.bins};
        rc = sar_create(&s->strip, &sd, &geo);
    }
    if (rc != B200FFT_OK) {
        if (s->whole) sar_rda_params_destroy(s->whole);
        delete s;
        return rc;
    }
    *out = s;
    return B200FFT_OK;
}

extern "C" int sar_rda_shard_get_geometry(sar_rda_shard_t s, sar_rda_shard_geometry* g) {
    if (!s || !g) return B200FFT_ERR_INVALID_ARG;
    *g = s->g;
    return B200FFT_OK;
}

extern "C" int sar_rda_shard_set_workspace(sar_rda_shard_t s, void* ptr, size_t bytes) {
    if (!s || !ptr) return B200FFT_ERR_INVALID_ARG;
    if (bytes < (size_t)s->g.workspace_bytes) return B200FFT_ERR_WORKSPACE;
    return sar_rda_set_workspace(s->strip, ptr, bytes);
}

extern "C" int sar_rda_shard_range_compress(sar_rda_shard_t s, const void* raw_rows, void* const* strips, void* stream) {
    if (!s || !raw_rows || !strips) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(raw_rows) % 16) return B200FFT_ERR_ALIGNMENT;
    const b200fft_sar_s* w = s->whole;
    SarArgs a{};
    a.in = raw_rows; a.out = nullptr; a.tw = w->tw_range;
    a.tab = SarTables{w->H, w->mig, w->phs, w->stp};
    a.tiles = s->g.pulses; a.ld = w->d.n_range; a.nr = (int)w->d.n_range; a.na = (int)w->d.n_azimuth; a.scale = 1.0f;
    for (int g = 0; g < s->world; ++g) {
        if (!strips[g]) return B200FFT_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(strips[g]) % 16) return B200FFT_ERR_ALIGNMENT;
        if (strips[g] == raw_rows) return B200FFT_ERR_INVALID_ARG;
        a.sh.strip[g] = (unsigned long long)reinterpret_cast<uintptr_t>(strips[g]);
    }
    a.sh.world = s->world;
    a.sh.strip_cols = (int)s->g.bins;
    a.sh.strip_shift = 0;
    while (((int64_t)1 << a.sh.strip_shift) < s->g.bins) ++a.sh.strip_shift;
    a.sh.halo_l = (int)s->g.halo_left;
    a.sh.halo_r = (int)s->g.halo_right;
    a.sh.sw = (int)s->g.strip_width;
    a.sh.row0 = s->g.first_pulse;
    return s->scatter->launch(a, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA;
}

extern "C" int sar_rda_shard_azimuth(sar_rda_shard_t s, void* image_strip, void* stream) {
    if (!s || !image_strip) return B200FFT_ERR_INVALID_ARG;
    if (!s->strip->workspace) return B200FFT_ERR_WORKSPACE;
    if (image_strip == s->strip->workspace) return B200FFT_ERR_INVALID_ARG;
    int rc = sar_rda_run_step(nullptr, s->strip, image_strip, 1, stream);
    if (rc != B200FFT_OK) return rc;
    return sar_rda_run_step(nullptr, s->strip, image_strip, 2, stream);
}

extern "C" int sar_rda_shard_destroy(sar_rda_shard_t s) {
    if (!s) return B200FFT_ERR_INVALID_ARG;
    sar_rda_params_destroy(s->whole);
    sar_rda_params_destroy(s->strip);
    delete s;
    return B200FFT_OK;
}
