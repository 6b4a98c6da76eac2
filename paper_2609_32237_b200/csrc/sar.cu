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
// The filter and the migration are affine in the range index with per-Doppler-bin
// coefficients, built once in float64. The paper's four numerical fixes are kept:
// baseband filter (D - 1); phase in cycles with a split that makes the fp32
// product exact; a continuous interpolator (evaluated directly, no table);
// the fractional shift taken from the migration alone.
#include <cuda_runtime.h>
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
};

// ---------------------------------------------------------------- step 0
template <class C, class TOut>
__global__ void __launch_bounds__(C::THREADS, C::MINB) sar_range_compress_kernel(const SarArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    static_assert(C::W == 1, "range compression works on contiguous rows");
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
    e.dit(sm, a.tw);
    if (active) e.template store_first<TOut, true>(a.out, base, a.ld, 1.0f);
}

// ---------------------------------------------------------------- step 2
// weights of the 8-tap sinc interpolator, taps j = -3..4, unit sum:
// sinc(mu - j) = (-1)^j sin(pi mu) / (pi (mu - j)); after normalisation the common
// factor drops out, and multiplying through by prod_i (mu - i) removes the divisions:
// w_j = (-1)^j P_j / sum_j' (-1)^j' P_j',  P_j = prod_{i != j} (mu - i).
__device__ __forceinline__ void sinc8_weights(float mu, float (&w)[8]) {
    float d[8], pre[8], suf[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) d[i] = mu - (float)(i - 3);
    pre[0] = 1.0f;
#pragma unroll
    for (int i = 1; i < 8; ++i) pre[i] = pre[i - 1] * d[i - 1];
    suf[7] = 1.0f;
#pragma unroll
    for (int i = 6; i >= 0; --i) suf[i] = suf[i + 1] * d[i + 1];
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float p = pre[i] * suf[i];
        w[i] = ((i - 3) & 1) ? -p : p;
        s += w[i];
    }
    const float inv = 1.0f / s;
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] *= inv;
}

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
    float s, c;
    sincospif(2.0f * (f - floorf(f)), &s, &c);
    return make_float2(c, s);
}

template <class C, class TIn>
__global__ void __launch_bounds__(C::THREADS, C::MINB) sar_rcmc_filter_ifft_kernel(const SarArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    constexpr int W = C::W;
    static_assert(W >= 2, "azimuth transforms work on column tiles");
    const int g = threadIdx.x / C::T, t = threadIdx.x % C::T;
    int64_t tile = (C::CL > 1) ? (int64_t)(blockIdx.x / C::CL) : (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    const int64_t base = tile * W;
    Engine<C> e;
    e.setup(t);
    {
        using G = Geo<C, 1>;
        constexpr int V = G::V, r = G::r;
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            const int c = C::template cidx<V>(e.t, v, e.rank);
            const int q = c % W, lo = c / W;
            const int n0 = (int)base + q;                  // range bins n0, n0 + 1
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const int k = j * G::Ls + lo;              // Doppler bin (row)
                const float4 mg = __ldg(a.tab.mig + k);
                const float4 ph = __ldg(a.tab.phs + k);
                int ia, ib;
                float mua, mub;
                migration(mg, n0, ia, mua);
                migration(mg, n0 + 1, ib, mub);
                float wa[8], wb[8];
                sinc8_weights(mua, wa);
                sinc8_weights(mub, wb);
                const int64_t row = (int64_t)k * a.ld;
                float2 sa = make_float2(0.f, 0.f), sb = make_float2(0.f, 0.f);
#pragma unroll
                for (int tap = 0; tap < 8; ++tap) {
                    const int ca = n0 + ia + tap - 3, cb = n0 + 1 + ib + tap - 3;
                    if (ca >= 0 && ca < a.nr) {
                        const float2 s = TIn::load1(a.in, row + ca);
                        sa.x = fmaf(wa[tap], s.x, sa.x);
                        sa.y = fmaf(wa[tap], s.y, sa.y);
                    }
                    if (cb >= 0 && cb < a.nr) {
                        const float2 s = TIn::load1(a.in, row + cb);
                        sb.x = fmaf(wb[tap], s.x, sb.x);
                        sb.y = fmaf(wb[tap], s.y, sb.y);
                    }
                }
                const float2 fa = filter_phase(ph, n0), fb = filter_phase(ph, n0 + 1);
                const float2 ya = cmul(sa, fa), yb = cmul(sb, fb);
                // conjugate: the inverse transform is conj(FFT(conj(.)))
                e.x[j * V + v] = make_float2(ya.x, -ya.y);
                e.x[j * V + v + 1] = make_float2(yb.x, -yb.y);
            });
        });
    }
    e.dif(sm, a.tw);
    if (active) e.template store_last<StoreC64, true>(a.out, base, a.ld, a.scale);
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

__global__ void sar_build_doppler_tables(float4* mig, float4* phs, int na, int nr, double wavelength,
                                         double prf, double velocity, double r_center, double dr) {
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
    const double a0 = (r_center / dr - (double)(nr / 2)) * gslope;
    const double g_hi = round_to_bits(gslope, 10);
    const double a_int = floor(a0);
    mig[k] = make_float4((float)g_hi, (float)(gslope - g_hi), (float)(a0 - a_int), __int_as_float((int)a_int));
    // filter phase in cycles: (2/lambda) R0(n) (D - 1) = A + n B
    const double A = (2.0 / wavelength) * (r_center - (double)(nr / 2) * dr) * d_minus_1;
    const double B = (2.0 * dr / wavelength) * d_minus_1;
    const double b_hi = round_to_bits(B, 10);
    phs[k] = make_float4((float)(A - floor(A)), (float)b_hi, (float)(B - b_hi), 0.0f);
}

// ---------------------------------------------------------------- host side
template <class C, class TOut>
cudaError_t launch_range(const SarArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(sar_range_compress_kernel<C, TOut>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    return launch_tiles<C>(sar_range_compress_kernel<C, TOut>, a, a.tiles, st);
}
template <class C, class TIn>
cudaError_t launch_rcmc(const SarArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(sar_rcmc_filter_ifft_kernel<C, TIn>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    return launch_tiles<C>(sar_rcmc_filter_ifft_kernel<C, TIn>, a, a.tiles, st);
}

struct SarEntry {
    int n, dtype, w, tw_total;
    cudaError_t (*launch)(const SarArgs&, cudaStream_t);
    cudaError_t (*build_tw)(float2*, cudaStream_t);
};
template <class C, class T, bool RANGE>
constexpr SarEntry sar_entry() {
    if constexpr (RANGE) return SarEntry{C::N, T::ELEM_BYTES == 8 ? 0 : 1, C::W, C::TW_TOTAL, &launch_range<C, T>, &launch_build_tw<C>};
    else return SarEntry{C::N, T::ELEM_BYTES == 8 ? 0 : 1, C::W, C::TW_TOTAL, &launch_rcmc<C, T>, &launch_build_tw<C>};
}
#define SAR_PAIR(C, RANGE) sar_entry<C, StoreC64, RANGE>(), sar_entry<C, StoreC32H, RANGE>()
static const SarEntry k_range[] = {SAR_PAIR(R1024, true), SAR_PAIR(R2048, true), SAR_PAIR(R4096, true), SAR_PAIR(R8192, true)};
static const SarEntry k_rcmc[] = {SAR_PAIR(T1024, false), SAR_PAIR(T2048, false), SAR_PAIR(T4096, false)};

template <size_t K>
static const SarEntry* find(const SarEntry (&tab)[K], int n, int dtype) {
    for (const SarEntry& e : tab)
        if (e.n == n && e.dtype == dtype) return &e;
    return nullptr;
}

}  // namespace b200fft

using namespace b200fft;

struct b200fft_sar_s {
    sar_rda_desc d;
    const SarEntry* range;
    const KernelEntry* azfft;
    const SarEntry* rcmc;
    float2 *tw_range, *tw_az, *H;
    float4 *mig, *phs;
    void* workspace;
    size_t workspace_bytes;
};

static void sar_release(b200fft_sar_s* p) {
    if (p->tw_range) cudaFree(p->tw_range);
    if (p->tw_az) cudaFree(p->tw_az);
    if (p->H) cudaFree(p->H);
    if (p->mig) cudaFree(p->mig);
    if (p->phs) cudaFree(p->phs);
}

extern "C" int sar_rda_params_create(sar_rda_params_t* params, const sar_rda_desc* d) {
    if (!params || !d) return B200FFT_ERR_INVALID_ARG;
    *params = nullptr;
    if (d->n_azimuth <= 0 || d->n_range <= 0 || d->carrier_hz <= 0 || d->bandwidth_hz <= 0 || d->fs_hz <= 0 ||
        d->pulse_s <= 0 || d->prf_hz <= 0 || d->velocity_mps <= 0 || d->r_center_m <= 0)
        return B200FFT_ERR_INVALID_ARG;
    if (d->intermediate_dtype != B200FFT_C64 && d->intermediate_dtype != B200FFT_C32H) return B200FFT_ERR_INVALID_ARG;
    if (d->rcmc_taps != 8) return B200FFT_ERR_UNSUPPORTED;
    const double wavelength = kLight / d->carrier_hz;
    if (wavelength * d->prf_hz / (4.0 * d->velocity_mps) >= 0.5) return B200FFT_ERR_INVALID_ARG;  // D must stay real
    const long long pulse_samples = llround(d->pulse_s * d->fs_hz);
    if (pulse_samples < 1 || pulse_samples > d->n_range) return B200FFT_ERR_INVALID_ARG;

    b200fft_sar_s* p = new (std::nothrow) b200fft_sar_s();
    if (!p) return B200FFT_ERR_ALLOC;
    p->d = *d;
    const int na = (int)d->n_azimuth, nr = (int)d->n_range, dt = d->intermediate_dtype;
    p->range = find(k_range, nr, dt);
    p->azfft = find_cols_kernel(na, false, dt, dt);
    p->rcmc = find(k_rcmc, na, dt);
    if (!p->range || !p->azfft || !p->rcmc || d->n_azimuth > 16384 || d->n_range > 16384 || nr % p->rcmc->w) {
        delete p;
        return B200FFT_ERR_UNSUPPORTED;
    }
    bool ok = cudaMalloc(&p->tw_range, sizeof(float2) * (size_t)p->range->tw_total) == cudaSuccess &&
              cudaMalloc(&p->tw_az, sizeof(float2) * (size_t)p->rcmc->tw_total) == cudaSuccess &&
              cudaMalloc(&p->H, sizeof(float2) * (size_t)nr) == cudaSuccess &&
              cudaMalloc(&p->mig, sizeof(float4) * (size_t)na) == cudaSuccess &&
              cudaMalloc(&p->phs, sizeof(float4) * (size_t)na) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        sar_release(p);
        delete p;
        return B200FFT_ERR_ALLOC;
    }
    const double dr = kLight / (2.0 * d->fs_hz);
    const double kappa = (d->bandwidth_hz / d->pulse_s) / (d->fs_hz * d->fs_hz);
    ok = p->range->build_tw(p->tw_range, 0) == cudaSuccess && p->rcmc->build_tw(p->tw_az, 0) == cudaSuccess;
    sar_build_matched_filter<<<(nr + 127) / 128, 128>>>(p->H, nr, (int)pulse_samples, kappa);
    sar_build_doppler_tables<<<(na + 127) / 128, 128>>>(p->mig, p->phs, na, nr, wavelength, d->prf_hz,
                                                       d->velocity_mps, d->r_center_m, dr);
    g_launch_count.fetch_add(2, std::memory_order_relaxed);
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
    *bytes = (size_t)p->d.n_azimuth * (size_t)p->d.n_range * (p->d.intermediate_dtype == B200FFT_C64 ? 8 : 4);
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
    if (step == 0) {
        if (!raw) return B200FFT_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(raw) % 16) return B200FFT_ERR_ALIGNMENT;
        SarArgs a{};
        a.in = raw; a.out = p->workspace; a.tw = p->tw_range;
        a.tab = SarTables{p->H, p->mig, p->phs};
        a.tiles = na; a.ld = nr; a.nr = (int)nr; a.scale = 1.0f;
        return p->range->launch(a, st) == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA;
    }
    if (step == 1) {
        FftArgs a{};
        a.in = p->workspace; a.out = p->workspace; a.tw = p->tw_az;
        a.tiles = nr / p->azfft->w; a.dist = nr;
        a.scale = (float)(1.0 / (double)na);
        return p->azfft->launch(a, st) == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA;
    }
    if (!out) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
    SarArgs a{};
    a.in = p->workspace; a.out = out; a.tw = p->tw_az;
    a.tab = SarTables{p->H, p->mig, p->phs};
    a.tiles = nr / p->rcmc->w; a.ld = nr; a.nr = (int)nr; a.scale = 1.0f;
    return p->rcmc->launch(a, st) == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA;
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
