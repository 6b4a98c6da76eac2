// Two-pass transform, n = n1 * n2, for n past the on-chip limit (paper, Section
// "One Pass": the two-pass "four-step" FFT is the usual remedy when a transform
// does not fit on chip; each extra pass through main memory divides the ceiling).
//
// View transform b as an n1 x n2 row-major matrix x[j1][j2].
//   pass 1: for every column j2, an n1-point transform over j1 (read in place at
//           stride n2, W adjacent columns per tile), then multiply element
//           (k1, j2) by exp(-2 pi i j2 k1 / n); written to the workspace as
//           A[k1][j2].
//   pass 2: for every row k1 of A, an n2-point transform over j2; X[k1 + n1 k2]
//           is stored transposed. A tile is W adjacent rows so that the
//           transposed store writes W*8-byte segments.
// The inverse conjugates on the way in and on the way out and scales by 1/n.
// Pass 2 reads its tile rows with one 64-bit load per element: a register pair is two adjacent ROWS of the
// workspace, n2 elements apart, so a warp-level load still covers whole sectors (consecutive elements of a row
// go to consecutive lane pairs), and a 128-bit form would only trade two loads for one load and two shuffles.
// Pass 2 on 16-row tiles, whose transposed store writes whole 128-byte lines, measured slower than the 4-row
// tiles (757 against 713 us for 2048 transforms of 65536 points) and is not used.
#include "../../include/b200fft.h"
#include "fourstep.h"
#include "configs.h"
#include "registry.h"

namespace b200fft {

struct FourStepArgs {
    const void* in;
    void* out;
    const float2* tw;       // stage twiddles of this pass's configuration
    const float2* tw_lo;
    const float2* tw_hi;
    int64_t tiles;          // batch * (columns or rows) / W
    int64_t groups;         // tiles per transform
    int64_t dist_in, dist_out;
    int64_t n, n1, n2;
    float scale;
};

struct FourStepEntry {
    int n, dtype;
    bool inverse;
    int w, g, tw_total;
    cudaError_t (*launch)(const FourStepArgs&, cudaStream_t);
    cudaError_t (*build_tw)(float2*, cudaStream_t);
};

template <class C, bool INV, class TIn, class TOut>
__global__ void __launch_bounds__(C::THREADS, C::MINB) fourstep_pass1_kernel(const FourStepArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    constexpr int W = C::W;
    const int g = threadIdx.x / C::T, t = threadIdx.x % C::T;
    int64_t tile = (C::CL > 1) ? (int64_t)(blockIdx.x / C::CL) : (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;
    const int64_t b = tile / a.groups, cg = tile % a.groups;
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    Engine<C> e;
    e.setup(t);
    e.template load_first<TIn, INV>(a.in, b * a.dist_in + cg * W, a.n2);
    e.template dif<false>(sm, a.tw);
    if (!active) return;
    using G = Geo<C, C::S>;
    constexpr int V = G::V, r = G::r, KS = C::N / r;
    static_assert(V >= 2, "register pairs");
    // k1 < n1 <= 1024, j2 < n2 and n1 * n2 <= 2^20: the products fit 32 bits
    const unsigned nmask = (unsigned)(a.n - 1), n2 = (unsigned)a.n2;
    const int64_t obase = b * a.dist_out;
    auto twiddle_and_store = [&](auto v_, auto j_, float2 pa, float2 pb) {
        constexpr int v = decltype(v_)::value, j = decltype(j_)::value;
        int b0, q;
        e.last_index(v, b0, q);
        const unsigned j2 = (unsigned)cg * W + q;
        const unsigned k1 = j * KS + b0;
        const unsigned m0 = (k1 * j2) & nmask;
        const float2 w0 = cmul(__ldg(a.tw_hi + (m0 >> 10)), __ldg(a.tw_lo + (m0 & 1023)));
        const float2 w1 = cmul(w0, __ldg(a.tw_lo + k1));     // one column on: times exp(-2 pi i k1 / n), k1 < 1024
        TOut::store2(a.out, obase + (k1 * n2 + j2), cmul(pa, w0), cmul(pb, w1));
    };
    if constexpr (r == 8 || r == 16 || r == 32) {
        e.template compute<C::S, false>(nullptr, twiddle_and_store);      // outputs leave as they complete
    } else {
        e.template compute<C::S, false>(nullptr);
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                twiddle_and_store(IntC<v>{}, j_, e.x[j * V + v], e.x[j * V + v + 1]);
            });
        });
    }
}

template <class C, bool INV, class TIn, class TOut>
__global__ void __launch_bounds__(C::THREADS, C::MINB) fourstep_pass2_kernel(const FourStepArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    constexpr int W = C::W;
    const int g = threadIdx.x / C::T, t = threadIdx.x % C::T;
    int64_t tile = (C::CL > 1) ? (int64_t)(blockIdx.x / C::CL) : (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;
    const int64_t b = tile / a.groups, rg = tile % a.groups;
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    Engine<C> e;
    e.setup(t);
    {
        using G = Geo<C, 1>;
        constexpr int V = G::V, r = G::r;
        const int64_t rowbase = b * a.dist_in + rg * W * a.n2;
        const unsigned n2 = (unsigned)a.n2;                 // W * n2 <= 16384: offsets within the tile fit 32 bits
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            const int c = C::template cidx<V>(e.t, v, e.rank);
            const unsigned q = c % W, lo = c / W;
            const int64_t pbase = rowbase + (q * n2 + lo);
            static_for<0, r>([&](auto i_) {
                constexpr int j = fetch_order<r>(decltype(i_)::value);
                e.x[j * V + v] = TIn::load1(a.in, pbase + j * G::Ls);
                e.x[j * V + v + 1] = TIn::load1(a.in, pbase + j * G::Ls + n2);
            });
        });
    }
    e.template dif<false>(sm, a.tw);
    if (active) e.template last_stage_and_store<TOut, INV>(a.out, b * a.dist_out + rg * W, a.n1, a.scale);
}

template <class C, bool INV, class TI, class TO, int PASS>
cudaError_t launch_fourstep(const FourStepArgs& a, cudaStream_t st) {
    static bool done[64] = {};
    if constexpr (PASS == 1) {          // (a ternary would instantiate both kernels for every configuration)
        cudaError_t e = ensure_smem(fourstep_pass1_kernel<C, INV, TI, TO>, C::SMEM_BYTES, done);
        if (e != cudaSuccess) return e;
        return launch_tiles<C>(fourstep_pass1_kernel<C, INV, TI, TO>, a, a.tiles, st);
    } else {
        cudaError_t e = ensure_smem(fourstep_pass2_kernel<C, INV, TI, TO>, C::SMEM_BYTES, done);
        if (e != cudaSuccess) return e;
        return launch_tiles<C>(fourstep_pass2_kernel<C, INV, TI, TO>, a, a.tiles, st);
    }
}

template <class C, bool INV, class TS, int PASS>
constexpr FourStepEntry make_fs_entry() {
    return FourStepEntry{C::N, TS::ELEM_BYTES == 8 ? 0 : 1, INV, C::W, C::G, C::TW_TOTAL,
                         &launch_fourstep<C, INV, TS, TS, PASS>, &launch_build_tw<C>};
}
#define FS_ENTRIES(C, PASS)                                                         \
    make_fs_entry<C, false, StoreC64, PASS>(), make_fs_entry<C, true, StoreC64, PASS>(), \
    make_fs_entry<C, false, StoreC32H, PASS>(), make_fs_entry<C, true, StoreC32H, PASS>()

static const FourStepEntry k_pass1[] = {FS_ENTRIES(F64, 1), FS_ENTRIES(F128, 1), FS_ENTRIES(F256, 1),
                                        FS_ENTRIES(F512, 1), FS_ENTRIES(F1024, 1)};
static const FourStepEntry k_pass2[] = {FS_ENTRIES(T64, 2), FS_ENTRIES(T128, 2), FS_ENTRIES(T256, 2),
                                        FS_ENTRIES(T512, 2), FS_ENTRIES(T1024, 2), FS_ENTRIES(T2048, 2),
                                        FS_ENTRIES(T4096, 2)};

template <size_t K>
static const FourStepEntry* find(const FourStepEntry (&tab)[K], int n, bool inv, int dtype) {
    for (const FourStepEntry& e : tab)
        if (e.n == n && e.inverse == inv && e.dtype == dtype) return &e;
    return nullptr;
}

// exp(-2 pi i m step / n) for m = 0..count-1, float64 then one rounding
__global__ void build_factor_table(float2* tab, int count, int64_t step, int64_t n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const int64_t m = ((int64_t)i * step) % n;
    double sn, cs;
    sincospi(-2.0 * (double)m / (double)n, &sn, &cs);
    tab[i] = make_float2((float)cs, (float)sn);
}

// n = n1 * n2. Default: n1 = 256 from n = 65536 on (pass 1 then runs on 32 KiB tiles, four CTAs per SM, and
// pass 2 carries the long transform along contiguous rows; measured for 512 MiB of complex64: 2^17 404 -> 394 us,
// 2^18 428 -> 402, 2^19 480 -> 441, 2^20 492 -> 476 against the near-square split), the near-square split with
// n1 >= n2 below. `n1_request` > 0 asks for another one (64 <= n1 <= 1024, 64 <= n2 <= 4096).
static int fourstep_split(int64_t n, int64_t n1_request, int64_t* n1, int64_t* n2) {
    int lg = 0;
    while (((int64_t)1 << lg) < n) ++lg;
    if (((int64_t)1 << lg) != n || lg < 12 || lg > 20) return B200FFT_ERR_UNSUPPORTED;
    *n1 = lg >= 16 ? 256 : (int64_t)1 << ((lg + 1) / 2);
    if (n1_request > 0) {
        if ((n1_request & (n1_request - 1)) || n1_request < 64 || n1_request > 1024 || n / n1_request < 64 ||
            n / n1_request > 4096)
            return B200FFT_ERR_UNSUPPORTED;
        *n1 = n1_request;
    }
    *n2 = n / *n1;
    return B200FFT_OK;
}

void fourstep_release(FourStep* fs) {
    if (fs->tw1) cudaFree(fs->tw1);
    if (fs->tw2) cudaFree(fs->tw2);
    if (fs->tw_lo) cudaFree(fs->tw_lo);
    if (fs->tw_hi) cudaFree(fs->tw_hi);
    *fs = FourStep();
}

int fourstep_build(FourStep* fs, int64_t n, int64_t batch, int64_t dist, int direction, int dtype, int64_t n1_request) {
    fourstep_release(fs);
    int64_t n1, n2;
    const int rc = fourstep_split(n, n1_request, &n1, &n2);
    if (rc != B200FFT_OK) return rc;
    fs->n = n;
    fs->n1 = n1;
    fs->n2 = n2;
    fs->batch = batch;
    fs->dist = dist;
    fs->direction = direction;
    fs->dtype = dtype;
    const bool inv = direction == B200FFT_INVERSE;
    fs->pass1 = find(k_pass1, (int)fs->n1, inv, dtype);
    fs->pass2 = find(k_pass2, (int)fs->n2, inv, dtype);
    if (!fs->pass1 || !fs->pass2) return B200FFT_ERR_UNSUPPORTED;
    const int hi_count = (int)(n / 1024);
    if (cudaMalloc(&fs->tw1, sizeof(float2) * (size_t)fs->pass1->tw_total) != cudaSuccess ||
        cudaMalloc(&fs->tw2, sizeof(float2) * (size_t)fs->pass2->tw_total) != cudaSuccess ||
        cudaMalloc(&fs->tw_lo, sizeof(float2) * 1024) != cudaSuccess ||
        cudaMalloc(&fs->tw_hi, sizeof(float2) * (size_t)hi_count) != cudaSuccess) {
        cudaGetLastError();
        fourstep_release(fs);
        return B200FFT_ERR_ALLOC;
    }
    bool ok = fs->pass1->build_tw(fs->tw1, 0) == cudaSuccess && fs->pass2->build_tw(fs->tw2, 0) == cudaSuccess;
    build_factor_table<<<4, 256>>>(fs->tw_lo, 1024, 1, n);
    build_factor_table<<<(hi_count + 255) / 256, 256>>>(fs->tw_hi, hi_count, 1024, n);
    g_launch_count.fetch_add(2, std::memory_order_relaxed);
    ok = ok && cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(0) == cudaSuccess;
    if (!ok) {
        fourstep_release(fs);
        return B200FFT_ERR_CUDA;
    }
    return B200FFT_OK;
}

size_t fourstep_table_elems(int64_t n, int direction, int dtype) {
    int64_t n1, n2;
    if (fourstep_split(n, 0, &n1, &n2) != B200FFT_OK) return 0;
    const bool inv = direction == B200FFT_INVERSE;
    const FourStepEntry* p1 = find(k_pass1, (int)n1, inv, dtype);
    const FourStepEntry* p2 = find(k_pass2, (int)n2, inv, dtype);
    if (!p1 || !p2) return 0;
    // each table starts on a 16-byte boundary (two float2)
    auto up = [](size_t v) { return (v + 1) & ~(size_t)1; };
    return up((size_t)p1->tw_total) + up((size_t)p2->tw_total) + 1024 + up((size_t)(n / 1024));
}

int fourstep_build_in_place(FourStep* fs, int64_t n, int64_t batch, int64_t dist, int direction, int dtype,
                            float2* tables, size_t table_elems, cudaStream_t st) {
    *fs = FourStep();
    int64_t n1, n2;
    int rc = fourstep_split(n, 0, &n1, &n2);
    if (rc != B200FFT_OK) return rc;
    const size_t need = fourstep_table_elems(n, direction, dtype);
    if (need == 0) return B200FFT_ERR_UNSUPPORTED;
    if (!tables || table_elems < need) return B200FFT_ERR_WORKSPACE;
    const bool inv = direction == B200FFT_INVERSE;
    fs->n = n; fs->n1 = n1; fs->n2 = n2; fs->batch = batch; fs->dist = dist;
    fs->direction = direction; fs->dtype = dtype;
    fs->pass1 = find(k_pass1, (int)n1, inv, dtype);
    fs->pass2 = find(k_pass2, (int)n2, inv, dtype);
    auto up = [](size_t v) { return (v + 1) & ~(size_t)1; };
    const int hi_count = (int)(n / 1024);
    fs->tw1 = tables;
    fs->tw2 = fs->tw1 + up((size_t)fs->pass1->tw_total);
    fs->tw_lo = fs->tw2 + up((size_t)fs->pass2->tw_total);
    fs->tw_hi = fs->tw_lo + 1024;
    bool ok = fs->pass1->build_tw(fs->tw1, st) == cudaSuccess && fs->pass2->build_tw(fs->tw2, st) == cudaSuccess;
    build_factor_table<<<4, 256, 0, st>>>(fs->tw_lo, 1024, 1, n);
    build_factor_table<<<(hi_count + 255) / 256, 256, 0, st>>>(fs->tw_hi, hi_count, 1024, n);
    g_launch_count.fetch_add(2, std::memory_order_relaxed);
    ok = ok && cudaGetLastError() == cudaSuccess;
    return ok ? B200FFT_OK : B200FFT_ERR_CUDA;
}

int fourstep_execute(const FourStep* fs, const void* in, void* out, void* workspace, cudaStream_t st) {
    FourStepArgs a;
    a.tw_lo = fs->tw_lo;
    a.tw_hi = fs->tw_hi;
    a.n = fs->n;
    a.n1 = fs->n1;
    a.n2 = fs->n2;
    a.scale = (fs->direction == B200FFT_INVERSE) ? (float)(1.0 / (double)fs->n) : 1.0f;
    // pass 1: columns of every n1 x n2 matrix
    a.in = in;
    a.out = workspace;
    a.tw = fs->tw1;
    a.groups = fs->n2 / fs->pass1->w;
    a.tiles = fs->batch * a.groups;
    a.dist_in = fs->dist;
    a.dist_out = fs->n;
    if (fs->pass1->launch(a, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    // pass 2: rows of the workspace, transposed store
    a.in = workspace;
    a.out = out;
    a.tw = fs->tw2;
    a.groups = fs->n1 / fs->pass2->w;
    a.tiles = fs->batch * a.groups;
    a.dist_in = fs->n;
    a.dist_out = fs->dist;
    if (fs->pass2->launch(a, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    return B200FFT_OK;
}

}  // namespace b200fft
