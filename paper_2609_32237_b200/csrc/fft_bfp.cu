// Block-floating-point variant of the single-pass row transform with fp16 storage: every
// transform carries one power-of-two exponent, so that coherent data (whose spectrum grows
// up to N times the input) keeps its precision and never overflows the fp16 range. The paper
// (Section "FP16 Storage") names block floating point as what real radar data needs and uses
// fixed shifts in its own chain; this is the per-transform form.
//
//   true input  x_b[n] = in_b[n]  * 2^in_exp[b]      (in_exp may be null: all zero)
//   true output X_b[k] = out_b[k] * 2^out_exp[b]
//
// The kernel transforms the stored fp16 values in fp32, takes the largest |Re|, |Im| of the
// result m_b, and stores X * 2^(-s_b) with s_b = floor(log2 m_b) - 14, i.e. the largest stored
// component lies in [2^14, 2^15) (one bit of headroom below the fp16 maximum). s_b comes from the
// exponent bits of m_b: no rounding decision is involved. out_exp[b] = in_exp[b] + s_b, minus
// log2 N for the inverse (its 1/N is folded into the exponent, not the mantissas).
#include "configs.h"
#include "registry.h"

namespace b200fft {

template <class C, bool INV>
__global__ void __launch_bounds__(C::THREADS, C::MINB) fft_rows_bfp_kernel(const FftArgs a, const int* in_exp,
                                                                          int* out_exp) {
    static_assert(C::W == 1 && C::CL == 1, "contiguous rows, one CTA per tile group");
    extern __shared__ __align__(16) float2 smem_dyn[];
    __shared__ float wmax[32];
    constexpr int T = C::T;
    const int g = threadIdx.x / T, t = threadIdx.x % T;
    int64_t tile = (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;          // keep the barriers uniform; results discarded
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    const int64_t base = tile * a.dist;
    Engine<C> e;
    e.setup(t);
    e.template load_first<StoreC32H, INV>(a.in, base, a.dist);
    e.dif(sm, a.tw);
    // largest component of this transform
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < C::P; ++i) m = fmaxf(m, fmaxf(fabsf(e.x[i].x), fabsf(e.x[i].y)));
    constexpr int LANES = T < 32 ? T : 32;    // a transform's threads are T consecutive lanes (T < 32) or whole warps
#pragma unroll
    for (int off = LANES / 2; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if constexpr (T > 32) {
        constexpr int WPT = T / 32;           // warps per transform
        const int warp = threadIdx.x >> 5;
        if ((threadIdx.x & 31) == 0) wmax[warp] = m;
        __syncthreads();
        const int w0 = g * WPT;
        m = wmax[w0];
#pragma unroll
        for (int i = 1; i < WPT; ++i) m = fmaxf(m, wmax[w0 + i]);
    }
    // s = floor(log2 m) - 14 from the exponent field; zero (or subnormal) data keep exponent 0
    const int ebits = (__float_as_int(m) >> 23) & 0xff;
    int s = (ebits == 0) ? 0 : (ebits - 127) - 14;
    s = max(s, -100);                                          // keeps 2^(-s) a finite fp32 for vanishing data
    const float scale = __int_as_float((127 - s) << 23);      // 2^(-s), exact
    if (active) {
        e.template store_last<StoreC32H, INV>(a.out, base, a.dist, scale);
        if (t == 0) {
            const int ein = in_exp ? in_exp[tile] : 0;
            out_exp[tile] = ein + s - (INV ? ilog2(C::N) : 0);
        }
    }
}

template <class C, bool INV>
cudaError_t launch_bfp(const FftArgs& a, const int* in_exp, int* out_exp, cudaStream_t st) {
    static bool done[64] = {};
    cudaError_t e = ensure_smem(fft_rows_bfp_kernel<C, INV>, C::SMEM_BYTES, done);
    if (e != cudaSuccess) return e;
    const int64_t grid = (a.tiles + C::G - 1) / C::G;
    fft_rows_bfp_kernel<C, INV><<<(unsigned)grid, C::THREADS, C::SMEM_BYTES, st>>>(a, in_exp, out_exp);
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

template <class C, bool INV>
constexpr BfpEntry make_bfp_entry() {
    return BfpEntry{C::N, INV, C::TW_TOTAL, &launch_bfp<C, INV>, &launch_build_tw<C>};
}
#define B200FFT_BFP(C) make_bfp_entry<C, false>(), make_bfp_entry<C, true>()

static const BfpEntry k_bfp[] = {B200FFT_BFP(R1024), B200FFT_BFP(R2048), B200FFT_BFP(R4096), B200FFT_BFP(R8192),
                                 B200FFT_BFP(R16384)};

const BfpEntry* find_bfp_kernel(int n, bool inverse) {
    for (const BfpEntry& e : k_bfp)
        if (e.n == n && e.inverse == inverse) return &e;
    return nullptr;
}

}  // namespace b200fft
