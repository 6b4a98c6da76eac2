// Register-resident mixed-radix FFT engine for sm_100a.
//
// One "tile" is W transforms of N points that share a CTA's shared memory
// (W = 1: a contiguous row; W > 1: W adjacent columns of a row-major matrix).
// Each thread keeps P complex values in registers. The transform is an
// in-place decimation-in-frequency network N = r1 * r2 * ... * rS: stage s
// combines, for every other digit fixed, the r_s values whose position differs
// in digit s (weight L_s = N / (r1..rs)), then multiplies output k by
// exp(-2 pi i lo k / L_{s-1}) (lo = the lower digits). Between stages the
// values go through shared memory, each thread writing back exactly the
// positions it read, so one barrier per exchange is enough. The first stage
// reads global memory directly in natural order; the last stage leaves
// X[d1 + r1 d2 + ...] at position (d1, d2, ..) and its threads are assigned
// with d1 fastest, so the global store is contiguous as well. The same
// network run backwards (twiddle first, then butterfly, stages S..1) is the
// decimation-in-time transform that consumes digit-reversed input: used to
// fuse FFT -> pointwise filter -> inverse FFT without reordering.
//
// Shared-memory positions are XOR-swizzled with the top digit so that both the
// lane-contiguous accesses of stages 1..S-1 and the d1-fastest accesses of the
// last stage are free of bank conflicts with 128-bit accesses.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <type_traits>

namespace b200fft {

// ---------------------------------------------------------------- utilities
template <int I>
using IntC = std::integral_constant<int, I>;

template <int B, int E, class F>
__device__ __forceinline__ void static_for(F&& f) {
    if constexpr (B < E) {
        f(IntC<B>{});
        static_for<B + 1, E>(f);
    }
}

__host__ __device__ constexpr int ilog2(int x) { return x <= 1 ? 0 : 1 + ilog2(x >> 1); }

// Complex add and subtract, optionally as one packed fp32 instruction each (sm_100 add/sub.f32x2: the
// same two IEEE roundings as the scalar pair, so results are bit-identical, in one issue slot instead of
// two). Measured on B200 the packed forms run at half the scalar rate per instruction, so only issue slots
// are saved, and the aligned register pairs they need cost the large kernels more than that: N = 4096
// +1.3 %, N = 8192 fp16 storage +2.8 %, but N = 8192 / 16384 complex64 -6 % / -7 %. Off by default;
// -DB200FFT_PACKED_ADDS builds the packed variant.
#ifdef B200FFT_PACKED_ADDS
__device__ __forceinline__ float2 operator+(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 operator-(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\t"
        "mov.b64 rb, {%4, %5};\n\t"
        "sub.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
#else
__device__ __forceinline__ float2 operator+(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 operator-(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
#endif
__device__ __forceinline__ float2 cmul(float2 a, float2 w) {
    return make_float2(fmaf(a.x, w.x, -a.y * w.y), fmaf(a.x, w.y, a.y * w.x));
}

// cos / sin of 2 pi m / 32, m = 0..8, as compile-time constants
__host__ __device__ constexpr double cos32_table(int m) {
    constexpr double t[9] = {1.0,
                             0.98078528040323044913,
                             0.92387953251128675613,
                             0.83146961230254523708,
                             0.70710678118654752440,
                             0.55557023301960222474,
                             0.38268343236508977173,
                             0.19509032201612826785,
                             0.0};
    return t[m];
}
__host__ __device__ constexpr double cos32(int m) {
    m &= 31;
    if (m <= 8) return cos32_table(m);
    if (m <= 16) return -cos32_table(16 - m);
    if (m <= 24) return -cos32_table(m - 16);
    return cos32_table(32 - m);
}
__host__ __device__ constexpr double sin32(int m) { return cos32(m - 8); }

// x * exp(-2 pi i M / 32), M a compile-time constant
template <int M_>
__device__ __forceinline__ float2 mulw32(float2 x) {
    constexpr int M = M_ & 31;
    if constexpr (M == 0) return x;
    else if constexpr (M == 8) return make_float2(x.y, -x.x);
    else if constexpr (M == 16) return make_float2(-x.x, -x.y);
    else if constexpr (M == 24) return make_float2(-x.y, x.x);
    else if constexpr (M == 4) {
        constexpr float h = 0.70710678118654752440f;
        return make_float2((x.x + x.y) * h, (x.y - x.x) * h);
    } else if constexpr (M == 12) {
        constexpr float h = 0.70710678118654752440f;
        return make_float2((x.y - x.x) * h, -(x.x + x.y) * h);
    } else if constexpr (M == 20) {
        constexpr float h = 0.70710678118654752440f;
        return make_float2(-(x.x + x.y) * h, (x.x - x.y) * h);
    } else if constexpr (M == 28) {
        constexpr float h = 0.70710678118654752440f;
        return make_float2((x.x - x.y) * h, (x.x + x.y) * h);
    } else {
        constexpr float c = (float)cos32(M), s = (float)sin32(M);
        // (a + ib)(c - is) = (ac + bs) + i(bc - as)
        return make_float2(fmaf(x.x, c, x.y * s), fmaf(x.y, c, -x.x * s));
    }
}

// ------------------------------------------------------- small DFTs in registers
// Dft<R>::run(v): v[k] <- sum_j v[j] exp(-2 pi i j k / R), natural order in and out.
template <int R>
struct Dft;

template <>
struct Dft<1> {
    static __device__ __forceinline__ void run(float2*) {}
};
template <>
struct Dft<2> {
    static __device__ __forceinline__ void run(float2* v) {
        float2 a = v[0], b = v[1];
        v[0] = a + b;
        v[1] = a - b;
    }
};
template <>
struct Dft<4> {
    static __device__ __forceinline__ void run(float2* v) {
        float2 a0 = v[0] + v[2], a1 = v[0] - v[2], a2 = v[1] + v[3], a3 = v[1] - v[3];
        v[0] = a0 + a2;
        v[2] = a0 - a2;
        v[1] = make_float2(a1.x + a3.y, a1.y - a3.x);  // a1 - i a3
        v[3] = make_float2(a1.x - a3.y, a1.y + a3.x);  // a1 + i a3
    }
};

// R = A * B: B-point transforms over j = a + A b, twiddle exp(-2 pi i a c / R),
// A-point transforms over a; output k = c + B d.
template <int R, int A, int B>
__device__ __forceinline__ void dft_composite(float2* v) {
    float2 y[R];
    static_for<0, A>([&](auto a_) {
        constexpr int a = decltype(a_)::value;
        float2 t[B];
        static_for<0, B>([&](auto b_) { constexpr int b = decltype(b_)::value; t[b] = v[a + A * b]; });
        Dft<B>::run(t);
        static_for<0, B>([&](auto c_) {
            constexpr int c = decltype(c_)::value;
            y[a * B + c] = mulw32<a * c * (32 / R)>(t[c]);
        });
    });
    static_for<0, B>([&](auto c_) {
        constexpr int c = decltype(c_)::value;
        float2 t[A];
        static_for<0, A>([&](auto a_) { constexpr int a = decltype(a_)::value; t[a] = y[a * B + c]; });
        Dft<A>::run(t);
        static_for<0, A>([&](auto d_) { constexpr int d = decltype(d_)::value; v[c + B * d] = t[d]; });
    });
}
// The same for two butterflies at once, handing every finished output pair (k, a_k, b_k) to `emit`
// as soon as its last small transform is done, so that stores can leave while the rest is computed.
template <int R, int A, int B, class F>
__device__ __forceinline__ void dft_composite_emit2(const float2* va, const float2* vb, F&& emit) {
    float2 ya[R], yb[R];
    static_for<0, A>([&](auto a_) {
        constexpr int a = decltype(a_)::value;
        float2 ta[B], tb[B];
        static_for<0, B>([&](auto b_) {
            constexpr int b = decltype(b_)::value;
            ta[b] = va[a + A * b];
            tb[b] = vb[a + A * b];
        });
        Dft<B>::run(ta);
        Dft<B>::run(tb);
        static_for<0, B>([&](auto c_) {
            constexpr int c = decltype(c_)::value;
            ya[a * B + c] = mulw32<a * c * (32 / R)>(ta[c]);
            yb[a * B + c] = mulw32<a * c * (32 / R)>(tb[c]);
        });
    });
    static_for<0, B>([&](auto c_) {
        constexpr int c = decltype(c_)::value;
        float2 ta[A], tb[A];
        static_for<0, A>([&](auto a_) {
            constexpr int a = decltype(a_)::value;
            ta[a] = ya[a * B + c];
            tb[a] = yb[a * B + c];
        });
        Dft<A>::run(ta);
        Dft<A>::run(tb);
        static_for<0, A>([&](auto d_) {
            constexpr int d = decltype(d_)::value;
            emit(IntC<c + B * d>{}, ta[d], tb[d]);
        });
    });
}
template <int R, int A, int B, class F>
__device__ __forceinline__ void dft_composite_emit1(const float2* va, F&& emit) {
    float2 ya[R];
    static_for<0, A>([&](auto a_) {
        constexpr int a = decltype(a_)::value;
        float2 ta[B];
        static_for<0, B>([&](auto b_) { constexpr int b = decltype(b_)::value; ta[b] = va[a + A * b]; });
        Dft<B>::run(ta);
        static_for<0, B>([&](auto c_) { constexpr int c = decltype(c_)::value; ya[a * B + c] = mulw32<a * c * (32 / R)>(ta[c]); });
    });
    static_for<0, B>([&](auto c_) {
        constexpr int c = decltype(c_)::value;
        float2 ta[A];
        static_for<0, A>([&](auto a_) { constexpr int a = decltype(a_)::value; ta[a] = ya[a * B + c]; });
        Dft<A>::run(ta);
        static_for<0, A>([&](auto d_) { constexpr int d = decltype(d_)::value; emit(IntC<c + B * d>{}, ta[d]); });
    });
}
template <int R>
struct Split { static constexpr int A = 1, B = R; };      // R = A * B as used by Dft<R> (8, 16, 32 below)
template <> struct Split<8> { static constexpr int A = 2, B = 4; };
template <> struct Split<16> { static constexpr int A = 4, B = 4; };
template <> struct Split<32> { static constexpr int A = 4, B = 8; };

template <>
struct Dft<8> {
    static __device__ __forceinline__ void run(float2* v) { dft_composite<8, 2, 4>(v); }
};
template <>
struct Dft<16> {
    static __device__ __forceinline__ void run(float2* v) { dft_composite<16, 4, 4>(v); }
};
template <>
struct Dft<32> {
    static __device__ __forceinline__ void run(float2* v) { dft_composite<32, 4, 8>(v); }
};

// Order in which the r inputs of a butterfly are fetched: the composite transforms work on the
// subsets j = a + A b first (a fixed), so fetching subset by subset lets the arithmetic on the
// first subset start while the rest are still in flight.
template <int R>
__host__ __device__ constexpr int fetch_order(int i) {
    constexpr int A = (R == 32 || R == 16) ? 4 : (R == 8 ? 2 : 1);
    constexpr int B = R / A;
    return (i / B) + A * (i % B);
}

// ------------------------------------------------------------ configuration
template <int N_, int W_, int P_, int G_, int CL_, int R1_, int R2_, int R3_ = 1, int R4_ = 1, int TW1_ = 1>
struct Cfg {
    static constexpr int N = N_, W = W_, P = P_, G = G_, CL = CL_;
    static constexpr int TW1_LOADS = TW1_;    // first-stage twiddle rows loaded from the table (rest computed)
    static constexpr int S = (R3_ == 1) ? 2 : ((R4_ == 1) ? 3 : 4);
    __host__ __device__ static constexpr int radix(int s) { return s == 1 ? R1_ : (s == 2 ? R2_ : (s == 3 ? R3_ : R4_)); }
    __host__ __device__ static constexpr int L(int s) {
        int l = N;
        for (int i = 1; i <= s; ++i) l /= radix(i);
        return l;
    }
    // A tile (W transforms of N points) is shared by a cluster of CL CTAs: each keeps
    // 1/CL of it in its own shared memory and 1/CL of the threads.
    static constexpr int T = N * W / P / CL;  // threads per tile per CTA
    static constexpr int THREADS = T * G;     // threads per CTA
    static constexpr int TILE_ELEMS = N * W;
    static constexpr int LOCAL_ELEMS = TILE_ELEMS / CL;
    static constexpr int SMEM_BYTES = LOCAL_ELEMS * G * 8;
    static constexpr int RC = R1_ / CL;       // values of the top digit a CTA owns after the first exchange
    // twiddle rows of stage s < S start here: (radix-1) rows of L(s) entries each
    __host__ __device__ static constexpr int tw_off(int s) {
        int o = 0;
        for (int i = 1; i < s; ++i) o += (radix(i) - 1) * L(i);
        return o;
    }
    static constexpr int TW_TOTAL = tw_off(S);
    // Index, within the whole tile, of butterfly v (0 .. V-1) of thread t of CTA `rank`
    // at a stage with V butterflies per thread. Butterflies go to threads in adjacent
    // pairs, and the pairs of one register slot are contiguous across the threads of a
    // CTA, so that a warp's shared-memory access is one contiguous run.
    template <int V>
    __host__ __device__ static constexpr int cidx(int t, int v, int rank) {
        if (V == 1) return rank * T + t;
        return rank * V * T + 2 * ((v >> 1) * T + t) + (v & 1);
    }
    // weight of digit i (1 .. S-1) in the last stage's local butterfly index (top digit fastest)
    __host__ __device__ static constexpr int blw(int i) {
        int w = 1;
        if (i >= 2) w = RC;
        for (int k = 2; k < i; ++k) w *= radix(k);
        return w;
    }
    static_assert(R1_ * R2_ * R3_ * R4_ == N_, "radices must multiply to N");
    // bits of the element index the swizzle may flip: bits 1..3, but only below the top digit
    static constexpr int SWZ = 14 & (L(1) * W_ - 1);
    // with one butterfly per thread in the last stage neighbouring lanes hold neighbouring butterflies (not
    // every other one), so the index is doubled before it is folded into bits 1..3
    static constexpr int SWM = (P_ / radix(S) == 1) ? 2 : 1;
    static_assert(L(1) * W_ >= 2, "at least two elements below the top digit");
    static_assert(CL_ == 1 || G_ == 1, "a cluster works on one tile");
    static_assert(CL_ >= 1 && R1_ % CL_ == 0 && RC >= 2, "the cluster splits the top digit");
    static_assert(CL_ == 1 || RC * W_ >= 16 || L(2) * W_ >= 16, "second digit must stay constant over 16 elements");
    // registers per thread are capped at 128 so that at least 65536 / (128 * THREADS) CTAs fit an SM
    static constexpr int MINB = (65536 / (128 * THREADS)) > 0 ? (65536 / (128 * THREADS)) : 1;
    static_assert(P_ % R1_ == 0 && P_ % R2_ == 0 && P_ % R3_ == 0 && P_ % R4_ == 0, "P must be a multiple of every radix");
    static_assert(P_ / radix(S) >= 2 || W_ == 1, "column tiles need two butterflies per thread in the last stage");
    static_assert((N_ * W_) % (P_ * CL_) == 0, "tile must divide among threads");
};

// Geometry of butterfly v of thread te (index within the whole tile: cluster rank * T + t)
// at stage s. Element indices are local to the owning CTA's shared memory.
template <class C, int s>
struct Geo {
    static constexpr int r = C::radix(s), V = C::P / r, Ls = C::L(s), Lp = C::L(s - 1), L1 = C::L(1);
    static constexpr bool last = (s == C::S);
    static constexpr int W = C::W, CL = C::CL, RC = C::RC;
    static constexpr int estep = last ? W : Ls * W;  // element step per register index j
    int e0;    // local element index (position * W + column) of j = 0, before swizzle
    int bl0;   // low bits of the last-stage butterfly index of these positions, digit s counted as 0
    int lo;    // twiddle column (stages < S); global output index low part (last stage)

    // low 4 bits of the last stage's local butterfly index that position p0 belongs to,
    // leaving out digit `skip`; the top digit is taken relative to the owning CTA
    template <int skip>
    static __device__ __forceinline__ int bl_of(int p0, int rank) {
        int bl = 0;
        static_for<1, C::S>([&](auto i_) {
            constexpr int i = decltype(i_)::value;
            if constexpr (i != skip && C::blw(i) < 16) {
                int d = (p0 / C::L(i)) % C::radix(i);
                if constexpr (i == 1) d -= rank * RC;
                bl += d * C::blw(i);
            }
        });
        return bl;
    }

    __device__ __forceinline__ void init(int t, int v, int rank) {
        const int c = C::template cidx<V>(t, v, rank);
        const int q = c % W;
        const int b = c / W;
        if constexpr (!last) {
            lo = b % Ls;
            const int hi = b / Ls;
            const int p0 = hi * Lp + lo;              // position with digit s = 0
            bl0 = bl_of<s>(p0, rank);
            e0 = p0 * W + q - ((s == 1) ? 0 : rank * C::LOCAL_ELEMS);
        } else {
            const int bloc = b - rank * (C::N / r / CL);   // local butterfly index, top digit fastest
            const int d1 = bloc % RC + rank * RC;
            int rem = bloc / RC, p0 = d1 * L1;
            lo = d1 + C::radix(1) * rem;
            static_for<2, C::S>([&](auto i_) {
                constexpr int i = decltype(i_)::value;
                p0 += (rem % C::radix(i)) * C::L(i);
                rem /= C::radix(i);
            });
            e0 = p0 * W + q - rank * C::LOCAL_ELEMS;
            bl0 = bloc & 15;
        }
    }
    // CTA (cluster rank) that owns position j of the first stage after the first exchange
    template <int j>
    __host__ __device__ static constexpr int dest() { return j / RC; }
    template <int j>
    __device__ __forceinline__ int elem() const {
        if constexpr (s == 1) {
            constexpr int jl = j % RC;                // top digit relative to the owner
            return (e0 + jl * estep) ^ (((bl0 + jl) * W * C::SWM) & C::SWZ);
        } else if constexpr (!last) {
            if constexpr (C::blw(s) < 16) return (e0 + j * estep) ^ (((bl0 + j * C::blw(s)) * W * C::SWM) & C::SWZ);
            else return (e0 + j * estep) ^ ((bl0 * W * C::SWM) & C::SWZ);
        } else {
            return (e0 + j * estep) ^ ((bl0 * W * C::SWM) & C::SWZ);
        }
    }
};

// ------------------------------------------------------------ cluster helpers
__device__ __forceinline__ unsigned cluster_ctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// store two complex values into the shared memory of CTA `rank` of this cluster, at the
// address that `local` has in this CTA (all CTAs of a cluster lay out shared memory alike)
__device__ __forceinline__ void st_cluster_f4(const float2* local, unsigned rank, float4 v) {
    const unsigned a = (unsigned)__cvta_generic_to_shared(local);
    unsigned ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(ra), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ void st_cluster_f2(const float2* local, unsigned rank, float2 v) {
    const unsigned a = (unsigned)__cvta_generic_to_shared(local);
    unsigned ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(ra), "f"(v.x), "f"(v.y) : "memory");
}

// ------------------------------------------------------------ storage types
struct StoreC64 {
    using pair_t = float4;  // two complex fp32
    static constexpr int ELEM_BYTES = 8;
    static __device__ __forceinline__ void load2(const void* base, int64_t idx, float2& a, float2& b) {
        const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float2*>(base) + idx);
        a = make_float2(v.x, v.y);
        b = make_float2(v.z, v.w);
    }
    static __device__ __forceinline__ void store2(void* base, int64_t idx, float2 a, float2 b) {
        *reinterpret_cast<float4*>(reinterpret_cast<float2*>(base) + idx) = make_float4(a.x, a.y, b.x, b.y);
    }
    static __device__ __forceinline__ float2 load1(const void* base, int64_t idx) {
        return reinterpret_cast<const float2*>(base)[idx];
    }
    static __device__ __forceinline__ void store1(void* base, int64_t idx, float2 a) {
        reinterpret_cast<float2*>(base)[idx] = a;
    }
};
struct StoreC32H {
    static constexpr int ELEM_BYTES = 4;
    static __device__ __forceinline__ void load2(const void* base, int64_t idx, float2& a, float2& b) {
        const uint2 v = *reinterpret_cast<const uint2*>(reinterpret_cast<const __half2*>(base) + idx);
        a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
        b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    }
    static __device__ __forceinline__ void store2(void* base, int64_t idx, float2 a, float2 b) {
        __half2 ha = __float22half2_rn(a), hb = __float22half2_rn(b);
        uint2 v;
        v.x = *reinterpret_cast<unsigned*>(&ha);
        v.y = *reinterpret_cast<unsigned*>(&hb);
        *reinterpret_cast<uint2*>(reinterpret_cast<__half2*>(base) + idx) = v;
    }
    static __device__ __forceinline__ float2 load1(const void* base, int64_t idx) {
        return __half22float2(reinterpret_cast<const __half2*>(base)[idx]);
    }
    static __device__ __forceinline__ void store1(void* base, int64_t idx, float2 a) {
        reinterpret_cast<__half2*>(base)[idx] = __float22half2_rn(a);
    }
};

// ------------------------------------------------------------ the engine
template <class C>
struct Engine {
    static constexpr int P = C::P, W = C::W, S = C::S, CL = C::CL;
    float2 x[P];
    int rank;   // CTA rank in its cluster (0 when CL == 1)
    int t;      // thread index within the tile's threads of this CTA

    __device__ __forceinline__ void setup(int t_) {
        rank = (CL > 1) ? (int)cluster_ctarank() : 0;
        t = t_;
        // every CTA of the cluster must be running before its shared memory is written remotely
        if constexpr (CL > 1) cluster_arrive();
    }

    // ---- shared-memory exchange -------------------------------------------------
    // Registers of stage s are x[j * V + v]: butterfly v, element j.
    template <int s, bool WR>
    __device__ __forceinline__ void smem_rw(float2* sm) {
        using G = Geo<C, s>;
        constexpr int V = G::V, r = G::r;
        constexpr bool REMOTE = (CL > 1 && s == 1);
        static_assert(!(REMOTE && !WR), "with a cluster the first stage reads global memory only");
        if constexpr (G::last && W == 1) {
            // the two butterflies of a thread sit L1 apart: go 128-bit along j instead
            static_for<0, V>([&](auto v_) {
                constexpr int v = decltype(v_)::value;
                G g;
                g.init(t, v, rank);
                static_for<0, r / 2>([&](auto h_) {
                    constexpr int j = 2 * decltype(h_)::value;
                    float4* p = reinterpret_cast<float4*>(sm + g.template elem<j>());
                    if constexpr (WR) {
                        *p = make_float4(x[j * V + v].x, x[j * V + v].y, x[(j + 1) * V + v].x, x[(j + 1) * V + v].y);
                    } else {
                        const float4 q = *p;
                        x[j * V + v] = make_float2(q.x, q.y);
                        x[(j + 1) * V + v] = make_float2(q.z, q.w);
                    }
                });
            });
        } else if constexpr (V >= 2) {
            static_for<0, V / 2>([&](auto h_) {
                constexpr int v = 2 * decltype(h_)::value;
                G g;
                g.init(t, v, rank);
                static_for<0, r>([&](auto i_) {
                    constexpr int j = WR ? decltype(i_)::value : fetch_order<r>(decltype(i_)::value);
                    float2* p2 = sm + g.template elem<j>();
                    if constexpr (WR) {
                        const float4 val = make_float4(x[j * V + v].x, x[j * V + v].y, x[j * V + v + 1].x, x[j * V + v + 1].y);
                        if constexpr (REMOTE) st_cluster_f4(p2, (unsigned)G::template dest<j>(), val);
                        else *reinterpret_cast<float4*>(p2) = val;
                    } else {
                        const float4 q = *reinterpret_cast<const float4*>(p2);
                        x[j * V + v] = make_float2(q.x, q.y);
                        x[j * V + v + 1] = make_float2(q.z, q.w);
                    }
                });
            });
        } else {
            G g;
            g.init(t, 0, rank);
            static_for<0, r>([&](auto i_) {
                constexpr int j = WR ? decltype(i_)::value : fetch_order<r>(decltype(i_)::value);
                float2* p2 = sm + g.template elem<j>();
                if constexpr (WR) {
                    if constexpr (REMOTE) st_cluster_f2(p2, (unsigned)G::template dest<j>(), x[j]);
                    else *p2 = x[j];
                } else {
                    x[j] = *p2;
                }
            });
        }
    }

    // barrier of exchange s -> s+1 (DIF) or s -> s-1 (DIT)
    template <bool CLUSTER>
    __device__ __forceinline__ void exchange_barrier() {
        if constexpr (CLUSTER) {
            cluster_arrive();
            cluster_wait();
        } else {
            __syncthreads();
        }
    }

    // ---- butterflies + twiddles ----------------------------------------------------
    // DIT = false: butterfly, then multiply output k by tw[k][lo]   (stages 1..S-1)
    // DIT = true : multiply input j by tw[j][lo], then butterfly     (transposed network)
    // With a sink (stages whose butterfly comes last: the DIF last stage, every DIT stage, two
    // butterflies per thread, radix 8/16/32) the outputs are not written back to the registers:
    // sink(v, k, a_k, b_k) receives output k of butterflies v and v + 1 as soon as it is final.
    struct NoSink {};
    template <int s, bool DIT, class Sink = NoSink>
    __device__ __forceinline__ void compute(const float2* __restrict__ tw, Sink&& sink = Sink{}) {
        using G = Geo<C, s>;
        constexpr bool SINK = !std::is_same<typename std::decay<Sink>::type, NoSink>::value;
        constexpr int V = G::V, r = G::r, Ls = G::Ls;
        constexpr bool has_tw = !G::last;
        // Rows of the stage's twiddle table that are loaded; the rest are products of loaded
        // ones (w^k = w^M w^(k-M)). Only the first stage of a one-transform tile trades
        // loads for arithmetic: there every lane needs different entries, so each table row
        // costs four L1 wavefronts per warp, and L1 is the busiest unit of these kernels.
        constexpr int M = (s == 1 && W == 1 && r > C::TW1_LOADS) ? C::TW1_LOADS : r - 1;
        auto twiddle_pair = [&](int lo0, float2* a, float2* b) {
            // a, b: the r values of butterflies v, v+1 (b == nullptr if V == 1)
            const float2* row = tw + C::tw_off(s) + lo0;
            if constexpr (M < r - 1 && V == 1) {
                float2 wa[r];
                static_for<1, r>([&](auto k_) {
                    constexpr int k = decltype(k_)::value;
                    if constexpr (k <= M) wa[k] = __ldg(row + (k - 1) * Ls);
                    else wa[k] = cmul(wa[M], wa[k - M]);
                    a[k] = cmul(a[k], wa[k]);
                });
            } else if constexpr (M < r - 1) {
                float2 wa[r], wb[r];
                static_for<1, r>([&](auto k_) {
                    constexpr int k = decltype(k_)::value;
                    if constexpr (k <= M) {
                        const float4 w = __ldg(reinterpret_cast<const float4*>(row + (k - 1) * Ls));
                        wa[k] = make_float2(w.x, w.y);
                        wb[k] = make_float2(w.z, w.w);
                    } else {
                        wa[k] = cmul(wa[M], wa[k - M]);
                        wb[k] = cmul(wb[M], wb[k - M]);
                    }
                    a[k] = cmul(a[k], wa[k]);
                    b[k] = cmul(b[k], wb[k]);
                });
            } else {
                static_for<1, r>([&](auto k_) {
                    constexpr int k = decltype(k_)::value;
                    // keep the compiler from hoisting all r-1 table loads above the arithmetic
                    // (that costs ~60 live registers on top of the 64 data registers)
                    if constexpr (DIT && (k % 4) == 1 && k > 1) asm volatile("" ::: "memory");
                    if constexpr (W == 1 && V >= 2) {
                        const float4 w = __ldg(reinterpret_cast<const float4*>(row + (k - 1) * Ls));
                        a[k] = cmul(a[k], make_float2(w.x, w.y));
                        b[k] = cmul(b[k], make_float2(w.z, w.w));
                    } else {
                        const float2 w = __ldg(row + (k - 1) * Ls);
                        a[k] = cmul(a[k], w);
                        if (b) b[k] = cmul(b[k], w);
                    }
                });
            }
        };
        if constexpr (V >= 2) {
            static_for<0, V / 2>([&](auto h_) {
                constexpr int v = 2 * decltype(h_)::value;
                float2 a[r], b[r];
                static_for<0, r>([&](auto j_) {
                    constexpr int j = decltype(j_)::value;
                    a[j] = x[j * V + v];
                    b[j] = x[j * V + v + 1];
                });
                [[maybe_unused]] int lo0 = 0;
                if constexpr (has_tw) {
                    lo0 = (C::template cidx<V>(t, v, rank) / W) % Ls;
                    if constexpr (DIT) twiddle_pair(lo0, a, b);
                }
                if constexpr (SINK) {
                    static_assert((DIT || !has_tw) && (r == 8 || r == 16 || r == 32), "a sink takes finished outputs");
                    dft_composite_emit2<r, Split<r>::A, Split<r>::B>(
                        a, b, [&](auto k_, float2 pa, float2 pb) { sink(IntC<v>{}, k_, pa, pb); });
                } else {
                    Dft<r>::run(a);
                    Dft<r>::run(b);
                    if constexpr (has_tw && !DIT) twiddle_pair(lo0, a, b);
                    static_for<0, r>([&](auto j_) {
                        constexpr int j = decltype(j_)::value;
                        x[j * V + v] = a[j];
                        x[j * V + v + 1] = b[j];
                    });
                }
            });
        } else {
            static_assert(!SINK, "sinks are for stages with two butterflies per thread");
            [[maybe_unused]] int lo0 = 0;
            if constexpr (has_tw) {
                lo0 = (C::template cidx<1>(t, 0, rank) / W) % Ls;
                if constexpr (DIT) twiddle_pair(lo0, x, nullptr);
            }
            Dft<r>::run(x);
            if constexpr (has_tw && !DIT) twiddle_pair(lo0, x, nullptr);
        }
    }

    // Butterfly, twiddle and shared-memory write of a stage s < S in one: output k is multiplied by its
    // twiddle and written as soon as its last small transform is done, so the write phase overlaps the
    // arithmetic. For stages whose twiddle rows are all loaded (any order of k), local shared memory.
    template <int s>
    __host__ __device__ static constexpr bool fused_write_ok() {
        constexpr int r = C::radix(s);
        constexpr int M = (s == 1 && W == 1 && r > C::TW1_LOADS) ? C::TW1_LOADS : r - 1;
        return s < S && M == r - 1 && !(CL > 1 && s == 1) && (r == 8 || r == 16 || r == 32);
    }
    template <int s>
    __device__ __forceinline__ void compute_and_write(float2* sm, const float2* __restrict__ tw) {
        using G = Geo<C, s>;
        constexpr int V = G::V, r = G::r, Ls = G::Ls;
        if constexpr (V >= 2) {
            static_for<0, V / 2>([&](auto h_) {
                constexpr int v = 2 * decltype(h_)::value;
                float2 a[r], b[r];
                static_for<0, r>([&](auto j_) {
                    constexpr int j = decltype(j_)::value;
                    a[j] = x[j * V + v];
                    b[j] = x[j * V + v + 1];
                });
                const int lo0 = (C::template cidx<V>(t, v, rank) / W) % Ls;
                const float2* row = tw + C::tw_off(s) + lo0;
                G g;
                g.init(t, v, rank);
                dft_composite_emit2<r, Split<r>::A, Split<r>::B>(a, b, [&](auto k_, float2 pa, float2 pb) {
                    constexpr int k = decltype(k_)::value;
                    if constexpr (k > 0) {
                        if constexpr (W == 1) {
                            const float4 w = __ldg(reinterpret_cast<const float4*>(row + (k - 1) * Ls));
                            pa = cmul(pa, make_float2(w.x, w.y));
                            pb = cmul(pb, make_float2(w.z, w.w));
                        } else {
                            const float2 w = __ldg(row + (k - 1) * Ls);
                            pa = cmul(pa, w);
                            pb = cmul(pb, w);
                        }
                    }
                    *reinterpret_cast<float4*>(sm + g.template elem<k>()) = make_float4(pa.x, pa.y, pb.x, pb.y);
                });
            });
        } else {
            const int lo0 = (C::template cidx<1>(t, 0, rank) / W) % Ls;
            const float2* row = tw + C::tw_off(s) + lo0;
            G g;
            g.init(t, 0, rank);
            dft_composite_emit1<r, Split<r>::A, Split<r>::B>(x, [&](auto k_, float2 pa) {
                constexpr int k = decltype(k_)::value;
                if constexpr (k > 0) pa = cmul(pa, __ldg(row + (k - 1) * Ls));
                sm[g.template elem<k>()] = pa;
            });
        }
    }

    // ---- global access with the stage-1 mapping (natural-order positions) --------------
    // position of register (j, v): p = j * L1 + lo; rows: index base + p (+1 for v odd);
    // columns: index base + p * ld + q.
    template <class ST, bool CONJ>
    __device__ __forceinline__ void load_first(const void* in, int64_t base, int64_t ld) {
        using G = Geo<C, 1>;
        constexpr int V = G::V, r = G::r;
        if constexpr (V == 1) {     // radix = values per thread: one butterfly per thread, 64-bit loads,
                                    // still one contiguous run per warp
            const int c = C::template cidx<1>(t, 0, rank);
            const int q = c % W, lo = c / W;
            static_for<0, r>([&](auto i_) {
                constexpr int j = fetch_order<r>(decltype(i_)::value);
                const int64_t idx = (W == 1) ? base + j * G::Ls + lo : base + (int64_t)(j * G::Ls + lo) * ld + q;
                x[j] = ST::load1(in, idx);
                if constexpr (CONJ) x[j].y = -x[j].y;
            });
        }
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            const int c = C::template cidx<V>(t, v, rank);
            const int q = c % W, lo = c / W;
            static_for<0, r>([&](auto i_) {
                constexpr int j = fetch_order<r>(decltype(i_)::value);
                const int64_t idx = (W == 1) ? base + j * G::Ls + lo : base + (int64_t)(j * G::Ls + lo) * ld + q;
                ST::load2(in, idx, x[j * V + v], x[j * V + v + 1]);
                if constexpr (CONJ) {
                    x[j * V + v].y = -x[j * V + v].y;
                    x[j * V + v + 1].y = -x[j * V + v + 1].y;
                }
            });
        });
    }
    template <class ST, bool CONJ>
    __device__ __forceinline__ void store_first(void* out, int64_t base, int64_t ld, float scale) {
        using G = Geo<C, 1>;
        constexpr int V = G::V, r = G::r;
        static_assert(V >= 2, "store_first writes register pairs");
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            const int c = C::template cidx<V>(t, v, rank);
            const int q = c % W, lo = c / W;
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const int64_t idx = (W == 1) ? base + j * G::Ls + lo : base + (int64_t)(j * G::Ls + lo) * ld + q;
                float2 a = x[j * V + v], b = x[j * V + v + 1];
                a = make_float2(a.x * scale, (CONJ ? -a.y : a.y) * scale);
                b = make_float2(b.x * scale, (CONJ ? -b.y : b.y) * scale);
                ST::store2(out, idx, a, b);
            });
        });
    }
    // output index (low part) and column of butterfly pair v of the last stage
    __device__ __forceinline__ void last_index(int v, int& b0, int& q) const {
        Geo<C, S> g;
        g.init(t, v, rank);
        b0 = g.lo;
        q = C::template cidx<Geo<C, S>::V>(t, v, rank) % W;
    }
    // ---- global store with the last-stage mapping: X[b0 + (N / r_S) j] ---------------------
    template <class ST, bool CONJ>
    __device__ __forceinline__ void store_last(void* out, int64_t base, int64_t ld, float scale) {
        // the unnormalised forward transform (scale 1) skips the two multiplications per value
        if (scale == 1.0f) store_last_impl<ST, CONJ, false>(out, base, ld, scale);
        else store_last_impl<ST, CONJ, true>(out, base, ld, scale);
    }
    template <class ST, bool CONJ, bool SCALE>
    __device__ __forceinline__ void store_last_impl(void* out, int64_t base, int64_t ld, float scale) {
        using G = Geo<C, S>;
        constexpr int V = G::V, r = G::r;
        constexpr int KS = C::N / r;
        if constexpr (V == 1) {     // one butterfly per thread: 64-bit stores, one contiguous run per warp
            int b0, q;
            last_index(0, b0, q);
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                float2 a = x[j];
                if constexpr (CONJ) a.y = -a.y;
                if constexpr (SCALE) a = make_float2(a.x * scale, a.y * scale);
                ST::store1(out, base + j * KS + b0, a);
            });
        }
        static_for<0, V / 2>([&](auto h_) {
            constexpr int v = 2 * decltype(h_)::value;
            int b0, q;
            last_index(v, b0, q);
            static_for<0, r>([&](auto j_) {
                constexpr int j = decltype(j_)::value;
                const int64_t idx = (W == 1) ? base + j * KS + b0 : base + (int64_t)(j * KS + b0) * ld + q;
                float2 a = x[j * V + v], b = x[j * V + v + 1];
                if constexpr (CONJ) {
                    a.y = -a.y;
                    b.y = -b.y;
                }
                if constexpr (SCALE) {
                    a = make_float2(a.x * scale, a.y * scale);
                    b = make_float2(b.x * scale, b.y * scale);
                }
                ST::store2(out, idx, a, b);
            });
        });
    }

    // Stage 1 of the backward network and the natural-order global store in one.
    template <class ST, bool CONJ>
    __device__ __forceinline__ void first_stage_dit_and_store(const float2* __restrict__ tw, void* out, int64_t base, int64_t ld,
                                                              float scale) {
        first_stage_dit_and_store_at<ST, CONJ>(tw, out, scale, [&](int p, int q) -> int64_t {
            return (W == 1) ? base + p : base + (int64_t)p * ld + q;
        });
    }
    // The same with the caller's map from (position p, column q) of a register pair to the element index
    // where the pair (positions p, p + 1 of a row tile; columns q, q + 1 of a column tile) is stored.
    template <class ST, bool CONJ, class Index>
    __device__ __forceinline__ void first_stage_dit_and_store_at(const float2* __restrict__ tw, void* out, float scale,
                                                                 Index&& index) {
        first_stage_dit_emit<CONJ>(tw, scale, [&](int p, int q, float2 pa, float2 pb) { ST::store2(out, index(p, q), pa, pb); });
    }
    // The same, handing every finished pair (position p, column q, the two values) to the caller's `emit`.
    template <bool CONJ, class Emit>
    __device__ __forceinline__ void first_stage_dit_emit(const float2* __restrict__ tw, float scale, Emit&& emit) {
        using G = Geo<C, 1>;
        constexpr int V = G::V;
        static_assert(V >= 2, "register pairs");
        compute<1, true>(tw, [&](auto v_, auto k_, float2 pa, float2 pb) {
            constexpr int v = decltype(v_)::value, k = decltype(k_)::value;
            const int c = C::template cidx<V>(t, v, rank);
            const int q = c % W, lo = c / W;
            pa = make_float2(pa.x * scale, (CONJ ? -pa.y : pa.y) * scale);
            pb = make_float2(pb.x * scale, (CONJ ? -pb.y : pb.y) * scale);
            emit(k * G::Ls + lo, q, pa, pb);
        });
    }

    // Last stage and global store in one: every output pair is stored as soon as it is final.
    template <class ST, bool CONJ>
    __device__ __forceinline__ void last_stage_and_store(void* out, int64_t base, int64_t ld, float scale) {
        using G = Geo<C, S>;
        constexpr int V = G::V, r = G::r, KS = C::N / r;
        if constexpr (V >= 2 && (r == 8 || r == 16 || r == 32)) {
            const bool scaled = scale != 1.0f;
            static_for<0, V / 2>([&](auto h_) {
                constexpr int v = 2 * decltype(h_)::value;
                int b0, q;
                last_index(v, b0, q);
                float2 a[r], b[r];
                static_for<0, r>([&](auto j_) {
                    constexpr int j = decltype(j_)::value;
                    a[j] = x[j * V + v];
                    b[j] = x[j * V + v + 1];
                });
                dft_composite_emit2<r, Split<r>::A, Split<r>::B>(a, b, [&](auto k_, float2 pa, float2 pb) {
                    constexpr int k = decltype(k_)::value;
                    const int64_t idx = (W == 1) ? base + k * KS + b0 : base + (int64_t)(k * KS + b0) * ld + q;
                    if constexpr (CONJ) {
                        pa.y = -pa.y;
                        pb.y = -pb.y;
                    }
                    if (scaled) {
                        pa = make_float2(pa.x * scale, pa.y * scale);
                        pb = make_float2(pb.x * scale, pb.y * scale);
                    }
                    ST::store2(out, idx, pa, pb);
                });
            });
        } else if constexpr (V == 1 && W == 1 && (r == 8 || r == 16 || r == 32)) {
            const bool scaled = scale != 1.0f;
            int b0, q;
            last_index(0, b0, q);
            dft_composite_emit1<r, Split<r>::A, Split<r>::B>(x, [&](auto k_, float2 pa) {
                constexpr int k = decltype(k_)::value;
                if constexpr (CONJ) pa.y = -pa.y;
                if (scaled) pa = make_float2(pa.x * scale, pa.y * scale);
                ST::store1(out, base + k * KS + b0, pa);
            });
        } else {
            compute<S, false>(nullptr);
            store_last<ST, CONJ>(out, base, ld, scale);
        }
    }

    // ---- whole networks ---------------------------------------------------------------
    // registers hold stage-1 layout on entry; on exit they hold the last stage's
    // layout: x[j*V + v] = X[b0 + (N/r_S) j] for butterfly pair v (digit-reversed positions)
    template <bool LAST_COMPUTE = true>
    __device__ __forceinline__ void dif(float2* sm, const float2* __restrict__ tw) {
        static_for<1, S + 1>([&](auto s_) {
            constexpr int s = decltype(s_)::value;
            if constexpr (fused_write_ok<s>()) {
                compute_and_write<s>(sm, tw);
                __syncthreads();
                smem_rw<s + 1, false>(sm);
            } else {
                if constexpr (s < S || LAST_COMPUTE) compute<s, false>(tw);
                if constexpr (s < S) {
                    if constexpr (CL > 1 && s == 1) cluster_wait();   // pairs with the arrive in setup()
                    smem_rw<s, true>(sm);
                    exchange_barrier<(CL > 1 && s == 1)>();
                    smem_rw<s + 1, false>(sm);
                }
            }
        });
    }
    // registers hold the last stage's layout (digit-reversed positions) on entry,
    // stage-1 layout in natural order on exit
    template <bool LAST_COMPUTE = true>
    __device__ __forceinline__ void dit(float2* sm, const float2* __restrict__ tw) {
        static_assert(CL == 1, "the backward network is built for single-CTA tiles");
        static_for<0, S>([&](auto i_) {
            constexpr int s = S - decltype(i_)::value;
            // Make the thread index opaque again at every stage: otherwise the compiler keeps
            // the address arithmetic of the forward network alive for reuse here and spills.
            asm volatile("" : "+r"(t));
            if constexpr (s > 1 || LAST_COMPUTE) compute<s, true>(tw);
            if constexpr (s > 1) {
                smem_rw<s, true>(sm);
                __syncthreads();
                smem_rw<s - 1, false>(sm);
            }
        });
    }
};

struct FftArgs {
    const void* in;
    void* out;
    const float2* tw;
    int64_t tiles;   // rows: batch; columns: batch / W
    int64_t dist;    // rows: elements between transforms; columns: elements between rows (ld)
    float scale;
    int prefetch_ahead;   // rows: tiles ahead whose input one thread asks L2 to fetch (0 = off)
    // Column tiles of a slab image (see slab_index): tpg = tiles per slab, slab_stride = elements per
    // slab, dist = columns per slab. tpg == 0: a plain row-major matrix (tile t starts at column t * W).
    int64_t tpg = 0, slab_stride = 0;
    // Output geometry where it differs from the input's (out_dist == 0: the same as the input's).
    int64_t out_dist = 0, out_tpg = 0, out_slab_stride = 0;
    // Kernels that wait on asynchronous copies: polls before a wait gives up (0 = the default), and a test
    // knob that makes the consumer wait on a barrier nothing ever completes, so that the give-up path runs.
    int wait_polls = 0, starve_wait = 0;
};

// Slab layout of an image with `rows` rows and G columns per granule: columns are grouped G at a time
// and every group (slab) is stored as its own contiguous rows x G matrix, so that the element of row k
// and column n lives at ((n / G) * rows + k) * G + n % G. A tile of W <= G adjacent columns is then
// row segments at a pitch of G elements inside one contiguous slab.
__host__ __device__ __forceinline__ int64_t slab_index(int64_t k, int64_t n, int64_t rows, int g) {
    return ((n / g) * rows + k) * g + (n % g);
}
// first element of column tile `tile` (W columns wide)
__device__ __forceinline__ int64_t column_tile_base(int64_t tile, int w, int64_t tpg, int64_t slab_stride) {
    return tpg ? (tile / tpg) * slab_stride + (tile % tpg) * w : tile * w;
}

// Ask L2 to start fetching `bytes` contiguous bytes (a multiple of 16, 16-byte aligned).
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, unsigned bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// One CTA = G tiles, or one cluster of CL CTAs = one tile. INV: inverse via
// conj(FFT(conj(x))) * scale.
template <class C, bool INV, class TIn, class TOut>
__global__ void __launch_bounds__(C::THREADS, C::MINB) fft_kernel(const FftArgs a) {
    extern __shared__ __align__(16) float2 smem_dyn[];
    const int g = threadIdx.x / C::T, t = threadIdx.x % C::T;
    int64_t tile = (C::CL > 1) ? (int64_t)(blockIdx.x / C::CL) : (int64_t)blockIdx.x * C::G + g;
    const bool active = tile < a.tiles;
    if (!active) tile = a.tiles - 1;          // keep the barriers uniform; results discarded
    float2* sm = smem_dyn + g * C::LOCAL_ELEMS;
    const int64_t base = (C::W == 1) ? tile * a.dist : column_tile_base(tile, C::W, a.tpg, a.slab_stride);
    int64_t obase = base, odist = a.dist;
    if constexpr (C::W > 1) {
        if (a.out_dist) {
            obase = column_tile_base(tile, C::W, a.out_tpg, a.out_slab_stride);
            odist = a.out_dist;
        }
    }
    Engine<C> e;
    e.setup(t);
    if constexpr (C::W == 1 && C::G == 1) {
        // A large tile leaves room for one or two CTAs per SM, so nothing overlaps this CTA's
        // load phase. One thread asks L2 for the input of the tile that will run where this
        // one runs now, some CTAs later; that tile's loads then hit L2. (Each CTA of a cluster
        // asks for its share of the transform.)
        constexpr unsigned SHARE = (unsigned)(C::N / C::CL * TIn::ELEM_BYTES);
        if (a.prefetch_ahead > 0 && threadIdx.x == 0 && tile + a.prefetch_ahead < a.tiles)
            prefetch_l2_bulk(reinterpret_cast<const char*>(a.in) + (tile + a.prefetch_ahead) * a.dist * TIn::ELEM_BYTES +
                                 (size_t)e.rank * SHARE,
                             SHARE);
    }
    e.template load_first<TIn, INV>(a.in, base, a.dist);
    e.template dif<false>(sm, a.tw);
    if (active) e.template last_stage_and_store<TOut, INV>(a.out, obase, odist, a.scale);
}

// Builds the per-stage twiddle rows of a configuration in float64, rounds once to fp32:
// row (k-1) of stage s holds exp(-2 pi i lo k / L_{s-1}), lo = 0 .. L_s - 1.
template <class C>
__global__ void build_twiddles_kernel(float2* tw) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= C::TW_TOTAL) return;
    int s = 1;
    static_for<1, C::S>([&](auto s_) {
        constexpr int ss = decltype(s_)::value;
        if (i >= C::tw_off(ss)) s = ss;
    });
    int off = 0, Ls = 1, Lp = 1;
    static_for<1, C::S>([&](auto s_) {
        constexpr int ss = decltype(s_)::value;
        if (s == ss) {
            off = C::tw_off(ss);
            Ls = C::L(ss);
            Lp = C::L(ss - 1);
        }
    });
    const int k = (i - off) / Ls + 1, lo = (i - off) % Ls;
    const int m = (lo * k) % Lp;                    // exact integer angle index
    double sn, cs;
    sincospi(-2.0 * (double)m / (double)Lp, &sn, &cs);
    tw[i] = make_float2((float)cs, (float)sn);
}

}  // namespace b200fft
