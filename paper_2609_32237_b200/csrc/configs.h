// Radix factorisations of the compiled sizes. Cfg<N, W, P, G, CL, r1, r2, r3, r4>:
// N points, W transforms per tile, P values per thread, G tiles per CTA, CL CTAs
// (one thread-block cluster) sharing a tile through distributed shared memory.
#pragma once
#include "fft_core.cuh"

namespace b200fft {

// contiguous rows, one transform per tile
// (the three smallest keep 16 values per thread: 8, 4 and 2 threads per transform)
using R128 = Cfg<128, 1, 16, 16, 1, 16, 8>;
using R64 = Cfg<64, 1, 16, 32, 1, 8, 8>;
using R32 = Cfg<32, 1, 16, 64, 1, 4, 8>;
// below the paper's range: one thread per transform (16 = 4 x 4, 8 = 2 x 4), 128 transforms per CTA
using R16 = Cfg<16, 1, 16, 128, 1, 4, 4>;
using R8 = Cfg<8, 1, 8, 128, 1, 2, 4>;
using R256 = Cfg<256, 1, 32, 16, 1, 16, 16>;
using R512 = Cfg<512, 1, 32, 8, 1, 16, 32>;
using R1024 = Cfg<1024, 1, 32, 4, 1, 32, 32>;
// for kernels that work on register pairs at both ends of the network (fused range compression)
using R1024p = Cfg<1024, 1, 32, 4, 1, 16, 4, 16>;
using R2048 = Cfg<2048, 1, 32, 2, 1, 16, 8, 16>;
using R4096 = Cfg<4096, 1, 32, 1, 1, 16, 16, 16>;
using R8192 = Cfg<8192, 1, 32, 1, 1, 16, 32, 16>;
// 16384 = 32 x 32 x 16: two exchanges instead of three; its radix-32 first stage has one
// butterfly per thread, so the global loads are 64 bits per thread (still one contiguous
// run per warp); measured 6-10 % faster than 16 x 4 x 16 x 16, which stays as a test knob
using R16384 = Cfg<16384, 1, 32, 1, 1, 32, 32, 16, 1, 4>;   // 4 of the 31 first-stage twiddle rows loaded
using R16384s4 = Cfg<16384, 1, 32, 1, 1, 16, 4, 16, 16>;
// the same transforms split over a cluster of 2 or 4 CTAs (smaller tiles per SM, more CTAs resident)
using R8192x2 = Cfg<8192, 1, 32, 1, 2, 16, 32, 16>;
using R8192x4 = Cfg<8192, 1, 32, 1, 4, 16, 32, 16>;
using R16384x2 = Cfg<16384, 1, 32, 1, 2, 32, 32, 16, 1, 4>;
using R16384x4 = Cfg<16384, 1, 32, 1, 4, 32, 32, 16, 1, 4>;
// past the single-CTA limit: one 32768-point transform over a cluster of 2 CTAs of 16384 points each, still
// one pass over main memory (the first exchange goes through distributed shared memory). Measured on B200
// against the two-pass split: 609 against 706 us for 4096 transforms, 16.8 against 21.2 us for 64, and no
// workspace (32 x 32 x 32: the last stage has one butterfly per thread and stores 64 bits per lane; the
// four-stage 32 x 4 x 16 x 16 took 693 us). The same with 4 CTAs at 65536 points (32 x 8 x 16 x 16) and 8 CTAs
// at 131072 (32 x 16 x 16 x 16) is correct but slower than two passes (876 against 745 us, 1134 against 831 us)
// and is not compiled.
using R32768x2 = Cfg<32768, 1, 32, 1, 2, 32, 32, 32, 1, 4>;
// the same with every first-stage twiddle row loaded from the table instead of computed
using R4096t15 = Cfg<4096, 1, 32, 1, 1, 16, 16, 16, 1, 15>;


// W adjacent columns (or rows, in the second pass of the two-pass split) per tile
using T64 = Cfg<64, 4, 32, 16, 1, 16, 4>;
using T128 = Cfg<128, 4, 32, 8, 1, 16, 8>;
using T256 = Cfg<256, 4, 32, 4, 1, 16, 16>;
using T512 = Cfg<512, 4, 32, 2, 1, 16, 2, 16>;
using T1024 = Cfg<1024, 4, 32, 1, 1, 16, 4, 16>;
using T2048 = Cfg<2048, 4, 32, 1, 1, 16, 8, 16>;
using T4096 = Cfg<4096, 4, 32, 1, 1, 16, 16, 16>;
using T8192 = Cfg<8192, 2, 32, 1, 1, 16, 32, 16>;
// two columns per tile: half the on-chip footprint of the 4-column tiles, so that two or three CTAs share a
// multiprocessor (used on the slab layout of the SAR chain, where a 16-byte row segment is half a granule)
using S1024 = Cfg<1024, 2, 32, 4, 1, 16, 4, 16>;
using S2048 = Cfg<2048, 2, 32, 2, 1, 16, 8, 16>;
using S4096 = Cfg<4096, 2, 32, 1, 1, 16, 16, 16>;
// wide tiles for the first pass of the two-pass split: whole 128-byte (or 64-byte) row segments
using F64 = Cfg<64, 16, 32, 4, 1, 16, 4>;
using F128 = Cfg<128, 16, 32, 2, 1, 16, 8>;
using F256 = Cfg<256, 16, 32, 1, 1, 16, 16>;
using F512 = Cfg<512, 16, 32, 1, 1, 16, 2, 16>;
using F1024 = Cfg<1024, 8, 32, 1, 1, 16, 4, 16>;
using T2048x2 = Cfg<2048, 4, 32, 1, 2, 16, 8, 16>;
using T4096x2 = Cfg<4096, 4, 32, 1, 2, 16, 16, 16>;
using T4096x4 = Cfg<4096, 4, 32, 1, 4, 16, 16, 16>;
using T8192x2 = Cfg<8192, 2, 32, 1, 2, 16, 32, 16>;
// wider tiles shared by a cluster of two CTAs (16384 points each): 64-byte row segments at n = 4096, 32-byte at 8192
using T4096w8x2 = Cfg<4096, 8, 32, 1, 2, 16, 16, 16>;
using T8192w4x2 = Cfg<8192, 4, 32, 1, 2, 16, 32, 16>;
using T2048w16x2 = Cfg<2048, 16, 32, 1, 2, 16, 8, 16>;

}  // namespace b200fft
