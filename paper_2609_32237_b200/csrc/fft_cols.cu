// Single-pass FFT along the columns of a row-major matrix: one tile = W adjacent
// columns, so every row of the tile is one contiguous W*8-byte segment in memory.
#include "configs.h"
#include "registry.h"

namespace b200fft {

static const KernelEntry k_cols[] = {
    B200FFT_ENTRIES_STD(T256),  B200FFT_ENTRIES_STD(T512),  B200FFT_ENTRIES_STD(T1024),
    B200FFT_ENTRIES_STD(T2048), B200FFT_ENTRIES_STD(T4096), B200FFT_ENTRIES_STD(T8192),
    B200FFT_ENTRIES_STD(T2048x2), B200FFT_ENTRIES_STD(T4096x2), B200FFT_ENTRIES_STD(T4096x4),
    B200FFT_ENTRIES_STD(T8192x2),
};

static int default_cluster(int n) { return 1; }

const KernelEntry* find_cols_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl) {
    if (cl == 0) cl = default_cluster(n);
    for (const KernelEntry& e : k_cols)
        if (e.n == n && e.cl == cl && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
    return nullptr;
}

}  // namespace b200fft
