// Single-pass batched FFT over contiguous rows: one tile = one transform.
#include "configs.h"
#include "registry.h"

namespace b200fft {

static const KernelEntry k_rows[] = {
    B200FFT_ENTRIES_STD(R32),   B200FFT_ENTRIES_STD(R64),   B200FFT_ENTRIES_STD(R128),
    B200FFT_ENTRIES_STD(R256),  B200FFT_ENTRIES_STD(R512),
    B200FFT_ENTRIES_STD(R1024), B200FFT_ENTRIES_STD(R2048), B200FFT_ENTRIES_STD(R4096),
    B200FFT_ENTRIES_STD(R8192), B200FFT_ENTRIES_STD(R16384),
    B200FFT_ENTRIES_STD(R8192x2), B200FFT_ENTRIES_STD(R8192x4),
    B200FFT_ENTRIES_STD(R16384x2), B200FFT_ENTRIES_STD(R16384x4),
};

static const KernelEntry k_rows_alt[] = {B200FFT_ENTRIES_STD(R4096t15), B200FFT_ENTRIES_STD(R16384s4)};

// Small batches leave most SMs idle with one CTA per transform (the paper's "when not to
// use it"): there a transform is split over a cluster of CTAs through distributed shared
// memory. Measured on B200: n = 16384, batch <= 32: 14.3 -> 10.2 us with 4 CTAs per transform;
// n = 8192, batch <= 16: 12.3 -> 10.2 us with 2. Large batches are faster with one CTA.
static int default_cluster(int n, int64_t batch) {
    if (n == 16384 && batch <= 32) return 4;
    if (n == 8192 && batch <= 16) return 2;
    return 1;
}

const KernelEntry* find_rows_kernel(int n, bool inverse, int in_dtype, int out_dtype, int cl, int64_t batch) {
    if (cl == 1015 || cl == 1016) {                   // test knobs: 1015 = all first-stage twiddle rows from
                                                      // the table (n = 4096); 1016 = four-stage n = 16384
        for (const KernelEntry& e : k_rows_alt)
            if (e.n == n && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
        return nullptr;
    }
    if (cl == 0) cl = default_cluster(n, batch);
    for (const KernelEntry& e : k_rows)
        if (e.n == n && e.cl == cl && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype) return &e;
    return nullptr;
}

}  // namespace b200fft
