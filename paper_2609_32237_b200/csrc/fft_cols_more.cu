// Column tiles on thread-block clusters, and wide column tiles for the shorter transforms.
#include "configs.h"
#include "registry.h"

namespace b200fft {

// Wide tiles (16 columns: whole 128-byte row segments; 8 at n = 1024) for the shorter transforms, taken
// by default when the batch is a multiple of the tile width. Measured on B200 for a 128 MiB matrix,
// complex64 / fp16 storage: n = 256: 64 -> 54 us / 58 -> 37 us; n = 512: 70 -> 62 us; n = 1024: 74 -> 68 us /
// 74 -> 55 us. At n = 2048 an 8-column tile fills the SM and gains nothing (80 us either way).
static const KernelEntry k_cols_more[] = {
    B200FFT_ENTRIES_STD(T2048x2), B200FFT_ENTRIES_STD(T4096x2), B200FFT_ENTRIES_STD(T4096x4), B200FFT_ENTRIES_STD(T8192x2),
    B200FFT_ENTRIES_STD(F64),     B200FFT_ENTRIES_STD(F128),
    B200FFT_ENTRIES_STD(F256),    B200FFT_ENTRIES_STD(F512),    B200FFT_ENTRIES_STD(F1024),
    B200FFT_ENTRIES_STD(T4096w8x2), B200FFT_ENTRIES_STD(T8192w4x2), B200FFT_ENTRIES_STD(T2048w16x2),
};

EntryList cols_entries_more() { return EntryList{k_cols_more, (int)(sizeof(k_cols_more) / sizeof(k_cols_more[0]))}; }

}  // namespace b200fft
