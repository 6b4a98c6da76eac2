// Single-pass row kernels, N = 8 .. 2048 (several transforms per CTA).
#include "configs.h"
#include "registry.h"

namespace b200fft {

static const KernelEntry k_rows_small[] = {
    B200FFT_ENTRIES_STD(R8),    B200FFT_ENTRIES_STD(R16),
    B200FFT_ENTRIES_STD(R32),   B200FFT_ENTRIES_STD(R64),   B200FFT_ENTRIES_STD(R128), B200FFT_ENTRIES_STD(R256),
    B200FFT_ENTRIES_STD(R512),  B200FFT_ENTRIES_STD(R1024), B200FFT_ENTRIES_STD(R2048),
};

EntryList rows_entries_small() { return EntryList{k_rows_small, (int)(sizeof(k_rows_small) / sizeof(k_rows_small[0]))}; }

}  // namespace b200fft
