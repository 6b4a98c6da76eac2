// Row transforms shared by a thread-block cluster of 2 or 4 CTAs through distributed shared memory.
#include "configs.h"
#include "registry.h"

namespace b200fft {

static const KernelEntry k_rows_cluster[] = {
    B200FFT_ENTRIES_STD(R8192x2),  B200FFT_ENTRIES_STD(R8192x4), B200FFT_ENTRIES_STD(R16384x2),
    B200FFT_ENTRIES_STD(R16384x4), B200FFT_ENTRIES_STD(R32768x2),
};

EntryList rows_entries_cluster() { return EntryList{k_rows_cluster, (int)(sizeof(k_rows_cluster) / sizeof(k_rows_cluster[0]))}; }

}  // namespace b200fft
