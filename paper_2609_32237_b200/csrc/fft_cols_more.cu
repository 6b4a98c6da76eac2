// Column tiles on thread-block clusters, and wide column tiles for the shorter transforms.
#include "configs.h"
#include "registry.h"

namespace b200fft {

// Wide tiles (16 columns: whole 128-byte row segments; 8 at n = 1024) for the shorter transforms, taken
// by default when the batch is a multiple of the tile width. Measured on B200 for a 128 MiB matrix,
// complex64 / fp16 storage: n = 256: 64 -> 54 us / 58 -> 37 us; n = 512: 70 -> 62 us; n = 1024: 74 -> 68 us /
// 74 -> 55 us. At n = 2048 an 8-column tile fills the SM and gains nothing (80 us either way).
template <class C, bool INV, class TS>
constexpr KernelEntry make_var_entry(int variant) {
    KernelEntry e = make_entry<C, INV, TS, TS>();
    e.variant = variant;
    return e;
}
#define B200FFT_ENTRIES_VAR(C, V)                                                           \
    make_var_entry<C, false, StoreC64>(V), make_var_entry<C, true, StoreC64>(V),           \
    make_var_entry<C, false, StoreC32H>(V), make_var_entry<C, true, StoreC32H>(V)

static const KernelEntry k_cols_more[] = {
    B200FFT_ENTRIES_STD(T2048x2), B200FFT_ENTRIES_STD(T4096x2), B200FFT_ENTRIES_STD(T4096x4), B200FFT_ENTRIES_STD(T8192x2),
    B200FFT_ENTRIES_VAR(F64, VAR_WIDE),     B200FFT_ENTRIES_VAR(F128, VAR_WIDE),
    B200FFT_ENTRIES_VAR(F256, VAR_WIDE),    B200FFT_ENTRIES_VAR(F512, VAR_WIDE),    B200FFT_ENTRIES_VAR(F1024, VAR_WIDE),
    B200FFT_ENTRIES_VAR(T4096w8x2, VAR_WIDE_CLUSTER), B200FFT_ENTRIES_VAR(T8192w4x2, VAR_WIDE_CLUSTER),
    B200FFT_ENTRIES_VAR(T2048w16x2, VAR_WIDE_CLUSTER),
};

EntryList cols_entries_more() { return EntryList{k_cols_more, (int)(sizeof(k_cols_more) / sizeof(k_cols_more[0]))}; }

}  // namespace b200fft
