// Single-pass row kernels, N = 4096 .. 16384 (one transform per CTA), and the alternative
// factorisations kept as test knobs (variants VAR_TW_TABLE, VAR_FOUR_STAGE).
#include "configs.h"
#include "registry.h"

namespace b200fft {

template <class C, bool INV, class TI, class TO>
constexpr KernelEntry make_alt_entry(int knob) {
    KernelEntry e = make_entry<C, INV, TI, TO>();
    e.variant = knob;
    return e;
}
#define B200FFT_ENTRIES_ALT(C, K)                                                                      \
    make_alt_entry<C, false, StoreC64, StoreC64>(K), make_alt_entry<C, true, StoreC64, StoreC64>(K),  \
    make_alt_entry<C, false, StoreC32H, StoreC32H>(K), make_alt_entry<C, true, StoreC32H, StoreC32H>(K)

static const KernelEntry k_rows_large[] = {
    B200FFT_ENTRIES_STD(R4096), B200FFT_ENTRIES_STD(R8192), B200FFT_ENTRIES_STD(R16384),
    B200FFT_ENTRIES_ALT(R4096t15, VAR_TW_TABLE), B200FFT_ENTRIES_ALT(R16384s4, VAR_FOUR_STAGE),
};

EntryList rows_entries_large() { return EntryList{k_rows_large, (int)(sizeof(k_rows_large) / sizeof(k_rows_large[0]))}; }

}  // namespace b200fft
