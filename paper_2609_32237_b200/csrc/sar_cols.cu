// Column-tile kernels of the SAR chain on the slab layout: tiles of 2 and of 4 range bins; forward with the
// intermediate type on both sides, inverse from the intermediate type to the complex64 image.
#include "configs.h"
#include "registry.h"

namespace b200fft {

#define SAR_COLS(C)                                                                        \
    make_entry<C, false, StoreC64, StoreC64>(), make_entry<C, false, StoreC32H, StoreC32H>(), \
    make_entry<C, true, StoreC64, StoreC64>(), make_entry<C, true, StoreC32H, StoreC64>()

static const KernelEntry k_sar_cols[] = {
    SAR_COLS(S1024), SAR_COLS(S2048), SAR_COLS(S4096), SAR_COLS(T1024), SAR_COLS(T2048), SAR_COLS(T4096),
};

const KernelEntry* find_sar_cols_kernel(int n, int w, bool inverse, int in_dtype, int out_dtype) {
    for (const KernelEntry& e : k_sar_cols)
        if (e.n == n && e.w == w && e.cl == 1 && e.inverse == inverse && e.in_dtype == in_dtype && e.out_dtype == out_dtype)
            return &e;
    return nullptr;
}

}  // namespace b200fft
