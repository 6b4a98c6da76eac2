// fft_execute_noalloc: a batched transform for callers that must not allocate.
//
// Who needs this: a processing loop that runs beside other GPU work and cannot
// afford the device-wide stall that cudaMalloc / cudaFree may cause; a process
// that has already handed all device memory to its own pool, where a late
// cudaMalloc would fail; an embedded deployment whose memory budget is fixed at
// load time. For them the two-pass transform's scratch image and its twiddle
// tables live in one file-scope device array of fixed size, which every GPU that
// loads this library holds until the process exits. The caller still passes the
// input and output buffers. The paper has no counterpart to this entry point.
#include <cuda_runtime.h>
#include "../../include/b200fft.h"
#include "fourstep.h"
#include "registry.h"

namespace b200fft {

// Scratch image: at most B200FFT_NOALLOC_MAX_ELEMS complex64 elements (2 MiB).
// Table region behind it: the largest table set of any supported size.
constexpr size_t kNoallocImageElems = B200FFT_NOALLOC_MAX_ELEMS;
constexpr size_t kNoallocTableElems = 8192;
static __device__ __align__(256) float2 g_noalloc_scratch[kNoallocImageElems + kNoallocTableElems];

// Device address of the array above, per device. In host code the array's name is
// only a handle; cudaGetSymbolAddress turns it into the pointer kernels can use.
static float2* g_noalloc_ptr[64] = {};

static int noalloc_scratch(float2** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return B200FFT_ERR_CUDA;
    if (dev < 0 || dev >= 64) return B200FFT_ERR_CUDA;
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return B200FFT_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = static_cast<float2*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return B200FFT_OK;
}

}  // namespace b200fft

using namespace b200fft;

extern "C" int fft_execute_noalloc(int64_t n, int64_t batch, int direction, const void* in, void* out,
                                   void* stream) {
    if (!in || !out || n <= 0 || batch <= 0) return B200FFT_ERR_INVALID_ARG;
    if (direction != B200FFT_FORWARD && direction != B200FFT_INVERSE) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(in) % 16 || reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
    const size_t tables = fourstep_table_elems(n, direction, B200FFT_C64);
    if (tables == 0) return B200FFT_ERR_UNSUPPORTED;            // n not a power of two in 2^12 .. 2^20
    if ((size_t)n > kNoallocImageElems || (size_t)batch > kNoallocImageElems / (size_t)n ||
        tables > kNoallocTableElems)
        return B200FFT_ERR_WORKSPACE;                            // beyond the fixed scratch: use a plan instead
    float2* scratch = nullptr;
    int rc = noalloc_scratch(&scratch);
    if (rc != B200FFT_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents. Nothing has to start at zero:
    // the tables are rebuilt for this n on this stream, and pass 1 overwrites every
    // scratch element that pass 2 reads.
    FourStep fs;
    rc = fourstep_build_in_place(&fs, n, batch, n, direction, B200FFT_C64, scratch + kNoallocImageElems,
                                 kNoallocTableElems, st);
    if (rc != B200FFT_OK) return rc;
    return fourstep_execute(&fs, in, out, scratch, st);
}
