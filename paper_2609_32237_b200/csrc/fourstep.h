// Two-pass ("four-step") transform for sizes past the single-pass limit.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace b200fft {

struct FourStepEntry;

struct FourStep {
    int64_t n = 0, n1 = 0, n2 = 0, batch = 0, dist = 0;
    int direction = 0, dtype = 0;
    const FourStepEntry* pass1 = nullptr;   // n2*batch column transforms of length n1 + twiddle
    const FourStepEntry* pass2 = nullptr;   // n1*batch row transforms of length n2, transposed store
    float2* tw1 = nullptr;                  // stage twiddles of the two configurations
    float2* tw2 = nullptr;
    float2* tw_lo = nullptr;                // exp(-2 pi i m / n), m = 0..1023
    float2* tw_hi = nullptr;                // exp(-2 pi i 1024 m / n), m = 0..n/1024-1
};

// n1_request = 0: the default split; otherwise n = n1_request * n2 if both passes exist for it.
int fourstep_build(FourStep* fs, int64_t n, int64_t batch, int64_t dist, int direction, int dtype,
                   int64_t n1_request = 0);
int fourstep_execute(const FourStep* fs, const void* in, void* out, void* workspace, cudaStream_t st);
void fourstep_release(FourStep* fs);

// Number of float2 table entries a FourStep of this size needs (0 if unsupported).
size_t fourstep_table_elems(int64_t n, int direction, int dtype);
// Like fourstep_build, but allocates nothing: the four tables are placed in
// caller-provided device memory `tables` (at least fourstep_table_elems entries)
// and built by kernels enqueued on `st`, without synchronising. The FourStep
// must not be passed to fourstep_release.
int fourstep_build_in_place(FourStep* fs, int64_t n, int64_t batch, int64_t dist, int direction, int dtype,
                            float2* tables, size_t table_elems, cudaStream_t st);

}  // namespace b200fft
