// C ABI of the FFT plans: argument validation, variant choice, table ownership.
#include <cuda_runtime.h>
#include <cstring>
#include <new>
#include "../../include/b200fft.h"
#include "registry.h"
#include "fourstep.h"

namespace b200fft {
std::atomic<int64_t> g_launch_count{0};
}

using namespace b200fft;

enum Layout { LAYOUT_ROWS = 0, LAYOUT_COLS = 1 };

struct b200fft_plan_s {
    int64_t n, batch, stride, dist;
    int direction, dtype;
    Layout layout;
    bool four_step;
    int cluster;                 // CTAs per tile requested by the "cluster" option (0 = default)
    int variant;                 // kernel family forced by an option (VAR_PLAIN = the default rules)
    int wait_polls, starve_wait; // test knobs of the kernels that wait on asynchronous copies
    int prefetch_ahead;          // "prefetch" option: tiles ahead to prefetch into L2 (-1 = default)
    bool via_transpose;          // "via_transpose" option (columns): transpose, row transforms, transpose back
    const KernelEntry* rows_kernel;   // its row variant and table
    float2* tw_rows;
    const BfpEntry* bfp;         // block-floating-point variant and its table, built on first use
    float2* tw_bfp;
    int staged;                  // "staged" option: persistent kernel fed by the copy engine (-1 = default)
    int stream;                  // "stream" option (columns): 0 forbids the streaming kernel, -1 = default rules
    const KernelEntry* kernel;   // single-pass variant
    float2* tw;                  // its twiddle rows (device)
    int device;
    int sms;                     // multiprocessors of that device
    FourStep fs;                 // two-pass variant
    void* workspace;
    size_t workspace_bytes;
    // host-buffer path: two copy streams and per-chunk events, created on first use
    static constexpr int kChunks = 16;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_start, ev_done, ev_in[kChunks], ev_k[kChunks];
    bool pipe_ready;
};

static int launch_single_pass(b200fft_plan_s* p, const void* in, void* out, int64_t tiles, cudaStream_t st);

static bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

static int elem_bytes(int dtype) { return dtype == B200FFT_C64 ? 8 : 4; }

static int build_single_pass(b200fft_plan_s* p) {
    const bool inv = p->direction == B200FFT_INVERSE;
    const int cl = p->cluster;
    int variant = p->variant;
    const KernelEntry* k = nullptr;
    if (p->layout == LAYOUT_ROWS && variant == VAR_PLAIN && cl == 0) {
        // Persistent staged kernel: measured on B200 at n = 16384 with fp16 storage, 379 -> 342 us for
        // 8192 transforms; with fp32 storage it is slower than the plain kernel (455 against 447 us:
        // only half of the tile can wait beside the exchange buffer), so there it is only taken on request.
        const bool by_default = p->n == 16384 && p->dtype == B200FFT_C32H && p->batch >= 2 * (int64_t)p->sms;
        if (p->staged == 1 || (p->staged == -1 && by_default)) variant = VAR_STAGED;
        // Transforms of at most 32 points packed back to back: one thread per transform, the CTA's chunk staged
        // through shared memory. Measured for 1 GiB in and 1 GiB out of complex64: 316 us at n = 8, 16 and 32
        // (104 % of the copy peak) against 551, 1010 and 521 us for the plain kernel; fp16 storage 160 us
        // (103 %) against 508 us at n = 32. The same staging for 64 <= n <= 2048 (several threads per
        // transform) measured slower than the plain kernels (fp16 storage: 62 % against 64-92 %).
        if (p->n <= 32 && p->dist == p->n && p->staged != 0) variant = VAR_TINY;
    }
    if (p->layout == LAYOUT_COLS && variant == VAR_PLAIN && cl == 0) {
        // default rules, widest first: 16-column tiles for n <= 1024 where they divide the batch ...
        k = find_cols_kernel((int)p->n, inv, p->dtype, p->dtype, 0, VAR_WIDE);
        if (k && p->batch % k->w) k = nullptr;
        // ... the persistent streaming kernel for tiles that fill a multiprocessor, when there is more than one
        // tile per multiprocessor to overlap ...
        if (!k && p->stream != 0 && p->batch / 4 > p->sms) {
            k = find_cols_kernel((int)p->n, inv, p->dtype, p->dtype, 0, VAR_STREAM);
            if (k && (p->batch % k->w || k->n < 4096)) k = nullptr;
        }
        // ... else a tile twice as wide on a cluster of two CTAs for n >= 2048
        // (measured: n = 2048 complex64 80 us with 4-column tiles against 84 us, fp16 storage 80 -> 70 us)
        if (!k && !(p->n == 2048 && p->dtype == B200FFT_C64)) {
            k = find_cols_kernel((int)p->n, inv, p->dtype, p->dtype, 0, VAR_WIDE_CLUSTER);
            if (k && p->batch % k->w) k = nullptr;
        }
    }
    if (!k)
        k = (p->layout == LAYOUT_ROWS) ? find_rows_kernel((int)p->n, inv, p->dtype, p->dtype, cl, p->batch, variant)
                                       : find_cols_kernel((int)p->n, inv, p->dtype, p->dtype, cl, variant);
    if (!k) return B200FFT_ERR_UNSUPPORTED;
    if (p->layout == LAYOUT_COLS && p->batch % k->w) return B200FFT_ERR_UNSUPPORTED;
    p->kernel = k;                  // the table depends on the factorisation: always rebuilt
    if (p->tw) cudaFree(p->tw);
    p->tw = nullptr;
    if (cudaMalloc(&p->tw, sizeof(float2) * (size_t)p->kernel->tw_total) != cudaSuccess) {
        cudaGetLastError();
        return B200FFT_ERR_ALLOC;
    }
    if (p->kernel->build_tw(p->tw, 0) != cudaSuccess) return B200FFT_ERR_CUDA;
    if (cudaStreamSynchronize(0) != cudaSuccess) return B200FFT_ERR_CUDA;
    return B200FFT_OK;
}

// set one selection field, rebuild, and put the old value back if no such kernel exists
static int reselect(b200fft_plan_s* p, int* field, int value) {
    const int old = *field;
    *field = value;
    int rc = build_single_pass(p);
    if (rc != B200FFT_OK) {
        *field = old;
        build_single_pass(p);
    }
    return rc;
}

static void release(b200fft_plan_s* p) {
    if (p->tw) cudaFree(p->tw);
    p->tw = nullptr;
    if (p->tw_rows) cudaFree(p->tw_rows);
    p->tw_rows = nullptr;
    if (p->tw_bfp) cudaFree(p->tw_bfp);
    p->tw_bfp = nullptr;
    fourstep_release(&p->fs);
    if (p->pipe_ready) {
        cudaStreamDestroy(p->s_in);
        cudaStreamDestroy(p->s_out);
        cudaEventDestroy(p->ev_start);
        cudaEventDestroy(p->ev_done);
        for (int i = 0; i < b200fft_plan_s::kChunks; ++i) {
            cudaEventDestroy(p->ev_in[i]);
            cudaEventDestroy(p->ev_k[i]);
        }
        p->pipe_ready = false;
    }
}

static bool pipe_setup(b200fft_plan_s* p) {
    if (p->pipe_ready) return true;
    bool ok = cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p->ev_start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&p->ev_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < b200fft_plan_s::kChunks; ++i)
        ok = cudaEventCreateWithFlags(&p->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&p->ev_k[i], cudaEventDisableTiming) == cudaSuccess;
    p->pipe_ready = ok;
    return ok;
}

extern "C" int fft_plan_create(fft_plan_t* plan, int64_t n, int64_t batch, int64_t stride,
                               int64_t dist, int direction, int storage_dtype) {
    if (!plan) return B200FFT_ERR_INVALID_ARG;
    *plan = nullptr;
    if (n <= 0 || batch <= 0 || stride <= 0 || dist <= 0) return B200FFT_ERR_INVALID_ARG;
    if (direction != B200FFT_FORWARD && direction != B200FFT_INVERSE) return B200FFT_ERR_INVALID_ARG;
    if (storage_dtype != B200FFT_C64 && storage_dtype != B200FFT_C32H) return B200FFT_ERR_INVALID_ARG;
    if (!is_pow2(n)) return B200FFT_ERR_UNSUPPORTED;
    if (n < 8 || n > (1 << 20)) return B200FFT_ERR_UNSUPPORTED;

    Layout layout;
    if (stride == 1 && dist >= n) layout = LAYOUT_ROWS;
    else if (dist == 1 && stride >= batch) layout = LAYOUT_COLS;
    else return B200FFT_ERR_UNSUPPORTED;
    // 128-bit (c64) or 64-bit (c32h) vector access: two elements at a time
    const int64_t align_elems = (storage_dtype == B200FFT_C64) ? 2 : 4;
    if (layout == LAYOUT_ROWS && dist % align_elems) return B200FFT_ERR_ALIGNMENT;
    if (layout == LAYOUT_COLS && (stride % align_elems || batch % 2)) return B200FFT_ERR_ALIGNMENT;

    b200fft_plan_s* p = new (std::nothrow) b200fft_plan_s();
    if (!p) return B200FFT_ERR_ALLOC;
    p->n = n; p->batch = batch; p->stride = stride; p->dist = dist;
    p->direction = direction; p->dtype = storage_dtype; p->layout = layout;
    p->prefetch_ahead = -1;
    p->staged = -1;
    p->stream = -1;
    p->variant = VAR_PLAIN;
    if (cudaGetDevice(&p->device) != cudaSuccess) { delete p; return B200FFT_ERR_CUDA; }
    p->sms = 148;
    cudaDeviceGetAttribute(&p->sms, cudaDevAttrMultiProcessorCount, p->device);

    int rc;
    if (n == 32768 && layout == LAYOUT_ROWS) {
        rc = build_single_pass(p);              // one pass on a cluster of two CTAs; "four_step" = 1 for the split
    } else if (n > 16384) {
        if (layout != LAYOUT_ROWS) { delete p; return B200FFT_ERR_UNSUPPORTED; }
        p->four_step = true;
        rc = fourstep_build(&p->fs, n, batch, dist, direction, storage_dtype);
    } else {
        if (layout == LAYOUT_COLS) {
            const KernelEntry* k = find_cols_kernel((int)n, false, storage_dtype, storage_dtype);
            if (!k) { delete p; return B200FFT_ERR_UNSUPPORTED; }
            if (batch % k->w) { delete p; return B200FFT_ERR_UNSUPPORTED; }
        }
        rc = build_single_pass(p);
    }
    if (rc != B200FFT_OK) { release(p); delete p; return rc; }
    *plan = p;
    return B200FFT_OK;
}

extern "C" int fft_plan_set_option(fft_plan_t p, const char* key, int64_t value) {
    if (!p || !key) return B200FFT_ERR_INVALID_ARG;
    if (std::strcmp(key, "four_step") == 0) {
        if (p->layout != LAYOUT_ROWS || p->n < 4096) return B200FFT_ERR_UNSUPPORTED;
        if (value && !p->four_step) {
            int rc = fourstep_build(&p->fs, p->n, p->batch, p->dist, p->direction, p->dtype);
            if (rc != B200FFT_OK) return rc;
            p->four_step = true;
            p->workspace = nullptr;
            p->workspace_bytes = 0;
        } else if (!value && p->four_step && p->n <= 32768) {
            if (!p->kernel) {
                int rc = build_single_pass(p);
                if (rc != B200FFT_OK) return rc;
            }
            p->four_step = false;
        }
        return B200FFT_OK;
    }
    if (std::strcmp(key, "split_n1") == 0) {       // two-pass plans: n = n1 * n2 with this n1 (0 = the default split)
        if (!p->four_step || value < 0) return B200FFT_ERR_UNSUPPORTED;
        FourStep fs;
        int rc = fourstep_build(&fs, p->n, p->batch, p->dist, p->direction, p->dtype, value);
        if (rc != B200FFT_OK) return rc;
        fourstep_release(&p->fs);
        p->fs = fs;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "prefetch") == 0) {
        if (value < -1 || value > (1 << 20)) return B200FFT_ERR_INVALID_ARG;
        p->prefetch_ahead = (int)value;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "via_transpose") == 0) {
        if (p->four_step || p->layout != LAYOUT_COLS) return B200FFT_ERR_UNSUPPORTED;
        if (!value) {
            p->via_transpose = false;
            return B200FFT_OK;
        }
        if (!p->rows_kernel) {
            const KernelEntry* k = find_rows_kernel((int)p->n, p->direction == B200FFT_INVERSE, p->dtype, p->dtype, 0, p->batch);
            if (!k) k = find_rows_kernel((int)p->n, p->direction == B200FFT_INVERSE, p->dtype, p->dtype, 1, p->batch);
            if (!k) return B200FFT_ERR_UNSUPPORTED;
            if (cudaMalloc(&p->tw_rows, sizeof(float2) * (size_t)k->tw_total) != cudaSuccess) {
                cudaGetLastError();
                p->tw_rows = nullptr;
                return B200FFT_ERR_ALLOC;
            }
            if (k->build_tw(p->tw_rows, 0) != cudaSuccess || cudaStreamSynchronize(0) != cudaSuccess) return B200FFT_ERR_CUDA;
            p->rows_kernel = k;
        }
        p->via_transpose = true;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "staged") == 0) {
        if (p->four_step || p->layout != LAYOUT_ROWS || value < -1 || value > 1) return B200FFT_ERR_UNSUPPORTED;
        return reselect(p, &p->staged, (int)value);
    }
    if (std::strcmp(key, "stream") == 0 || std::strcmp(key, "tma") == 0) {
        // 1: the persistent streaming column kernel; 0: never; -1: the default rules
        if (p->four_step || p->layout != LAYOUT_COLS || value < -1 || value > 1) return B200FFT_ERR_UNSUPPORTED;
        if (value == 1) {
            int rc = reselect(p, &p->variant, VAR_STREAM);
            if (rc == B200FFT_OK) p->cluster = 0;
            return rc;
        }
        p->variant = VAR_PLAIN;
        return reselect(p, &p->stream, (int)value);
    }
    if (std::strcmp(key, "cluster") == 0) {
        if (p->four_step || p->n > 32768) return B200FFT_ERR_UNSUPPORTED;
        if (value != 0 && value != 1 && value != 2 && value != 4) return B200FFT_ERR_INVALID_ARG;
        p->variant = VAR_PLAIN;
        return reselect(p, &p->cluster, (int)value);
    }
    if (std::strcmp(key, "alt_factorisation") == 0) {
        // test knob: the other compiled factorisation of a rows plan (n = 4096 with every first-stage
        // twiddle row loaded from its table; n = 16384 as 16 x 4 x 16 x 16)
        if (p->four_step || p->layout != LAYOUT_ROWS) return B200FFT_ERR_UNSUPPORTED;
        if (!value) return reselect(p, &p->variant, VAR_PLAIN);
        return reselect(p, &p->variant, p->n == 4096 ? VAR_TW_TABLE : VAR_FOUR_STAGE);
    }
    if (std::strcmp(key, "wait_polls") == 0) {
        if (value < 0 || value > (1 << 30)) return B200FFT_ERR_INVALID_ARG;
        p->wait_polls = (int)value;
        return B200FFT_OK;
    }
    if (std::strcmp(key, "starve_wait") == 0) {
        p->starve_wait = value != 0;
        return B200FFT_OK;
    }
    return B200FFT_ERR_INVALID_ARG;
}

extern "C" int fft_plan_workspace_bytes(fft_plan_t p, size_t* bytes) {
    if (!p || !bytes) return B200FFT_ERR_INVALID_ARG;
    *bytes = (p->four_step || p->via_transpose) ? (size_t)p->n * (size_t)p->batch * (size_t)elem_bytes(p->dtype) : 0;
    return B200FFT_OK;
}

extern "C" int fft_plan_set_workspace(fft_plan_t p, void* ptr, size_t bytes) {
    if (!p) return B200FFT_ERR_INVALID_ARG;
    size_t need = 0;
    fft_plan_workspace_bytes(p, &need);
    if (need == 0) { p->workspace = ptr; p->workspace_bytes = bytes; return B200FFT_OK; }
    if (!ptr) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(ptr) % 16) return B200FFT_ERR_ALIGNMENT;
    if (bytes < need) return B200FFT_ERR_WORKSPACE;
    p->workspace = ptr;
    p->workspace_bytes = bytes;
    return B200FFT_OK;
}

extern "C" int fft_execute(fft_plan_t p, const void* in, void* out, void* stream) {
    if (!p || !in || !out) return B200FFT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(in) % 16 || reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (p->four_step) {
        size_t need = 0;
        fft_plan_workspace_bytes(p, &need);
        if (!p->workspace || p->workspace_bytes < need) return B200FFT_ERR_WORKSPACE;
        return fourstep_execute(&p->fs, in, out, p->workspace, st);
    }
    if (p->via_transpose) {
        size_t need = 0;
        fft_plan_workspace_bytes(p, &need);
        if (!p->workspace || p->workspace_bytes < need) return B200FFT_ERR_WORKSPACE;
        if (p->workspace == in || p->workspace == out) return B200FFT_ERR_INVALID_ARG;
        const int eb = elem_bytes(p->dtype);
        // [n][batch] (row pitch stride) -> [batch][n], transform the rows in place, and back
        if (transpose_launch(in, p->workspace, (int)p->n, (int)p->batch, p->stride, p->n, eb, st) != cudaSuccess)
            return B200FFT_ERR_CUDA;
        FftArgs a;
        a.in = p->workspace;
        a.out = p->workspace;
        a.tw = p->tw_rows;
        a.prefetch_ahead = 0;
        a.scale = (p->direction == B200FFT_INVERSE) ? (float)(1.0 / (double)p->n) : 1.0f;
        a.tiles = p->batch;
        a.dist = p->n;
        if (p->rows_kernel->launch(a, st) != cudaSuccess) return B200FFT_ERR_CUDA;
        if (transpose_launch(p->workspace, out, (int)p->batch, (int)p->n, p->n, p->stride, eb, st) != cudaSuccess)
            return B200FFT_ERR_CUDA;
        return B200FFT_OK;
    }
    return launch_single_pass(p, in, out, p->layout == LAYOUT_ROWS ? p->batch : p->batch / p->kernel->w, st);
}

extern "C" int fft_execute_bfp(fft_plan_t p, const void* in, const int32_t* in_exp, void* out, int32_t* out_exp,
                               void* stream) {
    if (!p || !in || !out || !out_exp) return B200FFT_ERR_INVALID_ARG;
    if (p->layout != LAYOUT_ROWS || p->dtype != B200FFT_C32H || p->four_step) return B200FFT_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(in) % 16 || reinterpret_cast<uintptr_t>(out) % 16) return B200FFT_ERR_ALIGNMENT;
    if (!p->bfp) {
        const BfpEntry* k = find_bfp_kernel((int)p->n, p->direction == B200FFT_INVERSE);
        if (!k) return B200FFT_ERR_UNSUPPORTED;
        if (cudaMalloc(&p->tw_bfp, sizeof(float2) * (size_t)k->tw_total) != cudaSuccess) {
            cudaGetLastError();
            p->tw_bfp = nullptr;
            return B200FFT_ERR_ALLOC;
        }
        if (k->build_tw(p->tw_bfp, 0) != cudaSuccess || cudaStreamSynchronize(0) != cudaSuccess) return B200FFT_ERR_CUDA;
        p->bfp = k;
    }
    FftArgs a;
    a.in = in;
    a.out = out;
    a.tw = p->tw_bfp;
    a.prefetch_ahead = 0;
    a.scale = 1.0f;
    a.tiles = p->batch;
    a.dist = p->dist;
    return p->bfp->launch(a, in_exp, out_exp, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? B200FFT_OK
                                                                                                      : B200FFT_ERR_CUDA;
}

// one launch of the plan's single-pass kernel over `tiles` tiles starting at in/out
static int launch_single_pass(b200fft_plan_s* p, const void* in, void* out, int64_t tiles, cudaStream_t st) {
    FftArgs a;
    a.in = in;
    a.out = out;
    a.tw = p->tw;
    a.prefetch_ahead = 0;
    a.wait_polls = p->wait_polls;
    a.starve_wait = p->starve_wait;
    if (p->layout == LAYOUT_ROWS && p->kernel->variant != VAR_STAGED && p->kernel->g == 1) {
        // default: for tiles that fill an SM (one CTA resident), the tile one full wave ahead;
        // measured on B200: +13 % at n = 16384 rows, nothing to gain at n = 8192 and below,
        // and a loss for column tiles (their time goes to the lock-step compute, not the load)
        const bool fills_sm = p->kernel->smem_bytes > 100 * 1024;
        a.prefetch_ahead = (p->prefetch_ahead >= 0) ? p->prefetch_ahead : (fills_sm ? p->sms / p->kernel->cl : 0);
    }
    a.scale = (p->direction == B200FFT_INVERSE) ? (float)(1.0 / (double)p->n) : 1.0f;
    a.tiles = tiles;
    a.dist = (p->layout == LAYOUT_ROWS) ? p->dist : p->stride;
    return p->kernel->launch(a, st) == cudaSuccess ? B200FFT_OK : B200FFT_ERR_CUDA;
}

extern "C" int fft_execute_host(fft_plan_t p, const void* host_in, void* host_out,
                                void* dev_in, void* dev_out, void* stream) {
    if (!p || !host_in || !host_out || !dev_in || !dev_out) return B200FFT_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t elems = (size_t)((p->batch - 1) * p->dist + (p->n - 1) * p->stride + 1);
    const size_t bytes = elems * (size_t)elem_bytes(p->dtype);
    const int CH = b200fft_plan_s::kChunks;
    if (p->layout == LAYOUT_ROWS && !p->four_step && p->batch >= 4 * CH && bytes >= ((size_t)32 << 20) && pipe_setup(p)) {
        // Large row batches: cut the batch into chunks and overlap the copy in of chunk i+1,
        // the transform of chunk i and the copy out of chunk i-1 (PCIe is full duplex). The
        // caller's stream sees one ordered operation: the copy streams start after everything
        // already on `st`, and `st` ends up waiting for the last copy out.
        if (reinterpret_cast<uintptr_t>(dev_in) % 16 || reinterpret_cast<uintptr_t>(dev_out) % 16) return B200FFT_ERR_ALIGNMENT;
        const size_t eb = (size_t)elem_bytes(p->dtype);
        bool ok = cudaEventRecord(p->ev_start, st) == cudaSuccess &&
                  cudaStreamWaitEvent(p->s_in, p->ev_start, 0) == cudaSuccess &&
                  cudaStreamWaitEvent(p->s_out, p->ev_start, 0) == cudaSuccess;
        for (int i = 0; ok && i < CH; ++i) {
            const int64_t b0 = p->batch * i / CH, b1 = p->batch * (i + 1) / CH;
            const size_t off = (size_t)b0 * (size_t)p->dist * eb;
            const size_t len = (i + 1 < CH) ? (size_t)(b1 - b0) * (size_t)p->dist * eb : bytes - off;
            const char* hin = static_cast<const char*>(host_in) + off;
            char* hout = static_cast<char*>(host_out) + off;
            char* din = static_cast<char*>(dev_in) + off;
            char* dout = static_cast<char*>(dev_out) + off;
            ok = cudaMemcpyAsync(din, hin, len, cudaMemcpyHostToDevice, p->s_in) == cudaSuccess &&
                 cudaEventRecord(p->ev_in[i], p->s_in) == cudaSuccess &&
                 cudaStreamWaitEvent(st, p->ev_in[i], 0) == cudaSuccess &&
                 launch_single_pass(p, din, dout, b1 - b0, st) == B200FFT_OK &&
                 cudaEventRecord(p->ev_k[i], st) == cudaSuccess &&
                 cudaStreamWaitEvent(p->s_out, p->ev_k[i], 0) == cudaSuccess &&
                 cudaMemcpyAsync(hout, dout, len, cudaMemcpyDeviceToHost, p->s_out) == cudaSuccess;
        }
        ok = ok && cudaEventRecord(p->ev_done, p->s_out) == cudaSuccess && cudaStreamWaitEvent(st, p->ev_done, 0) == cudaSuccess;
        return ok ? B200FFT_OK : B200FFT_ERR_CUDA;
    }
    if (cudaMemcpyAsync(dev_in, host_in, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    int rc = fft_execute(p, dev_in, dev_out, stream);
    if (rc != B200FFT_OK) return rc;
    if (cudaMemcpyAsync(host_out, dev_out, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return B200FFT_ERR_CUDA;
    return B200FFT_OK;
}

extern "C" int fft_plan_destroy(fft_plan_t p) {
    if (!p) return B200FFT_ERR_INVALID_ARG;
    release(p);
    delete p;
    return B200FFT_OK;
}

extern "C" const char* fft_status_string(int status) {
    switch (status) {
    case B200FFT_OK: return "ok";
    case B200FFT_ERR_INVALID_ARG: return "invalid argument";
    case B200FFT_ERR_UNSUPPORTED: return "unsupported size or layout";
    case B200FFT_ERR_ALIGNMENT: return "pointer or stride not aligned for vector access";
    case B200FFT_ERR_ALLOC: return "allocation failed";
    case B200FFT_ERR_CUDA: return "CUDA runtime or launch error";
    case B200FFT_ERR_WORKSPACE: return "workspace missing or too small";
    default: return "unknown status";
    }
}

extern "C" int64_t b200fft_launch_count(void) { return g_launch_count.load(); }

extern "C" int b200fft_tma_timeouts(void) { return tma_timeouts() + rows_stage_timeouts(); }
