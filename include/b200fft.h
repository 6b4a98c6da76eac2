/*
 * b200fft — batched complex FFTs and range-Doppler SAR image formation on one
 * NVIDIA B200 (sm_100a). C ABI: plain pointers and sizes, no C++ or framework
 * types. Every DEVICE pointer is memory on the current CUDA device, owned by
 * the caller (for example a torch tensor's data_ptr()); the library allocates
 * only its own small tables. `stream` is a cudaStream_t passed as void*
 * (NULL = the default stream). No call synchronises the device unless it says
 * so; no call falls back to the CPU: what is not supported returns an error.
 *
 * Every function returns 0 (B200FFT_OK) or one of the B200FFT_ERR_* codes.
 */
#ifndef B200FFT_H
#define B200FFT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    B200FFT_OK = 0,
    B200FFT_ERR_INVALID_ARG = 1,   /* null pointer, n <= 0, batch <= 0, bad direction or dtype */
    B200FFT_ERR_UNSUPPORTED = 2,   /* not a power of two, size out of range, layout class */
    B200FFT_ERR_ALIGNMENT = 3,     /* pointer or stride breaks 128-bit access */
    B200FFT_ERR_ALLOC = 4,         /* device table allocation failed */
    B200FFT_ERR_CUDA = 5,          /* launch or runtime error */
    B200FFT_ERR_WORKSPACE = 6      /* plan needs a workspace that was not set or is too small */
};

#define B200FFT_FORWARD (-1)       /* exp(-2 pi i n k / N), unnormalised */
#define B200FFT_INVERSE (+1)       /* exp(+2 pi i n k / N), scaled by 1/N */

#define B200FFT_C64 0              /* interleaved (re, im) fp32, 8 bytes per element */
#define B200FFT_C32H 1             /* interleaved (re, im) fp16, 4 bytes per element; arithmetic stays fp32 */

typedef struct b200fft_plan_s *fft_plan_t;
typedef struct b200fft_sar_s *sar_rda_params_t;
typedef struct b200fft_sar_shard_s *sar_rda_shard_t;

/* ------------------------------------------------------------------------
 * Batched 1-D complex-to-complex transform (paper, Section "The M6 Memory
 * Hierarchy", the single-pass transform behind Eq. 1: each element is read
 * from main memory once and written once; Sections "One Pass for N=8192 and
 * 16384" and "FP16 Storage").
 *
 *   forward  X[b][k] =        sum_j x[b][j] exp(-2 pi i j k / n)
 *   inverse  x[b][j] = (1/n)  sum_k X[b][k] exp(+2 pi i j k / n)
 *
 * Element j of transform b lives at index b*dist + j*stride, counted in
 * complex elements, in the input and in the output alike. Output is in
 * natural order.
 *
 * Supported layouts:
 *   rows     stride == 1, dist >= n, dist even (dist a multiple of 4 for C32H)
 *   columns  dist == 1, stride >= batch, stride and batch even: the columns of
 *            a row-major matrix (paper, Section "End to End": the FFT that
 *            reads the columns directly)
 * Supported sizes: n a power of two, 8 <= n <= 32768 in a single pass over
 * memory (columns: 64 <= n <= 8192; rows of n = 32768 on a cluster of two
 * thread blocks that share the transform through distributed shared memory);
 * 2^16 <= n <= 2^20 (rows only) by a two-pass four-step split (the paper's
 * "usual remedy when a transform does not fit on chip"), which needs a
 * workspace of n*batch elements of the storage type.
 *
 * fft_plan_create allocates the plan's twiddle tables on the current device
 * (at most a few hundred KiB) and builds them there; it synchronises the
 * device once. The plan may be executed any number of times, on any stream of
 * that device; concurrent execution on several streams is allowed unless the
 * plan has a workspace.
 * ---------------------------------------------------------------------- */
int fft_plan_create(fft_plan_t *plan, int64_t n, int64_t batch, int64_t stride,
                    int64_t dist, int direction, int storage_dtype);

/* Bytes of caller-owned DEVICE workspace the plan needs (0 for single-pass plans). */
int fft_plan_workspace_bytes(fft_plan_t plan, size_t *bytes);

/* Hand the plan a DEVICE workspace (16-byte aligned, at least the size above).
 * The caller keeps ownership and must keep it alive while the plan executes. */
int fft_plan_set_workspace(fft_plan_t plan, void *device_ptr, size_t bytes);

/* Enqueue the transform on `stream`. `in` and `out` are DEVICE pointers,
 * 16-byte aligned, each holding (batch-1)*dist + (n-1)*stride + 1 elements of
 * the plan's storage type. in == out is allowed; partial overlap is not.
 * Returns after the launch; B200FFT_ERR_CUDA reports a launch error. */
int fft_execute(fft_plan_t plan, const void *in, void *out, void *stream);

/* The same transform from HOST buffers (paper's footprint: input plus output):
 * copies host_in -> dev_in, executes dev_in -> dev_out, copies dev_out ->
 * host_out. The host buffers should be pinned for the copies to be
 * asynchronous; the device staging buffers are caller-owned and sized like
 * in/out above. Large row batches are cut into 16 chunks whose copy in,
 * transform and copy out overlap on two internal copy streams (created on the
 * first such call); towards the caller it is still one operation ordered on
 * `stream`: it starts after the work already on `stream`, and `stream` waits
 * for the last copy out. Does not synchronise the host. */
int fft_execute_host(fft_plan_t plan, const void *host_in, void *host_out,
                     void *dev_in, void *dev_out, void *stream);

/* Free the plan's tables. The caller must have synchronised outstanding work. */
int fft_plan_destroy(fft_plan_t plan);

/* Variant choice and test knobs (paper, Section "One Pass": "a regression test forces N=8192 through
 * this path"). Every variant of a plan gives the same results to rounding. Unknown keys return
 * B200FFT_ERR_INVALID_ARG; a variant that is not compiled for the plan's size returns
 * B200FFT_ERR_UNSUPPORTED and leaves the plan as it was. Call before set_workspace.
 *   "four_step"  1 routes a rows plan of any supported n >= 4096 through the two-pass split; 0 brings a
 *                plan of n <= 32768 back to its single pass.
 *   "split_n1"   two-pass plans only: factor n = n1 * n2 with this n1 (a power of two, 64 <= n1 <= 1024,
 *                64 <= n2 <= 4096; 0 = the default, n1 = 256 for n >= 65536 and the near-square split
 *                with n1 >= n2 below). Pass 1 transforms the n2 columns of length n1, pass 2 the n1 rows
 *                of length n2.
 *   "cluster"    c = 1, 2 or 4 (0 = the default rules; other values are B200FFT_ERR_INVALID_ARG): the
 *                single-pass variant in which c CTAs of one thread-block cluster share a tile through
 *                distributed shared memory. Defaults: rows of n = 16384 and n = 8192 with at most 32
 *                transforms (4 CTAs each; n = 16384 up to 64 transforms: 2), and rows of n = 32768 (2),
 *                are split over clusters. Columns plans take, in
 *                this order, the widest tile that is compiled and divides the batch: 16 columns for
 *                n <= 512 and 8 for n = 1024; the streaming kernel (see "stream") for n = 4096 when the
 *                matrix has more than one 4-column tile per multiprocessor; for other n >= 2048 a
 *                tile of 32768 / n columns shared by a cluster of two CTAs (not complex64 at n = 2048);
 *                "cluster" = 1 forces the plain single-CTA 4-column tile (2 columns at n = 8192).
 *   "stream"     (columns plans; "tma" is an alias) 1 selects the persistent streaming kernel (n = 2048
 *                complex64, n = 4096 both storage types): one CTA per multiprocessor loops over
 *                4-column tiles, and the tensor memory accelerator brings the next tile into shared
 *                memory (2-D tiled bulk copies of this GPU's own memory, each addressed to one CTA) and takes the
 *                finished one out while the current one is transformed; 0 forbids it; -1 restores the
 *                default rules.
 *   "staged"     (rows plans) n = 16384: 1 selects the persistent kernel whose next transform arrives
 *                in shared memory through untiled bulk copies while the current one is computed; 0
 *                forbids it; -1 restores the default (on for fp16 storage with at least two transforms
 *                per multiprocessor). n <= 32 with dist == n: by default one thread per transform, the
 *                128 transforms of a CTA copied through shared memory in contiguous 16-byte pieces; 0
 *                selects the plain kernel (several threads per transform at n = 32, direct loads).
 *   "prefetch"   d makes each CTA of a rows plan ask L2 for the input of the transform d tiles ahead
 *                (0 = off, -1 = the default: one wave ahead for n = 16384).
 *   "via_transpose"  1 makes a columns plan work the way the paper's four-pass pipeline does (Section
 *                "End to End": a transpose, then the transform along rows): transpose into the
 *                workspace, row transforms in place there, transpose back into `out`; it then needs a
 *                workspace of n*batch elements of the storage type, which must be neither `in` nor
 *                `out`; kept as a measured comparison with the direct column kernels.
 *   "alt_factorisation"  (rows plans, test knob) 1 selects the other compiled factorisation: n = 4096
 *                with every first-stage twiddle row loaded from its table instead of multiplied up,
 *                n = 16384 as 16 x 4 x 16 x 16 instead of 32 x 32 x 16.
 *   "wait_polls", "starve_wait"  (test knobs of the kernels that wait on asynchronous copies) every such
 *                wait is bounded: after wait_polls polls (0 = the default, 2^22, a fraction of a second)
 *                the CTA gives up, raises the counter that b200fft_tma_timeouts() reads, waits for the
 *                copies it still has in flight and returns; the output of that call is then incomplete.
 *                starve_wait = 1 makes the streaming kernel poll a barrier that nothing completes, so
 *                that a test can see the give-up path run; never set it otherwise. */
int fft_plan_set_option(fft_plan_t plan, const char *key, int64_t value);

/* The paper has no counterpart to this call. It is for callers that must not
 * allocate device memory when they transform: a loop that cannot take the
 * device-wide stall cudaMalloc or cudaFree may cause, a process whose device
 * memory is already committed to its own pool, a deployment with a memory
 * budget fixed at load time. It runs the two-pass transform of `batch`
 * contiguous complex64 rows of n points (dist = n, in and out DEVICE pointers,
 * 16-byte aligned, n*batch elements each, in == out allowed) without a plan:
 * the scratch image and the twiddle tables live in a fixed device array inside
 * the library (B200FFT_NOALLOC_MAX_ELEMS elements of scratch, 2 MiB, plus
 * 64 KiB of tables, held by every GPU that loads the library until exit).
 * Limits: n a power of two, 4096 <= n <= 262144, n*batch <=
 * B200FFT_NOALLOC_MAX_ELEMS; anything larger returns B200FFT_ERR_WORKSPACE,
 * other sizes B200FFT_ERR_UNSUPPORTED. It calls no cudaMalloc, cudaFree or
 * other allocating routine. The first call on a device looks up the array's
 * device address; make that first call before any stream capture begins.
 * All calls share the one array: two calls that overlap on the GPU (different
 * streams, no ordering between them) race on it, so order them. The array keeps
 * the previous call's contents; each call rebuilds the tables it needs and
 * overwrites the scratch it reads, so no clearing is required of the caller.
 * Results equal those of a four-step plan of the same size. */
#define B200FFT_NOALLOC_MAX_ELEMS 262144
int fft_execute_noalloc(int64_t n, int64_t batch, int direction, const void *in, void *out, void *stream);

/* Block-floating-point form of fft_execute for rows plans with fp16 storage and
 * 1024 <= n <= 16384 (paper, Section "FP16 Storage": FFT outputs grow up to N
 * times for coherent data, so real radar data in fp16 needs block floating
 * point; the paper's own chain uses fixed shifts, see sar_rda_*). Every
 * transform b carries one power-of-two exponent:
 *   true input  x_b[n] = in_b[n]  * 2^in_exp[b]   (in_exp == NULL: all zero)
 *   true output X_b[k] = out_b[k] * 2^out_exp[b]
 * The transform is computed in fp32 from the stored fp16 values; the stored
 * output is scaled by the power of two that puts its largest real or imaginary
 * component in [2^14, 2^15) (all-zero output: unscaled), and out_exp[b] =
 * in_exp[b] + that shift (the inverse's 1/n goes into the exponent too).
 * in_exp, out_exp: device arrays of `batch` int32; in/out as for fft_execute
 * (in place allowed; in_exp may equal out_exp). No workspace. Errors:
 * B200FFT_ERR_UNSUPPORTED for other plans, B200FFT_ERR_ALIGNMENT,
 * B200FFT_ERR_INVALID_ARG for null pointers. */
int fft_execute_bfp(fft_plan_t plan, const void *in, const int32_t *in_exp, void *out, int32_t *out_exp,
                    void *stream);

/* Static description of a status code. */
const char *fft_status_string(int status);

/* Number of kernel launches the library has enqueued since it was loaded
 * (all plans, all streams); for launch accounting in benchmarks. */
int64_t b200fft_launch_count(void);

/* Number of bounded waits on asynchronous copies (streaming column kernel:
 * counted once per CTA; staged rows kernel) that gave up after their poll limit
 * since the library was loaded. Synchronises the device. 0 unless something is
 * badly wrong or a test asked for it: the waits are bounded so that a lost copy
 * can never hang the GPU. */
int b200fft_tma_timeouts(void);

/* ------------------------------------------------------------------------
 * Range-Doppler SAR image formation (paper, Section "End to End:
 * Range-Doppler SAR"): range compression (FFT, multiply by the conjugate
 * chirp spectrum, inverse FFT along each pulse, 1/n_range included); azimuth
 * FFT along each range bin; range cell migration correction with an 8-tap
 * sinc interpolator; the azimuth filter exp(+j 4 pi R0 (D - 1) / lambda),
 * D = sqrt(1 - (lambda f_a / 2 v)^2); azimuth inverse FFT. The chirp is an
 * up-chirp with its replica centred on t = 0, and range bin n_range/2 is the
 * scene centre (both fixed; the descriptor has no field for them). The default
 * form is four kernels: fused range compression; the azimuth FFT read as
 * columns in place (scaled 1/n_azimuth); RCMC + filter along the rows, written
 * to `out`; the inverse azimuth FFT as columns of `out` in place. The paper's
 * three-pass form (RCMC + filter + inverse FFT fused on column tiles) and two
 * other organisations are selectable: see sar_rda_set_option.
 * ---------------------------------------------------------------------- */
typedef struct {
    int64_t n_azimuth;          /* pulses (rows): 1024, 2048 or 4096 */
    int64_t n_range;            /* range samples per pulse (columns): 1024, 2048, 4096 or 8192 */
    double carrier_hz;
    double bandwidth_hz;        /* chirp bandwidth; up-chirp, replica centred on t = 0 */
    double fs_hz;               /* range sampling rate */
    double pulse_s;             /* pulse length */
    double prf_hz;
    double velocity_mps;
    double r_center_m;          /* slant range of range bin n_range/2 */
    int32_t intermediate_dtype; /* B200FFT_C64 or B200FFT_C32H for the two intermediate images */
    int32_t rcmc_taps;          /* must be 8 */
} sar_rda_desc;

/* Build the processing tables on the current device (conjugate chirp spectrum,
 * per-Doppler-bin migration and phase coefficients, computed in float64).
 * Synchronises the device once. */
int sar_rda_params_create(sar_rda_params_t *params, const sar_rda_desc *desc);

/* Bytes of DEVICE workspace: two intermediate images of n_azimuth*n_range
 * elements of the intermediate dtype (the default chain uses the first; the
 * slab and transposed forms use both). Its contents between calls are
 * unspecified; its layout is the library's own. */
int sar_rda_workspace_bytes(sar_rda_params_t params, size_t *bytes);
int sar_rda_set_workspace(sar_rda_params_t params, void *device_ptr, size_t bytes);

/* Variant choice; every form gives the same image to rounding.
 *   "fused_rcmc"   1 runs step 2 as the single fused kernel (RCMC + filter + inverse azimuth FFT on
 *                  column tiles: three passes over memory in all, the paper's best form); 0 runs it as a
 *                  row pass followed by the inverse column FFT (four passes, but faster on B200; with fp16
 *                  intermediates and 4096 pulses the row pass writes a second fp16 image, one more rounding,
 *                  else the complex64 output on which the column pass then runs in place; the
 *                  default whenever the scene allows it: B200FFT_ERR_UNSUPPORTED if the migration grows
 *                  by more than 112 bins over 2048 range bins).
 *   "layout"       0 (default) keeps the intermediate image row-major and transforms its columns
 *                  directly. 1 keeps it in slabs of 32-byte granules (4 complex64 or 8 complex-half range
 *                  bins; element (k, n) at ((n / G) * n_azimuth + k) * G + n % G), so that every column
 *                  tile is row segments inside one contiguous slab; step 2 then goes slab to slab (second
 *                  half of the workspace; with fp16 intermediates this image is fp16 as well, one more
 *                  rounding) and the inverse column FFT writes the row-major image. 2 is the paper's
 *                  four-pass form as a measured comparison: every azimuth transform is a transpose,
 *                  transforms along rows, and a transpose back. B200FFT_ERR_UNSUPPORTED if the scene's
 *                  shift spreads by more than 16 bins inside a block of 32 Doppler bins by 64 range bins
 *                  (layout 1) or the row pass cannot serve it (layout 2).
 *   "tile_columns" 2 or 4 (default): range bins per column tile on the slab layout. */
int sar_rda_set_option(sar_rda_params_t params, const char *key, int64_t value);

/* raw: DEVICE, n_azimuth x n_range interleaved complex fp32, row-major (row =
 * pulse). out: DEVICE, same shape and type, the focused image; must not alias
 * raw or the workspace. Enqueues four kernels on `stream` (three with
 * "fused_rcmc", eight with "layout" 2); does not
 * synchronise. Calls sharing one params object must not overlap on the GPU
 * (they share its workspace). */
int sar_rda_form_image(const void *raw, sar_rda_params_t params, void *out, void *stream);

/* Host-buffer variant: copies host_raw -> dev_raw, forms the image into
 * dev_out, copies dev_out -> host_out, all on `stream`. */
int sar_rda_form_image_host(const void *host_raw, sar_rda_params_t params, void *host_out,
                            void *dev_raw, void *dev_out, void *stream);

/* Run one step only, for tests: step 0 range compression (raw -> first image
 * of the workspace), 1 azimuth FFT (that image, in place), 2 RCMC + filter +
 * inverse FFT (-> out; one or more kernels, see sar_rda_set_option). `raw` is
 * read by step 0 only, `out` written by step 2 only. */
int sar_rda_run_step(const void *raw, sar_rda_params_t params, void *out, int step, void *stream);

int sar_rda_params_destroy(sar_rda_params_t params);

/* ------------------------------------------------------------------------
 * Image formation split over `world` devices, one process per device (not in
 * the paper, whose chain runs on one device; the decomposition follows from the
 * chain's structure in Section "End to End: Range-Doppler SAR": range
 * compression works on whole pulses, every later step on whole range-bin
 * columns, and the interpolator of step 2 reaches a bounded number of bins
 * along range). Rank r
 *   1. range-compresses pulses [first_pulse, first_pulse + pulses) and stores
 *      every compressed sample straight into the strip buffer of the rank that
 *      owns its range bin (its own memory or a peer's, through the addresses the
 *      caller passes in `strips`), and a second time into the neighbouring strip
 *      whose halo it falls into: the exchange is part of the kernel's epilogue,
 *      plain stores, no separate transpose or collective;
 *   2. after every rank has finished step 1 (the caller synchronises: a barrier
 *      of its process group after a stream synchronise), runs the azimuth FFT,
 *      RCMC + filter and the inverse azimuth FFT on its strip and writes range
 *      bins [first_bin, first_bin + bins) of the image, n_azimuth rows of `bins`
 *      complex64 values.
 * A strip buffer is n_azimuth rows of strip_width = halo_left + bins +
 * halo_right elements of the intermediate type: the strip's bins and, on both
 * sides, the neighbouring bins the interpolator reads (halo_right covers the
 * largest range migration of the frame plus the taps); halo bins outside the
 * frame are written as zeros by the rank that owns the pulse. The strip buffer
 * is the first strip_bytes of the rank's workspace (workspace_bytes in all).
 * world is 1, 2, 4 or 8; n_azimuth must be a multiple of world, n_range / world a
 * power of two (at least 8); halo_left + halo_right must not exceed bins (else
 * B200FFT_ERR_UNSUPPORTED). Results equal the single-device chain to rounding
 * (the per-bin coefficients are built in float64 for the strip's own origin).
 * ---------------------------------------------------------------------- */
typedef struct {
    int64_t first_pulse, pulses;     /* rows of the raw frame this rank range-compresses */
    int64_t first_bin, bins;         /* range bins of the image this rank forms */
    int64_t halo_left, halo_right;   /* neighbouring bins kept on each side of the strip */
    int64_t strip_width;             /* halo_left + bins + halo_right: row pitch of the strip buffer, in elements */
    int64_t strip_bytes;             /* n_azimuth * strip_width elements of the intermediate type */
    int64_t workspace_bytes;         /* the strip buffer followed by the second intermediate image */
} sar_rda_shard_geometry;

/* Host arithmetic only (no device needed): the geometry of rank `rank` of `world`. */
int sar_rda_shard_geometry_of(const sar_rda_desc *scene, int32_t rank, int32_t world, sar_rda_shard_geometry *geometry);
/* Tables and kernels for this rank on the current device. `scene` describes the whole frame. */
int sar_rda_shard_create(sar_rda_shard_t *shard, const sar_rda_desc *scene, int32_t rank, int32_t world);
int sar_rda_shard_get_geometry(sar_rda_shard_t shard, sar_rda_shard_geometry *geometry);
/* This rank's workspace (device memory, 16-byte aligned, at least workspace_bytes, caller-owned). Its start is
 * the strip buffer that every rank's step 1 stores into, so it must be memory the other ranks can address. */
int sar_rda_shard_set_workspace(sar_rda_shard_t shard, void *device_ptr, size_t bytes);
/* Step 1. raw_rows: this rank's pulses, `pulses` rows of n_range complex64 (device). strips: `world` device
 * addresses (host array), strips[g] = the workspace of rank g as this process addresses it. Asynchronous. */
int sar_rda_shard_range_compress(sar_rda_shard_t shard, const void *raw_rows, void *const *strips, void *stream);
/* Step 2, after all ranks completed step 1. image_strip: n_azimuth x bins complex64 (device), not the workspace. */
int sar_rda_shard_azimuth(sar_rda_shard_t shard, void *image_strip, void *stream);
int sar_rda_shard_destroy(sar_rda_shard_t shard);

#ifdef __cplusplus
}
#endif
#endif /* B200FFT_H */
