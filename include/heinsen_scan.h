/*
 * libheinsen_scan -- C ABI.
 *
 * Fused, single-pass evaluation on one NVIDIA B200 (sm_100a) of the first-order
 * linear recurrence
 *
 *         x_t = a_t * x_{t-1} + b_t ,   t = 1..n ,
 *
 * for `rows` independent sequences, through the two-prefix-sum log-space
 * expression of F. A. Heinsen, "Efficient Parallelization of a Ubiquitous
 * Sequential Computation" (2023):
 *
 *         a*_t      = cumsum_t(log a_t)                                  (Eq. 2, first prefix sum)
 *         log x_t   = a*_t + tail(LCSE(cat(log x_0, log b_t - a*_t)))    (Eq. 7, Eq. 8)
 *         x_t       = exp(log x_t)                                       (Eq. 3)
 *
 * Both prefix sums, the log-sum-exp and the final exponential are fused into one
 * pass over HBM: every input element is read once, every output element written
 * once.  Negative a_t, b_t, x_0 are carried as sign + magnitude, which is the
 * paper's complex-logarithm path on the principal branch (Summary, last
 * paragraph): log(-r) = log r + i*pi, the imaginary part is one sign bit.
 *
 * Conventions for every entry point
 *   - Layout: a, b, log_a, log_b, x, log_x, sign_*: [rows, n] row-major contiguous,
 *     element (r, t) of the paper (t = 1..n) at index r*n + (t-1).  x0, log_x0,
 *     sign_x0: [rows].  The output has n entries per row, x_1..x_n; x_0 is not part
 *     of it (Eq. 7's tail()).
 *   - Device entry points take DEVICE pointers owned by the caller.  The library
 *     never allocates or frees device memory and keeps none of the caller's.  Two
 *     things of its own live as long as the process: the fixed 1 MiB scratch array
 *     of heinsen_scan_log_static / scan_linear / scan_log (part of the library
 *     image on every GPU that loads it), and, per device, the two streams and three
 *     events that the *_host entry points create at their first call; *_host calls
 *     on one device run one at a time.  Work is enqueued on `stream` (a cudaStream_t
 *     passed as void*; NULL = legacy default stream) and the device entry points
 *     return without synchronising.
 *   - Pointers must be aligned to their element size.  When every base pointer is
 *     16-byte aligned and n * sizeof(element) is a multiple of 16 for every tensor,
 *     chunks move by TMA; otherwise a slower in-kernel path with plain loads is used
 *     (still entirely on the GPU).
 *   - The output may alias one input of the same type and shape exactly (in situ);
 *     partial overlap is undefined.
 *   - rows == 0 or n == 0: HS_OK, nothing is launched.
 *   - log 0 = -inf is a legal input.  +inf and NaN inputs give unspecified values in
 *     their own row from that element on and never affect other rows.
 *   - Limits: rows < 2^31, n < 2^31 - 2^20.
 *   - Errors found on the host (null pointer, negative size, size beyond the limits,
 *     unsupported type, bad workspace) return before any CUDA call.
 *   - Errors found on the device (a bounded wait that ran out) are written to a
 *     status word in `workspace` and are read back by heinsen_scan_check().
 *   - There is no CPU fallback: on a device that is not sm_100 the calls return
 *     HS_ERR_UNSUPPORTED_DEVICE.
 */
#ifndef HEINSEN_SCAN_H_
#define HEINSEN_SCAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { HS_F32 = 0, HS_BF16 = 1 } hs_dtype;

typedef enum {
    HS_OK = 0,
    HS_ERR_INVALID_ARG = 1,
    HS_ERR_UNSUPPORTED_DEVICE = 2,
    HS_ERR_WORKSPACE_TOO_SMALL = 3,
    HS_ERR_CUDA = 4,
    HS_ERR_LOOKBACK_TIMEOUT = 5, /* device: a tile's wait for its predecessors ran out */
    HS_ERR_COPY_TIMEOUT = 6      /* device: a wait for an asynchronous chunk copy ran out */
} hs_status;

/* Kernel selection for heinsen_scan_set_path(). */
typedef enum {
    HS_PATH_AUTO = 0,     /* rows >= a few per SM: batched kernel; else look-back kernel */
    HS_PATH_BATCHED = 1,  /* one warp walks one row, carry in registers */
    HS_PATH_LOOKBACK = 2  /* rows cut into tiles, single pass, the carry between tiles propagated beside the tiles' arithmetic */
} hs_path;

/*
 * Linear-domain entry point: Eq. 3 / Eq. 7 applied to linear inputs.
 *   x[r,t] = a[r,t] * x[r,t-1] + b[r,t],  x[r,0] = x0[r].
 * The kernel takes log|a|, log|b|, log|x0| and the sign bits itself (step "log a_t",
 * "log b_t", "log x_0" of Eq. 2 and Eq. 7), runs both prefix sums in log space and
 * writes x = +-exp(log|x|).
 *   a, b  : device, [rows,n], `dtype`;  x0: device, [rows], `dtype`;  x: device, [rows,n], `dtype`.
 *   dtype : HS_F32 only (HS_BF16 returns HS_ERR_INVALID_ARG).
 *   workspace, workspace_bytes: device scratch of at least
 *           heinsen_scan_workspace_bytes(rows, n) bytes, 256-byte aligned; contents
 *           need no initialisation; must not be shared by calls that overlap in time.
 */
hs_status heinsen_scan_linear(const void* a, const void* b, const void* x0, void* x,
                              int64_t rows, int64_t n, hs_dtype dtype,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * Comparison path, NOT the paper's method: the same recurrence scanned in the linear
 * domain as pairs (alpha, beta) = "x -> alpha x + beta" combined by
 * (alpha2 alpha1, alpha2 beta1 + beta2), i.e. the general two-operator formulation that
 * the section "Compared to Blelloch's Formulation" sets the log-space expression
 * against.  No logarithm or exponential is taken, so every prefix product and partial
 * sum must fit fp32's own range: a product of |a| over one part that overflows gives
 * inf/NaN, one that underflows drops what the log-space entry points still carry.
 * Arguments, layout, workspace and errors as for heinsen_scan_linear (HS_F32 only).
 * Always runs the row-batched kernel (one warp per row or per few rows); it is meant
 * for batches of rows and is slow for a single long row.
 */
hs_status heinsen_scan_linear_pairs(const void* a, const void* b, const void* x0, void* x,
                                    int64_t rows, int64_t n, hs_dtype dtype,
                                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * Log-domain entry point: Eq. 7 as printed, on log inputs, returning log x.
 *   log_x[r,t] = a*_t + logaddexp(log_x0[r], logcumsumexp(log_b - a*)_t),  a* = cumsum(log_a)
 * with an optional sign bit per value (sign + magnitude of a negative real).
 *   log_a, log_b : device, [rows,n], `dtype_in`;  log_x0: device, [rows], `dtype_in`.
 *   log_x        : device, [rows,n], `dtype_out`.  Supported (in,out): (F32,F32),
 *                  (BF16,BF16), (F32,BF16).  Arithmetic is fp32 throughout; bf16 is
 *                  storage only, rounded to nearest-even on store.
 *   sign_a, sign_b : device, [rows,n] uint8, 0 = '+', 1 = '-', or NULL (all positive).
 *   sign_x0        : device, [rows] uint8 or NULL.
 *   sign_x         : device, [rows,n] uint8 output; required iff any sign input is
 *                    non-NULL, ignored otherwise.  An exact zero reports sign 0.
 *   workspace      : as for heinsen_scan_linear.
 */
hs_status heinsen_scan_log(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                           const uint8_t* sign_a, const uint8_t* sign_b, const uint8_t* sign_x0,
                           uint8_t* sign_x,
                           int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Scratch size in bytes for a problem of this shape (any path, any type): a 256-byte
 * header (status words) plus three 16-byte words per tile of the look-back kernel (the
 * tile's aggregate, the value entering the tile), or one per warp slot of the batched
 * kernel when it shares rows out among its slots -- the carry between parts that the
 * associativity of prefix sums allows
 * (Summary, footnote on associativity).  Returns 0 only for invalid sizes.
 */
size_t heinsen_scan_workspace_bytes(int64_t rows, int64_t n);

/*
 * Synchronises `stream`, reads the status word of `workspace` (device pointer) and
 * returns it: HS_OK, or the device-side error recorded by the last call that used
 * this workspace.
 */
hs_status heinsen_scan_check(const void* workspace, void* stream);

/*
 * Host-buffer variants of the two entry points above, for callers whose data lives
 * in host memory (pinned memory recommended).  All tensor pointers are HOST pointers;
 * `device_scratch` is a DEVICE buffer of at least heinsen_scan_host_scratch_bytes(...)
 * bytes provided by the caller.  The call copies inputs to the device in row blocks,
 * runs the same kernels, copies results back, and returns after the last copy has
 * completed (it synchronises).  The recurrence itself runs only on the GPU.
 */
hs_status heinsen_scan_linear_host(const void* a, const void* b, const void* x0, void* x,
                                   int64_t rows, int64_t n, hs_dtype dtype,
                                   void* device_scratch, size_t device_scratch_bytes, void* stream);
hs_status heinsen_scan_log_host(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                                const uint8_t* sign_a, const uint8_t* sign_b, const uint8_t* sign_x0,
                                uint8_t* sign_x,
                                int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out,
                                void* device_scratch, size_t device_scratch_bytes, void* stream);
size_t heinsen_scan_host_scratch_bytes(int64_t rows, int64_t n, hs_dtype dtype_in, hs_dtype dtype_out,
                                       int with_signs);

/*
 * Allocation-free variant of heinsen_scan_log (the paper has no counterpart: this is a service
 * to callers, not a step of the method).
 *
 * Who needs it: code that runs where device memory cannot be requested -- a plug-in called from
 * another framework's execution callback under a fixed memory plan, a service that forbids
 * allocation after start-up because cudaMalloc synchronises the device and may fail under
 * fragmentation, or a host that simply has no allocator to hand this library a workspace.  Such
 * callers still own their inputs and outputs; what they cannot provide is the scratch that the
 * single-pass look-back kernel needs for its per-tile descriptors.
 *
 * What it does: the same computation as heinsen_scan_log with fp32 storage and no sign tensors
 * (log_a, log_b: [rows,n]; log_x0: [rows]; log_x: [rows,n]; all DEVICE pointers), always through
 * the look-back kernel, with the scratch taken from a fixed 1 MiB array that is part of the
 * library image.  Every GPU that loads the library carries that array until the process exits.
 * The call performs no cudaMalloc, cudaFree or other allocating call.
 *
 * Limits and rules:
 *   - rows and n must be small enough that heinsen_scan_workspace_bytes(rows, n) <= 1 MiB
 *     (one row: up to heinsen_scan_static_max_elements() elements, about 1.7e8); larger problems return
 *     HS_ERR_WORKSPACE_TOO_SMALL and launch nothing.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array and it keeps what the previous call wrote.  The entry point
 *     clears the part it uses on `stream` before launching, so calls issued one after another on
 *     one stream are safe; calls that can overlap on the GPU (different streams, or different
 *     host threads without ordering) race on the array and give undefined results.
 *   - Device-side errors of the last call are read with heinsen_scan_check_static(stream).
 */
hs_status heinsen_scan_log_static(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                                  int64_t rows, int64_t n, void* stream);
/* Synchronises `stream` and returns the device-side status of the last heinsen_scan_log_static call. */
hs_status heinsen_scan_check_static(void* stream);
/* Largest n that heinsen_scan_log_static accepts for a single row. */
size_t heinsen_scan_static_max_elements(void);

/*
 * Complex-logarithm form of heinsen_scan_log (Summary, last paragraph: with negative a_t, b_t
 * or x_0 the interim logarithms are complex while x_t stays real).  Every value is one complex64
 * (interleaved float pairs): real part log|v|, imaginary part an integer multiple of pi, odd for
 * a negative v (principal branch: log(-r) = log r + i*pi); log 0 = (-inf, anything).
 *   log_a, log_b : device, [rows,n] complex64;  log_x0: device, [rows] complex64.
 *   log_x        : device, [rows,n] complex64 = (log|x_t|, 0 or pi); an exact zero is (-inf, 0).
 *   workspace    : device, at least heinsen_scan_complex_workspace_bytes(rows, n) bytes, 256-byte
 *                  aligned: header and look-back descriptors only, as for heinsen_scan_log.  The kernels
 *                  read the complex elements themselves (magnitude from the real part, sign bit from the
 *                  parity of the imaginary part over pi) and write complex elements: 24 bytes of traffic
 *                  per element, nothing staged in between.
 *   n            : at most half the limit of the other entry points (a row is addressed as 2n floats).
 * Device-side errors: heinsen_scan_check(workspace, stream).
 */
hs_status heinsen_scan_log_complex(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                                   int64_t rows, int64_t n, void* workspace, size_t workspace_bytes, void* stream);
size_t heinsen_scan_complex_workspace_bytes(int64_t rows, int64_t n);

/*
 * The two calls in their shortest form: fp32 storage, legacy default stream, automatic kernel
 * selection, scratch from the library's fixed 1 MiB array (the rules of heinsen_scan_log_static
 * apply: problems whose look-back descriptors do not fit return HS_ERR_WORKSPACE_TOO_SMALL; calls
 * must not overlap on the GPU).  scan_linear: Eq. 3 / Eq. 7 on linear inputs, as
 * heinsen_scan_linear.  scan_log: Eq. 7 on log inputs with optional sign tensors (NULL = all
 * positive; sign_x required iff any sign input is given), as heinsen_scan_log.  Device pointers.
 * Device-side errors are read with heinsen_scan_check_static(NULL).
 */
hs_status scan_linear(const void* a, const void* b, const void* x0, void* x, int64_t rows, int64_t n);
hs_status scan_log(const void* log_a, const void* log_b, const void* log_x0, void* log_x,
                   const uint8_t* sign_a, const uint8_t* sign_b, const uint8_t* sign_x0, uint8_t* sign_x,
                   int64_t rows, int64_t n);

/* Process-wide kernel selection (default HS_PATH_AUTO); for tests and benchmarks. */
hs_status heinsen_scan_set_path(hs_path path);
/*
 * Test hook for the bounded waits of the look-back kernel (the only device-side waits on another
 * CTA).  `lookback_spin_limit` bounds the polls of a descriptor (0 restores the default);
 * `mute_tile` >= 0 makes that tile skip publishing its aggregate, so that the CTA that propagates
 * the carries and the tiles waiting for it run out of polls, record HS_ERR_LOOKBACK_TIMEOUT in the
 * workspace and leave;
 * -1 disables it.  Nothing faults or hangs: the kernel returns and the context stays usable.
 */
hs_status heinsen_scan_debug_config(uint32_t lookback_spin_limit, int64_t mute_tile);
/*
 * Checked build (the library compiled with -DHEINSEN_DEBUG; `python -m paper_2311_06281_b200.build_ext --debug`
 * writes it beside the normal one as libheinsen_scan_debug.so).  In that build every shared-memory access of
 * the kernels checks its address against the CTA's shared-memory window and its alignment, and the kernels
 * check the element, row, tile and TMA coordinates they are about to use.  A failed check never traps: it is
 * recorded and the access is skipped.
 *   heinsen_scan_debug_build()  : 1 in the checked build, 0 otherwise.
 *   heinsen_scan_debug_faults() : synchronises the device, copies the first recorded failure of the process to
 *                                 out[0..3] = {check code, detail (address or index), block, thread}, clears the
 *                                 record, and returns 1; 0 when nothing was recorded (always, in the normal
 *                                 build); -1 on a CUDA error.  `out` may be NULL.
 *   heinsen_scan_debug_window_ok(): the window predicate of those checks (addr, bytes inside [base, base + size),
 *                                 addr a multiple of align), exported so that it can be tested without a GPU.
 */
int heinsen_scan_debug_build(void);
int heinsen_scan_debug_faults(uint64_t out[4]);
int heinsen_scan_debug_window_ok(uint64_t addr, uint64_t bytes, uint64_t base, uint64_t size, uint64_t align);
/*
 * Tuning knobs, for sweeps and for tests that force a variant; every knob has a measured default
 * that is chosen per call.  `name` is one of "NO_TMA", "ROWS_PER_WARP", "WARPS", "STAGES",
 * "ROW_TICKETS", "SPANS", "NO_FLAT", "NO_PDL" (row-batched kernel), "LB_STAGES", "LB_WARPS",
 * "LB_SLEEP_IDLE", "LB_SLEEP_READY", "LB_CTAS_PER_SM" (look-back kernel); value >= 0 sets the knob
 * (clamped to its range), value < 0 returns it to its default.  The environment variables
 * HEINSEN_SCAN_<name> give the initial values; they are read once per process, not per call.
 * Unknown name: HS_ERR_INVALID_ARG.
 */
hs_status heinsen_scan_tune(const char* name, int value);
/*
 * Roofline probe (no passage of the paper: a measurement aid).  Runs a register-only kernel that does
 * nothing but ex2.approx / lg2.approx (the two transcendentals of Eq. 7-8 as the kernels evaluate them)
 * on every SM of the current device, on the legacy default stream, and returns after it has completed:
 * `results` = transcendental results produced, `seconds` = device time between two events around the
 * launch.  results / seconds / (SM count x SM clock) is the MUFU rate per clock and SM that bounds the
 * transcendental leg of the roofline.  iterations <= 0 or a null pointer: HS_ERR_INVALID_ARG.
 */
hs_status heinsen_scan_probe_mufu(int iterations, double* results, double* seconds);
/* Path taken by the most recent successful launch of this process (hs_path value), 0 if none. */
int heinsen_scan_last_path(void);
/* Number of kernels this library has launched in this process (memsets not counted). */
int64_t heinsen_scan_launch_count(void);

/* Static, NUL-terminated description of a status code. */
const char* heinsen_scan_strerror(hs_status status);

#ifdef __cplusplus
}
#endif
#endif /* HEINSEN_SCAN_H_ */
