/* bpdq.h -- C ABI of the BPDQ weight-only linear layer for NVIDIA B200 (sm_100a).
 *
 * The operation (paper: Methodology, Eq. 1; candidate values Eq. 7; Appendix A.2):
 *
 *     W^[r, j] = C0[r, G] + sum_{i=1..K} Ci[r, G] * Bi[r, j],   Bi in {0,1},  G = floor(j / g)
 *
 * a "variable grid": K bit-planes Bi of shape [out][in] plus K+1 scalar coefficients per
 * (output row r, input group G of g columns).  The layer output is the quantized weight
 * applied to the activations (paper: Section 3.1, the output-aligned objective compares W X
 * with W^ X), per token
 *
 *     y[m, r] = sum_j x[m, j] * W^[r, j].
 *
 * The paper fixes no inference arithmetic.  This library uses: coefficients stored as IEEE
 * binary16 (the paper's bits-per-weight figures, K + 16 (K+1) / g, leave room for nothing
 * else); a weight is decoded as float(c0), then for i = 1..K in order "if the bit is set add
 * float(ci)" in binary32, then rounded once to binary16 (bpdq_dequant returns exactly that
 * bit pattern); x and y are binary16, accumulation is binary32.
 *
 * Conventions
 *   - every function returns a status code (below) and never throws or aborts;
 *     bpdq_last_error() gives a thread-local text for the last non-OK status;
 *   - "host" / "device" says where a pointer must live.  Device pointers must be 16-byte
 *     aligned, tensors are dense row-major;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     that take a stream only enqueue work and do not synchronise, unless stated;
 *   - a handle owns its device copy of the packed weights and a scratch workspace.  Two calls
 *     on the same handle must not overlap on the GPU (issue them on one stream);
 *   - threads: calls that name the same handle (for bpdq_linear_batch: the same first handle,
 *     which keeps the launch plan) and all calls of bpdq_linear_noalloc on one device must be
 *     serialised by the caller; calls on different handles may run concurrently from
 *     different threads.  A handle is used with the device that was current when it was
 *     created: calling with another current device is BPDQ_ERR_INVALID, nothing is launched;
 *   - stream capture: once a handle has run a given kind of call outside a capture (its first use
 *     sets shared-memory limits, launch plans and tensor maps), bpdq_dequant, bpdq_linear,
 *     bpdq_linear_ex, bpdq_linear_batch and bpdq_gate_up_swiglu only enqueue kernels on `stream`
 *     (no allocation, no copy, no host wait) and may be recorded into a CUDA graph; x, y and the
 *     handles must then stay where they are for the replays.  The *_host calls, bpdq_get_status
 *     and bpdq_read_blob wait for the stream and cannot be recorded;
 *   - supported shapes: K in {1,2,3,4}; g in {64,128,256}; in % 128 == 0; out % 16 == 0.  Anything
 *     else is BPDQ_ERR_UNSUPPORTED.  With g = 256 and in % 256 == 128 the last group of a row holds the
 *     remaining 128 columns (ceil(in/g) groups per row; the paper applies g = 256 to a 29568-channel input
 *     and does not say how); the host producers take whole groups only.
 *
 * Logical tensors (what pack/unpack exchange with the caller)
 *   bits : uint8  [K][out][in], values 0/1; bits[i] is the paper's plane B_{i+1}
 *   coef : uint16 [K+1][out][ceil(in/g)], binary16 bit patterns; coef[0] is C0, coef[i] is Ci
 *
 * Packed blob (what lives in device memory), bpdq_packed_bytes() bytes, no padding:
 *   planes, then coefficients.
 *   planes : 32-bit words run along the input dimension; four words (128 columns, a "block")
 *            of one plane and one row form a 16-byte unit, and for a fixed block and plane
 *            the units of consecutive rows are adjacent, so that a warp reads 32 rows with one
 *            coalesced 512-byte request and a 128-row tile is one contiguous 2 KB run:
 *              unit(b, i, r) at byte ((b*K + i)*out + r)*16,   b = floor(j/128), i 0-based.
 *            Inside a unit: word k (k = 0..3, little-endian bytes 4k..4k+3) covers columns
 *            128*b + 32*k .. + 31, and bit 4*j + u of that word is column 128*b + 32*k + 8*u + j
 *            (j = 0..7, u = 0..3): eight consecutive columns sit one bit per nibble, which is the
 *            form the tensor-core kernel's byte-permute decode consumes.  Byte q of word k
 *            ("logical byte" L = 4*k + q) therefore holds, at bit 4*jj + u, column
 *            128*b + 32*k + 8*u + 2*q + jj (jj = 0..1).  The sixteen bytes are then rotated by
 *            the row number: physical byte p holds logical byte (p + r) mod 16.  Rows that a
 *            half-warp handles together therefore index sixteen different 8-column look-up
 *            tables at every step.
 *   coefs  : binary16 at byte planes_bytes + ((G*(K+1) + i)*out + r)*2.
 */
#ifndef BPDQ_H_
#define BPDQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BPDQ_API __attribute__((visibility("default")))
#else
#define BPDQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bpdq_handle_s* bpdq_handle_t;

enum {
    BPDQ_OK = 0,
    BPDQ_ERR_INVALID = 1,     /* null / misaligned pointer, bad size, M out of range          */
    BPDQ_ERR_UNSUPPORTED = 2, /* shape outside the supported set, or no sm_100 device         */
    BPDQ_ERR_ALLOC = 3,       /* device or host allocation failed                             */
    BPDQ_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed                          */
    BPDQ_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (read by bpdq_get_status) */
};

/* Which kernel bpdq_linear_ex runs. */
enum {
    BPDQ_KERNEL_AUTO = 0,     /* dispatch on M (what bpdq_linear does)                        */
    BPDQ_KERNEL_GEMV = 1,     /* look-up-table kernel, M <= BPDQ_GEMV_MAX_M                   */
    BPDQ_KERNEL_GEMM = 2,     /* tensor-core kernel (TMA + tcgen05), any M >= 1               */
    BPDQ_KERNEL_GEMV_SIMPLE = 3, /* one-bit-at-a-time kernel kept as an on-device cross-check */
    BPDQ_KERNEL_FEW = 4       /* few-token kernel (weights decoded in registers, warp-level
                                 tensor-core instructions), M <= BPDQ_FEW_MAX_M              */
};

#define BPDQ_GEMV_MAX_M 16
#define BPDQ_FEW_MAX_M 32
#define BPDQ_BATCH_MAX 16            /* most linears bpdq_linear_batch takes in one call */
#define BPDQ_NOALLOC_MAX_OUT 65536   /* most output rows bpdq_linear_noalloc accepts */

/* Storage accounting (paper: Table 1, column BPW = K + 16 (K+1) / g bits per weight).
 * Bytes of the packed blob: out*in*K/8 + out*ceil(in/g)*(K+1)*2.  Returns 0 for an unsupported
 * shape.  Host only, no CUDA call. */
BPDQ_API size_t bpdq_packed_bytes(int out, int in, int K, int group);

/* Host packer: logical tensors -> blob (layout above).  All pointers are host memory;
 * `blob` is caller-owned with bpdq_packed_bytes() bytes.  Every bit value must be 0 or 1
 * (BPDQ_ERR_INVALID otherwise).  Defines the storage of Eq. 1's B_i and C_i. */
BPDQ_API int bpdq_pack(const uint8_t* bits, const uint16_t* coef, int out, int in, int K, int group,
              void* blob);

/* Inverse of bpdq_pack: blob -> logical tensors.  unpack(pack(b, c)) == (b, c). */
BPDQ_API int bpdq_unpack(const void* blob, int out, int in, int K, int group, uint8_t* bits,
                uint16_t* coef);

/* Data-free producer of logical tensors from full-precision weights w (host, binary32 [out][in]): the
 * initialisation of the paper's quantizer without calibration data.  Per (row, group): asymmetric
 * round-to-nearest (ties to even) to an unsigned 8-bit code with scale (max - min) / 255 (paper:
 * Section 3.2, Eq. 5, Z = sum 2^i P_i); bits[i-1] = B_i = P_{7-K+i}, the K most significant planes;
 * coefficients by Eq. 6 with U_loc = I (least squares of the weights on [1, b_1, .., b_K], normal
 * equations in binary64, alpha * trace / (K+1) added to the diagonal; the paper uses alpha = 1e-4),
 * rounded to binary16.  bits / coef as for bpdq_pack.  Host only, no CUDA call.  NaN weights are
 * BPDQ_ERR_INVALID. */
BPDQ_API int bpdq_quantize_datafree(const float* w, int out, int in, int K, int group, double alpha, uint8_t* bits,
                           uint16_t* coef);

/* Multi-precision view (paper: closing section, serving several precisions from one stored model;
 * the mechanism is this library's reading): from logical tensors with K planes, those with the K2
 * most significant planes B_{K-K2+1}..B_K and their coefficients; every dropped plane adds half its
 * coefficient to the offset (binary32 adds in plane order, one rounding to binary16).  bits2
 * [K2][out][in], coef2 [K2+1][out][in/g] are caller-owned and may alias nothing.  Host only. */
BPDQ_API int bpdq_truncate_planes(const uint8_t* bits, const uint16_t* coef, int out, int in, int K, int group, int K2,
                         uint8_t* bits2, uint16_t* coef2);

/* Creates a layer on the current CUDA device.  `host_blob` (host memory, bpdq_packed_bytes()
 * bytes) is copied to the device; if it is NULL the blob is generated on the device from
 * `seed` with the counter-based generator of the synthetic workloads (plane bits iid
 * Bernoulli(1/2); c0 ~ N(0, 0.02); c1, c2 ~ U(0.005, 0.05); c3.. ~ U(0.002, 0.02)), which
 * reproduces the host generator bit for bit.  `max_M` (>= 1) bounds the token count of later
 * bpdq_linear calls and sizes the workspace.  Synchronises the device.  On failure *h is
 * NULL. */
BPDQ_API int bpdq_create(bpdq_handle_t* h, int out, int in, int K, int group, const void* host_blob,
                uint64_t seed, int max_M);

/* Eq. 1 materialised: writes W^ as binary16 [out][in] row-major to `w_fp16_dev` (device,
 * caller-owned, out*in*2 bytes).  Bit-exact with the decode rule stated at the top. */
BPDQ_API int bpdq_dequant(bpdq_handle_t h, void* w_fp16_dev, void* stream);

/* The quantized linear map y = x * W^T (paper: Eq. 1 applied to activations, Section 3.1).
 * x: device binary16 [M][in]; y: device binary16 [M][out]; 0 <= M <= max_M.  M == 0 returns
 * BPDQ_OK without a launch.  Picks the look-up-table kernel for the smallest M (default: up to
 * 2 tokens, 3 at K = 4 and g >= 128), the few-token kernel above that (default: up to 16 tokens) and the tcgen05 kernel
 * beyond (also below when the packed weights of the linear reach 4 GB, which the look-up-table
 * kernel's 32-bit offsets do not cover).  x and y must not alias. */
BPDQ_API int bpdq_linear(bpdq_handle_t h, const void* x_fp16_dev, void* y_fp16_dev, int M, void* stream);

/* Same map with the kernel chosen by the caller (BPDQ_KERNEL_*).  BPDQ_KERNEL_GEMV with
 * M > BPDQ_GEMV_MAX_M is BPDQ_ERR_INVALID. */
BPDQ_API int bpdq_linear_ex(bpdq_handle_t h, const void* x_fp16_dev, void* y_fp16_dev, int M, int kernel,
                   void* stream);

/* Several independent linears in one launch (decode: q, k, v of one token, or gate and up, or a
 * whole layer's linears when their inputs do not depend on each other).  y[k] = x[k] * W^[k]^T
 * for k = 0..n-1, each as bpdq_linear computes it for this M: the look-up-table kernel up to the
 * first handle's look-up-table threshold, the few-token kernel above it (up to its threshold,
 * when every linear allows it), else passes of the look-up-table kernel; the task spaces of the
 * n linears are concatenated, so launch ramp, set-up and tail are paid once instead of n times.  hs, xs, ys are HOST arrays of n
 * handles / device pointers (read before the call returns); 1 <= n <= BPDQ_BATCH_MAX; the
 * handles are distinct, live on the current device, share K, and either all or none of them
 * have group 64;
 * 0 <= M <= min(max_M of every handle, BPDQ_GEMV_MAX_M).  Inputs may be shared between
 * linears; outputs must not overlap anything else.  BPDQ_ERR_INVALID / BPDQ_ERR_UNSUPPORTED
 * otherwise, with nothing launched. */
BPDQ_API int bpdq_linear_batch(const bpdq_handle_t* hs, const void* const* xs_fp16_dev, void* const* ys_fp16_dev, int n,
                      int M, void* stream);

/* bpdq_linear_batch for callers whose activations live in HOST memory: brings every x[k] (host, [M][in_k])
 * into its handle's staging buffer, runs bpdq_linear_batch, returns every y[k] to host memory and waits for
 * the stream once.  Same argument rules as bpdq_linear_batch.  When every buffer is pinned (page-locked)
 * and 16-byte aligned, one gather kernel reads all x through their device-visible addresses and the
 * look-up-table kernel stores y straight into host memory: two launches and one wait per call.  Pageable
 * or unaligned buffers take one copy per buffer and direction instead. */
BPDQ_API int bpdq_linear_batch_host(const bpdq_handle_t* hs, const void* const* xs_fp16_host, void* const* ys_fp16_host, int n,
                           int M, void* stream);

/* Same map for callers whose activations live in HOST memory: copies x (host, [M][in]) to a
 * handle-owned staging buffer, runs bpdq_linear, copies y back to `y_fp16_host` and waits for
 * the stream.  Pinned host memory makes the copies asynchronous up to that wait; token counts that
 * go to the look-up-table kernel take bpdq_linear_batch_host's path with n = 1. */
BPDQ_API int bpdq_linear_host(bpdq_handle_t h, const void* x_fp16_host, void* y_fp16_host, int M,
                     void* stream);

/* The look-up-table kernel without a handle and without any allocation.  (The paper has no
 * counterpart: this entry point exists for callers that cannot allocate device memory at the
 * time they need the layer -- a plug-in whose host application reserves all device memory up
 * front and hands out one arena that already holds the packed weights, a process running under
 * a memory budget in which a later cudaMalloc may fail, or a latency-critical loop in which the
 * implicit device synchronisation of an allocation is not acceptable.)
 *
 * blob_dev is the packed blob (layout above, bpdq_packed_bytes() bytes) already in DEVICE memory,
 * caller-owned; x [M][in] and y [M][out] as for bpdq_linear, 0 <= M <= BPDQ_GEMV_MAX_M.  All
 * three pointers 16-byte aligned.  The kernel's scratch (binary32 row sums, arrival counters,
 * status word) is a static device array inside the library, about 0.5 MB, held by every GPU
 * that loads the library until the process exits; it bounds the layer at
 * out <= BPDQ_NOALLOC_MAX_OUT rows (larger: BPDQ_ERR_INVALID, nothing is launched).  Shapes as
 * for bpdq_create.
 *
 * The first call on a device looks up the array's device address and two device attributes;
 * make that first call outside any stream capture.  No call allocates or frees device or host
 * memory.  Every call on a device uses the same array: it is cleared on `stream` before the
 * kernel runs, so two calls that overlap on the GPU (different streams, different threads)
 * race on it -- issue them on one stream.  Asynchronous like bpdq_linear.  There is no handle, so
 * bpdq_get_status cannot report on these calls: the status word lives in the same array and is
 * cleared by the next call. */
BPDQ_API int bpdq_linear_noalloc(const void* blob_dev, int out, int in, int K, int group, const void* x_fp16_dev,
                        void* y_fp16_dev, int M, void* stream);

/* Input-channel permutation (paper: Section 4, the quantizer reorders channels with Group-Aware
 * Reordering and keeps the quantized matrix in that order; how inference undoes it is this
 * library's reading).  With perm set (host, int32 [in], a permutation of 0..in-1; copied), every
 * linear call on the handle computes y[m,r] = sum_j x[m, perm[j]] * W^[r,j]: the look-up-table
 * kernel reads x through perm while it builds its tables, the other kernels run on a gathered copy
 * of x that one extra launch writes into a handle-owned buffer.  NULL restores the identity.
 * Synchronises the device. */
BPDQ_API int bpdq_set_input_permutation(bpdq_handle_t h, const int32_t* perm_host);

/* Bias (not part of the paper's method; decoder layers carry one on q, k and v): binary16 [out] on
 * the host, copied; added in binary32 to every output row before the rounding to binary16, in
 * every kernel.  NULL removes it.  Synchronises the device. */
BPDQ_API int bpdq_set_bias(bpdq_handle_t h, const uint16_t* bias_fp16_host);

/* The gated unit around a (gate, up) pair that shares its input: h[m,r] = silu(g) * u with
 * g = x W^gate^T (+ bias), u = x W^up^T (+ bias), silu(v) = v / (1 + exp(-v)), evaluated in binary32
 * and rounded to binary16 (not part of the paper's method: the step that follows these two
 * linears in the decoder layers the paper measures).  Both handles have
 * the same out, in and K and live on the current device; 0 <= M <= min(max_M).  Up to the
 * few-token threshold the two linears run in one launch and the kernel that completes a block of
 * rows applies the unit to the unrounded binary32 sums (nothing but h is written); above it two
 * tcgen05 launches write g and u, rounded to binary16, to handle-owned buffers and a third launch
 * applies the unit.  x, h_out: device binary16 [M][in] /
 * [M][out], 16-byte aligned. */
BPDQ_API int bpdq_gate_up_swiglu(bpdq_handle_t gate, bpdq_handle_t up, const void* x_fp16_dev, void* h_fp16_dev, int M,
                        void* stream);

/* Sets the largest M that bpdq_linear sends to the look-up-table kernel (0 = always use the
 * tensor-core kernel; at most BPDQ_GEMV_MAX_M). */
BPDQ_API int bpdq_set_gemv_max_m(bpdq_handle_t h, int max_gemv_m);

/* Sets the largest M that bpdq_linear sends to the few-token kernel once M is above the look-up-table
 * threshold (0 = never; at most BPDQ_FEW_MAX_M and the handle's max_M). */
BPDQ_API int bpdq_set_few_max_m(bpdq_handle_t h, int max_few_m);

/* Copies the device blob back to host memory (bpdq_packed_bytes() bytes); synchronises. */
BPDQ_API int bpdq_read_blob(bpdq_handle_t h, void* host_blob);

/* Waits for `stream` and returns the handle's device status word: BPDQ_OK, or
 * BPDQ_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the result of that call is
 * then undefined; the context stays usable).  Clears the word. */
BPDQ_API int bpdq_get_status(bpdq_handle_t h, void* stream);

/* Diagnostic for the bounded device-side waits: enqueues a one-warp kernel that waits, with the bounded wait every
 * kernel of the library uses (cut to 50 ms; the kernels allow two seconds), on a barrier that nothing arrives at.  The wait gives up,
 * records BPDQ_ERR_TIMEOUT in the handle's status word and the kernel ends normally: the next bpdq_get_status
 * returns BPDQ_ERR_TIMEOUT once and the handle stays usable.  Nothing else is touched. */
BPDQ_API int bpdq_probe_wait_limit(bpdq_handle_t h, void* stream);

/* Number of kernels this handle has launched since creation (bookkeeping for benchmarks). */
BPDQ_API int bpdq_launch_count(bpdq_handle_t h, uint64_t* count);

/* Frees everything the handle owns; synchronises the device.  NULL is BPDQ_OK. */
BPDQ_API int bpdq_destroy(bpdq_handle_t h);

/* Text of the calling thread's last non-OK status ("" if none). */
BPDQ_API const char* bpdq_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BPDQ_H_ */
