/*
 * elutq.h - C ABI of the B200 (sm_100a) HLQ look-up-table GEMM/GEMV library.
 *
 * The library multiplies fp16 activations X[M,K] by Hierarchical-Linear-Quantized
 * weights W_hat[N,K] without dequantising them.  HLQ (paper Section 4.1, Eq. 3)
 * stores a weight as
 *
 *      W_hat[n,k] = sum_{j<q} s[n, k/G, j] * b_j[n,k] + z[n, k/G],   b_j in {0,1},
 *
 * with per-group, per-bit-plane fp16 scales s and per-group fp16 offsets z, groups
 * of G consecutive k (Algorithm 1: s in R^{N x K/G x q}, z in R^{N x K/G}).  The
 * product is evaluated with the bit-serial look-up-table procedure of Appendix B:
 * tables of partial activation sums are built in shared memory per call, each
 * bit-plane byte addresses a table entry, entries are summed per group in fp32,
 * multiplied by the group's per-plane scale, and the offset contributes
 * z[n,Gi] * sum_{k in Gi} x[k].
 *
 * Conventions
 *   - All entry points return an elutq_status (0 = ok, negative = error); none
 *     throws, aborts or traps.  Arguments are validated on the host before any
 *     launch; on error nothing is launched and outputs are untouched.
 *   - "device" pointers are CUDA device memory of the current device; the caller
 *     owns every buffer it passes.  `stream` is a cudaStream_t passed as void*
 *     (NULL = the legacy default stream).  Work is asynchronous on `stream`.
 *   - X, Y and `packed` must be 16-byte aligned; `planes` 8-byte aligned.
 *   - q in [1,4]; G in {32, 64, 128}; K a multiple of G; M, N >= 1 (any value).
 *   - Matrices are row-major and dense: X[M][K] fp16, Y[M][N] fp16 (or fp32).
 */
#ifndef ELUTQ_H_
#define ELUTQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum elutq_status {
    ELUTQ_OK = 0,
    ELUTQ_ERR_INVALID_ARG = -1,      /* null pointer, non-positive size, bad flag combination */
    ELUTQ_ERR_SHAPE = -2,            /* q/G out of range, K % G != 0, or (N,K) do not match the blob */
    ELUTQ_ERR_ALIGN = -3,            /* a pointer is not aligned as required */
    ELUTQ_ERR_BUFFER_TOO_SMALL = -4, /* packed_bytes / workspace_bytes below the required size */
    ELUTQ_ERR_UNSUPPORTED = -5,      /* valid request this build has no kernel for */
    ELUTQ_ERR_CUDA = -6              /* a CUDA call failed; see elutq_last_cuda_error() */
} elutq_status;

/* Flags of elutq_lut_gemm_ws / elutq_lut_gemm_f32. */
#define ELUTQ_FLAG_SKIP_OFFSET 0x1u /* leave out the z * sum(x) term (Eq. 3 with z = 0)            */
#define ELUTQ_FLAG_OFFSET_ONLY 0x2u /* only the z * sum(x) term; bit-planes are not read           */
#define ELUTQ_FLAG_OUT_F32     0x4u /* Y is float[M][N] instead of fp16 (no final fp16 rounding)   */
#define ELUTQ_FLAG_ACCUMULATE  0x8u /* Y += result (the sum is formed in fp32, rounded once)        */
#define ELUTQ_FLAG_PLAIN_G4    0x10u /* use two 16-entry (g = 4) tables per byte instead of the
                                        fused 256-entry table; same result up to fp32 rounding      */

#define ELUTQ_FLAG_CLUSTER_REDUCE 0x20u /* M = 1, K <= 4096 only: launch one thread-block cluster per row range
                                           (one CTA per 512-column chunk) and reduce the K split through
                                           distributed shared memory instead of the workspace + finalize
                                           kernel; same result bit for bit, measured equally fast          */

#define ELUTQ_FLAG_MIRROR 0x40u /* M = 1, G = 128: mirror storage of Appendix D - the weights are read as
                                   s^_j * b^_j + z^ with b^ = 2b - 1, s^ = s/2, z^ = z + (1/2) sum_j s_j
                                   (both formed in fp32), the tables hold the +-1 partial sums for the 128
                                   indices with the top bit clear and the other half is obtained by
                                   negation; same product up to fp32 rounding                              */

#define ELUTQ_TENSOR_MIN_M 9      /* batches of this many rows or more take the tensor-core path (G = 128, no
                                     look-up variant flag): the batched look-up kernel needs one pass per 4 rows,
                                     the tensor-core kernel's time does not depend on M up to 128              */
#define ELUTQ_TENSOR_MIN_M_NARROW 5   /* ... and so do batches of 5 to 8 rows when N <= ELUTQ_TENSOR_NARROW_N: there  */
#define ELUTQ_TENSOR_NARROW_N 8192    /* the second look-up pass already costs more than the tensor-core call (measured
                                         on the 8B shapes at M = 8, q = 2 / 3, us: qkv 6144 x 4096 17.1 / 20.8 against
                                         15.4 / 17.7, o 4096 x 4096 13.4 / 16.8 against 11.7 / 13.3, down 4096 x 14336
                                         27.3 / 36.3 against 26.3 / 32.0; gate_up 28672 x 4096 43.9 / 60.6 against
                                         48.8 / 66.5 stays on the look-up kernel).  elutq_takes_tensor_path says which
                                         path a call takes.                                                    */

#define ELUTQ_FLAG_LUT_ONLY 0x80u /* M >= 9: stay on the look-up-table kernels.  Without this flag batches of
                                     ELUTQ_TENSOR_MIN_M rows or more (G = 128) take the dequantise-and-contract path: the
                                     weight tile is rebuilt in fp16 from the bit-planes (BCQ form of
                                     Appendix D) and contracted on the tensor cores with fp32 accumulation;
                                     its results carry the fp16 rounding of W_hat (about 3e-4 relative)     */

#define ELUTQ_FLAG_TABLE_F16 0x100u /* M >= 2, G = 128: table quantisation of Appendix D, first form - the look-up
                                      tables hold fp16 entries (formed in fp32, rounded once), so one 16-byte
                                      load serves 8 activation rows instead of 4; accumulation stays fp32.  A
                                      lossy variant: each entry carries a 2^-11 relative rounding (about 3e-4
                                      on Y).  Stays on the look-up kernels at every M; ignored at M = 1          */

#define ELUTQ_FLAG_TABLE_I8 0x200u  /* M >= 2, G = 128: table quantisation of Appendix D, second form - the look-up
                                      tables hold int8 entries (round to nearest of entry / scale, one scale per
                                      activation row and 128-column group = largest possible |entry| / 127), 8 rows
                                      per 8-byte load, integer accumulation inside a group.  Lossy by design: about
                                      5e-3 relative error on Y, outside the 1e-3 bar of the other paths.  Not
                                      combinable with ELUTQ_FLAG_TABLE_F16; ignored at M = 1                     */

#define ELUTQ_HEADER_BYTES 128

/* Human-readable name of a status code (static string, never NULL). */
const char* elutq_status_string(int status);

/* The cudaError_t value of the most recent failed CUDA call on this thread (0 if none). */
int elutq_last_cuda_error(void);

/*
 * Size in bytes of the device layout of one layer (Appendix D "weight rearrange":
 * the one-bit matrices are rearranged offline so the kernel's loads are contiguous).
 * Pure function, no CUDA call.  The layout is q*N*K/8 bit-plane bytes +
 * 2*(q+1)*N*K/G parameter bytes (the paper's q + 16(q+1)/G bits per weight) + a
 * 128-byte header, with N rounded up to 16 and K to 512 by zero padding.
 */
int elutq_packed_bytes(int q, int G, int N, int K, size_t* bytes);

/*
 * Offline packing (Appendix B: the bit-plane split is given by the caller;
 * Appendix D: rearrangement).  Inputs, all device memory:
 *   planes   uint8 [q][N][K], a weight bit is (value != 0); plane j pairs with scale j
 *   scales   fp16  [N][K/G][q]
 *   offsets  fp16  [N][K/G]
 * Output: `packed`, a caller-owned device buffer of at least elutq_packed_bytes()
 * bytes, fully overwritten.  The blob is self-describing (header) and position
 * independent: it may be copied or stored and used at another address.
 */
int elutq_pack(const uint8_t* planes, const void* scales, const void* offsets,
               int q, int G, int N, int K, void* packed, size_t packed_bytes, void* stream);

/*
 * Inverse of elutq_pack (test/debug): recovers planes (uint8 0/1), scales and
 * offsets bit-exactly into caller-owned device buffers of the shapes above.
 */
int elutq_unpack(const void* packed, int N, int K, uint8_t* planes, void* scales,
                 void* offsets, void* stream);

/*
 * Reads q and G of the blob that is at `packed` now: the 128-byte header is copied
 * to the host (a synchronous cudaMemcpy - not during stream capture) and what the
 * library remembers about the address is refreshed.  Any of q, G may be NULL.
 * ELUTQ_ERR_SHAPE if the header is not a valid blob for (N, K).
 *
 * The GEMM entry points remember (q, G, N, K) per device address - from elutq_pack,
 * from this call, or from a header read on first use - so that a call costs no
 * copy.  A remembered description can go stale (the buffer was freed and its
 * address now holds another blob that arrived by a plain copy).  That is caught on
 * the device: every kernel that reads tiles first compares the blob's header with
 * the (q, G, N, K) it was launched for and, on a mismatch, raises the device status
 * ELUTQ_DEVICE_BLOB_MISMATCH and returns without reading a tile or writing Y.
 * Call elutq_describe (or elutq_forget) after replacing a blob in place.
 */
int elutq_describe(const void* packed, int N, int K, int* q, int* G);

/* Forget what the library remembers about `packed` (the next use reads the header). */
int elutq_forget(const void* packed);

/* Device status words (elutq_device_status, elutq_chain_status). */
#define ELUTQ_DEVICE_WAIT_EXPIRED  0x7C05 /* a bounded device-side wait ran out                        */
#define ELUTQ_DEVICE_BLOB_MISMATCH 0x7C0B /* a blob's header did not match what the kernel was given   */

/*
 * Scratch memory the GEMM needs for (M,N,K): a small reserved control area and the
 * fp32 partial sums of the K-split (one partial per 512-wide K chunk for M = 1, per
 * 256-wide half chunk for M > 1, summed in ascending chunk order by the finalize
 * kernel, so results are bit-reproducible).
 */
int elutq_workspace_bytes(int M, int N, int K, size_t* bytes);

/* Zero a caller-owned workspace.  Required once before its first use, and again
 * before it is used for a different (M, N, K): the kernels leave the counters at
 * zero after every call, but where they sit depends on the shape. */
int elutq_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Y[M,N] = X[M,K] * W_hat^T with scales and offsets applied (Eq. 3 under the
 * bit-serial LUT procedure of Appendix B), fp32 tables and accumulation, one
 * round-to-nearest-even conversion to fp16 at the end.
 *   X, Y, packed: device.  `packed` must be complete when the call is enqueued:
 *   the kernels start reading it before they wait for the work that precedes
 *   them on the stream (weights do not depend on the previous kernel; X, Y and the
 *   scratch do).  After elutq_pack on the same stream that holds - pack kernels
 *   run to completion before a dependent launch starts - but a producer of
 *   `packed` that triggers programmatic dependent launches early must be
 *   synchronised with first.
 *   Scratch comes from library-owned buffers per (device, stream), allocated with
 *   cudaMalloc on the first call that needs them or needs larger ones.  A buffer
 *   that has to grow is replaced, never freed: the old one stays allocated until
 *   elutq_release_scratch, because a CUDA graph captured earlier still carries its
 *   address.  While `stream` is being captured nothing is allocated: a call that
 *   would need more scratch than the stream has returns
 *   ELUTQ_ERR_BUFFER_TOO_SMALL.  So before capturing, make one warm-up call per
 *   shape or call elutq_reserve with the largest one; graph users who want no
 *   library-owned memory at all use elutq_lut_gemm_ws or elutq_lut_gemm_static.
 *   Calls that share a stream are ordered; calls on different streams use
 *   different scratch buffers.
 */
int elutq_lut_gemm(const void* X, const void* packed, void* Y, int M, int N, int K, void* stream);

/* Make the library-owned scratch of `stream` large enough for any call up to (M, N, K), including the
 * staging buffers of elutq_lut_gemm_host (allocates; not during capture). */
int elutq_reserve(int M, int N, int K, void* stream);

/* Address and size of one library-owned buffer of `stream` (kind 0 = control words, 1 = X staging,
 * 2 = Y staging, 3 = K-split partial sums); *ptr = NULL when none exists yet.  For tests and tools. */
int elutq_scratch_address(void* stream, int kind, void** ptr, size_t* bytes);

/*
 * Only the offset term of Eq. 3: Y[m,n] (+)= sum_Gi z[n,Gi] * sum_{k in Gi} X[m,k].
 * accumulate != 0 adds into the existing fp16 Y (fp32 sum, rounded once).
 */
int elutq_lut_gemm_bias(const void* X, const void* packed, void* Y, int M, int N, int K,
                        int accumulate, void* stream);

/* Same product with fp32 output (no fp16 rounding) and the ELUTQ_FLAG_* options
 * (OUT_F32 is implied).  Test/debug entry; scratch as elutq_lut_gemm. */
int elutq_lut_gemm_f32(const void* X, const void* packed, float* Y, int M, int N, int K,
                       unsigned flags, void* stream);

/*
 * The general entry: as above with explicit flags and a caller-owned workspace
 * (device, 16-byte aligned, >= elutq_workspace_bytes(M,N,K), initialised by
 * elutq_workspace_init for this shape).  Never allocates.  Two calls that run concurrently must
 * not share a workspace.
 */
int elutq_lut_gemm_ws(const void* X, const void* packed, void* Y, int M, int N, int K,
                      unsigned flags, void* workspace, size_t workspace_bytes, void* stream);

/*
 * End-to-end convenience for host callers: X_host (fp16 [M][K]) is copied to the
 * device, the product runs, and Y (fp16 [M][N]) is copied back to Y_host, all on
 * `stream` (use pinned host memory for the copies to be asynchronous).  `packed`
 * stays a device pointer.  Staging buffers are library-owned like the scratch of
 * elutq_lut_gemm.  The call returns without synchronising.  When both host buffers are pinned and
 * addressable by the device and together at most 1 MiB (decode, small batches), X is pulled across the
 * bus by a small kernel and Y is stored straight into host memory by the epilogue (no copy-engine
 * operations, which cost several microseconds each); otherwise two cudaMemcpyAsync are used.
 */
int elutq_lut_gemm_host(const void* X_host, const void* packed, void* Y_host,
                        int M, int N, int K, void* stream);

/*
 * (No counterpart in the paper: an addition for deployments that must not allocate.)
 * Same product as elutq_lut_gemm - Y[M,N] fp16 = X[M,K] * W_hat^T, all device pointers - for
 * callers that cannot allocate device memory: a component embedded in a runtime that owns the
 * whole device arena, a decode loop that cannot afford the device-wide stall of cudaMalloc or
 * cudaFree, a process held to a fixed memory budget.  The K-split scratch lives in a 4 MiB array
 * that is part of the library image on every GPU that loads it; the call never invokes
 * cudaMalloc, cudaFree or any allocating routine.
 *   - Limit: C * M * 16*ceil(N/16) * 4 bytes must not exceed 4 MiB, with C = ceil(K/512) K
 *     chunks for M = 1 and C = 2*ceil(K/512) for M > 1 (every M = 1 LLaMA-3.1 8B/70B shape
 *     fits); larger requests return ELUTQ_ERR_BUFFER_TOO_SMALL and launch nothing.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before any stream capture begins.
 *   - All calls on a device share the array, which keeps the previous call's contents (nothing
 *     needs clearing: every value read was written by the same call).  Calls that overlap on the
 *     GPU, e.g. on different streams, race on it: keep them stream-ordered.
 *   - Every M stays on the look-up kernels here (the tensor-core path needs more scratch than the array
 *     holds), so from M = 9 on the result differs from elutq_lut_gemm's in rounding (it is the more
 *     accurate of the two: W_hat is never rounded to fp16) and the call is slower.
 *   - `packed` must be known to the library (packed or described in this process) before a capture
 *     begins: an unknown address makes the call read the header with a synchronous copy.
 */
/* 1 when elutq_lut_gemm (and _f32, _ws, _host, _bias) runs a call of this shape on the tensor-core path, 0 when on the
 * look-up kernels; host-only, launches nothing.  (The tensor-core path's results carry the fp16 rounding of W_hat.) */
int elutq_takes_tensor_path(int M, int N, int K, int G, unsigned flags);

int elutq_lut_gemm_static(const void* X, const void* packed, void* Y, int M, int N, int K, void* stream);

/*
 * A decode step as one launch (Appendix B's procedure at M = 1, call after call).
 *
 * At M = 1 every linear of a decode step is one bit-serial LUT GEMV; launched one by one, each pays its own
 * kernel start, K-split reduction and kernel end, during which HBM idles.  A chain runs a fixed list of
 * such calls - typically all linears of a decode step, in model order - in ONE persistent launch (calls of
 * G = 128 may mix bit-widths freely; for other group sizes a launch takes a run of consecutive calls with equal
 * (q, G), and a list is cut where the group size changes):
 * Y_c[N_c] = X_c[K_c] * W_hat_c^T for c = 0 .. n_calls-1, each result identical in value to elutq_lut_gemm
 * up to the order of the fp32 K-chunk sum (chunks are always added in ascending order, so a chain is
 * bit-reproducible from launch to launch).
 *
 * Ordering: the results are those of the calls run one after another in list order.  The plan derives from
 * the buffer addresses which earlier calls a call really depends on - its X or Y overlaps their Y, or its Y
 * their X - and the launch waits exactly for those; calls whose buffers are disjoint overlap freely (a
 * decode step whose linears read separately produced activations streams without a pause, a chain in which
 * Y of one call is X of the next is run strictly in turn).
 *
 *   elutq_chain_plan_bytes  size of the plan buffer for a list on the current device (it depends on the SM count;
 *                           nothing is launched)
 *   elutq_chain_plan        validates the list, reads q and G of every blob (elutq_describe's rules) and
 *                           writes the plan into `plan`: caller-owned DEVICE memory, 256-byte aligned, of
 *                           at least that size.  It holds the descriptors, the K-split scratch and the
 *                           hand-over counters.  Synchronises `stream`; an offline step, once per list.
 *                           Pointers and shapes are frozen in the plan; the buffers they name may change
 *                           content between runs.  M is 1; flags per call: ELUTQ_FLAG_OUT_F32,
 *                           ELUTQ_FLAG_ACCUMULATE (others: ELUTQ_ERR_UNSUPPORTED).
 *   elutq_chain_run         one launch on `stream` per run, normally one in all (one CTA per SM; the first launch is
 *                           cooperative: the device must be able to hold its CTAs all at once, else
 *                           ELUTQ_ERR_CUDA and nothing runs).  Allocates nothing.  Runs of one plan must not
 *                           overlap on the GPU.  Every CTA first compares the header of each blob of its launch
 *                           with the plan; on a mismatch that launch ends with status 0x7C0B without reading a
 *                           tile or writing an output.
 *   elutq_chain_run_opts    the same with an explicit poll limit for the hand-over waits (0 = default, 2^22);
 *                           a test entry.
 *   elutq_chain_run_host    a run whose activations come from and whose outputs go to HOST memory, with one
 *                           transfer per direction: on `stream`, brings x_bytes from x_host to x_dev, runs the
 *                           plan, copies y_bytes from y_dev to y_host.  x_dev and y_dev are the caller's device
 *                           buffers that the plan's calls point into (typically one arena that holds every
 *                           call's X and one that holds every Y).  Page-locked x_host (16-byte aligned like
 *                           x_dev, x_bytes a multiple of 16 and at most 8 MiB) is fetched by a small kernel in
 *                           front of the chain, whose threads read it across the bus, instead of a copy
 *                           operation, which costs two hand-overs between copy engine and SMs (measured on the
 *                           twelve 8B calls, 160 KB of activations: 71.5 against 73.8 us per step); any other
 *                           x_host is copied with cudaMemcpyAsync (synchronous for pageable memory).
 *                           x_host must stay unchanged until the run has completed.  y_host should be pinned.
 *                           A size of 0 skips that transfer: the Y of a call may itself name pinned host memory
 *                           (it is device-accessible under unified addressing), in which case the reduction's
 *                           stores cross the bus while the launch runs and no copy out is needed (7 us per step
 *                           less than with the copy; the X of a CALL should not name host memory: every CTA
 *                           would read it across the bus, 144 us).  Returns as elutq_chain_run
 *                           (ELUTQ_ERR_INVALID_ARG for a null pointer with a non-zero size); the outputs are valid
 *                           on the host when `stream` has been synchronised.  The paper's decode loop keeps
 *                           activations on the device and has no counterpart of this call; it is the end-to-end
 *                           form of a step for a caller whose activations live on the host.
 *   elutq_chain_status      synchronises `stream` and reads the plan's status word: 0, or 0x7C05 after a
 *                           hand-over wait ran out (every wait is a bounded poll; the launch then finishes
 *                           without waiting any further and its results are undefined), or 0x7C0B.  After a
 *                           non-zero status the plan must be written again with elutq_chain_plan.
 */
typedef struct elutq_gemv_call {
    const void* X;        /* device fp16 [K]                                   */
    const void* packed;   /* device blob of elutq_pack for (N, K)              */
    void* Y;              /* device fp16 [N] (float [N] with ELUTQ_FLAG_OUT_F32) */
    int N, K;
    unsigned flags;
} elutq_gemv_call;

#define ELUTQ_CHAIN_MAX_CALLS 4096

int elutq_chain_plan_bytes(const elutq_gemv_call* calls, int n_calls, size_t* bytes);
int elutq_chain_plan(const elutq_gemv_call* calls, int n_calls, void* plan, size_t plan_bytes, void* stream);
int elutq_chain_run(void* plan, int n_calls, void* stream);
int elutq_chain_run_opts(void* plan, int n_calls, unsigned wait_limit, void* stream);
int elutq_chain_run_host(void* plan, int n_calls, void* x_dev, const void* x_host, size_t x_bytes, const void* y_dev,
                         void* y_host, size_t y_bytes, void* stream);
int elutq_chain_status(const void* plan, void* stream, int* status);
/* The library keeps a small host-side note per planned buffer (which runs of calls to launch);
 * elutq_chain_run returns ELUTQ_ERR_SHAPE for a buffer that this process has not planned.  Call this before
 * freeing a plan buffer. */
int elutq_chain_forget(const void* plan);
/* Host logic of elutq_chain_plan for ONE call, without any CUDA call (for tests and for sizing questions): how a call
 * of shape (N, K) is cut over the n_ctas_max CTAs of a launch.  shares: int [n_ctas_max][4], per CTA (first row
 * block, end row block, first chunk, chunks | chunk group << 16), zeros for a CTA without a share; row blocks are 16
 * rows, chunks 512 columns; the shares go to CTAs cta_first, cta_first + 1, ... modulo n_ctas_max, as in a plan, where
 * cta_first is the sum of the earlier calls' CTA counts.  independent != 0: the call neither waits for the call before
 * it nor is waited for by the call after it (a small such call takes fewer CTAs).  partition: int [4] = chunks per
 * CTA, row ranges, chunk groups, CTAs with a share.  ELUTQ_ERR_UNSUPPORTED: more chunk groups than CTAs. */
int elutq_chain_shares(int N, int K, int n_ctas_max, int cta_first, int independent, int* shares, int* partition);

/*
 * Algorithm 1 (Section 4.2): alternating optimisation of the HLQ parameters, the offline step that
 * produces what elutq_pack consumes.  For every group of G consecutive weights of a row: uniform
 * initialisation (Delta = (max - min) / (2^q - 1), s = [Delta, 2 Delta, ...], z = min), then t_max
 * rounds of bit-pattern selection (nearest of the 2^q candidates, Eq. 5; ties to the smallest code,
 * code digit j = b_j) and least squares for (s, z) on the selected bits.  A round whose normal
 * equations are singular (decided exactly, on the integer bit counts) keeps the previous parameters.
 * Arithmetic is fp64 in a fixed order, so planes and parameters are reproducible bit for bit.
 *   W          device fp16 [N][K], finite values
 *   planes     device uint8 [q][N][K], written 0 / 1 (B of the last round)
 *   scales     device fp16 [N][K/G][q]; offsets device fp16 [N][K/G] (s, z of the last round)
 *   err_trace  NULL, or device double [(t_max + 1)][N * K/G]: squared error of every group for the
 *              uniform initialisation (row 0) and after each round (fp64 parameters)
 * t_max in [1, 1000] (the paper uses 10).  All buffers are caller-owned; nothing is allocated.
 */
int elutq_hlq_fit(const void* W, int q, int G, int N, int K, int t_max, uint8_t* planes, void* scales,
                  void* offsets, double* err_trace, void* stream);

/*
 * Device-side status of the library-owned scratch of `stream` (synchronises the stream).
 * *status is 0 unless a kernel gave up on a bounded wait (then a non-zero code that stays set
 * until elutq_release_scratch).  Kernels never spin without a limit.
 */
int elutq_device_status(void* stream, int* status);

/*
 * Test entry for the bounded waits of the tensor-core kernel (9 <= M <= 128, G = 128, K >= 384): the call is
 * launched with the issuing thread told to issue no MMA and no completion signal and with the poll limit of the
 * device-side waits set to `wait_limit`, so that the waits for MMA completion run out: the kernel gives up
 * waiting, still joins every barrier, frees its tensor memory and returns; elutq_device_status then reads
 * ELUTQ_DEVICE_WAIT_EXPIRED.  Y (float [M][N]) receives undefined values.  Nothing faults and nothing waits
 * without a limit.  Call elutq_release_scratch afterwards to clear the status.
 */
int elutq_test_wait_expiry(const void* X, const void* packed, float* Y, int M, int N, int K,
                           unsigned wait_limit, void* stream);

/* Number of kernel launches the library has issued in this process (all entry
 * points); lets a benchmark count its launches. */
unsigned long long elutq_launch_count(void);

/* Release every library-owned scratch/staging buffer (synchronises the device). */
int elutq_release_scratch(void);

#ifdef __cplusplus
}
#endif
#endif /* ELUTQ_H_ */
