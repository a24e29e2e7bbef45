/*
 * lqer.h - C ABI of the B200 (sm_100a) LQER / L2QER inference linear layer.
 *
 *   Y = X W_q + (X A_k) B_k                        (paper Section 3.1, Section 3.2)
 *
 * W_q is the MXINT4 weight (4-bit mantissas, one shared power-of-two exponent per
 * block of 16 along K), X is quantised on the fly to MXINT8 (blocks of 16 along K),
 * A_k [K,k] and B_k [k,N] are the rank-k factors in MXINT8 (Section 2.2, Section 4.1).
 *
 * Conventions
 *  - Plain C.  Every function returns lqer_status_t (LQER_OK == 0) and never throws,
 *    aborts or prints.
 *  - Unless a parameter says "host", every data pointer is DEVICE memory owned by the
 *    caller.  The library allocates no device memory (the one exception is stated at
 *    its entry point) and never synchronises the stream except where stated.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *  - Matrices are dense row-major: X [M,K] fp32, W [K,N] fp32, A [K,k] fp32,
 *    B [k,N] fp32, Y [M,N] fp32.  Pointers must be 16-byte aligned.
 *  - Host-side argument checks run before any launch; on error nothing is launched
 *    and outputs are untouched.  Conditions that only the device can see (a bounded
 *    wait that ran out) are written to a status word at the head of `workspace` and
 *    read back with lqer_poll_status.
 *  - Element value convention: value = mantissa * 2^(e - (bits - 2)), e the block's
 *    shared exponent = clamp(floor(log2(max|v|)), exp_min, exp_max); mantissas are
 *    rounded half-to-even and clamped to +-(2^(bits-1) - 1).  Exponents are stored
 *    as one byte e + 127.
 */
#ifndef LQER_H
#define LQER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LQER_OK = 0,
  LQER_ERR_NULL = 1,             /* a required pointer is NULL */
  LQER_ERR_SHAPE = 2,            /* M/K/N/k out of range, K % 16 != 0, N % 8 != 0 */
  LQER_ERR_ALIGN = 3,            /* a pointer is not 16-byte aligned */
  LQER_ERR_CONFIG = 4,           /* unsupported lqer_config_t */
  LQER_ERR_BUFFER_TOO_SMALL = 5, /* packed / workspace buffer smaller than required */
  LQER_ERR_BAD_PACKED = 6,       /* not a packed buffer: no valid header at that (256-byte aligned, device) address */
  LQER_ERR_ARCH = 7,             /* current device is not compute capability 10.x */
  LQER_ERR_CUDA = 8,             /* a CUDA runtime / driver call failed */
  LQER_ERR_TIMEOUT = 9,          /* device side: a bounded wait ran out */
  LQER_ERR_BOUNDS = 10,          /* device side: an index check failed */
  LQER_ERR_STATIC_SCRATCH = 11   /* lqer_linear_static: the call needs more than LQER_STATIC_SCRATCH_BYTES */
} lqer_status_t;

/* Format parameters (Section 3.1: b_l, b_h; Section 4.1: block size, exponent width). */
typedef struct {
  int w_bits;        /* mantissa bits of W_q: 4 (default), or 2 (the W2A8 setting of Section 4.4: mantissas -1, 0, 1) */
  int a_bits;        /* mantissa bits of X and of T = X A_k: 3..8, default 8 (W4A8; 6 gives the W4A6 of Section 4.3) */
  int lr_bits;       /* mantissa bits of A_k, B_k: 8 */
  int block;         /* block size along the contraction dimension: 16 */
  int exp_min;       /* shared-exponent clamp window of X and T, default [-56, 55] */
  int exp_max;
  int deterministic; /* 1: fixed reduction order (the only mode implemented) */
  int w_exp_min;     /* shared-exponent clamp window of W_q, A_k, B_k, default [-56, 55]; Section 4.1 gives these a */
  int w_exp_max;     /* 4-bit shared exponent (16 values, e.g. [-12, 3]) and the activations an 8-bit one */
} lqer_config_t;

/* Element type of activations at the layer's boundary (Section 2.1: weight-only settings keep 16-bit activations
 * between layers; the w&a settings quantise them on entry, which the layer does itself either way). */
typedef enum {
  LQER_F32 = 0,
  LQER_BF16 = 1,
  LQER_MXINT8 = 2    /* MXINT activations in the layer's format: int8 mantissas, then exponent bytes; see lqer_linear_ex */
} lqer_dtype_t;

/* One call of a batch (Section 4.3: layers are independent). */
typedef struct {
  const float* X;     /* [M,K] */
  int M;
  const void* packed; /* prepared weights of this layer */
  float* Y;           /* [M,N] */
} lqer_call_t;

/* Human-readable name of a status code (static storage, never NULL). */
const char* lqer_status_string(lqer_status_t status);

/* Fill *cfg (host) with the defaults above. */
lqer_status_t lqer_default_config(lqer_config_t* cfg);

/* Size in bytes (host out) of the packed buffer for a [K,N] layer of rank k (k may be 0).
 * Storage follows Section 4.1: 4-bit mantissas + one exponent byte per 16 for W_q,
 * 8-bit mantissas + one exponent byte per 16 for A_k and B_k, plus a 256-byte header
 * and tile padding (N to a multiple of 128, K to a multiple of 64, k to a multiple of 16). */
lqer_status_t lqer_packed_bytes(int K, int N, int k, const lqer_config_t* cfg, size_t* bytes);

/* Size in bytes (host out) of the scratch `workspace` lqer_linear* needs for any call of up to
 * M_max rows.  The workspace holds a head of one fixed size that is all zero between calls (status
 * area, the kernels' arrival counters) followed by per-call scratch: the quantised activations
 * [X_q | T_q] (bf16, M rows) with the prologue's fp64 partial sums of X A_k and the GEMM's fp32
 * partial sums of Y where its K range is cut, or the decode kernel's partial sums of X A_k.  One
 * workspace may serve layers of different shapes in turn if it fits the largest. */
lqer_status_t lqer_workspace_bytes(int M_max, int K, int N, int k, const lqer_config_t* cfg, size_t* bytes);

/* Size in bytes (host out) that one call with exactly M rows uses of its workspace on the path the library
 * picks for it (column-owner decode kernel up to 4 rows, small-batch kernels up to 128, prologue + GEMM above): never more than
 * lqer_workspace_bytes(M_max, ...) for any M_max >= M.  This is the figure lqer_linear_static holds against
 * LQER_STATIC_SCRATCH_BYTES. */
lqer_status_t lqer_call_workspace_bytes(int M, int K, int N, int k, const lqer_config_t* cfg, size_t* bytes);

/* Weight preparation (Section 3.1: W_q = q(W); Section 4.1 formats): quantise W to MXINT4
 * (blocks of 16 along K), A and B to MXINT8 (A: blocks of 16 along K; B: blocks of 16 along
 * the rank, zero-padded to a multiple of 16) on the GPU and write the kernel layout into
 * `packed` (device, >= lqer_packed_bytes, 256-byte aligned).  A and B may be NULL iff k == 0.
 * Asynchronous on `stream`.  The buffer is registered with the library under its address. */
lqer_status_t lqer_prepare_weights(const float* W, const float* A, const float* B, int K, int N, int k,
                                   const lqer_config_t* cfg, void* packed, size_t packed_bytes, void* stream);

/* Weight preparation from the weight and a calibration batch alone (Section 3.1: E_q = W - W_q and its rank-k
 * factors A_k = U_k, B_k = Sigma_k V_k^T; Section 3.2: the SVD is taken of S E_q and A_k = S^-1 U'_k,
 * B_k = Sigma'_k V'_k^T; Appendix A: S from the calibration samples - mean |X| per channel over the tokens of a
 * sample, maximum over the samples, normalised by sqrt(min * max)).  All on the GPU: the truncated SVD is a
 * randomised subspace iteration (k + 16 columns, four rounds, fp64 accumulation), which approaches the optimal
 * rank-k residual of Section 3.2 from above; the factors are then rounded to fp32, quantised and packed with W
 * exactly as lqer_prepare_weights does.
 *  - W [K,N] fp32 (device).  samples: HOST array of n_samples DEVICE pointers, sample i is fp32 [sample_rows[i], K]
 *    (sample_rows: host array).  n_samples == 0 gives plain LQER (S = I, Section 3.1).
 *  - omega: the random test matrix, fp32 [N, columns] standard normal (device), columns from
 *    lqer_factor_sketch_columns; the caller draws it, so the run is reproducible with the caller's generator.
 *  - A_out [K,k], B_out [k,N] fp32 (device): the factors before quantisation, or NULL.
 *  - workspace (device, 256-byte aligned): lqer_prepare_workspace_bytes.  Asynchronous on `stream`.
 *  - lqer_prepare_status (synchronises) reads what only the device could see: 0 fine, 1 a calibration channel is
 *    identically zero (S not invertible; S = I was used), 2 a sketch lost rank (k larger than the rank of the
 *    error), 3 the small SVD did not converge. */
lqer_status_t lqer_factor_sketch_columns(int K, int N, int k, int* columns);
lqer_status_t lqer_prepare_workspace_bytes(int K, int N, int k, size_t* bytes);
lqer_status_t lqer_prepare_from_calibration(const float* W, const float* const* samples, const int* sample_rows, int n_samples,
                                            const float* omega, int K, int N, int k, const lqer_config_t* cfg, void* packed,
                                            size_t packed_bytes, float* A_out, float* B_out, void* workspace,
                                            size_t workspace_bytes, void* stream);
lqer_status_t lqer_prepare_status(const void* workspace, int K, int N, int k, void* stream, int* code);

/* Register a packed buffer that was produced earlier and copied to a new address
 * (save / restore).  Reads the header back from the device: synchronises `stream`.
 * Optional: every entry point that takes `packed` does the same on its own the first
 * time it meets an address it has not seen (one blocking 256-byte read, then cached). */
lqer_status_t lqer_attach_packed(const void* packed, size_t packed_bytes, void* stream);

/* Forget a packed buffer (call before freeing it).  Host only. */
lqer_status_t lqer_release_packed(const void* packed);

/* Shape of a registered packed buffer (host outs, any may be NULL). */
lqer_status_t lqer_packed_shape(const void* packed, int* K, int* N, int* k, int* k_pad);

/* Canonical read-back of the packed operands for bit-exact comparison: two's-complement
 * mantissas and exponent bytes (e + 127).  Any output pair may be NULL.  Device outputs:
 * Wm [K,N], We [K/16,N], Am [K,k], Ae [K/16,k], Bm [k_pad,N], Be [k_pad/16,N]. */
lqer_status_t lqer_export_weights(const void* packed, int8_t* Wm, uint8_t* We, int8_t* Am, uint8_t* Ae,
                                  int8_t* Bm, uint8_t* Be, void* stream);

/* Activation quantisation alone (Section 4.1: X_q in MXINT8, blocks [1,16]) with the same
 * device routine the layer uses.  Outputs Xm [M,K] int8, Xe [M,K/16] bytes. */
lqer_status_t lqer_quantize_activations(const float* X, int M, int K, const lqer_config_t* cfg,
                                        int8_t* Xm, uint8_t* Xe, void* stream);

/* The low-rank projection alone (Section 3.1: X A_k), re-quantised to the activation
 * format: T_q = q(X_q A_q), blocks of 16 along the rank.  Runs the layer's own prologue
 * kernel.  Outputs Tm [M,k_pad] int8, Te [M,k_pad/16] bytes.  Needs the same workspace
 * as lqer_linear. */
lqer_status_t lqer_project_lowrank(const float* X, int M, const void* packed, int8_t* Tm, uint8_t* Te,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* The layer (Section 3.1 last display, Section 3.2 last display):
 *   Y[M,N] = X_q W_q + q(X_q A_q) B_q,  fp32 accumulation of exactly represented products.
 * M <= 4 runs a fused decode kernel whose CTAs own output columns; M <= 128 a latency-oriented
 * prologue and a tensor-core GEMM that streams the weights once against a 64- or 128-row token tile;
 * larger M the activation prologue and the tensor-core GEMM over 256 x 256 tiles of the concatenated
 * contraction [X_q | T_q] . [W_q ; B_q].
 * lqer_linear uses the default stream. */
lqer_status_t lqer_linear(const float* X, int M, const void* packed, float* Y,
                          void* workspace, size_t workspace_bytes);
lqer_status_t lqer_linear_stream(const float* X, int M, const void* packed, float* Y,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* The same layer with a choice of element types at its boundary (Section 2.1: the layer sits between 16-bit
 * activations in the w-only setting and re-quantises them in the w&a setting): X [M,K] of x_dtype, Y [M,N] of
 * y_dtype, both dense row-major and 16-byte aligned.  bf16 X is quantised to MXINT like fp32 X (every bf16
 * value is an fp32 value); bf16 Y is the fp32 result rounded to nearest even.  Everything else - packed,
 * workspace, paths, device-side status - as for lqer_linear_stream.  lqer_linear_batched_ex is
 * lqer_linear_batched with every call's X and Y of the given types (cast the pointers of lqer_call_t).
 * y_dtype LQER_MXINT8 (Section 2.1, w&a setting: the activations between layers are quantised; Section 4.1:
 * MXINT, blocks [1,16]): the epilogue quantises Y itself, in blocks of 16 along N (the next layer's K), to the
 * layer's activation format (a_bits and exponent window of its lqer_config_t), exactly as the next layer's
 * prologue would quantise the fp32 Y.  Y then points to M*N + M*N/16 bytes: the int8 mantissas [M,N] followed
 * directly by the exponent bytes [M,N/16] (e + 127); N must be a multiple of 16.
 * x_dtype LQER_MXINT8: X is given in the same layout - mantissas [M,K], then exponent bytes [M,K/16], M*K + M*K/16
 * bytes - with the mantissa width and exponent window of the layer's lqer_config_t (what a previous layer's MXINT8
 * output holds if it has the same format; mantissas within the format's symmetric range, |m| <= 2^(a_bits-1) - 1).
 * It is taken at its value: a block that a quantiser would have produced passes through unchanged, any other block
 * stands for the same values as its normalised form, so the layer computes exactly what it computes on the fp32
 * tensor of those values - without reading 4 bytes per element. */
lqer_status_t lqer_linear_ex(const void* X, lqer_dtype_t x_dtype, int M, const void* packed, void* Y, lqer_dtype_t y_dtype,
                             void* workspace, size_t workspace_bytes, void* stream);
lqer_status_t lqer_linear_batched_ex(const lqer_call_t* calls, int n_calls, lqer_dtype_t x_dtype, lqer_dtype_t y_dtype,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* The same layer for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a property of the library, not of the method).  It is meant for code that runs
 * inside another component's memory plan - a plugin of a runtime that owns the whole device
 * and exposes no allocator, a path on which cudaMalloc's device-wide synchronisation is not
 * acceptable, a process whose memory budget was fixed before this library was loaded.  The
 * scratch that lqer_linear_stream takes from the caller lives here in a fixed array of
 * LQER_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds
 * that much memory until the process exits.  The call itself allocates and frees nothing.
 *  - X, Y, packed, stream: as for lqer_linear_stream (device pointers, caller owned).
 *  - Limit: what this call itself needs on the path it takes (lqer_call_workspace_bytes) must fit
 *    LQER_STATIC_SCRATCH_BYTES, otherwise LQER_ERR_STATIC_SCRATCH is returned and nothing is launched.  The
 *    need is smaller than lqer_workspace_bytes(M, ...), which covers every batch up to M: it is 2 M (K + k)
 *    bytes for [X_q | T_q] plus the partial sums of the path's K ranges (up to 128 rows: those of the
 *    small-batch GEMM, ceil(N / 256) x chunks x M x 1024 bytes; up to 256 rows: those of the split-K GEMM).  At
 *    K = N = 4096, rank 32 that admits M <= 57 and 257 <= M <= 487 and refuses the rest; M <= 16 fits for
 *    every K up to 131072.
 *  - The first call on a device looks up the array's device address (the device must be
 *    current); make that first call before any stream capture begins.
 *  - All calls on a device share the one array and it keeps the previous call's contents; the
 *    status area at its head is cleared at the start of every call.  Two calls that overlap on
 *    the GPU (different streams without an ordering between them) race on the array and give
 *    undefined results: keep calls of this entry point on one stream, or order them.
 *  - Device-side conditions (a bounded wait that ran out) cannot be polled for this variant;
 *    use lqer_linear_stream with a workspace where that matters. */
#define LQER_STATIC_SCRATCH_BYTES (8u << 20)
lqer_status_t lqer_linear_static(const float* X, int M, const void* packed, float* Y, void* stream);

/* n_calls independent layers back to back on one stream (`calls` is a HOST array).
 * The workspace is reused by consecutive calls (stream order makes that safe) and must
 * fit the largest of them.  Independent means that no call reads what another call of the
 * same batch writes; the library uses that, with the path left at 0, to share launches:
 *  - up to 16 consecutive calls with one M <= 4 (any shapes with N >= 32, one set of formats)
 *    run as ONE launch of the decode kernel that divides the SMs among them; consecutive such
 *    launches do not wait for one another, and a stretch of more than one launch first has the
 *    quantised activations and T_q of all its calls computed by one kernel, into the workspace;
 *  - up to 8 consecutive calls with one M > 256 (any shapes, one set of formats) run their
 *    prologues into separate slices of the workspace and then ONE GEMM launch over the tiles of
 *    all of them - if the workspace holds lqer_batched_workspace_bytes(calls, n_calls); with a
 *    smaller workspace (at least the largest lqer_workspace_bytes of the calls) fewer calls, or
 *    none, share a launch;
 *  - up to 16 consecutive calls with one M <= 128 that the decode kernel does not serve (any shapes,
 *    one set of formats) run as ONE launch of the small prologue and ONE launch of the small-batch
 *    GEMM over the work items of all of them, under the same condition on the workspace.
 * In the first two cases a result does not depend on the sharing, bit for bit.  In the third the
 * contraction of a tile is cut into fewer K chunks when layers share a launch, so a result may
 * differ from the single call's in its last bits (both within the layer's tolerance); it is
 * reproducible for the same sequence of calls. */
lqer_status_t lqer_batched_workspace_bytes(const lqer_call_t* calls, int n_calls, size_t* bytes);
lqer_status_t lqer_linear_batched(const lqer_call_t* calls, int n_calls,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Same layer with host buffers: copies X (host, [M,K]) to the device part of `workspace`,
 * runs the layer and copies Y back to Y_host ([M,N]); synchronises `stream` before it
 * returns.  workspace must hold lqer_workspace_bytes(M, ...) plus 4*M*K and 4*M*N, each rounded
 * up to a multiple of 256. */
lqer_status_t lqer_linear_host(const float* X_host, int M, const void* packed, float* Y_host,
                               void* workspace, size_t workspace_bytes, void* stream);

/* n_calls independent layers with HOST buffers (calls[i].X and calls[i].Y are host pointers; pinned
 * memory gives full copy speed; `calls` is a host array).  Copies in, layers and copies out are
 * pipelined: while layer i runs on `stream`, X of layer i+1 is on its way in and Y of layer i-1 on
 * its way out, on two internal streams made at the first call on a device.  Returns when every Y
 * is on the host.  workspace must hold lqer_linear_host_batched_bytes(calls, n_calls) bytes: the
 * largest lqer_workspace_bytes of the calls plus two X and two Y buffers of the largest sizes. */
lqer_status_t lqer_linear_host_batched_bytes(const lqer_call_t* calls, int n_calls, size_t* bytes);
lqer_status_t lqer_linear_host_batched(const lqer_call_t* calls, int n_calls, void* workspace,
                                       size_t workspace_bytes, void* stream);
/* The same with host X of x_dtype and host Y of y_dtype (Section 2.1: 16-bit activations between layers): bf16
 * halves the bytes that cross the host link in that direction.  The workspace size is the same. */
lqer_status_t lqer_linear_host_batched_ex(const lqer_call_t* calls, int n_calls, lqer_dtype_t x_dtype, lqer_dtype_t y_dtype,
                                          void* workspace, size_t workspace_bytes, void* stream);

/* Zero the head of a fresh workspace (status area, counters, accumulator; at most 168192 bytes;
 * asynchronous on `stream`).  Call once after allocating the workspace and again after
 * lqer_poll_status reported a device-side error (an interrupted call may leave counters behind). */
lqer_status_t lqer_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Read the device-side status word of `workspace` (synchronises `stream`). */
lqer_status_t lqer_poll_status(const void* workspace, void* stream, lqer_status_t* device_status);

/* Force a kernel path for tests: 0 auto, 1 plain CUDA-core reference kernel, 2 small-batch kernels
 * (column-owner kernel for M <= 4, small prologue + small-batch GEMM for M <= 128), 3 tensor-core GEMM behind the
 * activation prologue that runs the projection on int8 mma.sync (at every batch size), 4 tensor-core
 * GEMM with the prologue chosen as in 0, 5 small prologue + small-batch GEMM for every M <= 128 (the register-operand
 * kernel up to 16 rows - which paths 0 and 2 use only where several calls share its launches - and
 * the tensor-memory kernel otherwise), 6 as 4 with the
 * tcgen05 activation prologue at every batch size (ranks up to 64; by default it serves M >= 1024,
 * and paths 1 and 3 never use it), 7 as 5 with the tensor-memory kernel at every M <= 128.  Host only, process wide. */
lqer_status_t lqer_set_path(int path);

/* Test hooks for the device-side error path (host only, process wide; the paper has no counterpart: this is a
 * property of the library).  Every wait of a kernel on another CTA, warp or copy is bounded; a wait that runs out makes
 * the kernel give up, write LQER_ERR_TIMEOUT to the status word and return, so the context stays usable.
 *  - lqer_set_wait_limit_cycles: the bound in SM clock cycles (default 4e9, about two seconds; 1e3 .. 2^40).
 *  - lqer_inject_stall(family): the next launch of that kernel family (numbering of lqer_kernel_times_t:
 *    3 activation prologue, 6 tensor-core GEMM pair kernel, 7 decode kernels) is told to expect one arrival
 *    more than will ever come (3, 7) or has its last stage of operands withheld (6), so that its waits run
 *    out; no memory is touched that an ordinary launch would not touch.  -1 disarms.  After such a launch
 *    the outputs are undefined and the workspace needs lqer_workspace_init before its next use. */
lqer_status_t lqer_set_wait_limit_cycles(long long cycles);
lqer_status_t lqer_inject_stall(int kernel_family);

/* The checked build of the library (liblqer_dbg.so, compiled with -DLQER_DEBUG_BOUNDS; the paper has no counterpart).
 * Every global store of the inference kernels and every bulk copy of packed weights first checks its byte range
 * against the extent of the buffer it belongs to; the first violation is written to the status word
 * (LQER_ERR_BOUNDS; lqer_poll_status) and the access is skipped - nothing traps, nothing out of range is touched.
 * It stands in for a memory checker where none can be run.  lqer_debug_bounds_shrink (host, process wide) is its test
 * hook: the declared extent of every Y is made `bytes` smaller for the launches that follow, so that the checks at
 * the end of Y fire (the stores they guard are skipped; Y is then incomplete); 0 restores.  The ordinary build
 * returns LQER_ERR_CONFIG. */
lqer_status_t lqer_debug_bounds_shrink(long long bytes);

/* Number of kernels launched by the library in this process so far (host). */
unsigned long long lqer_launch_count(void);

/* Per-kernel timing for benchmarks.  While enabled (host, process wide), every kernel launch of
 * the library is bracketed by two CUDA events recorded on the launching stream; the events
 * serialise nothing but they do keep consecutive kernels from overlapping, so leave it off
 * when measuring end-to-end time.  lqer_profile_collect waits for the recorded launches,
 * sums launches and elapsed milliseconds per kernel family into *out (host) and forgets them.
 * Families: 0 weight pack, 1 export, 2 stand-alone activation quantiser, 3 activation prologue,
 * 4 CUDA-core reference GEMM, 5 factor preparation (calibration statistics, subspace iteration),
 * 6 tensor-core GEMM (CTA pair per tile), 7 decode kernels. */
#define LQER_NUM_KERNEL_FAMILIES 8
typedef struct {
  unsigned long long launches[LQER_NUM_KERNEL_FAMILIES];
  double milliseconds[LQER_NUM_KERNEL_FAMILIES];
} lqer_kernel_times_t;
lqer_status_t lqer_profile_enable(int on);
lqer_status_t lqer_profile_collect(lqer_kernel_times_t* out);

#ifdef __cplusplus
}
#endif
#endif /* LQER_H */
