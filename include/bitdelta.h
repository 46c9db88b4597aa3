/*
 * bitdelta.h -- C ABI of the B200 (sm_100a) BitDelta fused-GEMM library.
 *
 * The operation (multi-tenant BitDelta product; the paper's BitDelta paragraph
 * under "Recently Published Kernels" describes decoding packed binary weights,
 * s = 2*bit - 1, straight into tensor-core operands; the base-weight term, the
 * per-tenant scale and the packing order are the task's formula):
 *
 *   Y[b,t,n] = sum_k X[b,t,k] * W_base[n,k] + alpha[b] * sum_k X[b,t,k] * S[b,n,k]
 *
 * with S in {+1,-1} stored one bit per weight: word w of row (b,n) holds
 * k = 32w .. 32w+31, bit j (value 1<<j) belongs to k = 32w+j, a set bit means
 * +1 and a clear bit means -1.
 *
 * Conventions for every entry point
 *   - plain C types only; all arrays dense, row-major, no strides;
 *   - unless a parameter says "host", pointers are DEVICE pointers that the
 *     caller owns; the library never frees or reallocates them;
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream);
 *     work is queued on it and the call returns without synchronising, except
 *     where stated;
 *   - the return value is a bitdelta_status; on an argument error nothing is
 *     launched;
 *   - only compute capability 10.0 devices are served (BITDELTA_ERR_ARCH
 *     otherwise); there is no CPU fallback.
 */
#ifndef BITDELTA_H_
#define BITDELTA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BITDELTA_OK = 0,
    BITDELTA_ERR_NULL = 1,      /* a required pointer is NULL                         */
    BITDELTA_ERR_SHAPE = 2,     /* B, m, N <= 0, K <= 0 or K not a multiple of 32     */
    BITDELTA_ERR_ALIGN = 3,     /* a pointer is not 16-byte aligned                   */
    BITDELTA_ERR_WORKSPACE = 4, /* workspace missing or smaller than required         */
    BITDELTA_ERR_ARCH = 5,      /* current device is not compute capability 10.0      */
    BITDELTA_ERR_CUDA = 6,      /* a CUDA runtime / driver call failed                */
    BITDELTA_ERR_TIMEOUT = 7,   /* a bounded wait inside a kernel expired             */
    BITDELTA_ERR_OPTION = 8,    /* unknown data type or activation code               */
    BITDELTA_ERR_RANGE = 9      /* an activation beyond the decode schedules' range (reported by
                                   bitdelta_last_device_status, see bitdelta_gemm)    */
} bitdelta_status;

/*
 * Packing step (setup, before the GEMM):  bits[b,n,w] = sum_j [S[b,n,32w+j] > 0] << j.
 * S    : int8  [B,N,K]; any value > 0 packs as +1, zero and negatives as -1.
 * bits : uint32 [B,N,K/32] (output).  K must be a multiple of 32.
 * Integer work, bit-exact.  Asynchronous on the stream.
 */
int bitdelta_pack(const int8_t* S, uint32_t* bits, int B, int N, int K, void* cuda_stream);

/* Inverse of bitdelta_pack (test aid): S[b,n,k] = +1 if the bit is set, else -1. */
int bitdelta_unpack(const uint32_t* bits, int8_t* S, int B, int N, int K, void* cuda_stream);

/*
 * Compress step (setup, before the GEMM; the BitDelta method the paper cites in its BitDelta paragraph):
 * derives each tenant's 1-bit delta from its fine-tuned weights,
 *   bits[b,n,w] bit j = [W_fine[b,n,32w+j] - W_base[n,32w+j] > 0]   (zero and negative deltas pack as -1),
 *   alpha[b]          = mean over (n,k) of |W_fine[b,n,k] - W_base[n,k]|.
 * W_fine : bf16 [B,N,K]; W_base : bf16 [N,K]; bits : uint32 [B,N,K/32] (output); alpha : fp32 [B] (output).
 * workspace : at least bitdelta_compress_workspace_bytes(B,N,K) bytes of device memory, 8-byte aligned
 *             (per-block partial sums; needs no preparation, is fully rewritten).
 * The signs are exact (compared on the bf16 values); alpha is summed in double in a fixed order, so it is
 * reproducible bit for bit and within ~1e-7 relative of the exact mean.  K must be a multiple of 32;
 * W_fine, W_base and bits 16-byte aligned.  Asynchronous on the stream.
 */
size_t bitdelta_compress_workspace_bytes(int B, int N, int K);
int bitdelta_compress(const void* W_fine, const void* W_base, uint32_t* bits, float* alpha, int B, int N, int K,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Scratch memory bitdelta_gemm needs for this problem size (may depend on the
 * shape only, never on the data).  Returns 0 for invalid shapes.
 */
size_t bitdelta_gemm_workspace_bytes(int B, int m, int N, int K);

/*
 * Prepares a workspace for its first use (clears the arrival counters kept at
 * its start).  Call once after allocating the workspace; every completed
 * bitdelta_gemm leaves the workspace ready for the next call, so it need not
 * be repeated.  Asynchronous on the stream.
 */
int bitdelta_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The fused product defined at the top of this file.
 * X      : bf16 [B,m,K]      activations of B tenants, m tokens each
 * W_base : bf16 [N,K]        base weight shared by every tenant
 * bits   : uint32 [B,N,K/32] packed signs of each tenant's delta
 * alpha  : fp32 [B]          per-tenant scale (device memory)
 * Y      : bf16 [B,m,N]      output; fp32 accumulation, one round-to-nearest-even
 *                            conversion at the end
 * workspace / workspace_bytes : at least bitdelta_gemm_workspace_bytes(B,m,N,K),
 *          prepared once by bitdelta_workspace_init; calls that may overlap on
 *          the device must not share a workspace.
 * m <= 16 selects a decode schedule, larger m the tiled (prefill)
 * schedule (several tenants per tile up to m = 64; pairs of thread blocks with
 * 256-row MMAs for m > 64); all run on tcgen05 tensor cores with TMEM
 * accumulators, and bitdelta_gemm_plan tells which one a shape gets.  Shapes
 * whose K is not a multiple of 128 run on a plain CUDA-core kernel instead.
 * X, W_base, bits and Y must be 16-byte aligned; K a multiple of 32.
 * Asynchronous on the stream; a kernel-side wait that expires is reported by
 * bitdelta_last_device_status, not here.
 * Precision of X in the decode schedules (m <= 16): there the delta term runs on
 * a narrow-float tensor path.  bitdelta_gemm_plan tells which of two a shape gets.
 * 4-bit schedules (plan codes 7, 8; m <= 8, calls without options): every group
 * of 32 consecutive k of a token row is held as 16-bit fixed point relative to the
 * group's largest magnitude.  Values within a factor 2^8 of it are exact; smaller
 * ones lose what lies below 2^-16 of it (DELTA term only; the base term always
 * uses the bf16 value).  Nothing is clamped or flagged, whatever the magnitude.
 * 8-bit schedules (plan codes 1, 2): every activation is rewritten exactly
 * as a sum of e5m2 numbers, which have binary16's exponent range.  Finite bf16 activations
 * with |x| < 2^16 are exact down to 2^-16 (smaller parts of x, at most 2^-16 per
 * element, are dropped from the DELTA term only; the base term always uses the
 * bf16 value).  An activation with |x| >= 2^16 (or an infinity / NaN) is clamped
 * to +-65504 in the delta term, in every decode schedule alike, and the call is
 * flagged: bitdelta_last_device_status then returns BITDELTA_ERR_RANGE.  Inputs
 * like that need bitdelta_gemm_ex with BITDELTA_DTYPE_WIDE_RANGE, which runs any
 * m on the tiled schedule (bf16 operands for both terms: exact for every finite
 * input, and the route to take when neither narrow form is wanted).  The tiled
 * schedules (m > 16) have no such limit.
 * Early start: the kernel is queued so that it may begin (prologue, prefetch of
 * W_base, bits and alpha) while the kernel queued on the stream just before it
 * is still running; it reads X and writes Y and the workspace only after that
 * kernel has completed.  W_base, bits and alpha must therefore not be produced
 * by the kernel queued directly before the call (weights are static in the
 * intended use); X may be.  The library's own producers are covered: the
 * first bitdelta_gemm call after a bitdelta_pack or bitdelta_compress call is
 * launched without the early start.  BITDELTA_EARLY_START=0 in the environment
 * turns the early start off altogether.
 */
int bitdelta_gemm(const void* X, const void* W_base, const uint32_t* bits, const float* alpha,
                  void* Y, int B, int m, int N, int K,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same product with the paper's own operand type and a fused epilogue (the paper's BitDelta kernel
 * computes in FP16, and its suite fuses activations into GEMM epilogues, e.g. the fused GEMM-SiLU of
 * its evaluation; the paper fixes neither for this product, so the definition is the plain one):
 *
 *   Y[b,t,n] = act( sum_k X[b,t,k] W_base[n,k] + alpha[b] sum_k X[b,t,k] S[b,n,k] + bias[n] )
 *
 * dtype : BITDELTA_DTYPE_BF16 or BITDELTA_DTYPE_F16 (IEEE binary16): the element type of X, W_base,
 *         bias and Y; optionally OR-ed with BITDELTA_DTYPE_WIDE_RANGE, which plans every m on the tiled
 *         schedule (no 8-bit float operands: see the range note of bitdelta_gemm; slower for m <= 16).  Accumulation is fp32 in both; Y is rounded to nearest even once, after the
 *         epilogue.  With binary16 the delta term is exact for operands in the normal range (values
 *         below 2^-14 lose bits below 2^-16, in the delta term only).
 * bias  : device, [N] values of `dtype`, shared by all tenants, or NULL for none.  2-byte aligned.  Like
 *         alpha it is read during the early start (see bitdelta_gemm): it must not be produced by the kernel
 *         queued directly before the call.
 * act   : BITDELTA_ACT_NONE, or BITDELTA_ACT_SILU: y * sigmoid(y), applied after the bias (fp32,
 *         hardware exponential: relative error of a few 1e-7, far below the output rounding), or
 *         BITDELTA_ACT_SILU_GATE: the gate of a gated MLP whose gate and up projections are interleaved
 *         along N (row 2i of W_base, of every tenant's sign matrix and of bias: gate projection of
 *         feature i; row 2i+1: its up projection).  With z the sum above before any activation,
 *           Y[b,t,i] = SiLU(z[b,t,2i]) * z[b,t,2i+1],   i < N/2,
 *         so Y is [B,m,N/2] (N must be even: BITDELTA_ERR_SHAPE otherwise).
 * Everything else (shapes, layouts, workspace, stream semantics, errors, tolerance) is as for
 * bitdelta_gemm, which is this call with BITDELTA_DTYPE_BF16, no bias and no activation.  Unknown
 * codes return BITDELTA_ERR_OPTION and launch nothing.
 */
enum { BITDELTA_DTYPE_BF16 = 0, BITDELTA_DTYPE_F16 = 1, BITDELTA_DTYPE_WIDE_RANGE = 0x100 };
enum { BITDELTA_ACT_NONE = 0, BITDELTA_ACT_SILU = 1, BITDELTA_ACT_SILU_GATE = 2 };
int bitdelta_gemm_ex(const void* X, const void* W_base, const uint32_t* bits, const float* alpha,
                     const void* bias, void* Y, int B, int m, int N, int K, int dtype, int act,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * bitdelta_gemm for callers that must not allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for the deployment case below.)
 *
 * Some hosts of this library may not call cudaMalloc at all: code that runs inside a frozen,
 * pre-sized memory plan (a serving engine after start-up, a plug-in loaded into a process that owns
 * every byte of its memory pool, a real-time loop where an allocation can stall or fail).  They
 * cannot obtain the workspace bitdelta_gemm asks for.  This variant needs none from the caller: its
 * scratch is a fixed array of BITDELTA_NOALLOC_SCRATCH_BYTES that is part of the library's device
 * image, so every GPU that loads the library holds it from load until the process exits.  The call
 * itself allocates nothing (no cudaMalloc / cudaFree, no allocating library routine) and needs no
 * bitdelta_workspace_init.
 *
 * Arguments and result are those of bitdelta_gemm, without the workspace pair.
 *   - Shapes whose workspace (bitdelta_gemm_workspace_bytes) exceeds the array are refused with
 *     BITDELTA_ERR_WORKSPACE and nothing is launched; use bitdelta_gemm with your own buffer.
 *   - The first call on each device looks up the array's device address (the current device must be
 *     the one the call is for) and may be the moment the CUDA runtime binds this library's device image,
 *     array included, to that device: make that first call at start-up, before the memory plan is
 *     frozen and outside any stream capture.  Later calls allocate nothing.
 *   - All calls on a device share the one array.  Each call first clears, on the stream, the arrival
 *     counters at its start; the rest keeps whatever the previous call left and is fully rewritten
 *     before it is read.  Calls that can overlap on the device (issued on different streams) would
 *     race on it: keep all calls for one device on one stream, or order the streams with events.
 */
#define BITDELTA_NOALLOC_SCRATCH_BYTES (16u * 1024u * 1024u)
int bitdelta_gemm_noalloc(const void* X, const void* W_base, const uint32_t* bits, const float* alpha,
                          void* Y, int B, int m, int N, int K, void* cuda_stream);

/*
 * Diagnostic variant of bitdelta_gemm on plain CUDA cores (one warp per output
 * row, fp32 accumulation in k order per lane).  Same arguments and result
 * contract; needs no workspace.  Slow; used to triage the tensor-core path.
 */
int bitdelta_gemm_simt(const void* X, const void* W_base, const uint32_t* bits, const float* alpha,
                       void* Y, int B, int m, int N, int K, void* cuda_stream);

/*
 * End-to-end form for callers whose tensors live in HOST memory (pinned memory
 * makes the copies asynchronous).  Copies X, W_base, bits and alpha into the
 * device arena, runs bitdelta_gemm, copies Y back to Y_host and synchronises
 * the stream before returning, so Y_host is complete on return.
 * arena : DEVICE memory of at least bitdelta_gemm_host_arena_bytes(B,m,N,K)
 *         bytes, 256-byte aligned, owned by the caller.
 */
size_t bitdelta_gemm_host_arena_bytes(int B, int m, int N, int K);
int bitdelta_gemm_host(const void* X_host, const void* W_base_host, const uint32_t* bits_host,
                       const float* alpha_host, void* Y_host, int B, int m, int N, int K,
                       void* arena, size_t arena_bytes, void* cuda_stream);

/*
 * Plan queries (host only; no GPU is touched).  They report how bitdelta_gemm would run a shape on a
 * device with `num_sms` multiprocessors: which schedule, how many thread blocks, and which share of the
 * work list each block takes.  The work list is the flat list of (unit, k-step) items, unit-major: a unit
 * is one 128-row tile of W_base for one group of TB tenants (decode schedules) or one tenant's token tile
 * (tiled schedule), a k-step is 128 k; item = unit * P + k-step.
 *
 * bitdelta_gemm_plan fills info[0 .. BITDELTA_PLAN_INFO_INTS-1] (host pointer):
 *   [0] schedule: 0 tiled, 1 decode with a pre-pass activation split, 2 decode with the in-kernel split,
 *       3 CUDA-core kernel (K not a multiple of 128; all other entries are 0 then), 4 tiled on pairs of
 *       thread blocks (a unit is then two W_base tiles, [3] and the work list count such pairs, and [1] is
 *       twice the number of pairs that cut the list), 7 / 8 the 4-bit decode kernel on
 *       the flat work list / in clusters (8 is the default wherever it applies: m <= 8, one tenant group,
 *       2-8 blocks per W_base tile; BITDELTA_FP4=0 in the environment turns it off, =1 also takes 7)
 *   [1] thread blocks   [2] tenants per unit (tiled schedule: more than one in the middle regime,
 *       16 < m <= 64, where several tenants share a W_base tile)   [3] units   [4] P, k-steps per unit
 *   [5] work order: 0 one even cut of the list, 1 whole units round-robin (block b: units b, b+blocks, ...),
 *       2 teams (units numbered group-major, one team of blocks per tenant group, each cutting its
 *       group's items evenly)
 *   [6] teams (1 unless order 2)   [7] dynamic shared memory, bytes   [8] W_base ring depth
 *   [9] activation ring depth   [10] piece ring depth   [11] operand buffers in tensor memory (per decode
 *   group)   [12] hand-overs per k-step   [13] token tile (tiled schedule)   [14] tenant groups (decode) or
 *   tenant x token tiles (tiled) per W_base tile   [15] W_base tiles
 * bitdelta_gemm_plan_cta_items gives block `cta` its items [*first, *end) (orders 0 and 2; for order 1 the
 * items of its first unit; for schedule 4 both blocks of a pair report the pair's items).
 * bitdelta_gemm_plan_item_cta returns the block that owns `item` (schedule 4: the first block of the pair), or
 * -1 for a bad argument.  Errors: BITDELTA_ERR_NULL, BITDELTA_ERR_SHAPE (also: cta out of range, K % 128 != 0 for
 * the two item queries).
 */
#define BITDELTA_PLAN_INFO_INTS 16
int bitdelta_gemm_plan(int B, int m, int N, int K, int num_sms, int* info);
int bitdelta_gemm_plan_cta_items(int B, int m, int N, int K, int num_sms, int cta, int* first, int* end);
int bitdelta_gemm_plan_item_cta(int B, int m, int N, int K, int num_sms, int item);

/*
 * Synchronises the stream, then returns and clears the device-side status of
 * the current device: BITDELTA_OK; BITDELTA_ERR_TIMEOUT if a bounded wait in
 * one of this library's kernels expired since the last query (its output is
 * then undefined, and a workspace it used must be prepared again with
 * bitdelta_workspace_init: arrival counters may have been left non-zero); or
 * BITDELTA_ERR_RANGE if a decode-schedule call met an activation of magnitude
 * 2^16 or more (see bitdelta_gemm; a time-out takes precedence).  `site`, if not
 * NULL (host pointer), receives a code naming the wait that expired.
 */
int bitdelta_last_device_status(void* cuda_stream, int* site);

/*
 * Self-test of the time-out reporting (test aid; the paper's verifier section lists hangs on mbarrier phases
 * among the hazards of asynchronous kernels, and every wait in this library's kernels is bounded): queues a
 * one-warp kernel that waits, with the kernels' own bounded wait, on a barrier nobody signals, for
 * `limit_cycles` SM cycles (1e3 .. 2e9), then gives up and returns normally.  Afterwards
 * bitdelta_last_device_status returns BITDELTA_ERR_TIMEOUT with *site = `site`, once; the device and the
 * library stay usable.  Nothing else is touched.  Asynchronous on the stream.
 */
int bitdelta_selftest_timeout(long long limit_cycles, int site, void* cuda_stream);

/* Number of kernels this library has launched in this process (all entry points). */
unsigned long long bitdelta_kernel_launch_count(void);

/* Static, human-readable text for a status code. */
const char* bitdelta_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* BITDELTA_H_ */
