/*
 * fmm.h - C ABI of the B200 (sm_100a) library for block-scaled e4m3 fast matrix
 * multiplication  C = A * B  through a rank-R 2x2 realization (U, V, W).
 *
 * The operation (paper Sec. 2.1-2.2, App. D.1, App. E.2):
 *   split A (M x K) and B (K x N) into 2x2 blocks, row-vectorised in the order
 *   11, 12, 21, 22; for every term r form the encoded combinations
 *       S_r = sum_j U[r][j] A_j ,   T_r = sum_j V[r][j] B_j          (fp32)
 *   quantize S_r and T_r to e4m3 per block of `block_k` consecutive elements along
 *   the contracted axis (one scale per block, both sides), multiply the quantized
 *   operands with fp32 accumulation, and decode
 *       C_q = sum_r W[r][q] * (S_r^ * T_r^) .
 *   The raw operands are never quantized.  With `levels` > 1 the encoders and the
 *   decoder are applied recursively (Kronecker power) and only the R^levels leaf
 *   combinations are quantized (Sec. 3).  levels == 0 is the cubic fp8 product:
 *   A and B themselves are quantized and multiplied once.
 *
 * General rules
 *   - Every function returns fmm_status_t; nothing throws, aborts or traps the device.
 *   - "dev" pointers are device pointers of the current CUDA device, "host" pointers are
 *     host memory.  The caller owns every buffer it passes.  fmm_matmul, fmm_encode_only,
 *     fmm_ref_gemm_fp64 and fmm_error_stats allocate nothing and only enqueue work on
 *     `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream); they do not
 *     synchronise.  Inputs must be finite.
 *   - All matrices are dense row-major with no padding.
 *   - There is no CPU fallback: on a machine without a B200-class device the device
 *     functions return FMM_ERR_CUDA or FMM_ERR_ARCH.
 */
#ifndef FMM_B200_H
#define FMM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FMM_OK = 0,
    FMM_ERR_INVALID_ARG = 1,    /* null pointer, bad enum, bad rank / levels / block size */
    FMM_ERR_SHAPE = 2,          /* M, N, K not divisible as required (see fmm_matmul) */
    FMM_ERR_NOT_EXACT = 3,      /* (U, V, W) violates the Brent equations beyond 1e-5 */
    FMM_ERR_WORKSPACE = 4,      /* workspace missing, misaligned or too small */
    FMM_ERR_ALLOC = 5,          /* host or device allocation failed (plan creation only) */
    FMM_ERR_CUDA = 6,           /* a CUDA runtime / driver call failed (no device, bad stream, ...) */
    FMM_ERR_ARCH = 7,           /* current device is not compute capability 10.x */
    FMM_ERR_DEVICE_TIMEOUT = 8, /* a bounded device-side wait gave up (see fmm_device_status) */
    FMM_ERR_WRONG_DEVICE = 9    /* the current CUDA device is not the one the plan was created on */
} fmm_status_t;

typedef enum {
    /* Paper's quantizer (App. E.2): scale = amax / 448 kept in fp32. */
    FMM_SCALE_FP32_AMAX_DIV_448 = 0,
    /* Hardware-native deviation from the paper: the scale is rounded UP to a power of two
     * (UE8M0, e = ceil(log2(amax/448))) so that the tensor cores apply it themselves.
     * Requires block_k == 32.  Every number produced in this mode must be labelled as such. */
    FMM_SCALE_UE8M0_CEIL = 1
} fmm_scale_mode_t;

typedef struct {
    int block_k;                 /* 32 or 128: block length along the contracted axis */
    fmm_scale_mode_t scale_mode;
    float amax_floor;            /* minimum-scale clamp on the block amax; the paper uses 1e-12 */
    float fp8_max;               /* largest e4m3 magnitude; must be 448 */
    /* Deployment-matched weight-side options (App. E.5; both 0 for the paper's emulated protocol):
     * b_tile_n = 128 takes one scale per tile of 128 k x 128 columns of each encoded B-side
     * combination (the maximum is taken after the combination is formed), instead of one per column
     * and block; requires block_k == 128, FMM_SCALE_FP32_AMAX_DIV_448 and a leaf N divisible by 128.
     * b_preround_bf16 != 0 rounds each encoded B-side combination to bfloat16 (nearest even) before
     * the maximum and the e4m3 cast; same requirements on block_k and scale_mode.  The scale array keeps its shape: every column of a tile
     * carries the tile's scale. */
    int b_tile_n;
    int b_preround_bf16;
} fmm_quant_params_t;

typedef struct fmm_plan fmm_plan_t;   /* opaque */

/* Create a plan on the current CUDA device (Sec. 2.1: a realization is three R x 4 arrays).
 *   rank    number of terms R, 1..8 (7 for Strassen-type realizations, 8 for the cubic one);
 *           ignored when levels == 0.
 *   U, V, W host, rank x 4 row-major fp32, column order 11, 12, 21, 22.  W[r][q] is the weight of
 *           product r in output block C_q in that same order (NOT the paper's cyclic third
 *           factor w_r = rv(W_r^T); swap entries 12 and 21 to convert).  May be NULL when levels == 0.
 *   levels  0 (cubic fp8) .. 3.
 *   qp      quantizer parameters (copied).
 * Checks the Brent equations in fp64 (max residual <= 1e-5 else FMM_ERR_NOT_EXACT).  Allocates a few
 * KB of device memory for term tables and a status word; freed by fmm_plan_destroy. */
fmm_status_t fmm_plan_create(fmm_plan_t** plan, int rank, const float* U, const float* V,
                             const float* W, int levels, const fmm_quant_params_t* qp);
fmm_status_t fmm_plan_destroy(fmm_plan_t* plan);

/* Bytes of device workspace fmm_matmul / fmm_encode_only need for this problem size (host call).
 * The workspace holds what the fused regime of Sec. 2.2 / App. D.1 produces between its steps: the quantized
 * encoded combinations x_r, y_r of the R^levels leaves (e4m3 codes + one scale per block, App. E.2) and, for
 * levels >= 2, the fp32 combinations of the outer levels and the partially decoded products of the level-by-level
 * recursion (Sec. 3).  Never the products M_r themselves: those go from the tensor cores straight into C. */
fmm_status_t fmm_workspace_bytes(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K,
                                 size_t* bytes);

/* C = A * B through the plan's realization (whole hot path: pre-addition + quantization of both
 * sides, the R^levels block-scaled fp8 products on the tensor cores, post-addition into C).
 *   A dev, M x K fp32;  B dev, K x N fp32;  C dev, M x N fp32, overwritten.  All three 16-byte aligned
 *   (vector loads, tensor-map stores), else FMM_ERR_INVALID_ARG.
 *   Shape rule: with d = 2^levels, M/d and N/d must be multiples of 128 and K/d a multiple of 128
 *   (hence of block_k); otherwise FMM_ERR_SHAPE.
 *   workspace dev, 1024-byte aligned, at least fmm_workspace_bytes() bytes, caller-owned; its
 *   contents after the call are the quantized operands (see fmm_quantized_view).
 *   The plan's device (the one current at fmm_plan_create) must be the current device: FMM_ERR_WRONG_DEVICE otherwise;
 *   the same holds for every call that takes a plan and touches the device.
 * Asynchronous on cuda_stream.  Calls sharing a workspace must be stream-ordered; a plan may be shared by host
 * threads (it is read-only during a call, apart from the launch counter below).  Towards other work on the stream a
 * call is ordinary stream-ordered work: its first kernel starts after everything enqueued before it has completed, and
 * whatever is enqueued after it starts after all of its kernels have completed.  Between themselves the kernels of one
 * call overlap where they do not depend on each other (programmatic dependent launch: the B-side encoder starts under
 * the A-side encoder's last wave, the product kernel is set up under the B-side encoder's last blocks). */
fmm_status_t fmm_matmul(const fmm_plan_t* plan, const float* A, const float* B, float* C,
                        int64_t M, int64_t N, int64_t K, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/* The same product with HOST operands: uploads A and B, runs fmm_matmul on the device copies, downloads C.
 *   A host, M x K fp32;  B host, K x N fp32;  C host, M x N fp32, overwritten.  Page-locked (pinned) host
 *   memory makes the three copies asynchronous; pageable memory works but the copies then block the caller.
 *   workspace dev, 1024-byte aligned, at least fmm_host_workspace_bytes() bytes, caller-owned: the product's
 *   workspace followed by device staging for A, B and C.
 * Everything is enqueued on cuda_stream in order (upload A, upload B, product, download C) and nothing is
 * synchronised: C is valid once the stream has drained.  Calls on different streams with different workspaces
 * overlap one call's uploads with another's product and download (the links are full duplex); that is the
 * intended use for a sequence of products.  Errors as fmm_matmul, except that the host pointers need no
 * particular alignment; fmm_host_workspace_bytes returns FMM_ERR_INVALID_ARG for a null plan or bytes. */
fmm_status_t fmm_host_workspace_bytes(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K,
                                      size_t* bytes);
fmm_status_t fmm_matmul_host(const fmm_plan_t* plan, const float* A, const float* B, float* C,
                             int64_t M, int64_t N, int64_t K, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);

/* The encoder alone (Sec. 2.1: x_r = <U_r, a>, y_r = <V_r, b>, formed in fp32 from the unquantized blocks; Sec. 2.2 /
 * App. D.1: quantized only afterwards; App. E.2: scale and cast per block) for both sides, into the workspace.
 * Arguments, shape rule and errors as fmm_matmul; C is not touched. */
fmm_status_t fmm_encode_only(const fmm_plan_t* plan, const float* A, const float* B,
                             int64_t M, int64_t N, int64_t K, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/* The products and the decoder alone (Sec. 2.1: c = sum_r (x_r^ y_r^) W_r, fp32 accumulation) on operands a previous
 * fmm_encode_only / fmm_matmul left in the workspace.  Arguments, shape rule and errors as fmm_matmul. */
fmm_status_t fmm_multiply_only(const fmm_plan_t* plan, float* C, int64_t M, int64_t N, int64_t K,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Where the quantized encoded combination (App. E.2: e4m3 codes and one scale per block of block_k elements along
 * the contracted axis) of term `term` (depth-first order t = (r1*R + r2)*R + ..., the Kronecker order of Sec. 3;
 * r1 = outermost level; 0 for levels == 0) lives in the workspace (host call, byte offsets).  This is the view the
 * bit-parity tests read.
 *   side 'A': codes are q_rows x q_cols = (M/d) x (K/d) e4m3 bytes, row-major (K contiguous).
 *   side 'B': codes are stored TRANSPOSED, q_rows x q_cols = (N/d) x (K/d) (K contiguous).
 *   FP32 scale mode: fp32 scales, laid out as the product kernel fetches them per 128-k pipeline stage.
 *             side 'A': chunk-major, [c][i][g] = scale of K block c * (128/block_k) + g of row i, with c the 128-k
 *             chunk; reported as scale_rows x scale_cols = (K/d/128) x ((M/d) * (128/block_k)) row-major;
 *             side 'B': (K/d/block_k) x (N/d) row-major, entry [kb][j] = scale of block kb of column j.
 *   UE8M0 mode: one biased-exponent byte per block in 512-byte tiles of 128 rows x 4 blocks:
 *             tile index (block/4) * (rows/128) + (row/128), byte (row%32)*16 + ((row%128)/32)*4 + block%4
 *             where row is the M/d (side 'A') or N/d (side 'B') index; scale_rows x scale_cols then
 *             report that logical (rows x blocks) shape. */
fmm_status_t fmm_quantized_view(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K, int term,
                                char side, size_t* q_offset, int64_t* q_rows, int64_t* q_cols,
                                size_t* scale_offset, int64_t* scale_rows, int64_t* scale_cols);

/* Higher-precision reference of App. E.2: Cref (dev, M x N fp64) = A * B with fp64 accumulation of
 * the fp32 inputs (dev).  M, N multiples of 64; K a multiple of 16.  Off the timed path. */
fmm_status_t fmm_ref_gemm_fp64(const float* A, const float* B, double* Cref,
                               int64_t M, int64_t N, int64_t K, void* cuda_stream);

/* Error statistics of App. E.2 / Eq. (D.9): out3 (dev, 3 doubles) =
 * [ sum (C - Cref)^2, sum Cref^2, max |C - Cref| ] over the M x N entries; the relative Frobenius
 * error is sqrt(out3[0] / out3[1]).  Overwrites out3; deterministic (no floating-point atomics).
 * scratch: dev, at least fmm_error_stats_scratch_bytes() bytes, caller-owned. */
fmm_status_t fmm_error_stats(const float* C, const double* Cref, int64_t M, int64_t N,
                             double* out3, void* scratch, size_t scratch_bytes, void* cuda_stream);
size_t fmm_error_stats_scratch_bytes(void);

/* (No counterpart in the paper: a convenience for restricted callers.)
 * Same result as fmm_error_stats, for callers that are not allowed to allocate device memory at all -
 * code running inside a service whose memory pool is fixed up front, a plugin that must not touch the
 * host application's allocator, or a routine invoked where cudaMalloc would synchronise the device at a
 * bad moment.  The block partials go to a fixed 24 KB array compiled into the library (1024 slots of
 * three doubles, resident on every GPU that loads the library), so the call takes no scratch argument
 * and performs no allocation of any kind; C, Cref and out3 are still the caller's.
 *   Limit: M * N <= fmm_error_stats_noalloc_max_elements() (2^28, e.g. 16384 x 16384) and M * N even;
 *   larger problems are refused with FMM_ERR_SHAPE - use fmm_error_stats with your own scratch.
 *   The first call on each device looks up the array's device address (with that device current) and
 *   remembers it; make that first call outside any stream capture.
 *   All calls on a device share the one array.  Every slot is rewritten by each call, so stale contents
 *   are harmless, but two calls whose kernels overlap on the GPU (different streams, no ordering
 *   between them) would overwrite each other's partials: order such calls. */
fmm_status_t fmm_error_stats_noalloc(const float* C, const double* Cref, int64_t M, int64_t N,
                                     double* out3, void* cuda_stream);
int64_t fmm_error_stats_noalloc_max_elements(void);

/* (No counterpart in the paper: failure reporting of this implementation.)
 * Reads the plan's device status word after cudaDeviceSynchronize (all streams of the device, non-blocking
 * ones included, have drained).  *code == 0: no bounded wait has
 * given up since plan creation; otherwise a kernel-specific location code, and the results of the
 * call that set it are invalid.  Returns FMM_ERR_DEVICE_TIMEOUT when *code != 0. */
fmm_status_t fmm_device_status(const fmm_plan_t* plan, int* code);

/* Debug build (no counterpart in the paper).  The library can be built a second time with -DFMM_DEBUG
 * (libfmm_b200_debug.so): every global store of every kernel is then checked against the buffers the launch was
 * given (workspace slices, C, scratch); a store outside them is skipped and a location code is recorded - nothing
 * traps and the context stays usable.  fmm_debug_build() tells which build is loaded (1 = debug).
 * fmm_debug_violation synchronises the device and returns the first recorded code of the plan's launches (0 = none;
 * plan == NULL: of the statistics / reference kernels, which take no plan).  In the normal build it always reports 0. */
int fmm_debug_build(void);
fmm_status_t fmm_debug_violation(const fmm_plan_t* plan, int* code);
/* Self-test of that guard, safe in either build: enqueues a one-thread kernel that stores to a spare word of the
 * plan's own status array under a guard that does not include that word.  Debug build: the store is skipped and
 * fmm_debug_violation reports code 1901 until fmm_device_status_clear; normal build: no effect that a caller sees. */
fmm_status_t fmm_selftest_store_guard(const fmm_plan_t* plan, void* cuda_stream);

/* Resets the plan's status words to zero, after cudaDeviceSynchronize. */
fmm_status_t fmm_device_status_clear(const fmm_plan_t* plan);

/* Self-test of the failure-detection path (no counterpart in the paper): enqueues a one-warp kernel that
 * waits, with the library's bounded-wait routine, on a barrier that nothing signals.  After limit_ns
 * (1 .. 2e9 nanoseconds) the wait gives up, writes location code 901 into the status word and the kernel
 * ends normally - the context stays usable.  fmm_device_status then reports FMM_ERR_DEVICE_TIMEOUT until
 * fmm_device_status_clear is called. */
fmm_status_t fmm_selftest_bounded_wait(const fmm_plan_t* plan, int64_t limit_ns, void* cuda_stream);

/* Host utility (Sec. 2.1): Phi = sum_r |U_r|^2 |V_r|^2 |W_r|^2 and Gamma = sum_r |U_r| |V_r| |W_r|
 * with entrywise 2-norms, in fp64. */
fmm_status_t fmm_phi_gamma(int rank, const float* U, const float* V, const float* W,
                           double* phi, double* gamma);

/* Host utility: largest absolute residual of the 64 Brent equations of <2,2,2>, in fp64. */
fmm_status_t fmm_brent_residual(int rank, const float* U, const float* V, const float* W,
                                double* max_residual);

/* Number of kernels the last fmm_matmul / fmm_encode_only / fmm_multiply_only on this plan launched (with several
 * host threads on one plan: of whichever call finished last). */
fmm_status_t fmm_last_launch_count(const fmm_plan_t* plan, int* launches);

const char* fmm_status_string(fmm_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* FMM_B200_H */
