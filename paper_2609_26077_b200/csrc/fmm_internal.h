// Internal declarations shared by the translation units of the library (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <atomic>
#include "../../include/fmm.h"

#define FMM_MAX_RANK 8
#define FMM_MAX_LEVELS 3

// One destination of a leaf product in C: block origin, weight, and whether this is the first
// product written there (store) or a later one (accumulate).
struct FmmOutEntry {
    int row_off;   // element row of the destination block origin in C
    int col_off;   // element column
    float w;       // product of the W coefficients along the recursion path
    int first;     // 1: overwrite, 0: add
};

// Store guard of the FMM_DEBUG build (the stand-in for a memory checker, which this library cannot count on
// having): the address ranges a launch may write, and where to report a store that falls outside them.  Every
// launch fills it in; the kernels test it only when compiled with -DFMM_DEBUG - a bad store is then skipped and its
// location code goes to *status (first one wins, nothing traps).
struct FmmGuard {
    const char* lo[2];
    const char* hi[2];
    int* status;
};
#if defined(FMM_DEBUG) && defined(__CUDACC__)
__device__ __forceinline__ bool fmm_guard_ok(const FmmGuard& g, const void* ptr, size_t bytes, int code)
{
    const char* c = static_cast<const char*>(ptr);
    if ((c >= g.lo[0] && c + bytes <= g.hi[0]) || (c >= g.lo[1] && c + bytes <= g.hi[1])) return true;
    if (g.status) atomicCAS(g.status, 0, code);
    return false;
}
#define FMM_GUARD(g, ptr, bytes, code) fmm_guard_ok(g, ptr, bytes, code)
#else
#define FMM_GUARD(g, ptr, bytes, code) true
#endif
static inline FmmGuard fmm_make_guard(const void* a, size_t na, const void* b, size_t nb, int* status)
{
    FmmGuard g;
    g.lo[0] = static_cast<const char*>(a); g.hi[0] = g.lo[0] + na;
    g.lo[1] = static_cast<const char*>(b); g.hi[1] = g.lo[1] + nb;
    g.status = status;
    return g;
}
// status word that receives guard violations: plan->d_status[FMM_GUARD_WORD]
#define FMM_GUARD_WORD 2

// Pair-fused decoder (UE8M0 product kernel): the R products of a parent are walked in an order in which consecutive
// products (2s, 2s+1) form a step; the epilogue keeps product A on chip until product B is done and sends ONE weighted
// update wA * M_A + wB * M_B to every output block either of them feeds, which cuts the number of block updates that
// go through L2 (18 -> 11 for the Phi-optimal realization, 12 -> 9 for Strassen).  An unpaired last product is a step
// with wA = 0.
struct FmmPairEntry {
    int row_off, col_off;     // destination block, in units of leaf blocks
    float wA, wB;             // weights of the step's first and second product (wA = 0: first product absent / not used)
    int first;                // 1: overwrite, 0: add
};

struct FmmLayout {            // byte offsets into the workspace
    int64_t m, n, k;          // leaf dimensions
    int64_t terms;            // R^levels (1 for levels == 0)
    size_t qa, qb;            // e4m3 codes, terms x m x k and terms x n x k
    size_t sa, sb;            // scales
    size_t sa_term, sb_term;  // bytes of scales per term
    size_t inter_a[FMM_MAX_LEVELS], inter_b[FMM_MAX_LEVELS];  // fp32 combinations of outer levels
    size_t dec[FMM_MAX_LEVELS];   // dec[l]: R^l partially decoded products of (M/2^l) x (N/2^l) fp32, l = 1 .. levels-1
    size_t total;
};

struct fmm_plan {
    int rank, levels;
    fmm_quant_params_t qp;
    float U[FMM_MAX_RANK][4], V[FMM_MAX_RANK][4], W[FMM_MAX_RANK][4];
    int terms;
    int device;
    // device tables
    int* d_status;            // [64] status words (word 0: first bounded wait that gave up)
    int* d_out_start;         // [terms + 1]
    FmmOutEntry* d_out;       // [total entries], block offsets in units of leaf blocks (scaled at launch)
    int n_out_total;
    int order[FMM_MAX_RANK];  // walk order of the R products of a parent (identity unless the decoder is pair-fused)
    int steps;                // pair-fused decoder: steps per parent, ceil(R / 2)
    int* d_pair_start;        // [parents * steps + 1]
    FmmPairEntry* d_pair;     // entries of all steps
    // kernels launched by the most recent call on this plan; written once, at the end of a call (calls take the
    // plan as const, and two host threads may share one)
    mutable std::atomic<int> last_launches;
};

struct EncodeParams {
    const float* in;          // batch of matrices, each 2*rows x 2*cols (or rows x cols when nq == 1)
    int64_t in_batch_stride;  // elements between consecutive input matrices
    int64_t ld;               // leading dimension of the input matrices
    int batch;                // number of input matrices
    int rows, cols;           // leaf (output) dimensions per combination
    int64_t qoff[4];          // element offsets of the four input blocks that are combined
    int64_t qoff_outer[4];    // two-level kernels: offsets of the four blocks of the outer level
    int nq;                   // number of input blocks read (4, or 1 for a plain pass over one matrix)
    int R;                    // combinations per input matrix
    float coef[FMM_MAX_RANK][4];
    uint8_t* q_out;           // codes, term t = b * R + r at q_out + t * rows * cols
    void* s_out;              // scales
    int64_t s_term_stride;    // bytes between the scale arrays of consecutive terms
    int s_step;               // rows (A side) / columns (B side) by which combination r is shifted inside a shared scale array
    int s_ld;                 // fp32 scales: columns of B / rows of A that the shared scale array covers
    int sf_blocks;            // UE8M0: number of 128-row blocks of the scale-tile array
    float amax_floor;
    int b_tile;               // B side: 128 = one fp32 scale per 128 x 128 tile (blk 128 only), 0 = per column
    int preround_bf16;        // B side: round each combination to bfloat16 before the maximum and the cast
    FmmGuard guard;           // codes and scales of this side
    int overlap_prev;         // B side: the kernel launched just before on the stream is the A-side encoder of the same
                              // call (nothing this kernel reads): it may start while that one drains
};

struct CombParams {
    const float* in;
    int64_t in_batch_stride, ld;
    int batch, rows, cols, R;
    float coef[FMM_MAX_RANK][4];
    float* out;               // dense rows x cols per (b, r)
    FmmGuard guard;
};

// One outward step of the decoder: out[b] (2*rows x 2*cols, block q at (q>>1, q&1)) = sum_r W[r][q] * in[b*R + r]
struct DecodeParams {
    const float* in;          // batch * R matrices, rows x cols each, dense
    float* out;               // batch matrices, 2*rows x 2*cols each, dense
    int batch, rows, cols, R;
    float W[FMM_MAX_RANK][4];
    FmmGuard guard;
};
fmm_status_t fmm_launch_decode(const DecodeParams& p, cudaStream_t st);
fmm_status_t fmm_launch_comb(const CombParams& p, cudaStream_t st);
fmm_status_t fmm_launch_encode_a(const EncodeParams& p, int blk, int mode, cudaStream_t st);
fmm_status_t fmm_launch_encode_b(const EncodeParams& p, int blk, int mode, cudaStream_t st);
// last two recursion levels in one pass (p.rows x p.cols = leaf dimensions, inputs 4*rows x 4*cols)
bool fmm_encode2_supported(bool b_side, int blk, int b_tile, int preround_bf16);
fmm_status_t fmm_launch_encode2_a(const EncodeParams& p, int blk, int mode, cudaStream_t st);
fmm_status_t fmm_launch_encode2_b(const EncodeParams& p, int mode, cudaStream_t st);

struct GemmParams {
    const uint8_t* qa; const uint8_t* qb;   // terms x m x k, terms x n x k
    const void* sa; const void* sb;
    int64_t sa_term, sb_term;               // bytes per term
    float* C; int64_t ldc;                  // full output
    int64_t Mfull, Nfull;
    int m, n, k, terms;
    const int* out_start; const FmmOutEntry* out;
    const int* pair_start; const FmmPairEntry* pair;   // pair-fused decoder tables (UE8M0 kernel)
    int order[FMM_MAX_RANK]; int steps;
    int* status;
    int terms_per_group;                    // consecutive terms that feed the same output blocks (R at levels >= 2, else all)
    int sb_tile;                            // fp32 scales, blk 128: the B-side scale is constant over each 128-column tile
    int overlap_prev;                       // the kernel launched just before on the stream is the B-side encoder of the same call:
                                            // the product kernel may be set up while that one drains (its loads wait for it)
    FmmGuard guard;                         // the output matrix (C, or the stack of parent matrices)
};
// guard word of the statistics kernels, which have no plan (FMM_DEBUG build; always 0 otherwise)
fmm_status_t fmm_stats_guard_read(int* code);
fmm_status_t fmm_launch_bounded_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st);
fmm_status_t fmm_launch_guard_selftest(int* status, cudaStream_t st);
fmm_status_t fmm_launch_gemm(const GemmParams& p, int blk, int mode, cudaStream_t st, int* launches);

static inline int64_t fmm_ipow(int64_t b, int e) { int64_t r = 1; while (e-- > 0) r *= b; return r; }
