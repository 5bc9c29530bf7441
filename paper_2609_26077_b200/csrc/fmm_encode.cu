// Pre-addition + block quantization kernels (paper Sec. 2.2 / App. D.1: the encoded combinations
// S_r = sum_j U[r][j] A_j and T_r = sum_j V[r][j] B_j are formed in fp32 from the unquantized
// operand blocks and only then quantized; App. E.2: per block of `blk` elements along the
// contracted axis, scale = amax / 448 in fp32, round-to-nearest-even cast to e4m3).
//
// Arithmetic is pinned so that the bytes are reproducible: quadrant order 11,12,21,22, zero
// coefficients skipped, first term a rounded multiply, later terms single-rounded FMAs; the
// block is scaled by inv = 448 / max(amax, floor) (one IEEE division per block) and the stored
// scale is max(amax, floor) / 448.  In the power-of-two mode the scale is 2^ceil(log2(.)).
//
// Both kernels are HBM-bound streaming kernels: every input element is read once with
// full-line coalesced loads and every output byte is written once in whole 32-byte sectors.
#include <cuda_bf16.h>
#include <string.h>
#include "fmm_internal.h"
#include "fmm_ptx.cuh"

namespace {
using fmmptx::pack2; using fmmptx::unpack2; using fmmptx::mul2; using fmmptx::fma2;

__device__ __forceinline__ uint16_t cvt_e4m3x2(float hi, float lo)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint32_t pack4_e4m3(float a, float b, float c, float d)
{
    return (uint32_t)cvt_e4m3x2(b, a) | ((uint32_t)cvt_e4m3x2(d, c) << 16);
}

// Scale of one block from its amax.  Returns the multiplier applied before the cast and writes
// the stored scale (fp32 mode) or the biased power-of-two exponent (UE8M0 mode).
template <int MODE>
__device__ __forceinline__ float block_scale(float amax, float floor_, float& s_out, uint32_t& e8_out)
{
    const float amax_c = fmaxf(amax, floor_);
    if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
        s_out = __fdiv_rn(amax_c, 448.0f);
        e8_out = 0;
        return __fdiv_rn(448.0f, amax_c);
    } else {
        const float s0 = __fdiv_rn(amax_c, 448.0f);
        const uint32_t u = __float_as_uint(s0);
        const int ex = (int)(u >> 23);
        const uint32_t man = u & 0x7fffffu;
        int e;
        if (ex == 0) {
            const int hi = 31 - __clz((int)man);
            e = hi - 149 + ((man & (man - 1u)) ? 1 : 0);
        } else {
            e = ex - 127 + (man ? 1 : 0);
        }
        e = max(-127, min(127, e));
        e8_out = (uint32_t)(e + 127);
        s_out = 0.0f;
        // 2^-e, exact; -e == -127 is the subnormal 2^-127
        const int ne = -e;
        return ne >= -126 ? __uint_as_float((uint32_t)(ne + 127) << 23) : __uint_as_float(0x00400000u);
    }
}

// ---------------------------------------------------------------------------------------------
// A side.  One warp handles 128 consecutive k of one output row: 32 lanes x float4, a 512-byte
// coalesced read per quadrant.  A block of BLK elements is held by BLK/4 adjacent lanes.  All R
// combinations are formed first (two elements per fp32x2 instruction); their R block maxima are
// reduced with a transposing butterfly that leaves combination (lane & 7) in each lane, so the
// two IEEE divisions of a block are executed once per block instead of once per lane and
// combination; the multiplier is then broadcast back with one shuffle per combination.
//
// NZ is the zero pattern of the coefficients (bit 4r+j set when coef[r][j] != 0) when it is known at
// compile time - the named realizations are pre-instantiated so that the zero tests, the "first term"
// distinction and the rank guard cost nothing - or 0 for the generic run-time tests.
template <uint32_t NZ> __device__ __forceinline__ bool coef_used(int r, int j, float c)
{ return NZ ? ((NZ >> (4 * r + j)) & 1u) != 0 : (c != 0.0f); }
template <uint32_t NZ> __device__ __forceinline__ bool row_used(int r, int R)
{ return NZ ? ((NZ >> (4 * r)) & 15u) != 0 : (r < R); }

// The arithmetic of one chunk, shared by the one-level and two-level kernels.  x[j] holds four consecutive
// elements (along the contracted axis) of input block j; the GROUP lanes that share a quantization block are
// adjacent.  Forms the R combinations v[r], reduces their block maxima with a transposing butterfly over the
// 8 lanes (lane & 7) - afterwards each lane holds the maximum of combination (lane & 7) - and computes that
// combination's multiplier `inv` and stored scale (s or e8) once per block instead of once per lane.
template <int GROUP, int MODE, uint32_t NZ>
__device__ __forceinline__ void combine_chunk(const EncodeParams& p, const float4 (&x)[4], int lane,
                                              float4 (&v)[FMM_MAX_RANK], float& inv, float& s, uint32_t& e8)
{
    constexpr unsigned FULL = 0xffffffffu;
    const bool b2 = lane & 4, b1 = lane & 2, b0 = lane & 1;
    float am[FMM_MAX_RANK];
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) {
        v[r] = make_float4(0.f, 0.f, 0.f, 0.f); am[r] = 0.0f;
        if (row_used<NZ>(r, p.R)) {
            bool set = false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float cj = p.coef[r][j];
                if (coef_used<NZ>(r, j, cj)) {
                    if (!set) {
                        v[r].x = __fmul_rn(cj, x[j].x); v[r].y = __fmul_rn(cj, x[j].y);
                        v[r].z = __fmul_rn(cj, x[j].z); v[r].w = __fmul_rn(cj, x[j].w);
                        set = true;
                    } else {
                        v[r].x = __fmaf_rn(cj, x[j].x, v[r].x); v[r].y = __fmaf_rn(cj, x[j].y, v[r].y);
                        v[r].z = __fmaf_rn(cj, x[j].z, v[r].z); v[r].w = __fmaf_rn(cj, x[j].w, v[r].w);
                    }
                }
            }
            am[r] = fmaxf(fmaxf(fabsf(v[r].x), fabsf(v[r].y)), fmaxf(fabsf(v[r].z), fabsf(v[r].w)));
        }
    }
    float w[4], x2[2], mine;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float send = b2 ? am[j] : am[j + 4], keep = b2 ? am[j + 4] : am[j];
        w[j] = fmaxf(keep, __shfl_xor_sync(FULL, send, 4));
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const float send = b1 ? w[j] : w[j + 2], keep = b1 ? w[j + 2] : w[j];
        x2[j] = fmaxf(keep, __shfl_xor_sync(FULL, send, 2));
    }
    {
        const float send = b0 ? x2[0] : x2[1], keep = b0 ? x2[1] : x2[0];
        mine = fmaxf(keep, __shfl_xor_sync(FULL, send, 1));
    }
    if (GROUP == 32) {
        mine = fmaxf(mine, __shfl_xor_sync(FULL, mine, 8));
        mine = fmaxf(mine, __shfl_xor_sync(FULL, mine, 16));
    }
    inv = block_scale<MODE>(mine, p.amax_floor, s, e8);
}

// One combination of the outer level, in registers: the same rounded-multiply / FMA chain as above.
template <uint32_t NZ>
__device__ __forceinline__ float4 combine_outer(const EncodeParams& p, int r, const float4 (&raw)[4][4], int q2)
{
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    bool set = false;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float cj = p.coef[r][j];
        if (coef_used<NZ>(r, j, cj)) {
            const float4 a = raw[j][q2];
            if (!set) {
                o.x = __fmul_rn(cj, a.x); o.y = __fmul_rn(cj, a.y); o.z = __fmul_rn(cj, a.z); o.w = __fmul_rn(cj, a.w);
                set = true;
            } else {
                o.x = __fmaf_rn(cj, a.x, o.x); o.y = __fmaf_rn(cj, a.y, o.y);
                o.z = __fmaf_rn(cj, a.z, o.z); o.w = __fmaf_rn(cj, a.w, o.w);
            }
        }
    }
    return o;
}

// A-side stores of one chunk: four code bytes per lane and combination; the scale of combination (lane & 7).
// b = index of the input matrix (terms b*R .. b*R + R-1), i = leaf row, c = 128-k chunk.
template <int BLK, int MODE, uint32_t NZ>
__device__ __forceinline__ void store_chunk_a(const EncodeParams& p, const float4 (&v)[FMM_MAX_RANK], float inv, float s,
                                              uint32_t e8, int b, int i, int c, int lane)
{
    constexpr int GROUP = BLK / 4;
    constexpr unsigned FULL = 0xffffffffu;
    const int64_t term_codes = (int64_t)p.rows * p.cols;
    const int my_r = lane & 7;
    uint8_t* qp = p.q_out + ((int64_t)b * p.R) * term_codes + (int64_t)i * p.cols + c * 128 + lane * 4;
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) {
        if (row_used<NZ>(r, p.R)) {
            const float inv_r = __shfl_sync(FULL, inv, (GROUP == 32) ? r : ((lane & 24) | r));
            if (FMM_GUARD(p.guard, qp, 4, 1101))
            *reinterpret_cast<uint32_t*>(qp) = pack4_e4m3(__fmul_rn(v[r].x, inv_r), __fmul_rn(v[r].y, inv_r),
                                                          __fmul_rn(v[r].z, inv_r), __fmul_rn(v[r].w, inv_r));
        }
        qp += term_codes;
    }
    // scales: lane holds the scale of combination my_r, block (lane / GROUP) of this chunk
    if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
        if (my_r < p.R && (GROUP == 8 || lane < 8)) {
            // chunk-major: [128-k chunk c][row i][K block of the chunk], so the scales one pipeline stage of the
            // product kernel needs for 128 rows are contiguous, and this warp's (up to four) scales are adjacent;
            // combination my_r is shifted by my_r * s_step rows when several combinations share one array
            // (row panels of a plain pass)
            float* so = reinterpret_cast<float*>(reinterpret_cast<char*>(p.s_out) + ((int64_t)b * p.R + my_r) * p.s_term_stride);
            float* sp = so + ((int64_t)c * p.s_ld + i + my_r * p.s_step) * (128 / BLK) + (GROUP == 8 ? (lane >> 3) : 0);
            if (FMM_GUARD(p.guard, sp, 4, 1102)) *sp = s;
        }
    } else {
        // four exponent bytes of this row (blocks 4c .. 4c+3) form one aligned word of the scale tile
        uint32_t wv = e8 << (8 * (lane >> 3));
        wv |= __shfl_xor_sync(FULL, wv, 8);
        wv |= __shfl_xor_sync(FULL, wv, 16);
        if (lane < 8 && lane < p.R) {
            char* so = reinterpret_cast<char*>(p.s_out) + ((int64_t)b * p.R + lane) * p.s_term_stride;
            const int ig = i + lane * p.s_step;            // row inside the scale-tile array
            const int64_t tile = (int64_t)c * p.sf_blocks + (ig >> 7);
            char* sp = so + tile * 512 + (ig & 31) * 16 + ((ig & 127) >> 5) * 4;
            if (FMM_GUARD(p.guard, sp, 4, 1103)) *reinterpret_cast<uint32_t*>(sp) = wv;
        }
    }
}

template <int BLK, int MODE, uint32_t NZ>
__global__ void __launch_bounds__(256) encode_a_kernel(const EncodeParams p)
{
    fmmptx::griddep_launch_dependents();           // the B-side encoder of the same call reads nothing written here
    constexpr int GROUP = BLK / 4;                 // lanes per block
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const uint32_t warp_gid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const int chunks = p.cols / 128;
    // a task is CPT consecutive 128-k chunks of one output row (two adjacent rows at block 32 with fp32 scales).  Tasks
    // are dealt to warps round-robin (32-bit index arithmetic only: one division per task, none per chunk).  The fp32
    // scales of a chunk are stored row after row (16 bytes per row at block 32, 4 at block 128), so partial sectors
    // are avoided this way: block 32 walks two rows per task, the two rows of a chunk back to back (one 32-byte sector
    // per pair of stores); block 128 makes the ROW the fastest task index, so that the eight warps of a block hold
    // eight consecutive rows of the same chunks.  Both choices are the measured better one for their block size
    // (n = 8192, both sides: 0.160 vs 0.165 ms, and 0.158 vs 0.162 ms).  The power-of-two mode writes its exponent
    // bytes in row-major tiles: one row per task, chunk group fastest.
    const int CPT = (chunks % 8 == 0) ? 8 : ((chunks % 4 == 0) ? 4 : 1);
    constexpr bool FP32S = (MODE == FMM_SCALE_FP32_AMAX_DIV_448);
    const int RPT = (FP32S && BLK == 32 && p.rows % 2 == 0) ? 2 : 1;
    constexpr bool ROW_FASTEST = FP32S && BLK == 128;
    const uint32_t tasks_per_row = (uint32_t)(chunks / CPT);
    const uint32_t row_groups = (uint32_t)(p.rows / RPT);
    const uint32_t rows_all = (uint32_t)p.batch * row_groups;
    const uint32_t tasks = rows_all * tasks_per_row;

    for (uint32_t task = warp_gid; task < tasks; task += nwarps) {
      const uint32_t cgrp = ROW_FASTEST ? task / rows_all : 0u;
      const uint32_t row_id = ROW_FASTEST ? task - cgrp * rows_all : task / tasks_per_row;
      const int c0 = (int)(ROW_FASTEST ? cgrp : task - row_id * tasks_per_row) * CPT;
      const int b = (int)(row_id / row_groups);
      const int i0 = (int)(row_id - (uint32_t)b * row_groups) * RPT;
      // the loads of step n+1 are issued before step n is processed (two steps in flight per warp); step = (chunk, row)
      const float* row_base = p.in + (int64_t)b * p.in_batch_stride + (int64_t)i0 * p.ld + lane * 4;
      const int steps = CPT * RPT;
      float4 xn[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
          if (j < p.nq) xn[j] = __ldcs(reinterpret_cast<const float4*>(row_base + c0 * 128 + p.qoff[j]));
      for (int st = 0; st < steps; ++st) {
        const int c = c0 + st / RPT, i = i0 + st % RPT;
        float4 x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) x[j] = xn[j];
        if (st + 1 < steps) {
            const int cn = c0 + (st + 1) / RPT, rn = (st + 1) % RPT;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < p.nq) xn[j] = __ldcs(reinterpret_cast<const float4*>(row_base + (int64_t)rn * p.ld + cn * 128 + p.qoff[j]));
        }

        float4 v[FMM_MAX_RANK];
        float inv, s; uint32_t e8;
        combine_chunk<GROUP, MODE, NZ>(p, x, lane, v, inv, s, e8);

        store_chunk_a<BLK, MODE, NZ>(p, v, inv, s, e8, b, i, c, lane);
      }
    }
}

// ---------------------------------------------------------------------------------------------
// B side.  Blocks run along k, the strided axis of row-major B, and the output is K-major (the
// tensor-core operand layout).  A thread owns 16 consecutive k of one column n; lanes l and l+16
// hold the two halves of a 32-element (sub-)block, so one shuffle completes the amax.  Each load
// is two 64-byte row segments per warp; each thread writes 16 contiguous code bytes and the two
// lanes of a block fill one 32-byte sector.  BLK == 128 takes a second pass over the four
// 32-element sub-blocks (served by L1/L2).
//
// TILE (App. E.5, the deployment-matched weight grouping; BLK == 128, FP32 scales): one scale per tile of
// 128 k x 128 columns of each encoded combination.  A block of 256 threads then covers a whole tile, the
// column maxima of the first pass are reduced across the block, and every column stores the tile's scale,
// so the scale array keeps its per-column shape.  p.preround_bf16 rounds each encoded combination to
// bfloat16 (nearest even) before the maximum and the cast, as the paper's real kernel does.
template <int MODE>
__device__ __forceinline__ void store_b_scale(const EncodeParams& p, int64_t t, int r, int j, int kb, int kc,
                                              float s, uint32_t e8word, bool last_of_word)
{
    char* so = reinterpret_cast<char*>(p.s_out) + t * p.s_term_stride;
    const int jg = j + r * p.s_step;                   // column inside the scale array
    if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
        float* sp = reinterpret_cast<float*>(so) + (int64_t)kb * p.s_ld + jg;
        if (FMM_GUARD(p.guard, sp, 4, 1201)) *sp = s;
    } else if (last_of_word) {
        const int64_t tile = (int64_t)kc * p.sf_blocks + (jg >> 7);
        char* sp = so + tile * 512 + (jg & 31) * 16 + ((jg & 127) >> 5) * 4;
        if (FMM_GUARD(p.guard, sp, 4, 1202)) *reinterpret_cast<uint32_t*>(sp) = e8word;
    }
}

template <int BLK, int MODE, uint32_t NZ, bool TILE, bool PRE>
__global__ void __launch_bounds__(TILE ? 256 : 128, TILE ? 2 : 4) encode_b_kernel(const EncodeParams p)
{
    static_assert(!(TILE || PRE) || (BLK == 128 && MODE == FMM_SCALE_FP32_AMAX_DIV_448), "weight-side options: blk 128, fp32");
    // here p.rows = leaf k (contracted), p.cols = leaf n
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int WARPS = TILE ? 8 : 4;
    __shared__ float tile_amax[TILE ? WARPS : 1][FMM_MAX_RANK];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j = blockIdx.x * (WARPS * 16) + warp * 16 + (lane & 15);
    const int khalf = lane >> 4;
    const int kc = blockIdx.y;                      // chunk of 128 k
    const int b = blockIdx.z;
    const float* base = p.in + (int64_t)b * p.in_batch_stride + j;
    const int64_t term_codes = (int64_t)p.rows * p.cols;

    float raw[4][16];
    float blk_amax[FMM_MAX_RANK], blk_inv[FMM_MAX_RANK];
    uint32_t e8word[FMM_MAX_RANK];
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) { blk_amax[r] = 0.0f; blk_inv[r] = 0.0f; e8word[r] = 0; }

    constexpr int PASSES = (BLK == 32) ? 1 : 2;
#pragma unroll 1
    for (int pass = 0; pass < PASSES; ++pass) {
#pragma unroll 1
        for (int sub = 0; sub < 4; ++sub) {
            const int k0 = kc * 128 + sub * 32 + khalf * 16;
#pragma unroll
            for (int jq = 0; jq < 4; ++jq)
                if (jq < p.nq) {
#pragma unroll
                    for (int kk = 0; kk < 16; ++kk)
                        raw[jq][kk] = __ldg(base + p.qoff[jq] + (int64_t)(k0 + kk) * p.ld);
                }
#pragma unroll
            for (int r = 0; r < FMM_MAX_RANK; ++r) {
                if (row_used<NZ>(r, p.R)) {
                    float v[16];
                    bool set = false;
#pragma unroll
                    for (int jq = 0; jq < 4; ++jq) {
                        const float cj = p.coef[r][jq];
                        if (coef_used<NZ>(r, jq, cj)) {
                            if (!set) {
#pragma unroll
                                for (int kk = 0; kk < 16; ++kk) v[kk] = __fmul_rn(cj, raw[jq][kk]);
                                set = true;
                            } else {
#pragma unroll
                                for (int kk = 0; kk < 16; ++kk) v[kk] = __fmaf_rn(cj, raw[jq][kk], v[kk]);
                            }
                        }
                    }
                    if (!set) {
#pragma unroll
                        for (int kk = 0; kk < 16; ++kk) v[kk] = 0.0f;
                    }
                    if (PRE) {
#pragma unroll
                        for (int kk = 0; kk < 16; ++kk) v[kk] = __bfloat162float(__float2bfloat16_rn(v[kk]));
                    }
                    const int64_t t = (int64_t)b * p.R + r;
                    if (BLK == 32 || pass == 0) {
                        float amax = 0.0f;
#pragma unroll
                        for (int kk = 0; kk < 16; ++kk) amax = fmaxf(amax, fabsf(v[kk]));
                        amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 16));
                        if (BLK == 32) blk_amax[r] = amax; else blk_amax[r] = fmaxf(blk_amax[r], amax);
                    }
                    if (!TILE && (BLK == 32 || (pass == 0 && sub == 3))) {
                        float sc; uint32_t e8;
                        blk_inv[r] = block_scale<MODE>(blk_amax[r], p.amax_floor, sc, e8);
                        const int kb = (BLK == 32) ? (kc * 4 + sub) : kc;
                        e8word[r] |= e8 << (8 * (kb & 3));
                        if (khalf == 0) store_b_scale<MODE>(p, t, r, j, kb, kc, sc, e8word[r], (kb & 3) == 3);
                    }
                    if (BLK == 32 || pass == 1) {
                        const float inv = blk_inv[r];
                        uint32_t wv[4];
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            wv[g] = pack4_e4m3(__fmul_rn(v[4 * g], inv), __fmul_rn(v[4 * g + 1], inv),
                                               __fmul_rn(v[4 * g + 2], inv), __fmul_rn(v[4 * g + 3], inv));
                        uint8_t* qp = p.q_out + t * term_codes + (int64_t)j * p.rows + k0;
                        if (FMM_GUARD(p.guard, qp, 16, 1203)) *reinterpret_cast<uint4*>(qp) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
                    }
                }
            }
        }
        if (TILE && pass == 0) {
            // column maxima -> tile maximum: 16 columns per warp by shuffles, 8 warps through shared memory
#pragma unroll
            for (int r = 0; r < FMM_MAX_RANK; ++r) {
                float a = blk_amax[r];
#pragma unroll
                for (int d = 8; d >= 1; d >>= 1) a = fmaxf(a, __shfl_xor_sync(FULL, a, d));
                if (lane == 0) tile_amax[warp][r] = a;
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < FMM_MAX_RANK; ++r) {
                if (row_used<NZ>(r, p.R)) {
                    float a = tile_amax[0][r];
#pragma unroll
                    for (int w = 1; w < WARPS; ++w) a = fmaxf(a, tile_amax[w][r]);
                    float sc; uint32_t e8;
                    blk_inv[r] = block_scale<MODE>(a, p.amax_floor, sc, e8);
                    if (khalf == 0) store_b_scale<MODE>(p, (int64_t)b * p.R + r, r, j, kc, kc, sc, 0u, false);
                }
            }
        }
    }
    // the product kernel, launched behind this one by the same call, may be scheduled as soon as every block has got
    // here: its launch latency and set-up then fall under this grid's last blocks (signalling at the start instead lets
    // its CTAs take SMs from this grid's tail: 0.5 % slower back to back)
    fmmptx::griddep_launch_dependents();
    // a launch that overlapped the A-side encoder must not end before it (what follows on the stream needs both):
    // the last block of the grid waits for it, the others leave as they finish
    if (blockIdx.x + 1 == gridDim.x && blockIdx.y + 1 == gridDim.y && blockIdx.z + 1 == gridDim.z) fmmptx::griddep_wait();
}

// B side, block 32, one 32-k block of 16 columns per warp (thread = 16 k of one column, lanes l and l+16 the two
// halves of a block), so every thread issues all its loads at once.  A thread block is a single warp: the warps
// share nothing, and one-warp blocks let the scheduler replace each finished warp on its own (2 % faster than four
// warps of one 128-k chunk per block; blocks of two to eight warps side by side, covering 128- to 512-byte row
// segments, are within 1 %).  Grid: (cols / 16, rows / 32, batch), 32 threads.
template <int MODE, uint32_t NZ>
__global__ void __launch_bounds__(32, 16) encode_b32_kernel(const EncodeParams p)
{
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x;
    const int col = lane & 15, khalf = lane >> 4;
    const int j = blockIdx.x * 16 + col;
    const int kb = blockIdx.y;                      // this warp's quantization block
    const int kc = kb >> 2;                         // its chunk of 128 k
    const int b = blockIdx.z;
    const int k0 = kb * 32 + khalf * 16;
    const float* base = p.in + (int64_t)b * p.in_batch_stride + j;
    const int64_t term_codes = (int64_t)p.rows * p.cols;

    float raw[4][16];
#pragma unroll
    for (int jq = 0; jq < 4; ++jq)
        if (jq < p.nq) {
#pragma unroll
            for (int kk = 0; kk < 16; ++kk)
                raw[jq][kk] = __ldg(base + p.qoff[jq] + (int64_t)(k0 + kk) * p.ld);
        }
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) {
        if (row_used<NZ>(r, p.R)) {
            float v[16];
            bool set = false;
#pragma unroll
            for (int jq = 0; jq < 4; ++jq) {
                const float cj = p.coef[r][jq];
                if (coef_used<NZ>(r, jq, cj)) {
                    if (!set) {
#pragma unroll
                        for (int kk = 0; kk < 16; ++kk) v[kk] = __fmul_rn(cj, raw[jq][kk]);
                        set = true;
                    } else {
#pragma unroll
                        for (int kk = 0; kk < 16; ++kk) v[kk] = __fmaf_rn(cj, raw[jq][kk], v[kk]);
                    }
                }
            }
            if (!set) {
#pragma unroll
                for (int kk = 0; kk < 16; ++kk) v[kk] = 0.0f;
            }
            float amax = 0.0f;
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) amax = fmaxf(amax, fabsf(v[kk]));
            amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 16));
            float sc; uint32_t e8;
            const float inv = block_scale<MODE>(amax, p.amax_floor, sc, e8);
            const int64_t t = (int64_t)b * p.R + r;
            if (khalf == 0) {
                char* so = reinterpret_cast<char*>(p.s_out) + t * p.s_term_stride;
                const int jg = j + r * p.s_step;                   // column inside the scale array
                if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
                    float* sp = reinterpret_cast<float*>(so) + (int64_t)kb * p.s_ld + jg;
                    if (FMM_GUARD(p.guard, sp, 4, 1205)) *sp = sc;
                } else {
                    const int64_t tile = (int64_t)kc * p.sf_blocks + (jg >> 7);
                    char* sp = so + tile * 512 + (jg & 31) * 16 + ((jg & 127) >> 5) * 4 + (kb & 3);
                    if (FMM_GUARD(p.guard, sp, 1, 1206)) *reinterpret_cast<uint8_t*>(sp) = (uint8_t)e8;
                }
            }
            uint32_t wv[4];
#pragma unroll
            for (int g = 0; g < 4; ++g)
                wv[g] = pack4_e4m3(__fmul_rn(v[4 * g], inv), __fmul_rn(v[4 * g + 1], inv),
                                   __fmul_rn(v[4 * g + 2], inv), __fmul_rn(v[4 * g + 3], inv));
            uint8_t* qp = p.q_out + t * term_codes + (int64_t)j * p.rows + k0;
            if (FMM_GUARD(p.guard, qp, 16, 1207)) *reinterpret_cast<uint4*>(qp) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
    }
    // the product kernel, launched behind this one by the same call, may be scheduled as soon as every block has got
    // here: its launch latency and set-up then fall under this grid's last blocks (signalling at the start instead lets
    // its CTAs take SMs from this grid's tail: 0.5 % slower back to back)
    fmmptx::griddep_launch_dependents();
    // a launch that overlapped the A-side encoder must not end before it (what follows on the stream needs both):
    // the last block of the grid waits for it, the others leave as they finish
    if (blockIdx.x + 1 == gridDim.x && blockIdx.y + 1 == gridDim.y && blockIdx.z + 1 == gridDim.z) fmmptx::griddep_wait();
}

// B side, block 128, per-column scales, one pass.  The four warps of a block take the four 32-k sub-blocks of one
// 128-k block of the same 16 columns; every thread forms the combinations of its 16 k x 1 column, the sub-block
// maxima meet in shared memory, and each warp then quantizes its own sub-block from the raw values it still holds
// (the combinations are formed a second time in registers - the same rounded-multiply / FMA chain, so the same bits -
// instead of reading the operand a second time).  Grid: (cols / 16, rows / 128, batch), 128 threads.
template <uint32_t NZ>
__global__ void __launch_bounds__(128, 4) encode_b128_kernel(const EncodeParams p)
{
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int MODE = FMM_SCALE_FP32_AMAX_DIV_448;
    __shared__ float sub_amax[4][FMM_MAX_RANK][16];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = lane & 15, khalf = lane >> 4;
    const int j = blockIdx.x * 16 + col;
    const int kc = blockIdx.y;                      // chunk of 128 k = one quantization block
    const int b = blockIdx.z;
    const int k0 = kc * 128 + warp * 32 + khalf * 16;
    const float* base = p.in + (int64_t)b * p.in_batch_stride + j;
    const int64_t term_codes = (int64_t)p.rows * p.cols;

    float raw[4][16];
#pragma unroll
    for (int jq = 0; jq < 4; ++jq)
        if (jq < p.nq) {
#pragma unroll
            for (int kk = 0; kk < 16; ++kk)
                raw[jq][kk] = __ldg(base + p.qoff[jq] + (int64_t)(k0 + kk) * p.ld);
        }
    auto combine = [&](int r, float (&v)[16]) {
        bool set = false;
#pragma unroll
        for (int jq = 0; jq < 4; ++jq) {
            const float cj = p.coef[r][jq];
            if (coef_used<NZ>(r, jq, cj)) {
                if (!set) {
#pragma unroll
                    for (int kk = 0; kk < 16; ++kk) v[kk] = __fmul_rn(cj, raw[jq][kk]);
                    set = true;
                } else {
#pragma unroll
                    for (int kk = 0; kk < 16; ++kk) v[kk] = __fmaf_rn(cj, raw[jq][kk], v[kk]);
                }
            }
        }
        if (!set) {
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) v[kk] = 0.0f;
        }
    };
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) {
        if (row_used<NZ>(r, p.R)) {
            float v[16];
            combine(r, v);
            float amax = 0.0f;
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) amax = fmaxf(amax, fabsf(v[kk]));
            amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 16));
            if (khalf == 0) sub_amax[warp][r][col] = amax;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) {
        if (row_used<NZ>(r, p.R)) {
            const float amax = fmaxf(fmaxf(sub_amax[0][r][col], sub_amax[1][r][col]), fmaxf(sub_amax[2][r][col], sub_amax[3][r][col]));
            float sc; uint32_t e8;
            const float inv = block_scale<MODE>(amax, p.amax_floor, sc, e8);
            const int64_t t = (int64_t)b * p.R + r;
            if (warp == 0 && khalf == 0) store_b_scale<MODE>(p, t, r, j, kc, kc, sc, 0u, false);
            float v[16];
            combine(r, v);
            uint32_t wv[4];
#pragma unroll
            for (int g = 0; g < 4; ++g)
                wv[g] = pack4_e4m3(__fmul_rn(v[4 * g], inv), __fmul_rn(v[4 * g + 1], inv),
                                   __fmul_rn(v[4 * g + 2], inv), __fmul_rn(v[4 * g + 3], inv));
            uint8_t* qp = p.q_out + t * term_codes + (int64_t)j * p.rows + k0;
            if (FMM_GUARD(p.guard, qp, 16, 1204)) *reinterpret_cast<uint4*>(qp) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
    }
    // the product kernel, launched behind this one by the same call, may be scheduled as soon as every block has got
    // here: its launch latency and set-up then fall under this grid's last blocks (signalling at the start instead lets
    // its CTAs take SMs from this grid's tail: 0.5 % slower back to back)
    fmmptx::griddep_launch_dependents();
    // a launch that overlapped the A-side encoder must not end before it (what follows on the stream needs both):
    // the last block of the grid waits for it, the others leave as they finish
    if (blockIdx.x + 1 == gridDim.x && blockIdx.y + 1 == gridDim.y && blockIdx.z + 1 == gridDim.z) fmmptx::griddep_wait();
}

// ---------------------------------------------------------------------------------------------
// Two recursion levels in one pass (levels >= 2): the combinations of the second-to-last level are formed in
// registers from the 16 sub-blocks and fed to the leaf-level arithmetic above, so the 7 fp32 intermediate
// matrices of that level are neither written nor read back.  The rounding sequence is the one of the
// level-by-level evaluation (Sec. 3: recursion = Kronecker power; each level a rounded multiply / FMA chain
// in fp32), so the bytes are identical.  p.rows x p.cols are the leaf dimensions, the input matrices are
// 4*rows x 4*cols, p.qoff_outer[] / p.qoff[] the block offsets of the two levels; terms are numbered
// (b * R + r1) * R + r2.
template <int BLK, int MODE, uint32_t NZ>
__global__ void __launch_bounds__(256) encode2_a_kernel(const EncodeParams p)
{
    fmmptx::griddep_launch_dependents();           // as encode_a_kernel
    constexpr int GROUP = BLK / 4;
    const int lane = threadIdx.x & 31;
    const uint32_t warp_gid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t chunks = (uint32_t)(p.cols / 128);
    const uint32_t tasks = (uint32_t)p.batch * (uint32_t)p.rows * chunks;       // one 128-k chunk of one leaf row
    for (uint32_t task = warp_gid; task < tasks; task += nwarps) {
        const uint32_t row_id = task / chunks;
        const int c = (int)(task - row_id * chunks);
        const int b = (int)(row_id / (uint32_t)p.rows);
        const int i = (int)(row_id - (uint32_t)b * (uint32_t)p.rows);
        const float* base = p.in + (int64_t)b * p.in_batch_stride + (int64_t)i * p.ld + c * 128 + lane * 4;
        float4 raw[4][4];                                   // [outer block][inner block]
#pragma unroll
        for (int q1 = 0; q1 < 4; ++q1)
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2)
                raw[q1][q2] = __ldcs(reinterpret_cast<const float4*>(base + p.qoff_outer[q1] + p.qoff[q2]));
#pragma unroll
        for (int r1 = 0; r1 < FMM_MAX_RANK; ++r1) {
            if (row_used<NZ>(r1, p.R)) {
                float4 x[4];
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2) x[q2] = combine_outer<NZ>(p, r1, raw, q2);
                float4 v[FMM_MAX_RANK];
                float inv, s; uint32_t e8;
                combine_chunk<GROUP, MODE, NZ>(p, x, lane, v, inv, s, e8);
                store_chunk_a<BLK, MODE, NZ>(p, v, inv, s, e8, b * p.R + r1, i, c, lane);
            }
        }
    }
}

// B side, block 32: a thread owns 4 consecutive k of one column, the 8 lanes (lane & 7) of a column hold one
// 32-element block, a warp covers 4 adjacent columns (16-byte row segments; the neighbouring warp of the block
// uses the other half of each 32-byte sector).  The eight lanes of a column write 32 contiguous code bytes of
// the K-major output.  Grid: (cols / 32, rows / 32, batch), 256 threads.
template <int MODE, uint32_t NZ>
__global__ void __launch_bounds__(256) encode2_b_kernel(const EncodeParams p)
{
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + warp * 4 + (lane >> 3);        // leaf column
    const int kb = blockIdx.y;                                      // 32-k block
    const int k0 = kb * 32 + (lane & 7) * 4;
    const int b = blockIdx.z;
    const int64_t term_codes = (int64_t)p.rows * p.cols;
    const int my_r = lane & 7;
    // The block's 32 k x 32 columns of each of the 16 sub-blocks go through shared memory: the global loads are
    // whole 128-byte row segments (a thread reading its own 4 k x 1 column directly touches eight lines per warp
    // instruction with 16 bytes each and is bound by L1 wavefronts), the transposed reads are conflict-free with
    // rows padded to 33 words.  Two passes of eight sub-blocks keep the buffer under the static 48 KB.
    __shared__ float tile[8][32][33];
    float4 raw[4][4];
    {
        const int lrow = threadIdx.x >> 3, lc = (threadIdx.x & 7) * 4;
        const float* blk = p.in + (int64_t)b * p.in_batch_stride + ((int64_t)kb * 32 + lrow) * p.ld + blockIdx.x * 32 + lc;
        const int rk = (lane & 7) * 4, rc = warp * 4 + (lane >> 3);
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
            if (pass) __syncthreads();
            float4 v[8];
#pragma unroll
            for (int sblk = 0; sblk < 8; ++sblk)
                v[sblk] = __ldg(reinterpret_cast<const float4*>(blk + p.qoff_outer[2 * pass + (sblk >> 2)] + p.qoff[sblk & 3]));
#pragma unroll
            for (int sblk = 0; sblk < 8; ++sblk) {
                tile[sblk][lrow][lc] = v[sblk].x; tile[sblk][lrow][lc + 1] = v[sblk].y;
                tile[sblk][lrow][lc + 2] = v[sblk].z; tile[sblk][lrow][lc + 3] = v[sblk].w;
            }
            __syncthreads();
#pragma unroll
            for (int sblk = 0; sblk < 8; ++sblk)
                raw[2 * pass + (sblk >> 2)][sblk & 3] = make_float4(tile[sblk][rk][rc], tile[sblk][rk + 1][rc],
                                                                    tile[sblk][rk + 2][rc], tile[sblk][rk + 3][rc]);
        }
    }
#pragma unroll
    for (int r1 = 0; r1 < FMM_MAX_RANK; ++r1) {
        if (row_used<NZ>(r1, p.R)) {
            float4 x[4];
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) x[q2] = combine_outer<NZ>(p, r1, raw, q2);
            float4 v[FMM_MAX_RANK];
            float inv, s; uint32_t e8;
            combine_chunk<8, MODE, NZ>(p, x, lane, v, inv, s, e8);
            const int64_t t0 = ((int64_t)b * p.R + r1) * p.R;
            uint8_t* qp = p.q_out + t0 * term_codes + (int64_t)j * p.rows + k0;
#pragma unroll
            for (int r = 0; r < FMM_MAX_RANK; ++r) {
                if (row_used<NZ>(r, p.R)) {
                    const float inv_r = __shfl_sync(FULL, inv, (lane & 24) | r);
                    if (FMM_GUARD(p.guard, qp, 4, 1301))
                    *reinterpret_cast<uint32_t*>(qp) = pack4_e4m3(__fmul_rn(v[r].x, inv_r), __fmul_rn(v[r].y, inv_r),
                                                                  __fmul_rn(v[r].z, inv_r), __fmul_rn(v[r].w, inv_r));
                }
                qp += term_codes;
            }
            if (my_r < p.R) {
                char* so = reinterpret_cast<char*>(p.s_out) + (t0 + my_r) * p.s_term_stride;
                if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
                    float* sp = reinterpret_cast<float*>(so) + (int64_t)kb * p.s_ld + j;
                    if (FMM_GUARD(p.guard, sp, 4, 1302)) *sp = s;
                } else {
                    const int64_t tile = (int64_t)(kb >> 2) * p.sf_blocks + (j >> 7);
                    char* sp = so + tile * 512 + (j & 31) * 16 + ((j & 127) >> 5) * 4 + (kb & 3);
                    if (FMM_GUARD(p.guard, sp, 1, 1303)) *reinterpret_cast<uint8_t*>(sp) = (uint8_t)e8;
                }
            }
        }
    }
    // the product kernel, launched behind this one by the same call, may be scheduled as soon as every block has got
    // here: its launch latency and set-up then fall under this grid's last blocks (signalling at the start instead lets
    // its CTAs take SMs from this grid's tail: 0.5 % slower back to back)
    fmmptx::griddep_launch_dependents();
    // a launch that overlapped the A-side encoder must not end before it (what follows on the stream needs both):
    // the last block of the grid waits for it, the others leave as they finish
    if (blockIdx.x + 1 == gridDim.x && blockIdx.y + 1 == gridDim.y && blockIdx.z + 1 == gridDim.z) fmmptx::griddep_wait();
}

// fp32 combinations of the outer recursion levels (levels >= 3): out[b*R + r] = sum_j coef[r][j] X_j
__global__ void __launch_bounds__(256) comb_kernel(const CombParams p)
{
    const int c4 = p.cols / 4;
    const int64_t units = (int64_t)p.batch * p.rows * c4;
    const int64_t qoff[4] = {0, (int64_t)p.cols, (int64_t)p.rows * p.ld, (int64_t)p.rows * p.ld + p.cols};
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(u % c4);
        const int64_t bi = u / c4;
        const int i = (int)(bi % p.rows);
        const int b = (int)(bi / p.rows);
        const float* base = p.in + (int64_t)b * p.in_batch_stride + (int64_t)i * p.ld + c * 4;
        float4 x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) x[j] = __ldcs(reinterpret_cast<const float4*>(base + qoff[j]));
        for (int r = 0; r < p.R; ++r) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            bool set = false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float cj = p.coef[r][j];
                if (cj != 0.0f) {
                    if (!set) {
                        v.x = __fmul_rn(cj, x[j].x); v.y = __fmul_rn(cj, x[j].y);
                        v.z = __fmul_rn(cj, x[j].z); v.w = __fmul_rn(cj, x[j].w);
                        set = true;
                    } else {
                        v.x = __fmaf_rn(cj, x[j].x, v.x); v.y = __fmaf_rn(cj, x[j].y, v.y);
                        v.z = __fmaf_rn(cj, x[j].z, v.z); v.w = __fmaf_rn(cj, x[j].w, v.w);
                    }
                }
            }
            float* o = p.out + ((int64_t)b * p.R + r) * p.rows * p.cols + (int64_t)i * p.cols + c * 4;
            if (FMM_GUARD(p.guard, o, 16, 1401)) *reinterpret_cast<float4*>(o) = v;
        }
    }
}

// Outward step of the decoder for levels >= 2: the R partially decoded products of a parent are
// combined into the four blocks of the parent's matrix, out_q = sum_r W[r][q] * in_r (fp32, r ascending,
// zero weights skipped, first term a multiply, later terms FMAs).
__global__ void __launch_bounds__(256) decode_kernel(const DecodeParams p)
{
    const int c4 = p.cols / 4;
    const int64_t units = (int64_t)p.batch * p.rows * c4;
    const int64_t in_stride = (int64_t)p.rows * p.cols;
    const int64_t out_ld = 2 * (int64_t)p.cols;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(u % c4);
        const int64_t bi = u / c4;
        const int i = (int)(bi % p.rows);
        const int b = (int)(bi / p.rows);
        float4 acc[4];
        bool set[4] = {false, false, false, false};
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* src = p.in + ((int64_t)b * p.R) * in_stride + (int64_t)i * p.cols + c * 4;
        // all R loads are issued before the first use (R x 16 bytes in flight per thread)
        float4 xs[FMM_MAX_RANK];
#pragma unroll
        for (int r = 0; r < FMM_MAX_RANK; ++r)
            if (r < p.R) xs[r] = __ldcs(reinterpret_cast<const float4*>(src + r * in_stride));
#pragma unroll
        for (int r = 0; r < FMM_MAX_RANK; ++r) {
            if (r >= p.R) break;
            const float4 x = xs[r];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float w = p.W[r][q];
                if (w != 0.0f) {
                    if (!set[q]) {
                        acc[q].x = __fmul_rn(w, x.x); acc[q].y = __fmul_rn(w, x.y);
                        acc[q].z = __fmul_rn(w, x.z); acc[q].w = __fmul_rn(w, x.w);
                        set[q] = true;
                    } else {
                        acc[q].x = __fmaf_rn(w, x.x, acc[q].x); acc[q].y = __fmaf_rn(w, x.y, acc[q].y);
                        acc[q].z = __fmaf_rn(w, x.z, acc[q].z); acc[q].w = __fmaf_rn(w, x.w, acc[q].w);
                    }
                }
            }
        }
        float* dst = p.out + (int64_t)b * 4 * in_stride;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float* o = dst + ((int64_t)(q >> 1) * p.rows + i) * out_ld + (q & 1) * p.cols + c * 4;
            if (FMM_GUARD(p.guard, o, 16, 1501)) *reinterpret_cast<float4*>(o) = acc[q];
        }
    }
}

int sm_count()
{
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);      // a cached host-side attribute: cheap
    return n > 0 ? n : 148;
}

}  // namespace

fmm_status_t fmm_launch_decode(const DecodeParams& p, cudaStream_t st)
{
    const int64_t units = (int64_t)p.batch * p.rows * (p.cols / 4);
    int64_t blocks = (units + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    decode_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_comb(const CombParams& p, cudaStream_t st)
{
    const int64_t units = (int64_t)p.batch * p.rows * (p.cols / 4);
    int64_t blocks = (units + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    comb_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

namespace {
uint32_t coef_mask(const EncodeParams& p)
{
    uint32_t m = 0;
    for (int r = 0; r < p.R; ++r)
        for (int j = 0; j < 4; ++j)
            if (p.coef[r][j] != 0.0f) m |= 1u << (4 * r + j);
    return m;
}

// zero patterns with pre-instantiated kernels: U and V of Strassen, the Winograd form and the
// Phi-optimal realization, and the identity used to quantize a matrix as four panels
#define FMM_KNOWN_MASKS(X) X(0x0a5381c9u) X(0x0c385a19u) X(0x05dc8f21u) X(0x0ab3f841u) X(0x0f5fc5c9u) X(0x0cfc5f59u) X(0x00008421u)

// Launch of a B-side encoder.  With p.overlap_prev it carries the programmatic-serialization attribute: the kernel
// before it on the stream (the A-side encoder, which signals at its start) need not have drained when this one
// begins, so its blocks fill the SMs that the other's last wave leaves idle (6 % of the encode phase at n = 8192).
template <typename K>
void launch_b_kernel(K kernel, dim3 grid, unsigned threads, cudaStream_t st, const EncodeParams& p)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = dim3(threads, 1, 1); cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = p.overlap_prev ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int BLK, int MODE>
void launch_a(const EncodeParams& p, unsigned g, cudaStream_t st)
{
    const uint32_t m = (p.nq == 4) ? coef_mask(p) : 0u;
    switch (m) {
#define X(M) case M: encode_a_kernel<BLK, MODE, M><<<g, 256, 0, st>>>(p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: encode_a_kernel<BLK, MODE, 0u><<<g, 256, 0, st>>>(p); return;
    }
}
template <int BLK, int MODE>
void launch_b(const EncodeParams& p, dim3 grid, cudaStream_t st)
{
    const uint32_t m = (p.nq == 4) ? coef_mask(p) : 0u;
    switch (m) {
#define X(M) case M: launch_b_kernel(encode_b_kernel<BLK, MODE, M, false, false>, grid, 128, st, p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: launch_b_kernel(encode_b_kernel<BLK, MODE, 0u, false, false>, grid, 128, st, p); return;
    }
}
template <int MODE>
void launch_b32(const EncodeParams& p, dim3 grid, cudaStream_t st)
{
    const uint32_t m = (p.nq == 4) ? coef_mask(p) : 0u;
    switch (m) {
#define X(M) case M: launch_b_kernel(encode_b32_kernel<MODE, M>, grid, 32, st, p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: launch_b_kernel(encode_b32_kernel<MODE, 0u>, grid, 32, st, p); return;
    }
}
void launch_b128(const EncodeParams& p, dim3 grid, cudaStream_t st)
{
    const uint32_t m = (p.nq == 4) ? coef_mask(p) : 0u;
    switch (m) {
#define X(M) case M: launch_b_kernel(encode_b128_kernel<M>, grid, 128, st, p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: launch_b_kernel(encode_b128_kernel<0u>, grid, 128, st, p); return;
    }
}
template <int BLK, int MODE>
void launch_a2(const EncodeParams& p, unsigned g, cudaStream_t st)
{
    switch (coef_mask(p)) {
#define X(M) case M: encode2_a_kernel<BLK, MODE, M><<<g, 256, 0, st>>>(p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: encode2_a_kernel<BLK, MODE, 0u><<<g, 256, 0, st>>>(p); return;
    }
}
template <int MODE>
void launch_b2(const EncodeParams& p, dim3 grid, cudaStream_t st)
{
    switch (coef_mask(p)) {
#define X(M) case M: launch_b_kernel(encode2_b_kernel<MODE, M>, grid, 256, st, p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: launch_b_kernel(encode2_b_kernel<MODE, 0u>, grid, 256, st, p); return;
    }
}
// weight-side options (tile scales and / or bf16 pre-round): blk 128, fp32 scales
template <bool TILE, bool PRE>
void launch_b_opt(const EncodeParams& p, dim3 grid, cudaStream_t st)
{
    constexpr int F = FMM_SCALE_FP32_AMAX_DIV_448;
    constexpr int T = TILE ? 256 : 128;
    const uint32_t m = (p.nq == 4) ? coef_mask(p) : 0u;
    switch (m) {
#define X(M) case M: launch_b_kernel(encode_b_kernel<128, F, M, TILE, PRE>, grid, T, st, p); return;
        FMM_KNOWN_MASKS(X)
#undef X
        default: launch_b_kernel(encode_b_kernel<128, F, 0u, TILE, PRE>, grid, T, st, p); return;
    }
}
}  // namespace

fmm_status_t fmm_launch_encode_a(const EncodeParams& p, int blk, int mode, cudaStream_t st)
{
    // one task (8, 4 or 1 chunks of 128 k of one row) per warp; the block scheduler balances the SMs
    const int chunks = p.cols / 128;
    const int cpt = (chunks % 8 == 0) ? 8 : ((chunks % 4 == 0) ? 4 : 1);
    const int64_t tasks = (int64_t)p.batch * p.rows * (chunks / cpt);
    int64_t blocks = (tasks + 7) / 8;
    if (blocks > 0x7fffffff) blocks = 0x7fffffff;
    const unsigned g = (unsigned)blocks;
    if (mode == FMM_SCALE_FP32_AMAX_DIV_448) {
        if (blk == 32) launch_a<32, FMM_SCALE_FP32_AMAX_DIV_448>(p, g, st);
        else launch_a<128, FMM_SCALE_FP32_AMAX_DIV_448>(p, g, st);
    } else {
        launch_a<32, FMM_SCALE_UE8M0_CEIL>(p, g, st);
    }
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_encode_b(const EncodeParams& p, int blk, int mode, cudaStream_t st)
{
    dim3 grid((unsigned)(p.cols / 64), (unsigned)(p.rows / 128), (unsigned)p.batch);
    if (p.b_tile || p.preround_bf16) {
        if (p.b_tile) grid.x = (unsigned)(p.cols / 128);
        if (p.b_tile && p.preround_bf16) launch_b_opt<true, true>(p, grid, st);
        else if (p.b_tile) launch_b_opt<true, false>(p, grid, st);
        else launch_b_opt<false, true>(p, grid, st);
    } else if (mode == FMM_SCALE_FP32_AMAX_DIV_448) {
        grid.x = (unsigned)(p.cols / 16);
        if (blk == 32) { grid.y = (unsigned)(p.rows / 32); launch_b32<FMM_SCALE_FP32_AMAX_DIV_448>(p, grid, st); }
        else launch_b128(p, grid, st);
    } else {
        grid.x = (unsigned)(p.cols / 16); grid.y = (unsigned)(p.rows / 32);
        launch_b32<FMM_SCALE_UE8M0_CEIL>(p, grid, st);
    }
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

bool fmm_encode2_supported(bool b_side, int blk, int b_tile, int preround_bf16)
{
    // A side: every block size; B side: block 32 (a 128-element block along the strided axis would leave one
    // column per warp), no weight-side options
    return !b_side || (blk == 32 && !b_tile && !preround_bf16);
}

fmm_status_t fmm_launch_encode2_a(const EncodeParams& p, int blk, int mode, cudaStream_t st)
{
    const int64_t tasks = (int64_t)p.batch * p.rows * (p.cols / 128);
    int64_t blocks = (tasks + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 64;
    if (blocks > cap) blocks = cap;
    const unsigned g = (unsigned)blocks;
    if (mode == FMM_SCALE_FP32_AMAX_DIV_448) {
        if (blk == 32) launch_a2<32, FMM_SCALE_FP32_AMAX_DIV_448>(p, g, st);
        else launch_a2<128, FMM_SCALE_FP32_AMAX_DIV_448>(p, g, st);
    } else {
        launch_a2<32, FMM_SCALE_UE8M0_CEIL>(p, g, st);
    }
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_encode2_b(const EncodeParams& p, int mode, cudaStream_t st)
{
    dim3 grid((unsigned)(p.cols / 32), (unsigned)(p.rows / 32), (unsigned)p.batch);
    if (mode == FMM_SCALE_FP32_AMAX_DIV_448) launch_b2<FMM_SCALE_FP32_AMAX_DIV_448>(p, grid, st);
    else launch_b2<FMM_SCALE_UE8M0_CEIL>(p, grid, st);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}
