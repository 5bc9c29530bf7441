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
#include "fmm_internal.h"

namespace {

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
// coalesced read per quadrant.  A block of BLK elements is held by BLK/4 adjacent lanes, so the
// amax is a short butterfly.  Codes leave as one 128-byte store per warp and combination.
template <int BLK, int MODE>
__global__ void __launch_bounds__(256) encode_a_kernel(const EncodeParams p)
{
    constexpr int GROUP = BLK / 4;                 // lanes per block
    const int lane = threadIdx.x & 31;
    const int64_t warp_gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int chunks = p.cols / 128;
    const int nkb = p.cols / BLK;
    const int64_t units = (int64_t)p.batch * p.rows * chunks;
    const int64_t qoff[4] = {0, (int64_t)p.cols, (int64_t)p.rows * p.ld, (int64_t)p.rows * p.ld + p.cols};
    const int64_t term_codes = (int64_t)p.rows * p.cols;

    for (int64_t u = warp_gid; u < units; u += nwarps) {
        const int c = (int)(u % chunks);
        const int64_t bi = u / chunks;
        const int i = (int)(bi % p.rows);
        const int b = (int)(bi / p.rows);
        const float* base = p.in + (int64_t)b * p.in_batch_stride + (int64_t)i * p.ld + c * 128 + lane * 4;
        float4 x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < p.nq) x[j] = __ldcs(reinterpret_cast<const float4*>(base + qoff[j]));

        for (int r = 0; r < p.R; ++r) {
            float v0 = 0.f, v1 = 0.f, v2 = 0.f, v3 = 0.f;
            bool set = false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float cj = p.coef[r][j];
                if (cj != 0.0f) {
                    if (!set) {
                        v0 = __fmul_rn(cj, x[j].x); v1 = __fmul_rn(cj, x[j].y);
                        v2 = __fmul_rn(cj, x[j].z); v3 = __fmul_rn(cj, x[j].w);
                        set = true;
                    } else {
                        v0 = __fmaf_rn(cj, x[j].x, v0); v1 = __fmaf_rn(cj, x[j].y, v1);
                        v2 = __fmaf_rn(cj, x[j].z, v2); v3 = __fmaf_rn(cj, x[j].w, v3);
                    }
                }
            }
            float amax = fmaxf(fmaxf(fabsf(v0), fabsf(v1)), fmaxf(fabsf(v2), fabsf(v3)));
#pragma unroll
            for (int o = 1; o < GROUP; o <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            float s; uint32_t e8;
            const float inv = block_scale<MODE>(amax, p.amax_floor, s, e8);
            const uint32_t packed = pack4_e4m3(__fmul_rn(v0, inv), __fmul_rn(v1, inv),
                                               __fmul_rn(v2, inv), __fmul_rn(v3, inv));
            const int64_t t = (int64_t)b * p.R + r;
            *reinterpret_cast<uint32_t*>(p.q_out + t * term_codes + (int64_t)i * p.cols + c * 128 + lane * 4) = packed;
            if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
                if ((lane % GROUP) == 0) {
                    float* so = reinterpret_cast<float*>(reinterpret_cast<char*>(p.s_out) + t * p.s_term_stride);
                    so[(int64_t)i * nkb + c * (128 / BLK) + lane / GROUP] = s;
                }
            } else {
                // four exponent bytes of this row (blocks 4c .. 4c+3) form one aligned word of the scale tile
                uint32_t w = __shfl_sync(0xffffffffu, e8, 0) | (__shfl_sync(0xffffffffu, e8, 8) << 8) |
                             (__shfl_sync(0xffffffffu, e8, 16) << 16) | (__shfl_sync(0xffffffffu, e8, 24) << 24);
                if (lane == 0) {
                    char* so = reinterpret_cast<char*>(p.s_out) + t * p.s_term_stride;
                    const int64_t tile = (int64_t)(i >> 7) * (nkb >> 2) + c;
                    *reinterpret_cast<uint32_t*>(so + tile * 512 + (i & 31) * 16 + ((i & 127) >> 5) * 4) = w;
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// B side.  Blocks run along k, the strided axis of row-major B, and the output is K-major (the
// tensor-core operand layout).  One thread owns one column n: each of its loads is part of a
// 128-byte coalesced warp read of a B row; the amax is thread-local; the 32 codes of a block
// leave as 32 contiguous bytes.  BLK == 128 takes a second pass over the four 32-element
// sub-blocks (served by L1/L2) because the whole block does not fit in registers.
template <int MODE>
__device__ __forceinline__ void store_b_scale(const EncodeParams& p, int64_t t, int j, int kb, int nkb,
                                              float s, uint32_t e8word, bool last_of_word)
{
    char* so = reinterpret_cast<char*>(p.s_out) + t * p.s_term_stride;
    if (MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
        reinterpret_cast<float*>(so)[(int64_t)kb * p.cols + j] = s;
    } else if (last_of_word) {
        const int64_t tile = (int64_t)(j >> 7) * (nkb >> 2) + (kb >> 2);
        *reinterpret_cast<uint32_t*>(so + tile * 512 + (j & 31) * 16 + ((j & 127) >> 5) * 4) = e8word;
    }
}

template <int BLK, int MODE>
__global__ void __launch_bounds__(128) encode_b_kernel(const EncodeParams p)
{
    // here p.rows = leaf k (contracted), p.cols = leaf n
    const int j = blockIdx.x * 128 + threadIdx.x;
    const int kc = blockIdx.y;                      // chunk of 128 k
    const int b = blockIdx.z;
    const int nkb = p.rows / BLK;
    const int64_t qoff[4] = {0, (int64_t)p.cols, (int64_t)p.rows * p.ld, (int64_t)p.rows * p.ld + p.cols};
    const float* base = p.in + (int64_t)b * p.in_batch_stride + j;
    const int64_t term_codes = (int64_t)p.rows * p.cols;

    float raw[4][32];
    float blk_amax[FMM_MAX_RANK];
    float blk_inv[FMM_MAX_RANK];
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) { blk_amax[r] = 0.0f; blk_inv[r] = 0.0f; }
    uint32_t e8word[FMM_MAX_RANK];
#pragma unroll
    for (int r = 0; r < FMM_MAX_RANK; ++r) e8word[r] = 0;

    constexpr int PASSES = (BLK == 32) ? 1 : 2;
#pragma unroll 1
    for (int pass = 0; pass < PASSES; ++pass) {
#pragma unroll 1
        for (int sub = 0; sub < 4; ++sub) {
            const int k0 = kc * 128 + sub * 32;
#pragma unroll
            for (int jq = 0; jq < 4; ++jq)
                if (jq < p.nq) {
#pragma unroll
                    for (int kk = 0; kk < 32; ++kk)
                        raw[jq][kk] = __ldg(base + qoff[jq] + (int64_t)(k0 + kk) * p.ld);
                }
#pragma unroll
            for (int r = 0; r < FMM_MAX_RANK; ++r) {
                if (r < p.R) {
                    float v[32];
                    bool set = false;
#pragma unroll
                    for (int jq = 0; jq < 4; ++jq) {
                        const float cj = p.coef[r][jq];
                        if (cj != 0.0f) {
                            if (!set) {
#pragma unroll
                                for (int kk = 0; kk < 32; ++kk) v[kk] = __fmul_rn(cj, raw[jq][kk]);
                                set = true;
                            } else {
#pragma unroll
                                for (int kk = 0; kk < 32; ++kk) v[kk] = __fmaf_rn(cj, raw[jq][kk], v[kk]);
                            }
                        }
                    }
                    if (!set) {
#pragma unroll
                        for (int kk = 0; kk < 32; ++kk) v[kk] = 0.0f;
                    }
                    const int64_t t = (int64_t)b * p.R + r;
                    if (BLK == 32 || pass == 0) {
                        float amax = 0.0f;
#pragma unroll
                        for (int kk = 0; kk < 32; ++kk) amax = fmaxf(amax, fabsf(v[kk]));
                        if (BLK == 32) blk_amax[r] = amax; else blk_amax[r] = fmaxf(blk_amax[r], amax);
                    }
                    if (BLK == 32 || (pass == 0 && sub == 3)) {
                        float s; uint32_t e8;
                        blk_inv[r] = block_scale<MODE>(blk_amax[r], p.amax_floor, s, e8);
                        const int kb = (BLK == 32) ? (kc * 4 + sub) : kc;
                        e8word[r] |= e8 << (8 * (kb & 3));
                        store_b_scale<MODE>(p, t, j, kb, nkb, s, e8word[r], (kb & 3) == 3);
                    }
                    if (BLK == 32 || pass == 1) {
                        const float inv = blk_inv[r];
                        uint32_t w[8];
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            w[g] = pack4_e4m3(__fmul_rn(v[4 * g], inv), __fmul_rn(v[4 * g + 1], inv),
                                              __fmul_rn(v[4 * g + 2], inv), __fmul_rn(v[4 * g + 3], inv));
                        uint4* dst = reinterpret_cast<uint4*>(p.q_out + t * term_codes + (int64_t)j * p.rows + k0);
                        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                    }
                }
            }
        }
    }
}

// fp32 combinations of the outer recursion levels (levels >= 2): out[b*R + r] = sum_j coef[r][j] X_j
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
            *reinterpret_cast<float4*>(o) = v;
        }
    }
}

int sm_count()
{
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

}  // namespace

fmm_status_t fmm_launch_comb(const CombParams& p, cudaStream_t st)
{
    const int64_t units = (int64_t)p.batch * p.rows * (p.cols / 4);
    int64_t blocks = (units + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    comb_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_encode_a(const EncodeParams& p, int blk, int mode, cudaStream_t st)
{
    const int64_t units = (int64_t)p.batch * p.rows * (p.cols / 128);
    int64_t blocks = (units + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    const unsigned g = (unsigned)blocks;
    if (mode == FMM_SCALE_FP32_AMAX_DIV_448) {
        if (blk == 32) encode_a_kernel<32, FMM_SCALE_FP32_AMAX_DIV_448><<<g, 256, 0, st>>>(p);
        else encode_a_kernel<128, FMM_SCALE_FP32_AMAX_DIV_448><<<g, 256, 0, st>>>(p);
    } else {
        encode_a_kernel<32, FMM_SCALE_UE8M0_CEIL><<<g, 256, 0, st>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_encode_b(const EncodeParams& p, int blk, int mode, cudaStream_t st)
{
    dim3 grid((unsigned)(p.cols / 128), (unsigned)(p.rows / 128), (unsigned)p.batch);
    if (mode == FMM_SCALE_FP32_AMAX_DIV_448) {
        if (blk == 32) encode_b_kernel<32, FMM_SCALE_FP32_AMAX_DIV_448><<<grid, 128, 0, st>>>(p);
        else encode_b_kernel<128, FMM_SCALE_FP32_AMAX_DIV_448><<<grid, 128, 0, st>>>(p);
    } else {
        encode_b_kernel<32, FMM_SCALE_UE8M0_CEIL><<<grid, 128, 0, st>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}
