// The R^levels block-scaled fp8 sub-products and the fused post-addition (paper Sec. 2.1:
// c = sum_r <U_r,a><V_r,b> W_r; the products M_r = S_r^ * T_r^ of the quantized combinations are
// accumulated in fp32 and carried into the output blocks by the decoder W_r).
//
// One persistent CTA per SM owns an output tile POSITION (the same 128 x BN tile in every output
// block of C) and walks all terms for it, so the W-weighted accumulation into C is race-free and
// deterministic without atomics between CTAs.
//
//   warp 0      TMA producer: K-major e4m3 tiles of S_r and T_r (128-byte swizzle) + their scales
//   warp 1      tcgen05.mma issuer, fp32 accumulators in TMEM
//   warps 2..9  epilogue: TMEM -> registers -> (x W[r][q]) -> swizzled smem -> TMA store / TMA
//               add-reduce into the C blocks (the read-modify-write happens in L2, not in the SM)
//
// Scale handling:
//   UE8M0 mode  kind::mxf8f6f4.block_scale: the power-of-two block scales are copied to TMEM with
//               tcgen05.cp and applied by the tensor core; one accumulation over the whole K.
//   FP32 mode   (the paper's scale = amax/448 in fp32 on BOTH sides, per 1 x blk block): no
//               tensor-core path can apply a per-row x per-column fp32 factor per K block, so
//               each K block's partial product is accumulated on its own in TMEM
//               (kind::f8f6f4) and promoted on the CUDA cores: acc += P * (sA[row] * sB[col]).
//
// Every wait is bounded: on time-out a status word is set and all roles leave the kernel.
#include <stdio.h>
#include "fmm_internal.h"

namespace {

constexpr int BM = 128;
constexpr int BK = 128;                 // K elements (= bytes) per pipeline stage: one swizzle row
constexpr int EPI_WARPS = 8;
constexpr int NUM_THREADS = (2 + EPI_WARPS) * 32;
constexpr int STAGING_BYTES = 32 * 128; // 32 rows x 32 fp32 per epilogue warp and buffer
constexpr int STAGING_BUFS = 2;

template <int BN, int MODE, int BLK>
struct Cfg {
    static constexpr bool MX = (MODE == FMM_SCALE_UE8M0_CEIL);
    static constexpr int STAGES = (BN == 256) ? 3 : 4;
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int SF_STAGE_BYTES = MX ? (512 + (BN / 128) * 512) : 0;
    static constexpr int KB_PER_STAGE = BK / BLK;
    static constexpr int SB_STAGES = STAGES + 1;
    static constexpr int SB_STAGE_BYTES = MX ? 0 : KB_PER_STAGE * BN * 4;
    static constexpr int TX_BYTES = A_BYTES + B_BYTES + SF_STAGE_BYTES;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + STAGES * A_BYTES;
    static constexpr int OFF_STG = OFF_B + STAGES * B_BYTES;
    static constexpr int OFF_SF = OFF_STG + EPI_WARPS * STAGING_BUFS * STAGING_BYTES;
    static constexpr int OFF_SB = OFF_SF + STAGES * SF_STAGE_BYTES;
    static constexpr int OFF_BAR = OFF_SB + SB_STAGES * SB_STAGE_BYTES;
    static constexpr int NUM_BARS = 2 * STAGES + 2 * SB_STAGES + 8;
    static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16 + 1024;   // + alignment slack
    // TMEM: MX: one BN-column accumulator, then per stage 4 SFA + 4*(BN/128) SFB columns.
    //       FP32: ring of 512/BN accumulators, one per K block in flight.
    static constexpr int ACC_BUFS = MX ? 1 : (512 / BN);
    static constexpr int SF_COLS = 4 + 4 * (BN / 128);
    static constexpr int CW = BN / 2;      // columns per epilogue warp
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(!MX || BN + STAGES * SF_COLS <= 512, "TMEM budget");
};

// ------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{ asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count)); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{ asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{ asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer()
{ uint64_t t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* tm, int x, int y, uint32_t src)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{ asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void tc_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc)
{ asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory"); }
__device__ __forceinline__ void mma_f8f6f4(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_mxf8(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate,
                                         uint32_t tsfa, uint32_t tsfb)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Scale-factor chunk for tcgen05.cp 32x128b: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t make_sf_desc(uint32_t saddr)
{
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(128 >> 4) << 32) | ((uint64_t)1 << 46);
}

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s: far beyond any legitimate wait

struct Ctl {
    volatile int* abort_flag;   // shared memory
    int* status;                // global status words
};

// Bounded mbarrier wait.  Returns false after WAIT_LIMIT_NS or when another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Ctl& ctl, int where)
{
    uint32_t spins = 0;
    uint64_t t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*ctl.abort_flag) return false;
            const uint64_t now = global_timer();
            if (t0 == 0) t0 = now;
            else if (now - t0 > WAIT_LIMIT_NS) {
                *ctl.abort_flag = 1;
                atomicCAS(ctl.status, 0, where);
                return false;
            }
        }
    }
    return true;
}

// Same, with a warp-uniform verdict (the epilogue warps execute .sync.aligned instructions afterwards).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const Ctl& ctl, int where)
{
    const bool ok = mbar_wait(bar, parity, ctl, where);
    return __all_sync(0xffffffffu, ok);
}

struct KParams {
    const uint8_t* sa; const uint8_t* sb;   // scale arrays (bytes)
    long long sa_term, sb_term;
    int m, n, k, terms;
    const int* out_start; const FmmOutEntry* out;
    int* status;
};

template <int BN, int MODE, int BLK>
__global__ void __launch_bounds__(NUM_THREADS, 1)
fmm_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmC, const KParams p)
{
    using C = Cfg<BN, MODE, BLK>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw_addr);

    const uint32_t bar0 = base + C::OFF_BAR;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
    auto bar_sfull = [&](int s) { return bar0 + 8u * (2 * C::STAGES + s); };
    auto bar_sempty = [&](int s) { return bar0 + 8u * (2 * C::STAGES + C::SB_STAGES + s); };
    auto bar_tfull = [&](int b) { return bar0 + 8u * (2 * C::STAGES + 2 * C::SB_STAGES + b); };
    auto bar_tempty = [&](int b) { return bar0 + 8u * (2 * C::STAGES + 2 * C::SB_STAGES + 4 + b); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + C::OFF_BAR + C::NUM_BARS * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const Ctl ctl{abort_flag, p.status};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int s = 0; s < C::SB_STAGES; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sempty(s), EPI_WARPS); }
        for (int b = 0; b < 4; ++b) { mbar_init(bar_tfull(b), 1); mbar_init(bar_tempty(b), EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_n = p.n / BN;
    const int positions = (p.m / BM) * tiles_n;
    const int kstages = p.k / BK;
    const int nkb = p.k / BLK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            int ss = 0; uint32_t sphase = 0;
            bool ok = true;
            for (int pos = blockIdx.x; pos < positions && ok; pos += gridDim.x) {
                const int tm = pos / tiles_n, tn = pos % tiles_n;
                for (int t = 0; t < p.terms && ok; ++t) {
                    for (int ks = 0; ks < kstages; ++ks) {
                        if (!mbar_wait(bar_empty(stage), phase ^ 1u, ctl, 101)) { ok = false; break; }
                        mbar_expect_tx(bar_full(stage), C::TX_BYTES);
                        tma_load_2d(base + C::OFF_A + stage * C::A_BYTES, &tmA, ks * BK, t * p.m + tm * BM, bar_full(stage));
                        tma_load_2d(base + C::OFF_B + stage * C::B_BYTES, &tmB, ks * BK, t * p.n + tn * BN, bar_full(stage));
                        if (C::MX) {
                            const uint32_t sf = base + C::OFF_SF + stage * C::SF_STAGE_BYTES;
                            const uint8_t* ga = p.sa + (long long)t * p.sa_term + ((long long)tm * (nkb >> 2) + ks) * 512;
                            bulk_load(sf, ga, 512, bar_full(stage));
#pragma unroll
                            for (int h = 0; h < BN / 128; ++h) {
                                const uint8_t* gb = p.sb + (long long)t * p.sb_term +
                                                    ((long long)(tn * (BN / 128) + h) * (nkb >> 2) + ks) * 512;
                                bulk_load(sf + 512 + h * 512, gb, 512, bar_full(stage));
                            }
                        } else {
                            if (!mbar_wait(bar_sempty(ss), sphase ^ 1u, ctl, 102)) { ok = false; break; }
                            mbar_expect_tx(bar_sfull(ss), C::SB_STAGE_BYTES);
#pragma unroll
                            for (int g = 0; g < C::KB_PER_STAGE; ++g) {
                                const uint8_t* gb = p.sb + (long long)t * p.sb_term +
                                                    ((long long)(ks * C::KB_PER_STAGE + g) * p.n + tn * BN) * 4;
                                bulk_load(base + C::OFF_SB + ss * C::SB_STAGE_BYTES + g * BN * 4, gb, BN * 4, bar_sfull(ss));
                            }
                            if (++ss == C::SB_STAGES) { ss = 0; sphase ^= 1u; }
                        }
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            int buf = 0; uint32_t bphase = 0;
            bool ok = true;
            uint32_t idesc;
            if (C::MX) idesc = (1u << 23) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            else idesc = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            for (int pos = blockIdx.x; pos < positions && ok; pos += gridDim.x) {
                for (int t = 0; t < p.terms && ok; ++t) {
                    if (C::MX) {
                        if (!mbar_wait(bar_tempty(0), bphase ^ 1u, ctl, 201)) { ok = false; break; }
                        tc_fence_after();
                    }
                    for (int ks = 0; ks < kstages; ++ks) {
                        if (!mbar_wait(bar_full(stage), phase, ctl, 202)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t adesc = make_kmajor_sw128_desc(base + C::OFF_A + stage * C::A_BYTES);
                        const uint64_t bdesc = make_kmajor_sw128_desc(base + C::OFF_B + stage * C::B_BYTES);
                        if (C::MX) {
                            const uint32_t sf = base + C::OFF_SF + stage * C::SF_STAGE_BYTES;
                            const uint32_t tsfa = tmem_base + BN + stage * C::SF_COLS;
                            const uint32_t tsfb = tsfa + 4;
                            tc_cp_32x128b_warpx4(tsfa, make_sf_desc(sf));
#pragma unroll
                            for (int h = 0; h < BN / 128; ++h) tc_cp_32x128b_warpx4(tsfb + 4 * h, make_sf_desc(sf + 512 + h * 512));
#pragma unroll
                            for (int j = 0; j < BK / 32; ++j) {
                                const uint32_t id = idesc | ((uint32_t)j << 29) | ((uint32_t)j << 4);
                                mma_mxf8(tmem_base, adesc + 2 * j, bdesc + 2 * j, id, (ks > 0 || j > 0) ? 1u : 0u, tsfa, tsfb);
                            }
                        } else {
#pragma unroll
                            for (int g = 0; g < C::KB_PER_STAGE; ++g) {
                                if (!mbar_wait(bar_tempty(buf), bphase ^ 1u, ctl, 203)) { ok = false; break; }
                                tc_fence_after();
#pragma unroll
                                for (int j = 0; j < BLK / 32; ++j) {
                                    const int jj = g * (BLK / 32) + j;
                                    mma_f8f6f4(tmem_base + buf * BN, adesc + 2 * jj, bdesc + 2 * jj, idesc, j > 0 ? 1u : 0u);
                                }
                                tc_commit(bar_tfull(buf));
                                if (++buf == C::ACC_BUFS) { buf = 0; bphase ^= 1u; }
                            }
                            if (!ok) break;
                        }
                        tc_commit(bar_empty(stage));
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (C::MX && ok) { tc_commit(bar_tfull(0)); bphase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int e = warp - 2;
        const int q = warp & 3;            // TMEM lane quadrant this warp may access
        const int h = e >> 2;              // column half
        const uint32_t stg = base + C::OFF_STG + e * STAGING_BUFS * STAGING_BYTES;
        uint8_t* stg_ptr = base_ptr + C::OFF_STG + e * STAGING_BUFS * STAGING_BYTES;
        const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + h * C::CW;
        int buf = 0; uint32_t bphase = 0;
        int ss = 0; uint32_t sphase = 0;
        uint32_t store_cnt = 0;
        bool ok = true;
        float acc[C::CW];
        for (int pos = blockIdx.x; pos < positions && ok; pos += gridDim.x) {
            const int tm = pos / tiles_n, tn = pos % tiles_n;
            for (int t = 0; t < p.terms && ok; ++t) {
                if (C::MX) {
                    if (!mbar_wait_warp(bar_tfull(0), bphase, ctl, 301)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < C::CW / 32; ++c) tmem_ld32(lane_taddr + c * 32, &acc[c * 32]);
                    tmem_ld_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty(0));
                    bphase ^= 1u;
                } else {
#pragma unroll
                    for (int i = 0; i < C::CW; ++i) acc[i] = 0.0f;
                    const float* sa_row = reinterpret_cast<const float*>(p.sa + (long long)t * p.sa_term) +
                                          (long long)(tm * BM + q * 32 + lane) * nkb;
                    for (int ks = 0; ks < kstages && ok; ++ks) {
                        if (!mbar_wait_warp(bar_sfull(ss), sphase, ctl, 302)) { ok = false; break; }
                        float sa[C::KB_PER_STAGE];
#pragma unroll
                        for (int g = 0; g < C::KB_PER_STAGE; ++g) sa[g] = __ldg(sa_row + ks * C::KB_PER_STAGE + g);
                        const float* sbs = reinterpret_cast<const float*>(base_ptr + C::OFF_SB + ss * C::SB_STAGE_BYTES);
#pragma unroll
                        for (int g = 0; g < C::KB_PER_STAGE; ++g) {
                            if (!mbar_wait_warp(bar_tfull(buf), bphase, ctl, 303)) { ok = false; break; }
                            tc_fence_after();
                            const float* sbg = sbs + g * BN + h * C::CW;
#pragma unroll
                            for (int c = 0; c < C::CW / 32; ++c) {
                                float tmp[32];
                                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN + h * C::CW + c * 32, tmp);
                                tmem_ld_wait();
#pragma unroll
                                for (int i = 0; i < 32; i += 4) {
                                    const float4 s4 = *reinterpret_cast<const float4*>(sbg + c * 32 + i);
                                    acc[c * 32 + i + 0] = fmaf(tmp[i + 0], sa[g] * s4.x, acc[c * 32 + i + 0]);
                                    acc[c * 32 + i + 1] = fmaf(tmp[i + 1], sa[g] * s4.y, acc[c * 32 + i + 1]);
                                    acc[c * 32 + i + 2] = fmaf(tmp[i + 2], sa[g] * s4.z, acc[c * 32 + i + 2]);
                                    acc[c * 32 + i + 3] = fmaf(tmp[i + 3], sa[g] * s4.w, acc[c * 32 + i + 3]);
                                }
                            }
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_tempty(buf));
                            if (++buf == C::ACC_BUFS) { buf = 0; bphase ^= 1u; }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_sempty(ss));
                        if (++ss == C::SB_STAGES) { ss = 0; sphase ^= 1u; }
                    }
                    if (!ok) break;
                }
                // ---- post-addition: W-weighted scatter of this product into its C blocks
                const int o0 = p.out_start[t], o1 = p.out_start[t + 1];
                if (lane == 0) bulk_wait<0>();     // the previous term's writes to these tiles have landed
                __syncwarp();
                for (int o = o0; o < o1; ++o) {
                    const FmmOutEntry ent = p.out[o];
                    const int row0 = ent.row_off * p.m + tm * BM + q * 32;
                    const int col0 = ent.col_off * p.n + tn * BN + h * C::CW;
#pragma unroll
                    for (int c = 0; c < C::CW / 32; ++c) {
                        const uint32_t b = store_cnt & (STAGING_BUFS - 1);
                        if (lane == 0) bulk_wait_read<STAGING_BUFS - 1>();
                        __syncwarp();
                        uint8_t* dst = stg_ptr + b * STAGING_BYTES + lane * 128;
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            float4 v;
                            v.x = acc[c * 32 + i4 * 4 + 0] * ent.w; v.y = acc[c * 32 + i4 * 4 + 1] * ent.w;
                            v.z = acc[c * 32 + i4 * 4 + 2] * ent.w; v.w = acc[c * 32 + i4 * 4 + 3] * ent.w;
                            *reinterpret_cast<float4*>(dst + ((i4 ^ (lane & 7)) << 4)) = v;
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            if (ent.first) tma_store_2d(&tmC, col0 + c * 32, row0, stg + b * STAGING_BYTES);
                            else tma_reduce_add_2d(&tmC, col0 + c * 32, row0, stg + b * STAGING_BYTES);
                            bulk_commit();
                        }
                        ++store_cnt;
                    }
                }
            }
        }
        if (lane == 0) bulk_wait<0>();
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {
        // let copies that are still in flight towards this CTA's shared memory land
        const uint64_t t0 = global_timer();
        while (global_timer() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

// --------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

bool make_map_2d(CUtensorMap* tm, CUtensorMapDataType dt, int elt_bytes, const void* ptr, uint64_t inner, uint64_t outer,
                 uint32_t box_inner, uint32_t box_outer)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * (uint64_t)elt_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int MODE, int BLK>
fmm_status_t launch(const GemmParams& g, cudaStream_t st)
{
    using C = Cfg<BN, MODE, BLK>;
    CUtensorMap tmA, tmB, tmC;
    if (!make_map_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, g.qa, (uint64_t)g.k, (uint64_t)g.terms * g.m, BK, BM)) return FMM_ERR_CUDA;
    if (!make_map_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, g.qb, (uint64_t)g.k, (uint64_t)g.terms * g.n, BK, BN)) return FMM_ERR_CUDA;
    if (!make_map_2d(&tmC, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, g.C, (uint64_t)g.Nfull, (uint64_t)g.Mfull, 32, 32)) return FMM_ERR_CUDA;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(fmm_gemm_kernel<BN, MODE, BLK>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return FMM_ERR_CUDA;
        }
        attr_set = true;
    }
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int positions = (g.m / BM) * (g.n / BN);
    const int grid = positions < sms ? positions : sms;
    KParams kp;
    kp.sa = static_cast<const uint8_t*>(g.sa); kp.sb = static_cast<const uint8_t*>(g.sb);
    kp.sa_term = g.sa_term; kp.sb_term = g.sb_term;
    kp.m = g.m; kp.n = g.n; kp.k = g.k; kp.terms = g.terms;
    kp.out_start = g.out_start; kp.out = g.out; kp.status = g.status;
    fmm_gemm_kernel<BN, MODE, BLK><<<grid, NUM_THREADS, C::SMEM_BYTES, st>>>(tmA, tmB, tmC, kp);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

}  // namespace

fmm_status_t fmm_launch_gemm(const GemmParams& g, int blk, int mode, cudaStream_t st, int* launches)
{
    const bool wide = (g.n % 256) == 0;
    fmm_status_t s;
    if (mode == FMM_SCALE_UE8M0_CEIL) {
        s = wide ? launch<256, FMM_SCALE_UE8M0_CEIL, 32>(g, st) : launch<128, FMM_SCALE_UE8M0_CEIL, 32>(g, st);
    } else if (blk == 32) {
        s = wide ? launch<256, FMM_SCALE_FP32_AMAX_DIV_448, 32>(g, st) : launch<128, FMM_SCALE_FP32_AMAX_DIV_448, 32>(g, st);
    } else {
        s = wide ? launch<256, FMM_SCALE_FP32_AMAX_DIV_448, 128>(g, st) : launch<128, FMM_SCALE_FP32_AMAX_DIV_448, 128>(g, st);
    }
    if (s == FMM_OK && launches) *launches += 1;
    return s;
}
