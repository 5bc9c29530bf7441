// The R^levels block-scaled fp8 sub-products and the fused post-addition (paper Sec. 2.1:
// c = sum_r <U_r,a><V_r,b> W_r; the products M_r = S_r^ * T_r^ of the quantized combinations are
// accumulated in fp32 and carried into the output blocks by the decoder W_r).
//
// A persistent CTA (NCTA == 1) or CTA pair on two adjacent SMs (NCTA == 2, tcgen05 cta_group::2)
// owns an output tile POSITION - the same (NCTA*128) x BN tile in every output block of C - and
// walks all terms for it, so the W-weighted accumulation into C is race-free and deterministic.
//
//   warp 0      TMA producer: K-major e4m3 tiles of S_r and T_r (128-byte swizzle) + their scales.
//               In a pair each CTA loads its own 128 rows of S_r and its own half of the T_r tile.
//   warp 1      tcgen05.mma issuer (the even CTA of a pair issues for both), fp32 accumulators in TMEM
//   warps 4..11 epilogue (two warpgroups, given most of the register file with setmaxnreg): TMEM -> registers -> (x W[r][q]) -> swizzled smem -> TMA store / TMA
//               add-reduce into the C blocks (the read-modify-write happens in L2, not in the SM)
//
// Scale handling:
//   UE8M0 mode  kind::mxf8f6f4.block_scale: the power-of-two block scales are copied to TMEM with
//               tcgen05.cp and applied by the tensor core; one accumulation over the whole K.
//   FP32 mode   (the paper's scale = amax/448 in fp32 on BOTH sides, per 1 x blk block): no
//               tensor-core path can apply a per-row x per-column fp32 factor per K block, so
//               each K block's partial product is accumulated on its own in TMEM
//               (kind::f8f6f4) and promoted on the CUDA cores: acc += P * (sA[row] * sB[col]),
//               two columns per instruction (fp32x2), overlapped with the next TMEM load.
//
// Every wait is bounded: on time-out a status word is set and all roles leave the kernel.
#include <string.h>
#include <atomic>
#include "fmm_internal.h"
#include "fmm_ptx.cuh"

namespace {
using namespace fmmptx;

// Internal third mode of the product kernel: FP32 scales whose B-side value is constant over each
// 128-column tile (the 128 x 128 weight tiles of App. E.5).  The promotion then needs one multiply per row
// and K block (s = sA * sB_tile) and one FMA per element, instead of a multiply and an FMA per element.
constexpr int MODE_FP32_SB_TILE = 2;
// Internal fourth mode: FP32 scales (per column, as mode 0) with a dedicated output warp.  The promoting warps hand
// a finished product to it through a shared-memory copy of the (unweighted) accumulators and go straight on with
// the next term; the W-weighted stores / add-reductions then overlap the next term's promotion instead of stalling
// it.  The output warp needs a fixed time per term, so this pays only when a term has many K stages (measured
// cross-over near 16 stages of 128 k); the dispatcher picks the mode per launch.
constexpr int MODE_FP32_OUT_WARP = 3;

constexpr int BM = 128;                 // rows per CTA
constexpr int BK = 128;                 // K elements (= bytes) per pipeline stage: one swizzle row
constexpr int EPI_WARPS = 8;               // two per TMEM lane quadrant, each half of the tile's columns
constexpr int EPI_WARP0 = 4;               // warps 0..3: operand producer, MMA issuer, scale producer (FP32 modes), idle
constexpr int NUM_THREADS = (EPI_WARP0 + EPI_WARPS) * 32;
// setmaxnreg budget: the CTA's register pool is NUM_THREADS x (registers at launch); an increase
// beyond what the decrease freed would block forever, so every split is checked (see Cfg).
constexpr int REGS_AT_LAUNCH = 168;
static_assert(NUM_THREADS * (REGS_AT_LAUNCH + 8) > 65536, "REGS_AT_LAUNCH must be the launch-bound maximum");

template <int BN, int MODE, int BLK, int NCTA>
struct Cfg {
    static constexpr bool MX = (MODE == FMM_SCALE_UE8M0_CEIL);
    // Register split between the four control warps and the eight epilogue warps.  The FP32-scale kernels give the
    // promoting warps all they can (accumulators + a TMEM chunk + scales); the UE8M0 kernel's epilogue needs less and
    // its producer and issuer, which also handle the scale tiles, spilled at 56.
    static constexpr int REGS_CTRL = (MX || MODE == MODE_FP32_OUT_WARP) ? 72 : 56, REGS_EPI = (MX || MODE == MODE_FP32_OUT_WARP) ? 208 : 224;
    static_assert(EPI_WARP0 * 32 * REGS_CTRL + EPI_WARPS * 32 * REGS_EPI <= NUM_THREADS * REGS_AT_LAUNCH, "register pool");
    static constexpr int BROWS = BN / NCTA;                  // T_r rows this CTA loads per stage
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BROWS * BK;
    // The UE8M0 pair kernel keeps one staging chunk per epilogue warp: its shared memory goes to the operand stages,
    // and a second chunk in flight per warp was measured slower (more output traffic competing with the loads).
    static constexpr int STAGING_BUFS = (MX && NCTA == 2) ? 1 : 2;
    static constexpr bool DUMP = (MODE == MODE_FP32_OUT_WARP);
    // FP32 scales per column: the promoting warps read the accumulators with the 16-lane load shape, four rows x
    // CW/4 columns per thread (see the promotion loop).  The weight-tile mode has no per-column scale loads to
    // save and is faster with one row per thread.
    static constexpr bool ROWS4 = !MX && MODE != MODE_FP32_SB_TILE;
    static_assert(!DUMP || (BN == 128 && BK / BLK == 4), "output-warp mode: 128-column tiles, block 32");
    static constexpr int STAGES = (MX && NCTA == 2) ? 5 : ((A_BYTES + B_BYTES) > 40000 || DUMP ? 3 : 4);
    // DUMP (output-warp mode): shared-memory copy of a finished product, BM x BN fp32
    static constexpr int DUMP_BYTES = DUMP ? BM * BN * 4 : 0;
    // output chunk of one epilogue warp: 32 rows x CH fp32, staged in shared memory for one TMA store.  Rows of 128
    // bytes everywhere: a TMA add-reduction of 64-byte rows runs at half the bytes per clock (11 against 21 per SM,
    // measured; plain stores 25 either way), which costs the UE8M0 pair kernel more than its sixth operand stage,
    // bought with 16-column chunks, gave (two levels at n = 8192: 0.579 -> 0.556 ms; one level 0.451 -> 0.447 ms).
    static constexpr int CH = 32;
    static constexpr int STAGING_BYTES = 32 * CH * 4;
    static constexpr int SFB_ATOMS = BN / 128;
    static constexpr int SF_STAGE_BYTES = MX ? (512 + SFB_ATOMS * 512) : 0;
    static constexpr int KB_PER_STAGE = BK / BLK;
    // depth of the scale ring: scales are small, so in the block-32 kernel with the output warp, which has the room,
    // they run several stages ahead of the operand tiles (2.5 % for the cubic product at n = 8192, neutral for rank 7)
    static constexpr int SB_STAGES = STAGES + (DUMP ? 5 : 1);
    // FP32 modes: one stage of the scale ring = the B-side scales of the stage's K blocks (KB x BN fp32, stored
    // K-block-major) followed by the A-side scales of this CTA's 128 rows (128 x KB fp32: the A side stores the KB
    // scales of a 128-k chunk next to each other per row, one contiguous piece per stage)
    static constexpr int SB_PART_BYTES = MX ? 0 : KB_PER_STAGE * BN * 4;
    static constexpr int SB_STAGE_BYTES = MX ? 0 : KB_PER_STAGE * (BN + BM) * 4;
    static constexpr int TX_BYTES = NCTA * (A_BYTES + B_BYTES + SF_STAGE_BYTES);
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + STAGES * A_BYTES;
    static constexpr int OFF_STG = OFF_B + STAGES * B_BYTES;
    static constexpr int OUT_BUFS = 8;          // DUMP: staging chunks of the output warp (TMA stores in flight)
    static constexpr int OFF_DUMP = OFF_STG + (DUMP ? OUT_BUFS * 4096 : EPI_WARPS * STAGING_BUFS * STAGING_BYTES);
    static constexpr int OFF_SF = OFF_DUMP + DUMP_BYTES;
    static constexpr int OFF_SB = OFF_SF + STAGES * SF_STAGE_BYTES;
    static constexpr int OFF_BAR = OFF_SB + SB_STAGES * SB_STAGE_BYTES;
    static constexpr int NUM_BARS = 2 * STAGES + 2 * SB_STAGES + 8 + 2;
    static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16 + 1024;   // + alignment slack
    // TMEM: MX: one BN-column accumulator, then per stage 4 SFA + 4*(BN/128) SFB columns.
    //       FP32: ring of 512/BN accumulators, one per K block in flight.
    // FP32: GPB consecutive K blocks ("granules") share one completion signal: their MMAs are issued back to
    // back into adjacent TMEM buffers and committed once, so the tensor pipe is not drained per K block.
    static constexpr int GPB = MX ? 1 : ((KB_PER_STAGE >= 2 && 512 / BN >= 4) ? 2 : 1);
    static constexpr int ACC_BUFS = MX ? 1 : (512 / BN) / GPB;        // ring of (GPB x BN)-column super-buffers
    static constexpr int SF_COLS = 4 + 4 * SFB_ATOMS;
    // UE8M0: TMEM columns [0, BN) accumulator, [BN, BN + SF_COLS) the scale factors of the stage being multiplied (one
    // slot: tcgen05.cp and tcgen05.mma execute in issue order), then the HOLD area of the pair-fused decoder: every
    // epilogue warp parks CW - 16 columns of a finished product there (the other 16 stay in registers) until the
    // product it is paired with is done.
    static constexpr int HOLD_T = MX ? (BN / 2 - 16) : 0;          // parked columns per warp
    static constexpr int OFF_HOLD = BN + 16;
    static constexpr int CW = BN / 2;      // columns per epilogue warp
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(!MX || (SF_COLS <= 16 && OFF_HOLD + 2 * HOLD_T <= 512), "TMEM budget");
    static_assert(!MX || HOLD_T == 112 || HOLD_T == 48, "hold area is parked with 32- and 16-column stores");
};

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s: far beyond any legitimate wait

struct Ctl {
    volatile int* abort_flag;   // shared memory
    int* status;                // global status words
    unsigned long long limit_ns = WAIT_LIMIT_NS;
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
            else if (now - t0 > ctl.limit_ns) {
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

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever signals; the wait must
// give up after limit_ns, record `where` in the status word and let the kernel end normally.
__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns, int where)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); abort_flag = 0; fence_barrier_init(); }
    __syncthreads();
    Ctl ctl{&abort_flag, status, limit_ns};
    const bool ok = mbar_wait_warp(smem_u32(&bar), 0, ctl, where);
    if (threadIdx.x == 0 && ok) atomicExch(status + 1, 1);      // must not happen: nothing arrives on the barrier
}

struct KParams {
    const uint8_t* sa; const uint8_t* sb;   // scale arrays (bytes); fp32 mode only
    long long sa_term, sb_term;
    int m, n, k, terms;
    // Work items.  A slot is (term group, tile position): the terms of one group (the R products of one parent
    // at the innermost level; all terms at one level) feed one set of output blocks and are walked by one CTA
    // (pair) in order.  (Cutting the slots of a short last wave into narrower items does not pay: a tcgen05.mma of
    // half the width takes as long to issue, measured 4 % slower at n = 8192.)
    int positions, terms_per_group, items;
    const int* out_start; const FmmOutEntry* out;
    const int* pair_start; const FmmPairEntry* pair;   // pair-fused decoder (UE8M0): steps of two products, see FmmPairEntry
    int order[FMM_MAX_RANK]; int steps; int R;         // walk order of the R products of a parent; steps = ceil(R / 2)
    int* status;
    const float* c_base; long long ldc;       // the output matrix as plain memory: used by the FMM_DEBUG store guard only
    FmmGuard guard;
};

template <int BN, int MODE, int BLK, int NCTA>
__global__ void __launch_bounds__(NUM_THREADS, 1)
fmm_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmSFA,
                const __grid_constant__ CUtensorMap tmSFB, const KParams p)
{
    using C = Cfg<BN, MODE, BLK, NCTA>;
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
    const uint32_t bar_dfull = bar0 + 8u * (2 * C::STAGES + 2 * C::SB_STAGES + 8);      // accumulator copy written
    const uint32_t bar_dempty = bar_dfull + 8u;                                           // ... and consumed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + C::OFF_BAR + C::NUM_BARS * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const Ctl ctl{abort_flag, p.status};

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta_rank = (NCTA == 2) ? (int)cluster_ctarank() : 0;
    const bool leader = (cta_rank == 0);
    const int unit = blockIdx.x / NCTA;            // CTA or CTA pair index
    const int units = gridDim.x / NCTA;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int s = 0; s < C::SB_STAGES; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_sempty(s), EPI_WARPS); }
        for (int b = 0; b < 4; ++b) { mbar_init(bar_tfull(b), 1); mbar_init(bar_tempty(b), NCTA * EPI_WARPS); }
        mbar_init(bar_dfull, EPI_WARPS); mbar_init(bar_dempty, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc<NCTA>(smem_u32(tmem_slot), 512);
        tmem_relinquish<NCTA>();
    }
    tc_fence_before();
    __syncthreads();
    if (NCTA == 2) cluster_sync();                 // the peer's barriers are initialised before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_n = p.n / BN;
    const int kstages = p.k / BK;
    const int nkb = p.k / BLK;
    // ti-th product a CTA (pair) walks in work-item group grp: the parents of the group one after the other, the R
    // products of a parent in the plan's walk order (identity unless the decoder is pair-fused)
    auto term_of = [&](int grp, int ti) {
        if constexpr (C::MX) return grp * p.terms_per_group + (ti / p.R) * p.R + p.order[ti % p.R];
        else return grp * p.terms_per_group + ti;
    };
    const int row_blocks_a = p.m / 128, row_blocks_b = p.n / 128;

    if (warp < EPI_WARP0) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::REGS_CTRL));
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // (all lanes walk the loops, one elected lane issues: see the note on warp-collective issue in fmm_ptx.cuh)
        {
            griddep_wait();        // the encoders' output is complete and visible (no-op unless launched to overlap them)
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int w = unit; w < p.items && ok; w += units) {
                const int slot = w;
                const int grp = slot / p.positions, pos = slot - grp * p.positions;
                const int tm = pos / tiles_n, tn = pos % tiles_n;
                const int row_blk = tm * NCTA + cta_rank;                 // 128-row block of S_r this CTA owns
                for (int ti = 0; ti < p.terms_per_group && ok; ++ti) {
                    const int t = term_of(grp, ti);
                    for (int ks = 0; ks < kstages; ++ks) {
                        if (!mbar_wait_warp(bar_empty(stage), phase ^ 1u, ctl, 101)) { ok = false; break; }
                        // completion is counted on the even CTA's barrier; only that CTA arms it
                        const uint32_t fb = (NCTA == 2) ? (bar_full(stage) & PEER_BIT_MASK) : bar_full(stage);
                        if (elect_one()) {
                            if (leader) mbar_expect_tx(bar_full(stage), C::TX_BYTES);
                            tma_load_2d<NCTA>(base + C::OFF_A + stage * C::A_BYTES, &tmA, ks * BK, t * p.m + row_blk * BM, fb);
                            tma_load_2d<NCTA>(base + C::OFF_B + stage * C::B_BYTES, &tmB, ks * BK,
                                              t * p.n + tn * BN + cta_rank * C::BROWS, fb);
                            if (C::MX) {
                                // scale tiles: 512-byte atoms, ordered [term][k quad][128-row block]
                                const uint32_t sf = base + C::OFF_SF + stage * C::SF_STAGE_BYTES;
                                tma_load_2d<NCTA>(sf, &tmSFA, 0, (t * (nkb >> 2) + ks) * row_blocks_a + row_blk, fb);
                                tma_load_2d<NCTA>(sf + 512, &tmSFB, 0, (t * (nkb >> 2) + ks) * row_blocks_b + tn * C::SFB_ATOMS, fb);
                            }
                        }
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ FP32 modes: producer of the B-side scales
        // (its own thread and ring: the operand producer above has no registers to spare, and the scale ring is
        // released by the promoting warps, not by the tensor pipe)
        if (!C::MX) {
            griddep_wait();        // as the operand producer
            int ss = 0; uint32_t sphase = 0;
            bool ok = true;
            for (int w = unit; w < p.items && ok; w += units) {
                const int slot = w;
                const int grp = slot / p.positions, pos = slot - grp * p.positions;
                const int tn = pos % tiles_n;
                const int t_end = (grp + 1) * p.terms_per_group;
                const int tm = pos / tiles_n;
                for (int t = t_end - p.terms_per_group; t < t_end && ok; ++t) {
                    const uint8_t* sb_t = p.sb + (long long)t * p.sb_term + (long long)tn * BN * 4;
                    const uint8_t* sa_t = p.sa + (long long)t * p.sa_term + (long long)(tm * NCTA + cta_rank) * BM * (C::KB_PER_STAGE * 4);
                    for (int ks = 0; ks < kstages; ++ks) {
                        if (!mbar_wait_warp(bar_sempty(ss), sphase ^ 1u, ctl, 102)) { ok = false; break; }
                        if (elect_one()) {
                            mbar_expect_tx(bar_sfull(ss), C::SB_STAGE_BYTES);
#pragma unroll
                            for (int g = 0; g < C::KB_PER_STAGE; ++g)
                                bulk_load(base + C::OFF_SB + ss * C::SB_STAGE_BYTES + g * BN * 4,
                                          sb_t + (long long)(ks * C::KB_PER_STAGE + g) * p.n * 4, BN * 4, bar_sfull(ss));
                            bulk_load(base + C::OFF_SB + ss * C::SB_STAGE_BYTES + C::SB_PART_BYTES,
                                      sa_t + (long long)ks * p.m * (C::KB_PER_STAGE * 4), BM * C::KB_PER_STAGE * 4, bar_sfull(ss));
                        }
                        if (++ss == C::SB_STAGES) { ss = 0; sphase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ FP32 modes, 128-column tiles: output warp
        if (C::DUMP) {
            const uint32_t stg = base + C::OFF_STG + lane * 128;          // this lane's row of a staging chunk
            const uint32_t dump = base + C::OFF_DUMP + lane * 128;        // ... and of a chunk of the accumulator copy
            uint32_t dphase = 0, store_cnt = 0;
            bool ok = true;
            for (int w = unit; w < p.items && ok; w += units) {
                const int slot = w;
                const int grp = slot / p.positions, pos = slot - grp * p.positions;
                const int tm = pos / tiles_n, tn = pos % tiles_n;
                const int t_end = (grp + 1) * p.terms_per_group;
                for (int t = t_end - p.terms_per_group; t < t_end && ok; ++t) {
                    if (!mbar_wait_warp(bar_dfull, dphase, ctl, 401)) { ok = false; break; }
                    dphase ^= 1u;
                    const int o0 = p.out_start[t], o1 = p.out_start[t + 1];
                    if (lane == 0) bulk_wait<0>();     // the previous term's writes to these tiles have landed
                    __syncwarp();
                    for (int o = o0; o < o1; ++o) {
                        const FmmOutEntry ent = p.out[o];
                        const int row0 = ent.row_off * p.m + (tm * NCTA + cta_rank) * BM;
                        const int col0 = ent.col_off * p.n + tn * BN;
                        // A weight of exactly 1 needs no copy: the promoting warps stored the chunks in the swizzled layout
                        // the tensor map expects (and made them visible to the TMA engine), so they go out as they are.
                        const bool direct = (ent.w == 1.0f);
#pragma unroll 1
                        for (int ch0 = 0; ch0 < (BM / 32) * (BN / 32); ch0 += C::OUT_BUFS / 2) {
                            // OUT_BUFS/2 chunks of 32 rows x 32 columns per round (one proxy fence and one bulk group per
                            // round, two rounds in flight); other weights are applied on the way through registers.
                            const uint32_t b0 = (store_cnt & 1u) * (C::OUT_BUFS / 2);
                            if (!direct) {
                                if (lane == 0) bulk_wait_read<1>();
                                __syncwarp();
#pragma unroll 1
                                for (int k = 0; k < C::OUT_BUFS / 2; ++k) {
                                    const uint32_t src = dump + (ch0 + k) * 4096;
                                    const uint32_t dst = stg + (b0 + k) * 4096;
                                    // same physical piece on both sides (the swizzle is kept); the lane-dependent order only
                                    // spreads the 32 rows over the shared-memory banks.  All loads are issued before the
                                    // first store.
                                    float4 v[8];
#pragma unroll
                                    for (int i4 = 0; i4 < 8; ++i4) v[i4] = lds128(src + ((i4 ^ (lane & 7)) << 4));
#pragma unroll
                                    for (int i4 = 0; i4 < 8; ++i4) {
                                        v[i4].x *= ent.w; v[i4].y *= ent.w; v[i4].z *= ent.w; v[i4].w *= ent.w;
                                        sts128(dst + ((i4 ^ (lane & 7)) << 4), v[i4]);
                                    }
                                }
                                fence_proxy_async();
                                __syncwarp();
                            }
                            if (lane == 0) {
                                const uint64_t pol_c = policy_evict_last();     // see the note on the C tiles' L2 policy below
                                const uint32_t src0 = direct ? (base + C::OFF_DUMP + ch0 * 4096) : (base + C::OFF_STG + b0 * 4096);
#pragma unroll 1
                                for (int k = 0; k < C::OUT_BUFS / 2; ++k) {
                                    const int ch = ch0 + k;
                                    const int r = row0 + (ch / (BN / 32)) * 32, c = col0 + (ch % (BN / 32)) * 32;
                                    if (!FMM_GUARD(p.guard, p.c_base + (long long)r * p.ldc + c, (31 * p.ldc + 32) * 4, 1701)) continue;
                                    if (ent.first) tma_store_2d_hint(&tmC, c, r, src0 + k * 4096, pol_c);
                                    else tma_reduce_add_2d_hint(&tmC, c, r, src0 + k * 4096, pol_c);
                                }
                                bulk_commit();
                            }
                            if (!direct) ++store_cnt;
                        }
                    }
                    // the TMA engine has read the copy for the last time (chunks sent as they are), and so has every lane
                    if (lane == 0) bulk_wait_read<0>();
                    // every lane has read the copy for the last time
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_dempty);
                }
            }
            if (lane == 0) bulk_wait<0>();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only in a pair)
        // The whole warp walks the loops (convergent, warp-uniform operands); each tcgen05 instruction is issued by
        // one elected lane inside its wrapper.
        if (leader) {
            int stage = 0; uint32_t phase = 0;
            int buf = 0; uint32_t bphase = 0;
            bool ok = true;
            constexpr uint32_t MDIM = (uint32_t)(BM * NCTA) >> 4;
            uint32_t idesc_full;
            if (C::MX) idesc_full = (1u << 23) | ((uint32_t)(BN >> 3) << 17) | (MDIM << 24);
            else idesc_full = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | (MDIM << 24);
            for (int w = unit; w < p.items && ok; w += units) {
                const uint32_t idesc = idesc_full;
                for (int t = 0; t < p.terms_per_group && ok; ++t) {
                    if (C::MX) {
                        if (!mbar_wait_warp(bar_tempty(0), bphase ^ 1u, ctl, 201)) { ok = false; break; }
                        tc_fence_after();
                    }
                    for (int ks = 0; ks < kstages; ++ks) {
                        if (!mbar_wait_warp(bar_full(stage), phase, ctl, 202)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t adesc = make_kmajor_sw128_desc(base + C::OFF_A + stage * C::A_BYTES);
                        const uint64_t bdesc = make_kmajor_sw128_desc(base + C::OFF_B + stage * C::B_BYTES);
                        if (C::MX) {
                            const uint32_t sf = base + C::OFF_SF + stage * C::SF_STAGE_BYTES;
                            const uint32_t tsfa = tmem_base + BN;          // one slot: cp and mma execute in issue order
                            const uint32_t tsfb = tsfa + 4;
                            tc_cp_32x128b_warpx4<NCTA>(tsfa, make_sf_desc(sf));
#pragma unroll
                            for (int h = 0; h < C::SFB_ATOMS; ++h)
                                tc_cp_32x128b_warpx4<NCTA>(tsfb + 4 * h, make_sf_desc(sf + 512 + h * 512));
#pragma unroll
                            for (int j = 0; j < BK / 32; ++j) {
                                const uint32_t id = idesc | ((uint32_t)j << 29) | ((uint32_t)j << 4);
                                mma_mxf8<NCTA>(tmem_base, adesc + 2 * j, bdesc + 2 * j, id, (ks > 0 || j > 0) ? 1u : 0u, tsfa, tsfb);
                            }
                        } else {
#pragma unroll
                            for (int g0 = 0; g0 < C::KB_PER_STAGE; g0 += C::GPB) {
                                if (!mbar_wait_warp(bar_tempty(buf), bphase ^ 1u, ctl, 203)) { ok = false; break; }
                                tc_fence_after();
#pragma unroll
                                for (int gi = 0; gi < C::GPB; ++gi) {
#pragma unroll
                                    for (int j = 0; j < BLK / 32; ++j) {
                                        const int jj = (g0 + gi) * (BLK / 32) + j;
                                        mma_f8f6f4<NCTA>(tmem_base + (buf * C::GPB + gi) * BN, adesc + 2 * jj, bdesc + 2 * jj, idesc, j > 0 ? 1u : 0u);
                                    }
                                }
                                tc_commit<NCTA>(bar_tfull(buf));
                                if (++buf == C::ACC_BUFS) { buf = 0; bphase ^= 1u; }
                            }
                            if (!ok) break;
                        }
                        tc_commit<NCTA>(bar_empty(stage));
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (C::MX && ok) { tc_commit<NCTA>(bar_tfull(0)); bphase ^= 1u; }
                }
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::REGS_EPI));
        const int e = warp - EPI_WARP0;
        const int q = warp & 3;            // TMEM lane quadrant this warp may access
        const int h = e >> 2;              // column half
        const uint32_t stg = base + C::OFF_STG + e * C::STAGING_BUFS * C::STAGING_BYTES;
        // the accumulator-free signal goes to the MMA issuer, which lives in the even CTA
        auto release_acc = [&](int b) {
            if (NCTA == 2) mbar_arrive_cluster(bar_tempty(b) & PEER_BIT_MASK); else mbar_arrive(bar_tempty(b));
        };
        int buf = 0; uint32_t bphase = 0;
        int ss = 0; uint32_t sphase = 0;
        uint32_t store_cnt = 0;
        uint32_t dphase = 0;
        bool ok = true;
        uint32_t accu[C::MX ? C::CW : 1];               // UE8M0: raw fp32 bits drained from TMEM
        uint32_t kept[C::MX ? 16 : 1];                  // ... and the 16 columns of a parked product that stay in registers
        unsigned long long acc2[C::MX ? 1 : C::CW / 2]; // FP32: promoted accumulators, two columns per register pair
        for (int w = unit; w < p.items && ok; w += units) {
            const int slot = w;
            const int grp = slot / p.positions, pos = slot - grp * p.positions;
            const int tm = pos / tiles_n, tn = pos % tiles_n;
            const int row_in_leaf = (tm * NCTA + cta_rank) * BM + q * 32;
            // columns this warp owns, in 32-column chunks
            constexpr int cw = C::CW;
            const int nch = cw / 32;
            const uint32_t lane_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + h * cw;
            for (int ti = 0, left = p.terms_per_group; left > 0 && ok; ++ti, --left) {
                const int t = C::MX ? term_of(grp, ti) : grp * p.terms_per_group + ti;
                if (C::MX) {
                    if (!mbar_wait_warp(bar_tfull(0), bphase, ctl, 301)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < C::CW / 32; ++c)
                        if (c < nch) tmem_ld32(lane_taddr + c * 32, &accu[c * 32]);
                    tmem_ld_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) release_acc(0);
                    bphase ^= 1u;
                    // ---- pair-fused post-addition (see FmmPairEntry).  First product of a step: park it - CW - 16
                    // columns in this warp's part of the TMEM hold area, 16 in registers - and go on to the next product.
                    const int ri = ti % p.R;
                    const uint32_t hold_taddr = tmem_base + ((uint32_t)(q * 32) << 16) + C::OFF_HOLD + h * C::HOLD_T;
                    if ((ri & 1) == 0 && ri + 1 < p.R) {
#pragma unroll
                        for (int c = 0; c < C::HOLD_T / 32; ++c) tmem_st32(hold_taddr + c * 32, &accu[c * 32]);
                        tmem_st16(hold_taddr + (C::HOLD_T / 32) * 32, &accu[(C::HOLD_T / 32) * 32]);
#pragma unroll
                        for (int i = 0; i < 16; ++i) kept[i] = accu[C::HOLD_T + i];
                        tmem_st_wait();
                        continue;
                    }
                    // second product of a step, or an unpaired one: one weighted update per destination block
                    const uint64_t pol_c = policy_evict_last();
                    const int sidx = (t / p.R) * p.steps + (ri >> 1);
                    const int o0 = p.pair_start[sidx], o1 = p.pair_start[sidx + 1];
                    if (lane == 0) bulk_wait<0>();     // the previous step's writes to these tiles have landed
                    __syncwarp();
                    for (int o = o0; o < o1; ++o) {
                        const FmmPairEntry ent = p.pair[o];
                        const int row0 = ent.row_off * p.m + row_in_leaf;
                        const int col0 = ent.col_off * p.n + tn * BN + h * cw;
                        const bool useA = (ent.wA != 0.0f);
#pragma unroll
                        for (int c = 0; c < C::CW / C::CH; ++c) {
                            const uint32_t b = store_cnt & (C::STAGING_BUFS - 1);
                            if (lane == 0) bulk_wait_read<C::STAGING_BUFS - 1>();   // the buffer about to be rewritten has been read
                            __syncwarp();
                            const uint32_t dst = stg + b * C::STAGING_BYTES + lane * (C::CH * 4);
                            const int swz = (C::CH == 32) ? (lane & 7) : ((lane >> 1) & 3);
#pragma unroll
                            for (int s16 = 0; s16 < C::CH / 16; ++s16) {
                                const int col = c * C::CH + s16 * 16;          // first of 16 columns, within this warp's CW
                                uint32_t av[16];
                                if (useA) {
                                    if (col < C::HOLD_T) { tmem_ld16(hold_taddr + col, av); tmem_ld_wait(); }
                                    else {
#pragma unroll
                                        for (int i = 0; i < 16; ++i) av[i] = kept[i];
                                    }
                                }
#pragma unroll
                                for (int i4 = 0; i4 < 4; ++i4) {
                                    float4 v;
                                    v.x = __uint_as_float(accu[col + i4 * 4 + 0]) * ent.wB; v.y = __uint_as_float(accu[col + i4 * 4 + 1]) * ent.wB;
                                    v.z = __uint_as_float(accu[col + i4 * 4 + 2]) * ent.wB; v.w = __uint_as_float(accu[col + i4 * 4 + 3]) * ent.wB;
                                    if (useA) {
                                        v.x = fmaf(__uint_as_float(av[i4 * 4 + 0]), ent.wA, v.x); v.y = fmaf(__uint_as_float(av[i4 * 4 + 1]), ent.wA, v.y);
                                        v.z = fmaf(__uint_as_float(av[i4 * 4 + 2]), ent.wA, v.z); v.w = fmaf(__uint_as_float(av[i4 * 4 + 3]), ent.wA, v.w);
                                    }
                                    sts128(dst + (((s16 * 4 + i4) ^ swz) << 4), v);
                                }
                            }
                            fence_proxy_async();
                            __syncwarp();
                            if (lane == 0) {
                                if (FMM_GUARD(p.guard, p.c_base + (long long)row0 * p.ldc + col0 + c * C::CH, (31 * p.ldc + C::CH) * 4, 1703)) {
                                    if (ent.first) tma_store_2d_hint(&tmC, col0 + c * C::CH, row0, stg + b * C::STAGING_BYTES, pol_c);
                                    else tma_reduce_add_2d_hint(&tmC, col0 + c * C::CH, row0, stg + b * C::STAGING_BYTES, pol_c);
                                }
                                bulk_commit();
                            }
                            ++store_cnt;
                        }
                    }
                    continue;
                } else if (C::ROWS4) {
                    // ---- per-column fp32 scales.  The accumulators are read with the
                    // 16-lane load shape: a thread owns four rows (lane/4 + 8k) x CW/4 columns (8j + 2(lane%4), +1)
                    // instead of one row x CW columns, so it needs CW/4 B-side scales per K block instead of CW (a
                    // broadcast 16-byte shared-memory load returns 512 bytes to the register file; at one per four
                    // elements those loads were a quarter of the promotion) and four A-side scales instead of one.
                    static_assert(!C::ROWS4 || C::KB_PER_STAGE == 4 || C::KB_PER_STAGE == 1, "block 32 or 128");
                    static_assert(!C::DUMP || C::ROWS4, "the output warp expects the four-row register layout");
#pragma unroll
                    for (int i = 0; i < C::CW / 2; ++i) acc2[i] = 0ull;         // acc2[k * (CW/8) + j]: row slot k, column group j
                    constexpr int JG = C::CW / 8;                               // column groups of eight per warp
                    constexpr int KB = C::KB_PER_STAGE;
                    // A-side scales of the thread's four rows (q*32 + lane/4 + 8k of this CTA's 128), per K block
                    const uint32_t sa_lane = base + C::OFF_SB + C::SB_PART_BYTES + (q * 32 + (lane >> 2)) * (KB * 4);
                    const uint32_t sb_lane = base + C::OFF_SB + (h * C::CW + 2 * (lane & 3)) * 4;
                    for (int ks = 0; ks < kstages && ok; ++ks) {
                        if (!mbar_wait_warp(bar_sfull(ss), sphase, ctl, 302)) { ok = false; break; }
                        const uint32_t sbs32 = sb_lane + ss * C::SB_STAGE_BYTES;
                        // the stage's K blocks for the thread's four rows, from the scale ring (a global load here, even
                        // issued a stage early, stalled the promotion: 14 % of the block-32 kernel)
                        float sa4[4][KB];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if constexpr (KB == 4) {
                                const float4 v4 = lds128(sa_lane + ss * C::SB_STAGE_BYTES + 8 * k * 16);
                                sa4[k][0] = v4.x; sa4[k][1] = v4.y; sa4[k][2] = v4.z; sa4[k][3] = v4.w;
                            } else {
                                sa4[k][0] = lds32f(sa_lane + ss * C::SB_STAGE_BYTES + 8 * k * 4);
                            }
                        }
#pragma unroll
                        for (int g0 = 0; g0 < C::KB_PER_STAGE; g0 += C::GPB) {
                            if (!mbar_wait_warp(bar_tfull(buf), bphase, ctl, 303)) { ok = false; break; }
                            tc_fence_after();
#pragma unroll
                            for (int gi = 0; gi < C::GPB; ++gi) {
                                const int g = g0 + gi;
                                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (buf * C::GPB + gi) * BN + h * C::CW;
                                float sbt = 1.0f;
                                if (MODE == MODE_FP32_SB_TILE) sbt = *reinterpret_cast<const float*>(base_ptr + C::OFF_SB + ss * C::SB_STAGE_BYTES + (g * BN + h * C::CW) * 4);
#pragma unroll
                                for (int c = 0; c < C::CW / 32; ++c) {   // chunks of 32 columns
                                    uint32_t lo[16], hi[16];
                                    tmem_ld_16x256b_x4(taddr + c * 32, lo);                       // rows lane/4, lane/4 + 8
                                    tmem_ld_16x256b_x4(taddr + c * 32 + (16u << 16), hi);         // rows lane/4 + 16, lane/4 + 24
                                    unsigned long long sb2[4];
                                    if (MODE != MODE_FP32_SB_TILE) {
#pragma unroll
                                        for (int j = 0; j < 4; ++j) sb2[j] = lds64(sbs32 + (g * BN + c * 32 + 8 * j) * 4);
                                    }
                                    tmem_ld_wait();
                                    if (gi + 1 == C::GPB && c + 1 == C::CW / 32) {
                                        // the last chunk is in registers: hand the TMEM buffers back before the arithmetic
                                        tc_fence_before();
                                        __syncwarp();
                                        if (lane == 0) release_acc(buf);
                                    }
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        const float sak = sa4[k][g] * sbt;       // tile mode: sA * sB_tile; else sbt = 1 (folded away)
                                        const unsigned long long sa2 = pack2(sak, sak);
                                        const uint32_t* src = (k < 2) ? lo : hi;
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            const uint32_t* tp = src + 4 * j + 2 * (k & 1);
                                            const unsigned long long s2 = (MODE == MODE_FP32_SB_TILE) ? sa2 : mul2(sa2, sb2[j]);
                                            acc2[k * JG + c * 4 + j] = fma2(pack2u(tp[0], tp[1]), s2, acc2[k * JG + c * 4 + j]);
                                        }
                                    }
                                }
                            }
                            if (++buf == C::ACC_BUFS) { buf = 0; bphase ^= 1u; }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_sempty(ss));
                        if (++ss == C::SB_STAGES) { ss = 0; sphase ^= 1u; }
                    }
                    if (!ok) break;
                } else {
#pragma unroll
                    for (int i = 0; i < C::CW / 2; ++i) acc2[i] = 0ull;
                    // this thread's row (q*32 + lane of the CTA's 128) in the A-side part of a scale stage
                    const uint32_t sa_lane = base + C::OFF_SB + C::SB_PART_BYTES + (q * 32 + lane) * (C::KB_PER_STAGE * 4);
                    for (int ks = 0; ks < kstages && ok; ++ks) {
                        if (!mbar_wait_warp(bar_sfull(ss), sphase, ctl, 302)) { ok = false; break; }
                        float sa[C::KB_PER_STAGE];
#pragma unroll
                        for (int g = 0; g < C::KB_PER_STAGE; ++g) sa[g] = lds32f(sa_lane + ss * C::SB_STAGE_BYTES + g * 4);
                        const uint8_t* sbs = base_ptr + C::OFF_SB + ss * C::SB_STAGE_BYTES;
#pragma unroll
                        for (int g0 = 0; g0 < C::KB_PER_STAGE; g0 += C::GPB) {
                            if (!mbar_wait_warp(bar_tfull(buf), bphase, ctl, 303)) { ok = false; break; }
                            tc_fence_after();
#pragma unroll
                            for (int gi = 0; gi < C::GPB; ++gi) {
                                const int g = g0 + gi;
                                const ulonglong2* sbg = reinterpret_cast<const ulonglong2*>(sbs + (g * BN + h * C::CW) * 4);
                                float sab = sa[g];
                                if (MODE == MODE_FP32_SB_TILE) sab *= *reinterpret_cast<const float*>(sbs + (g * BN + h * C::CW) * 4);
                                const unsigned long long sa2 = pack2(sab, sab);
                                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (buf * C::GPB + gi) * BN + h * C::CW;
                                uint32_t tmp[32];
#pragma unroll
                                for (int c = 0; c < C::CW / 32; ++c) {
                                    tmem_ld32(taddr + c * 32, tmp);      // a TMEM load round trip is a few tens of cycles
                                    tmem_ld_wait();
                                    if (gi + 1 == C::GPB && c + 1 == C::CW / 32) {
                                        // the last chunk is in registers: hand the TMEM buffers back before the arithmetic
                                        tc_fence_before();
                                        __syncwarp();
                                        if (lane == 0) release_acc(buf);
                                    }
#pragma unroll
                                    for (int i = 0; i < 8; ++i) {
                                        const uint32_t* tp = tmp + 4 * i;
                                        unsigned long long s01 = sa2, s23 = sa2;        // tile mode: sA * sB_tile
                                        if (MODE != MODE_FP32_SB_TILE) {
                                            const ulonglong2 s4 = sbg[c * 8 + i];        // four column scales
                                            s01 = mul2(sa2, s4.x); s23 = mul2(sa2, s4.y);
                                        }
                                        acc2[c * 16 + 2 * i] = fma2(pack2u(tp[0], tp[1]), s01, acc2[c * 16 + 2 * i]);
                                        acc2[c * 16 + 2 * i + 1] = fma2(pack2u(tp[2], tp[3]), s23, acc2[c * 16 + 2 * i + 1]);
                                    }
                                }
                            }
                            if (++buf == C::ACC_BUFS) { buf = 0; bphase ^= 1u; }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_sempty(ss));
                        if (++ss == C::SB_STAGES) { ss = 0; sphase ^= 1u; }
                    }
                    if (!ok) break;
                }
                if (C::DUMP) {
                    // ---- hand the finished product to the output warp: rows q*32 + lane, columns h*CW .. of the tile,
                    // as 32 x 32 chunks in the 128-byte-swizzled layout of the output tensor map
                    if (!mbar_wait_warp(bar_dempty, dphase ^ 1u, ctl, 304)) { ok = false; break; }
                    dphase ^= 1u;
                    // thread: rows lane/4 + 8k of the warp's 32-row chunk, column pairs 8j + 2(lane%4) of its 64 columns
                    const uint32_t dchunk = base + C::OFF_DUMP + (q * (BN / 32) + h * (C::CW / 32)) * 4096 + (lane & 1) * 8;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int rr = (lane >> 2) + 8 * k;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int pc = 2 * (j & 3) + ((lane & 3) >> 1);        // 16-byte piece of the 128-byte row
                            sts64(dchunk + (j >> 2) * 4096 + rr * 128 + ((pc ^ (rr & 7)) << 4), acc2[k * 8 + j]);
                        }
                    }
                    fence_proxy_async();          // the output warp may hand these chunks to the TMA engine as they are
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_dfull);
                    continue;
                }
                // ---- post-addition: W-weighted scatter of this product into its C blocks
                // Each C tile is updated once per term that feeds it, and between two updates a whole term's operands
                // stream through L2: the tiles are marked evict-last (at n = 8192: fewer write-backs of
                // half-accumulated tiles, product kernel 3 % faster; evict-first on the operand loads was slower).
                // The policy word is rebuilt here so that it is not live across the promotion loop.
                const uint64_t pol_c = policy_evict_last();
                const int o0 = p.out_start[t], o1 = p.out_start[t + 1];
                if (lane == 0) bulk_wait<0>();     // the previous term's writes to these tiles have landed
                __syncwarp();
                for (int o = o0; o < o1; ++o) {
                    const FmmOutEntry ent = p.out[o];
                    const int row0 = ent.row_off * p.m + row_in_leaf;
                    const int col0 = ent.col_off * p.n + tn * BN + h * cw;
#pragma unroll
                    for (int c = 0; c < C::CW / C::CH; ++c) {
                        if (c * C::CH >= cw) break;
                        const uint32_t b = store_cnt & (C::STAGING_BUFS - 1);
                        if (lane == 0) bulk_wait_read<C::STAGING_BUFS - 1>();   // the buffer about to be rewritten has been read
                        __syncwarp();
                        // one row of the chunk per lane; 16-byte pieces permuted as the tensor map's swizzle expects
                        const uint32_t dst = stg + b * C::STAGING_BYTES + lane * (C::CH * 4);
                        const int swz = (C::CH == 32) ? (lane & 7) : ((lane >> 1) & 3);
                        if (C::ROWS4) {
                            // four-row layout: rows lane/4 + 8k, column pairs 8j + 2(lane%4) of this 32-column chunk
                            const uint32_t sdst = stg + b * C::STAGING_BYTES + (lane & 1) * 8;
                            const unsigned long long w2 = pack2(ent.w, ent.w);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const int rr = (lane >> 2) + 8 * k;
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const int pc = 2 * j + ((lane & 3) >> 1);
                                    sts64(sdst + rr * 128 + ((pc ^ (rr & 7)) << 4), mul2(acc2[k * (C::CW / 8) + c * 4 + j], w2));
                                }
                            }
                        } else
#pragma unroll
                        for (int i4 = 0; i4 < C::CH / 4; ++i4) {
                            float4 v;
                            if (C::MX) {
                                v.x = __uint_as_float(accu[c * C::CH + i4 * 4 + 0]); v.y = __uint_as_float(accu[c * C::CH + i4 * 4 + 1]);
                                v.z = __uint_as_float(accu[c * C::CH + i4 * 4 + 2]); v.w = __uint_as_float(accu[c * C::CH + i4 * 4 + 3]);
                            } else {
                                unpack2(acc2[c * (C::CH / 2) + i4 * 2], v.x, v.y);
                                unpack2(acc2[c * (C::CH / 2) + i4 * 2 + 1], v.z, v.w);
                            }
                            v.x *= ent.w; v.y *= ent.w; v.z *= ent.w; v.w *= ent.w;
                            sts128(dst + ((i4 ^ swz) << 4), v);
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            if (FMM_GUARD(p.guard, p.c_base + (long long)row0 * p.ldc + col0 + c * C::CH, (31 * p.ldc + C::CH) * 4, 1702)) {
                                if (ent.first) tma_store_2d_hint(&tmC, col0 + c * C::CH, row0, stg + b * C::STAGING_BYTES, pol_c);
                                else tma_reduce_add_2d_hint(&tmC, col0 + c * C::CH, row0, stg + b * C::STAGING_BYTES, pol_c);
                            }
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
    if (NCTA == 2) cluster_sync();      // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<NCTA>(tmem_base, 512);
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
                 uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * (uint64_t)elt_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int MODE, int BLK, int NCTA>
fmm_status_t launch(const GemmParams& g, cudaStream_t st)
{
    using C = Cfg<BN, MODE, BLK, NCTA>;
    CUtensorMap tmA, tmB, tmC, tmSFA, tmSFB;
    const CUtensorMapSwizzle SW = CU_TENSOR_MAP_SWIZZLE_128B;
    if (!make_map_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, g.qa, (uint64_t)g.k, (uint64_t)g.terms * g.m, BK, BM, SW)) return FMM_ERR_CUDA;
    if (!make_map_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, g.qb, (uint64_t)g.k, (uint64_t)g.terms * g.n, BK, C::BROWS, SW)) return FMM_ERR_CUDA;
    if (!make_map_2d(&tmC, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, g.C, (uint64_t)g.Nfull, (uint64_t)g.Mfull, C::CH, 32,
                     C::CH == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B)) return FMM_ERR_CUDA;
    if (C::MX) {
        // scale tiles as rows of 128 uint32 (one 512-byte atom per row)
        const uint64_t atoms_a = (uint64_t)g.terms * (g.k / 128) * (g.m / 128), atoms_b = (uint64_t)g.terms * (g.k / 128) * (g.n / 128);
        if (!make_map_2d(&tmSFA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, g.sa, 128, atoms_a, 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE)) return FMM_ERR_CUDA;
        if (!make_map_2d(&tmSFB, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, g.sb, 128, atoms_b, 128, C::SFB_ATOMS, CU_TENSOR_MAP_SWIZZLE_NONE)) return FMM_ERR_CUDA;
    } else {
        tmSFA = tmA; tmSFB = tmB;       // unused in this mode
    }
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // the dynamic shared memory limit is a per-device attribute of the function: set once per device
    static std::atomic<bool> attr_set[64];
    if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(fmm_gemm_kernel<BN, MODE, BLK, NCTA>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return FMM_ERR_CUDA;
        }
        if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
    }
    const int positions = (g.m / (BM * NCTA)) * (g.n / BN);
    const int max_units = sms / NCTA;
    // Term groups as separate work items only where that shortens the longest CTA's list of terms (many terms on
    // few tile positions); otherwise one CTA (pair) walks all terms of its position.
    int tpg = (g.terms_per_group > 0 && g.terms % g.terms_per_group == 0) ? g.terms_per_group : g.terms;
    {
        const long long one = (long long)((positions + max_units - 1) / max_units) * g.terms;
        const long long many = (long long)((positions * (g.terms / tpg) + max_units - 1) / max_units) * tpg;
        if (many >= one) tpg = g.terms;
    }
    const int slots = positions * (g.terms / tpg);
    // as few CTAs (pairs) as finish in the same number of waves: every unit then gets the same number of items, and
    // fewer units contend for L2 (256 positions: 64 pairs in 4 waves instead of 74 pairs with a ragged fourth wave)
    const int waves = (slots + max_units - 1) / max_units;
    const int units = (slots + waves - 1) / waves;
    KParams kp;
    kp.sa = static_cast<const uint8_t*>(g.sa); kp.sb = static_cast<const uint8_t*>(g.sb);
    kp.sa_term = g.sa_term; kp.sb_term = g.sb_term;
    kp.m = g.m; kp.n = g.n; kp.k = g.k; kp.terms = g.terms;
    kp.positions = positions; kp.terms_per_group = tpg;
    kp.items = slots;
    kp.out_start = g.out_start; kp.out = g.out; kp.status = g.status;
    kp.pair_start = g.pair_start; kp.pair = g.pair; kp.steps = g.steps;
    for (int r = 0; r < FMM_MAX_RANK; ++r) kp.order[r] = g.order[r];
    kp.R = g.terms_per_group > 0 ? g.terms_per_group : 1;       // products per parent (1 for the cubic product)
    kp.c_base = g.C; kp.ldc = g.Nfull; kp.guard = g.guard;

    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(units * NCTA), 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = NCTA; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    // right behind the encoders of the same call: the CTAs may be set up (barriers, TMEM, tensor maps) while the B-side
    // encoder drains; the two producer warps wait for it before their first load
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = g.overlap_prev ? 2 : 1;
    cudaError_t ce = cudaLaunchKernelEx(&cfg, fmm_gemm_kernel<BN, MODE, BLK, NCTA>, tmA, tmB, tmC, tmSFA, tmSFB, kp);
    if (ce != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    return FMM_OK;
}

template <int MODE, int BLK>
fmm_status_t launch_shape(const GemmParams& g, cudaStream_t st)
{
    // Pairs of CTAs whenever the leaf shape allows it; single CTAs otherwise.  The UE8M0 kernel wants the
    // widest tile (least operand traffic per MMA); the FP32-scale kernels are bound by the promotion
    // on the CUDA cores and use 128-column tiles, whose four TMEM accumulators let the MMA issuer run
    // further ahead of the promoting warps.
    if constexpr (MODE != FMM_SCALE_UE8M0_CEIL) {
        if constexpr (BLK == 32 && MODE == FMM_SCALE_FP32_AMAX_DIV_448) {
            // long terms: post-addition by the output warp.  (Block 128 does not gain from it: with 128-column tiles and
            // the output warp it runs as fast as with 256-column tiles and none, 0.81 ms at n = 8192, and the cubic
            // product, which has a single store per tile, is 20 % slower.)
            if (g.k / BK >= 16) {
                if ((g.m % 256) == 0) return launch<128, MODE_FP32_OUT_WARP, BLK, 2>(g, st);
                return launch<128, MODE_FP32_OUT_WARP, BLK, 1>(g, st);
            }
        }
        if constexpr (BLK == 128) {
            // one promotion per 128 k: 256-column tiles with two TMEM accumulators
            if ((g.m % 256) == 0 && (g.n % 256) == 0) return launch<256, MODE, BLK, 2>(g, st);
        }
        if ((g.m % 256) == 0) return launch<128, MODE, BLK, 2>(g, st);
        return launch<128, MODE, BLK, 1>(g, st);
    } else {
        if ((g.m % 256) == 0 && (g.n % 256) == 0) return launch<256, MODE, 32, 2>(g, st);
        if ((g.n % 256) == 0) return launch<256, MODE, 32, 1>(g, st);
        return launch<128, MODE, 32, 1>(g, st);
    }
}

}  // namespace

fmm_status_t fmm_launch_bounded_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st)
{
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns, 901);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_launch_gemm(const GemmParams& g, int blk, int mode, cudaStream_t st, int* launches)
{
    fmm_status_t s;
    if (mode == FMM_SCALE_UE8M0_CEIL) s = launch_shape<FMM_SCALE_UE8M0_CEIL, 32>(g, st);
    else if (blk == 128 && g.sb_tile) s = launch_shape<MODE_FP32_SB_TILE, 128>(g, st);
    else if (blk == 32) s = launch_shape<FMM_SCALE_FP32_AMAX_DIV_448, 32>(g, st);
    else s = launch_shape<FMM_SCALE_FP32_AMAX_DIV_448, 128>(g, st);
    if (s == FMM_OK && launches) *launches += 1;
    return s;
}
