// Host side of the C ABI: plan validation, workspace layout, the recursion driver that turns
// (levels, realization) into kernel launches.  No device allocation happens after plan creation.
#include <math.h>
#include <stdlib.h>
#include <string.h>
#include <new>
#include <vector>
#include "fmm_internal.h"

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool finite_all(const float* p, int n)
{
    for (int i = 0; i < n; ++i)
        if (!isfinite(p[i])) return false;
    return true;
}

// Largest residual of the Brent equations of <2,2,2> (Sec. 2.1: the decomposition must equal the
// matrix-multiplication tensor): sum_r U[r][ij] V[r][kl] W[r][mn] = [j==k][i==m][l==n].
double brent_residual(int rank, const float* U, const float* V, const float* W)
{
    double worst = 0.0;
    for (int a = 0; a < 4; ++a)
        for (int b = 0; b < 4; ++b)
            for (int c = 0; c < 4; ++c) {
                double s = 0.0;
                for (int r = 0; r < rank; ++r)
                    s += (double)U[r * 4 + a] * (double)V[r * 4 + b] * (double)W[r * 4 + c];
                const int i = a >> 1, j = a & 1, k = b >> 1, l = b & 1, m = c >> 1, n = c & 1;
                const double target = (j == k && i == m && l == n) ? 1.0 : 0.0;
                worst = fmax(worst, fabs(s - target));
            }
    return worst;
}

fmm_status_t check_shape(const fmm_plan* plan, int64_t M, int64_t N, int64_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return FMM_ERR_SHAPE;
    const int64_t d = (int64_t)1 << plan->levels;
    if (M % d || N % d || K % d) return FMM_ERR_SHAPE;
    if ((M / d) % 128 || (N / d) % 128 || (K / d) % 128) return FMM_ERR_SHAPE;
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return FMM_ERR_SHAPE;
    return FMM_OK;
}

void make_layout(const fmm_plan* plan, int64_t M, int64_t N, int64_t K, FmmLayout* L)
{
    const int64_t d = (int64_t)1 << plan->levels;
    L->m = M / d; L->n = N / d; L->k = K / d;
    L->terms = plan->terms;
    const int64_t nkb = L->k / plan->qp.block_k;
    size_t off = 0;
    L->qa = off; off = align_up(off + (size_t)(L->terms * L->m * L->k), 1024);
    L->qb = off; off = align_up(off + (size_t)(L->terms * L->n * L->k), 1024);
    const size_t sbytes = plan->qp.scale_mode == FMM_SCALE_FP32_AMAX_DIV_448 ? 4 : 1;
    L->sa_term = (size_t)(L->m * nkb) * sbytes;
    L->sb_term = (size_t)(L->n * nkb) * sbytes;
    L->sa = off; off = align_up(off + L->sa_term * L->terms, 1024);
    L->sb = off; off = align_up(off + L->sb_term * L->terms, 1024);
    for (int lv = 0; lv < FMM_MAX_LEVELS; ++lv) { L->inter_a[lv] = 0; L->inter_b[lv] = 0; L->dec[lv] = 0; }
    // fp32 combinations of the outer levels 1 .. levels-1
    for (int lv = 1; lv < plan->levels; ++lv) {
        const int64_t cnt = fmm_ipow(plan->rank, lv);
        const int64_t dd = (int64_t)1 << lv;
        // the innermost of these levels is formed in registers by the two-level encoder where that exists
        const bool last = (lv == plan->levels - 1);
        const bool need_a = !(last && fmm_encode2_supported(false, plan->qp.block_k, 0, 0));
        const bool need_b = !(last && fmm_encode2_supported(true, plan->qp.block_k, plan->qp.b_tile_n, plan->qp.b_preround_bf16));
        if (need_a) { L->inter_a[lv] = off; off = align_up(off + (size_t)(cnt * (M / dd) * (K / dd)) * 4, 1024); }
        if (need_b) { L->inter_b[lv] = off; off = align_up(off + (size_t)(cnt * (K / dd) * (N / dd)) * 4, 1024); }
        L->dec[lv] = off; off = align_up(off + (size_t)(cnt * (M / dd) * (N / dd)) * 4, 1024);
    }
    L->total = off;
}

// the kernels read the operands with 16-byte vector loads and write C through a tensor map
bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// a plan's device tables live on the device that was current at fmm_plan_create
fmm_status_t check_device(const fmm_plan* plan)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    return dev == plan->device ? FMM_OK : FMM_ERR_WRONG_DEVICE;
}

fmm_status_t check_ws(const fmm_plan* plan, int64_t M, int64_t N, int64_t K, void* ws, size_t ws_bytes,
                      FmmLayout* L)
{
    fmm_status_t s = check_device(plan);
    if (s != FMM_OK) return s;
    s = check_shape(plan, M, N, K);
    if (s != FMM_OK) return s;
    make_layout(plan, M, N, K, L);
    if (!ws || ((uintptr_t)ws & 1023) || ws_bytes < L->total) return FMM_ERR_WORKSPACE;
    return FMM_OK;
}

void fill_coef(float dst[FMM_MAX_RANK][4], const float src[FMM_MAX_RANK][4], int R)
{
    memset(dst, 0, sizeof(float) * FMM_MAX_RANK * 4);
    for (int r = 0; r < R; ++r)
        for (int j = 0; j < 4; ++j) dst[r][j] = src[r][j];
}

// One side of steps 1-2: outer levels as fp32 combinations, last level fused with the quantizer.
fmm_status_t encode_side(const fmm_plan* plan, const FmmLayout& L, char* ws, const float* X,
                         int64_t rows, int64_t cols, bool b_side, cudaStream_t st, int* launches)
{
    const int R = plan->rank, lv = plan->levels;
    const int blk = plan->qp.block_k, mode = (int)plan->qp.scale_mode;
    const float (*coef)[4] = b_side ? plan->V : plan->U;
    EncodeParams e;
    memset(&e, 0, sizeof(e));
    e.q_out = reinterpret_cast<uint8_t*>(ws + (b_side ? L.qb : L.qa));
    e.s_out = ws + (b_side ? L.sb : L.sa);
    e.s_term_stride = (int64_t)(b_side ? L.sb_term : L.sa_term);
    e.amax_floor = plan->qp.amax_floor;
    e.b_tile = b_side ? plan->qp.b_tile_n : 0;
    e.preround_bf16 = (b_side && plan->qp.b_preround_bf16) ? 1 : 0;
    e.guard = fmm_make_guard(e.q_out, (size_t)L.terms * (size_t)((b_side ? L.n : L.m) * L.k),
                             e.s_out, (size_t)L.terms * (b_side ? L.sb_term : L.sa_term), plan->d_status + FMM_GUARD_WORD);
    fmm_status_t s;
    if (lv == 0) {
        // Plain quantization of the matrix itself.  The matrix is cut into four panels (row panels of A,
        // column panels of B) that are handled like four "combinations" with identity coefficients, so
        // each thread keeps four independent loads in flight; the outputs land where the unsplit
        // matrix would put them.
        const bool panels = b_side ? (cols % (e.b_tile ? 512 : 256) == 0) : (rows % 4 == 0);
        e.in = X; e.in_batch_stride = 0; e.ld = cols; e.batch = 1;
        e.overlap_prev = b_side ? 1 : 0;
        if (panels) {
            e.nq = 4; e.R = 4;
            for (int r = 0; r < 4; ++r) e.coef[r][r] = 1.0f;
            if (b_side) {
                e.rows = (int)rows; e.cols = (int)(cols / 4);
                for (int j = 0; j < 4; ++j) e.qoff[j] = (int64_t)j * (cols / 4);
                e.s_step = (int)(cols / 4); e.s_ld = (int)cols; e.sf_blocks = (int)(cols / 128);
            } else {
                e.rows = (int)(rows / 4); e.cols = (int)cols;
                for (int j = 0; j < 4; ++j) e.qoff[j] = (int64_t)j * (rows / 4) * cols;
                e.s_step = (int)(rows / 4); e.s_ld = (int)rows; e.sf_blocks = (int)(rows / 128);
            }
            // the four panels share one scale array (panel r is shifted by r * s_step rows / columns inside it)
            e.s_term_stride = 0;
        } else {
            e.rows = (int)rows; e.cols = (int)cols; e.nq = 1; e.R = 1;
            e.coef[0][0] = 1.0f;
            e.s_step = 0; e.s_ld = (int)(b_side ? cols : rows); e.sf_blocks = (int)((b_side ? cols : rows) / 128);
        }
    } else {
        const float* cur = X;
        int64_t cur_rows = rows, cur_cols = cols, cur_ld = cols, cur_stride = 0;
        int batch = 1;
        // the last two levels run as one kernel where that is supported: the combinations of level lv-1 stay
        // in registers
        const bool fused2 = lv >= 2 && fmm_encode2_supported(b_side, blk, e.b_tile, e.preround_bf16);
        for (int level = 1; level < (fused2 ? lv - 1 : lv); ++level) {
            CombParams c;
            memset(&c, 0, sizeof(c));
            c.in = cur; c.in_batch_stride = cur_stride; c.ld = cur_ld; c.batch = batch;
            c.rows = (int)(cur_rows / 2); c.cols = (int)(cur_cols / 2); c.R = R;
            fill_coef(c.coef, coef, R);
            c.out = reinterpret_cast<float*>(ws + (b_side ? L.inter_b[level] : L.inter_a[level]));
            c.guard = fmm_make_guard(c.out, (size_t)batch * R * (size_t)(c.rows * (int64_t)c.cols) * 4, nullptr, 0,
                                     plan->d_status + FMM_GUARD_WORD);
            s = fmm_launch_comb(c, st);
            if (s != FMM_OK) return s;
            ++*launches;
            cur = c.out; cur_rows /= 2; cur_cols /= 2; cur_ld = cur_cols; cur_stride = cur_rows * cur_cols;
            batch *= R;
        }
        e.in = cur; e.in_batch_stride = cur_stride; e.ld = cur_ld; e.batch = batch;
        // the B-side leaf encoder may start under the tail of the A-side one (launched just before it by fmm_matmul /
        // fmm_encode_only) when it reads the caller's matrix itself, i.e. nothing a kernel of this call has written
        e.overlap_prev = (b_side && cur == X) ? 1 : 0;
        const int div = fused2 ? 4 : 2;
        e.rows = (int)(cur_rows / div); e.cols = (int)(cur_cols / div); e.nq = 4; e.R = R;
        e.qoff[0] = 0; e.qoff[1] = e.cols; e.qoff[2] = (int64_t)e.rows * e.ld; e.qoff[3] = (int64_t)e.rows * e.ld + e.cols;
        for (int j = 0; j < 4; ++j) e.qoff_outer[j] = 2 * e.qoff[j];
        fill_coef(e.coef, coef, R);
        e.s_step = 0; e.s_ld = b_side ? e.cols : e.rows; e.sf_blocks = (b_side ? e.cols : e.rows) / 128;
        if (fused2) {
            s = b_side ? fmm_launch_encode2_b(e, mode, st) : fmm_launch_encode2_a(e, blk, mode, st);
            if (s == FMM_OK) ++*launches;
            return s;
        }
    }
    s = b_side ? fmm_launch_encode_b(e, blk, mode, st) : fmm_launch_encode_a(e, blk, mode, st);
    if (s == FMM_OK) ++*launches;
    return s;
}

fmm_status_t multiply(const fmm_plan* plan, const FmmLayout& L, char* ws, float* C, int64_t M, int64_t N,
                      cudaStream_t st, int* launches, bool after_encode)
{
    GemmParams g;
    memset(&g, 0, sizeof(g));
    g.overlap_prev = after_encode ? 1 : 0;
    g.qa = reinterpret_cast<const uint8_t*>(ws + L.qa);
    g.qb = reinterpret_cast<const uint8_t*>(ws + L.qb);
    g.sa = ws + L.sa; g.sb = ws + L.sb;
    g.sa_term = (int64_t)L.sa_term; g.sb_term = (int64_t)L.sb_term;
    // The product kernel applies the innermost decoder only: leaf products of parent p land in the four
    // blocks of parent p's (2m x 2n) matrix.  For one level that matrix is C itself; for more levels the
    // parents' matrices are stacked in the workspace and decoded outwards level by level (the same
    // two-stage order as the recursion in Sec. 3), which moves far fewer bytes than scattering every
    // leaf product into all of its R^(levels-1)-fold weighted destinations.
    const int lv = plan->levels;
    const int64_t parents = lv >= 2 ? fmm_ipow(plan->rank, lv - 1) : 1;
    const int64_t pm = lv >= 1 ? 2 * L.m : L.m, pn = lv >= 1 ? 2 * L.n : L.n;      // a parent's matrix
    float* dest = lv >= 2 ? reinterpret_cast<float*>(ws + L.dec[lv - 1]) : C;
    g.C = dest; g.ldc = pn; g.Mfull = parents * pm; g.Nfull = pn;
    g.m = (int)L.m; g.n = (int)L.n; g.k = (int)L.k; g.terms = (int)L.terms;
    g.terms_per_group = plan->levels >= 2 ? plan->rank : (int)L.terms;
    g.out_start = plan->d_out_start; g.out = plan->d_out; g.status = plan->d_status;
    g.pair_start = plan->d_pair_start; g.pair = plan->d_pair; g.steps = plan->steps;
    // the pair-fused walk order belongs to the UE8M0 kernel; the fp32-scale kernels keep the products in term order
    for (int r = 0; r < FMM_MAX_RANK; ++r)
        g.order[r] = (plan->qp.scale_mode == FMM_SCALE_UE8M0_CEIL && plan->levels >= 1) ? plan->order[r] : r;
    g.sb_tile = plan->qp.b_tile_n == 128 ? 1 : 0;
    g.guard = fmm_make_guard(dest, (size_t)g.Mfull * (size_t)g.Nfull * 4, nullptr, 0, plan->d_status + FMM_GUARD_WORD);
    fmm_status_t s = fmm_launch_gemm(g, plan->qp.block_k, (int)plan->qp.scale_mode, st, launches);
    if (s != FMM_OK) return s;
    for (int l = lv - 1; l >= 1; --l) {
        DecodeParams d;
        memset(&d, 0, sizeof(d));
        d.in = reinterpret_cast<const float*>(ws + L.dec[l]);
        d.out = l == 1 ? C : reinterpret_cast<float*>(ws + L.dec[l - 1]);
        d.batch = (int)fmm_ipow(plan->rank, l - 1);
        d.rows = (int)(M >> l); d.cols = (int)(N >> l); d.R = plan->rank;
        for (int r = 0; r < plan->rank; ++r)
            for (int q = 0; q < 4; ++q) d.W[r][q] = plan->W[r][q];
        d.guard = fmm_make_guard(d.out, (size_t)d.batch * 4 * (size_t)d.rows * (size_t)d.cols * 4, nullptr, 0,
                                 plan->d_status + FMM_GUARD_WORD);
        s = fmm_launch_decode(d, st);
        if (s != FMM_OK) return s;
        ++*launches;
    }
    return FMM_OK;
}

}  // namespace

extern "C" {

const char* fmm_status_string(fmm_status_t s)
{
    switch (s) {
        case FMM_OK: return "ok";
        case FMM_ERR_INVALID_ARG: return "invalid argument";
        case FMM_ERR_SHAPE: return "shape not supported (M, N, K must be 2^levels * multiples of 128)";
        case FMM_ERR_NOT_EXACT: return "realization violates the Brent equations";
        case FMM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FMM_ERR_ALLOC: return "allocation failed";
        case FMM_ERR_CUDA: return "CUDA call failed";
        case FMM_ERR_ARCH: return "device is not compute capability 10.x (B200)";
        case FMM_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait timed out";
        case FMM_ERR_WRONG_DEVICE: return "the current device is not the one the plan was created on";
    }
    return "unknown status";
}

fmm_status_t fmm_phi_gamma(int rank, const float* U, const float* V, const float* W, double* phi, double* gamma)
{
    if (rank < 1 || rank > FMM_MAX_RANK || !U || !V || !W || !phi || !gamma) return FMM_ERR_INVALID_ARG;
    double p = 0.0, g = 0.0;
    for (int r = 0; r < rank; ++r) {
        double nu = 0, nv = 0, nw = 0;
        for (int j = 0; j < 4; ++j) {
            nu += (double)U[r * 4 + j] * U[r * 4 + j];
            nv += (double)V[r * 4 + j] * V[r * 4 + j];
            nw += (double)W[r * 4 + j] * W[r * 4 + j];
        }
        p += nu * nv * nw;
        g += sqrt(nu * nv * nw);
    }
    *phi = p; *gamma = g;
    return FMM_OK;
}

fmm_status_t fmm_brent_residual(int rank, const float* U, const float* V, const float* W, double* out)
{
    if (rank < 1 || rank > FMM_MAX_RANK || !U || !V || !W || !out) return FMM_ERR_INVALID_ARG;
    *out = brent_residual(rank, U, V, W);
    return FMM_OK;
}

fmm_status_t fmm_plan_create(fmm_plan_t** out, int rank, const float* U, const float* V, const float* W,
                             int levels, const fmm_quant_params_t* qp)
{
    if (!out) return FMM_ERR_INVALID_ARG;
    *out = nullptr;
    if (!qp || levels < 0 || levels > FMM_MAX_LEVELS) return FMM_ERR_INVALID_ARG;
    if (qp->block_k != 32 && qp->block_k != 128) return FMM_ERR_INVALID_ARG;
    if (qp->scale_mode != FMM_SCALE_FP32_AMAX_DIV_448 && qp->scale_mode != FMM_SCALE_UE8M0_CEIL) return FMM_ERR_INVALID_ARG;
    if (qp->scale_mode == FMM_SCALE_UE8M0_CEIL && qp->block_k != 32) return FMM_ERR_INVALID_ARG;
    if (qp->fp8_max != 448.0f || !(qp->amax_floor > 0.0f) || !isfinite(qp->amax_floor)) return FMM_ERR_INVALID_ARG;
    if (qp->b_tile_n != 0 && qp->b_tile_n != 128) return FMM_ERR_INVALID_ARG;
    if ((qp->b_tile_n == 128 || qp->b_preround_bf16) &&
        (qp->block_k != 128 || qp->scale_mode != FMM_SCALE_FP32_AMAX_DIV_448)) return FMM_ERR_INVALID_ARG;
    if (levels > 0) {
        if (rank < 1 || rank > FMM_MAX_RANK || !U || !V || !W) return FMM_ERR_INVALID_ARG;
        if (!finite_all(U, rank * 4) || !finite_all(V, rank * 4) || !finite_all(W, rank * 4)) return FMM_ERR_INVALID_ARG;
        if (brent_residual(rank, U, V, W) > 1e-5) return FMM_ERR_NOT_EXACT;
    } else {
        rank = 1;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (major != 10) return FMM_ERR_ARCH;

    fmm_plan* p = new (std::nothrow) fmm_plan;
    if (!p) return FMM_ERR_ALLOC;
    memset(static_cast<void*>(p), 0, sizeof(*p));
    p->last_launches.store(0, std::memory_order_relaxed);
    p->rank = rank; p->levels = levels; p->qp = *qp; p->device = dev;
    if (levels > 0)
        for (int r = 0; r < rank; ++r)
            for (int j = 0; j < 4; ++j) { p->U[r][j] = U[r * 4 + j]; p->V[r][j] = V[r * 4 + j]; p->W[r][j] = W[r * 4 + j]; }
    p->terms = (int)fmm_ipow(rank, levels);

    // Decoder table of the product kernel: leaf product t = parent * R + r goes to block q of its parent's
    // matrix with weight W[r][q] (Sec. 2.1 decode, innermost level; outer levels are decoded afterwards).
    // row_off / col_off are in units of leaf blocks inside the stack of parent matrices.
    std::vector<int> start(p->terms + 1, 0);
    std::vector<FmmOutEntry> entries;
    const int parents = levels >= 1 ? p->terms / rank : 1;
    std::vector<char> touched((size_t)parents * 4, 0);
    for (int t = 0; t < p->terms; ++t) {
        start[t] = (int)entries.size();
        if (levels == 0) {
            FmmOutEntry e; e.row_off = 0; e.col_off = 0; e.w = 1.0f; e.first = 1;
            entries.push_back(e);
            continue;
        }
        const int parent = t / rank, r = t % rank;
        for (int q = 0; q < 4; ++q) {
            const float w = p->W[r][q];
            if (w == 0.0f) continue;
            FmmOutEntry e;
            e.row_off = parent * 2 + (q >> 1); e.col_off = q & 1; e.w = w;
            e.first = touched[(size_t)parent * 4 + q] ? 0 : 1;
            touched[(size_t)parent * 4 + q] = 1;
            entries.push_back(e);
        }
    }
    start[p->terms] = (int)entries.size();
    p->n_out_total = (int)entries.size();

    // Pair-fused decoder: pair up the R products of a parent so that the pairs' unions of destination blocks are as
    // small as possible in total (exhaustive over the matchings: R <= 8), walk the pairs one after the other.
    for (int r = 0; r < FMM_MAX_RANK; ++r) p->order[r] = r;
    p->steps = levels >= 1 ? (rank + 1) / 2 : 1;
    std::vector<int> pstart;
    std::vector<FmmPairEntry> pentries;
    if (levels >= 1) {
        auto mask = [&](int r) { int m = 0; for (int q = 0; q < 4; ++q) if (p->W[r][q] != 0.0f) m |= 1 << q; return m; };
        auto bits = [](int m) { return (m & 1) + ((m >> 1) & 1) + ((m >> 2) & 1) + ((m >> 3) & 1); };
        int best_cost = 1 << 30, best[FMM_MAX_RANK], cur[FMM_MAX_RANK];
        bool used[FMM_MAX_RANK] = {false};
        // recursive matching: always pair the lowest unused product with some other one (or leave it single once)
        struct Rec {
            static void go(int n, int R, int cost, bool single_used, bool* used, int* cur, int& best_cost, int* best,
                           const int* masks, int (*bitsf)(int))
            {
                if (cost >= best_cost) return;
                int a = -1;
                for (int r = 0; r < R; ++r) if (!used[r]) { a = r; break; }
                if (a < 0) { best_cost = cost; for (int i = 0; i < R; ++i) best[i] = cur[i]; return; }
                used[a] = true;
                for (int b = a + 1; b < R; ++b) {
                    if (used[b]) continue;
                    used[b] = true; cur[n] = a; cur[n + 1] = b;
                    go(n + 2, R, cost + bitsf(masks[a] | masks[b]), single_used, used, cur, best_cost, best, masks, bitsf);
                    used[b] = false;
                }
                if ((R & 1) && !single_used) {
                    // the single product goes last in the walk: remember it at the end of cur
                    cur[R - 1] = a;
                    // shift: pairs fill cur[0 .. R-2]
                    go(n, R, cost + bitsf(masks[a]), true, used, cur, best_cost, best, masks, bitsf);
                }
                used[a] = false;
            }
        };
        int masks[FMM_MAX_RANK];
        for (int r = 0; r < rank; ++r) masks[r] = mask(r);
        Rec::go(0, rank, 0, false, used, cur, best_cost, best, masks, +bits);
        for (int r = 0; r < rank; ++r) p->order[r] = best[r];
        std::vector<char> ptouched((size_t)parents * 4, 0);
        for (int parent = 0; parent < parents; ++parent)
            for (int s = 0; s < p->steps; ++s) {
                pstart.push_back((int)pentries.size());
                const bool pairstep = 2 * s + 1 < rank;
                const int ra = pairstep ? p->order[2 * s] : -1, rb = pairstep ? p->order[2 * s + 1] : p->order[2 * s];
                for (int q = 0; q < 4; ++q) {
                    const float wa = ra >= 0 ? p->W[ra][q] : 0.0f, wb = p->W[rb][q];
                    if (wa == 0.0f && wb == 0.0f) continue;
                    FmmPairEntry e;
                    e.row_off = parent * 2 + (q >> 1); e.col_off = q & 1; e.wA = wa; e.wB = wb;
                    e.first = ptouched[(size_t)parent * 4 + q] ? 0 : 1;
                    ptouched[(size_t)parent * 4 + q] = 1;
                    pentries.push_back(e);
                }
            }
    } else {
        pstart.push_back(0);
        FmmPairEntry e; e.row_off = 0; e.col_off = 0; e.wA = 0.0f; e.wB = 1.0f; e.first = 1;
        pentries.push_back(e);
    }
    pstart.push_back((int)pentries.size());

    cudaError_t ce = cudaMalloc(&p->d_status, 64 * sizeof(int));
    if (ce == cudaSuccess) ce = cudaMalloc(&p->d_out_start, sizeof(int) * start.size());
    if (ce == cudaSuccess) ce = cudaMalloc(&p->d_out, sizeof(FmmOutEntry) * (entries.size() + 1));
    if (ce == cudaSuccess) ce = cudaMemset(p->d_status, 0, 64 * sizeof(int));
    if (ce == cudaSuccess) ce = cudaMemcpy(p->d_out_start, start.data(), sizeof(int) * start.size(), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess && !entries.empty())
        ce = cudaMemcpy(p->d_out, entries.data(), sizeof(FmmOutEntry) * entries.size(), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMalloc(&p->d_pair_start, sizeof(int) * pstart.size());
    if (ce == cudaSuccess) ce = cudaMalloc(&p->d_pair, sizeof(FmmPairEntry) * (pentries.size() + 1));
    if (ce == cudaSuccess) ce = cudaMemcpy(p->d_pair_start, pstart.data(), sizeof(int) * pstart.size(), cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemcpy(p->d_pair, pentries.data(), sizeof(FmmPairEntry) * pentries.size(), cudaMemcpyHostToDevice);
    if (ce != cudaSuccess) {
        cudaGetLastError();
        fmm_plan_destroy(p);
        return ce == cudaErrorMemoryAllocation ? FMM_ERR_ALLOC : FMM_ERR_CUDA;
    }
    *out = p;
    return FMM_OK;
}

fmm_status_t fmm_plan_destroy(fmm_plan_t* p)
{
    if (!p) return FMM_ERR_INVALID_ARG;
    if (p->d_status) cudaFree(p->d_status);
    if (p->d_out_start) cudaFree(p->d_out_start);
    if (p->d_out) cudaFree(p->d_out);
    if (p->d_pair_start) cudaFree(p->d_pair_start);
    if (p->d_pair) cudaFree(p->d_pair);
    delete p;
    return FMM_OK;
}

fmm_status_t fmm_workspace_bytes(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K, size_t* bytes)
{
    if (!plan || !bytes) return FMM_ERR_INVALID_ARG;
    fmm_status_t s = check_shape(plan, M, N, K);
    if (s != FMM_OK) return s;
    FmmLayout L;
    make_layout(plan, M, N, K, &L);
    *bytes = L.total;
    return FMM_OK;
}

fmm_status_t fmm_quantized_view(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K, int term, char side,
                                size_t* q_offset, int64_t* q_rows, int64_t* q_cols,
                                size_t* scale_offset, int64_t* scale_rows, int64_t* scale_cols)
{
    if (!plan || !q_offset || !q_rows || !q_cols || !scale_offset || !scale_rows || !scale_cols) return FMM_ERR_INVALID_ARG;
    if (side != 'A' && side != 'B') return FMM_ERR_INVALID_ARG;
    fmm_status_t s = check_shape(plan, M, N, K);
    if (s != FMM_OK) return s;
    if (term < 0 || term >= plan->terms) return FMM_ERR_INVALID_ARG;
    FmmLayout L;
    make_layout(plan, M, N, K, &L);
    const int64_t nkb = L.k / plan->qp.block_k;
    const bool fp32 = plan->qp.scale_mode == FMM_SCALE_FP32_AMAX_DIV_448;
    if (side == 'A') {
        *q_offset = L.qa + (size_t)term * L.m * L.k; *q_rows = L.m; *q_cols = L.k;
        *scale_offset = L.sa + (size_t)term * L.sa_term;
        if (fp32) { *scale_rows = L.k / 128; *scale_cols = L.m * (128 / plan->qp.block_k); } else { *scale_rows = L.m; *scale_cols = nkb; }
    } else {
        *q_offset = L.qb + (size_t)term * L.n * L.k; *q_rows = L.n; *q_cols = L.k;
        *scale_offset = L.sb + (size_t)term * L.sb_term;
        if (fp32) { *scale_rows = nkb; *scale_cols = L.n; } else { *scale_rows = L.n; *scale_cols = nkb; }
    }
    return FMM_OK;
}

fmm_status_t fmm_encode_only(const fmm_plan_t* plan, const float* A, const float* B, int64_t M, int64_t N, int64_t K,
                             void* ws, size_t ws_bytes, void* stream)
{
    if (!plan || !A || !B || !aligned16(A) || !aligned16(B)) return FMM_ERR_INVALID_ARG;
    FmmLayout L;
    fmm_status_t s = check_ws(plan, M, N, K, ws, ws_bytes, &L);
    if (s != FMM_OK) return s;
    int launches = 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    s = encode_side(plan, L, static_cast<char*>(ws), A, M, K, false, st, &launches);
    if (s == FMM_OK) s = encode_side(plan, L, static_cast<char*>(ws), B, K, N, true, st, &launches);
    plan->last_launches.store(launches, std::memory_order_relaxed);
    return s;
}

fmm_status_t fmm_multiply_only(const fmm_plan_t* plan, float* C, int64_t M, int64_t N, int64_t K,
                               void* ws, size_t ws_bytes, void* stream)
{
    if (!plan || !C || !aligned16(C)) return FMM_ERR_INVALID_ARG;
    FmmLayout L;
    fmm_status_t s = check_ws(plan, M, N, K, ws, ws_bytes, &L);
    if (s != FMM_OK) return s;
    int launches = 0;
    s = multiply(plan, L, static_cast<char*>(ws), C, M, N, reinterpret_cast<cudaStream_t>(stream), &launches, false);
    plan->last_launches.store(launches, std::memory_order_relaxed);
    return s;
}

fmm_status_t fmm_matmul(const fmm_plan_t* plan, const float* A, const float* B, float* C,
                        int64_t M, int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream)
{
    if (!plan || !A || !B || !C || !aligned16(A) || !aligned16(B) || !aligned16(C)) return FMM_ERR_INVALID_ARG;
    FmmLayout L;
    fmm_status_t s = check_ws(plan, M, N, K, ws, ws_bytes, &L);
    if (s != FMM_OK) return s;
    int launches = 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    s = encode_side(plan, L, static_cast<char*>(ws), A, M, K, false, st, &launches);
    if (s == FMM_OK) s = encode_side(plan, L, static_cast<char*>(ws), B, K, N, true, st, &launches);
    if (s == FMM_OK) s = multiply(plan, L, static_cast<char*>(ws), C, M, N, st, &launches, true);
    plan->last_launches.store(launches, std::memory_order_relaxed);
    return s;
}

// Host-operand variant: [product workspace | A | B | C] in the caller's device buffer, 1024-byte aligned parts.
static size_t host_align(size_t x) { return (x + 1023) & ~(size_t)1023; }

fmm_status_t fmm_host_workspace_bytes(const fmm_plan_t* plan, int64_t M, int64_t N, int64_t K, size_t* bytes)
{
    if (!bytes) return FMM_ERR_INVALID_ARG;
    size_t ws = 0;
    fmm_status_t s = fmm_workspace_bytes(plan, M, N, K, &ws);
    if (s != FMM_OK) return s;
    *bytes = host_align(ws) + host_align((size_t)M * K * 4) + host_align((size_t)K * N * 4) + host_align((size_t)M * N * 4);
    return FMM_OK;
}

fmm_status_t fmm_matmul_host(const fmm_plan_t* plan, const float* A, const float* B, float* C,
                             int64_t M, int64_t N, int64_t K, void* ws, size_t ws_bytes, void* stream)
{
    if (!plan || !A || !B || !C) return FMM_ERR_INVALID_ARG;
    size_t need = 0, inner = 0;
    fmm_status_t s = fmm_host_workspace_bytes(plan, M, N, K, &need);
    if (s != FMM_OK) return s;
    if (!ws || ((uintptr_t)ws & 1023) || ws_bytes < need) return FMM_ERR_WORKSPACE;
    fmm_workspace_bytes(plan, M, N, K, &inner);
    char* base = static_cast<char*>(ws);
    float* dA = reinterpret_cast<float*>(base + host_align(inner));
    float* dB = reinterpret_cast<float*>(reinterpret_cast<char*>(dA) + host_align((size_t)M * K * 4));
    float* dC = reinterpret_cast<float*>(reinterpret_cast<char*>(dB) + host_align((size_t)K * N * 4));
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(dA, A, (size_t)M * K * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dB, B, (size_t)K * N * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return FMM_ERR_CUDA;
    }
    s = fmm_matmul(plan, dA, dB, dC, M, N, K, ws, inner, stream);
    if (s != FMM_OK) return s;
    if (cudaMemcpyAsync(C, dC, (size_t)M * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        cudaGetLastError();
        return FMM_ERR_CUDA;
    }
    return FMM_OK;
}

fmm_status_t fmm_device_status(const fmm_plan_t* plan, int* code)
{
    if (!plan || !code) return FMM_ERR_INVALID_ARG;
    fmm_status_t sd = check_device(plan);
    if (sd != FMM_OK) return sd;
    int h[4] = {0, 0, 0, 0};
    // every stream, including non-blocking ones that the copy below would not wait for
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (cudaMemcpy(h, plan->d_status, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    *code = h[0];
    return h[0] ? FMM_ERR_DEVICE_TIMEOUT : FMM_OK;
}

int fmm_debug_build(void)
{
#ifdef FMM_DEBUG
    return 1;
#else
    return 0;
#endif
}

fmm_status_t fmm_debug_violation(const fmm_plan_t* plan, int* code)
{
    if (!code) return FMM_ERR_INVALID_ARG;
    if (!plan) return fmm_stats_guard_read(code);
    fmm_status_t sd = check_device(plan);
    if (sd != FMM_OK) return sd;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (cudaMemcpy(code, plan->d_status + FMM_GUARD_WORD, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    return FMM_OK;
}

fmm_status_t fmm_device_status_clear(const fmm_plan_t* plan)
{
    if (!plan) return FMM_ERR_INVALID_ARG;
    fmm_status_t sd = check_device(plan);
    if (sd != FMM_OK) return sd;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (cudaMemset(plan->d_status, 0, 64 * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    return FMM_OK;
}

fmm_status_t fmm_selftest_bounded_wait(const fmm_plan_t* plan, int64_t limit_ns, void* stream)
{
    if (!plan || limit_ns <= 0 || limit_ns > 2000000000ll) return FMM_ERR_INVALID_ARG;
    fmm_status_t sd = check_device(plan);
    if (sd != FMM_OK) return sd;
    return fmm_launch_bounded_wait_selftest(plan->d_status, (unsigned long long)limit_ns, reinterpret_cast<cudaStream_t>(stream));
}

fmm_status_t fmm_selftest_store_guard(const fmm_plan_t* plan, void* stream)
{
    if (!plan) return FMM_ERR_INVALID_ARG;
    fmm_status_t sd = check_device(plan);
    if (sd != FMM_OK) return sd;
    return fmm_launch_guard_selftest(plan->d_status, reinterpret_cast<cudaStream_t>(stream));
}

fmm_status_t fmm_last_launch_count(const fmm_plan_t* plan, int* launches)
{
    if (!plan || !launches) return FMM_ERR_INVALID_ARG;
    *launches = plan->last_launches.load(std::memory_order_relaxed);
    return FMM_OK;
}

}  // extern "C"
