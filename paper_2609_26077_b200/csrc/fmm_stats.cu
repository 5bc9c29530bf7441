// Error measurement (paper App. E.2: relative Frobenius error against an fp64 product;
// Eq. (D.9) compares the RMS of that error across realizations).
//   fmm_ref_gemm_fp64 : Cref = A * B with fp64 multiply-accumulate of the fp32 inputs (DFMA tiles).
//   fmm_error_stats   : sum (C - Cref)^2, sum Cref^2, max |C - Cref| with fp64 accumulation,
//                       warp-shuffle + shared-memory tree per block, fixed block partition and a
//                       single-block second stage, hence bit-reproducible.
#include <mutex>
#include "fmm_internal.h"

// Scratch of fmm_error_stats_noalloc: one partial triple per reduction block.  It lives in the
// library image, so every GPU that loads the library carries these 24 KB until the process exits.
// In host code this name is only a stand-in for the symbol; the device address comes from
// cudaGetSymbolAddress (see noalloc_scratch below).
static __device__ __align__(256) double g_noalloc_partials[3 * 1024];
// where the statistics kernels of the FMM_DEBUG build report a store outside their output buffers
static __device__ int g_stats_guard_code;

namespace {

constexpr int STAT_BLOCKS = 592;      // 4 x 148 SMs, all resident at 512 threads; at most the 1024 slots of g_noalloc_partials
constexpr int STAT_THREADS = 512;
constexpr int64_t STATS_MAX_DIM = (int64_t)1 << 30;    // per dimension, as for the product itself: M * N cannot overflow
static_assert(STAT_BLOCKS <= 1024, "one scratch slot per reduction block");

__device__ __forceinline__ void warp_reduce3(double& a, double& b, double& c)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
        c = fmax(c, __shfl_xor_sync(0xffffffffu, c, o));
    }
}

__device__ __forceinline__ void block_reduce3(double& a, double& b, double& c, double* sm)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    warp_reduce3(a, b, c);
    if (lane == 0) { sm[warp * 3] = a; sm[warp * 3 + 1] = b; sm[warp * 3 + 2] = c; }
    __syncthreads();
    if (warp == 0) {
        const int nw = blockDim.x >> 5;
        a = lane < nw ? sm[lane * 3] : 0.0;
        b = lane < nw ? sm[lane * 3 + 1] : 0.0;
        c = lane < nw ? sm[lane * 3 + 2] : 0.0;
        warp_reduce3(a, b, c);
    }
}

__global__ void __launch_bounds__(STAT_THREADS) error_partial_kernel(const float* __restrict__ C,
                                                                    const double* __restrict__ Cref,
                                                                    int64_t count, double* __restrict__ partial,
                                                                    const FmmGuard guard)
{
    __shared__ double sm[3 * (STAT_THREADS / 32)];
    double sd = 0.0, sr = 0.0, mx = 0.0;
    // each thread takes pairs: one 8-byte load of C, one 16-byte load of Cref (count is even); four pairs per
    // trip with all loads issued first, so that every thread keeps 96 bytes in flight
    const int64_t pairs = count >> 1;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float2* C2 = reinterpret_cast<const float2*>(C);
    const double2* R2 = reinterpret_cast<const double2*>(Cref);
    auto add = [&](float2 c, double2 r) {
        const double d0 = (double)c.x - r.x, d1 = (double)c.y - r.y;
        sd = fma(d0, d0, sd); sd = fma(d1, d1, sd);
        sr = fma(r.x, r.x, sr); sr = fma(r.y, r.y, sr);
        mx = fmax(mx, fmax(fabs(d0), fabs(d1)));
    };
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < pairs; i += 4 * stride) {
        float2 c[4]; double2 r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { c[u] = __ldcs(C2 + i + u * stride); r[u] = __ldcs(R2 + i + u * stride); }
#pragma unroll
        for (int u = 0; u < 4; ++u) add(c[u], r[u]);
    }
    for (; i < pairs; i += stride) add(__ldcs(C2 + i), __ldcs(R2 + i));
    block_reduce3(sd, sr, mx, sm);
    if (threadIdx.x == 0 && FMM_GUARD(guard, partial + blockIdx.x * 3, 24, 1601)) {
        partial[blockIdx.x * 3] = sd; partial[blockIdx.x * 3 + 1] = sr; partial[blockIdx.x * 3 + 2] = mx;
    }
}

__global__ void __launch_bounds__(STAT_THREADS) error_final_kernel(const double* __restrict__ partial, int n,
                                                                  double* __restrict__ out3, const FmmGuard guard)
{
    __shared__ double sm[3 * (STAT_THREADS / 32)];
    double sd = 0.0, sr = 0.0, mx = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        sd += partial[i * 3]; sr += partial[i * 3 + 1]; mx = fmax(mx, partial[i * 3 + 2]);
    }
    block_reduce3(sd, sr, mx, sm);
    if (threadIdx.x == 0 && FMM_GUARD(guard, out3, 24, 1602)) { out3[0] = sd; out3[1] = sr; out3[2] = mx; }
}

// 64x64 output tile per block of 16x16 threads, 4x4 outputs per thread, K step 16.
__global__ void __launch_bounds__(256) ref_gemm_fp64_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                           double* __restrict__ C, int64_t M, int64_t N, int64_t K,
                                                           const FmmGuard guard)
{
    __shared__ float As[16][64 + 1];   // [k][m]
    __shared__ float Bs[16][64];       // [k][n]
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
    for (int64_t k0 = 0; k0 < K; k0 += 16) {
        // A tile: 64 rows x 16 k = 1024 floats, 4 per thread
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = threadIdx.x + e * 256;
            const int r = idx >> 4, kk = idx & 15;
            As[kk][r] = A[(m0 + r) * K + k0 + kk];
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = threadIdx.x + e * 256;
            const int kk = idx >> 6, c = idx & 63;
            Bs[kk][c] = B[(k0 + kk) * N + n0 + c];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = (double)As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = (double)Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        double* c = C + (m0 + ty * 4 + i) * N + n0 + tx * 4;
        if (!FMM_GUARD(guard, c, 32, 1603)) continue;
        reinterpret_cast<double2*>(c)[0] = make_double2(acc[i][0], acc[i][1]);
        reinterpret_cast<double2*>(c)[1] = make_double2(acc[i][2], acc[i][3]);
    }
}

// Device address of g_stats_guard_code on the current device (FMM_DEBUG build; the release build passes no word and
// never resolves the symbol, so its calls stay free of runtime lookups).
int* stats_guard_word()
{
#ifdef FMM_DEBUG
    int* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_stats_guard_code) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return ptr;
#else
    return nullptr;
#endif
}

}  // namespace

// Self-test of the store guard: one thread stores to status word 40 under a guard that allows words 32..39 only.
// Both addresses lie inside the plan's 64-word status array, so nothing is ever written out of bounds; the checked
// build must skip the store and record code 1901, the normal build has no guard and simply writes the spare word.
__global__ void guard_selftest_kernel(int* status, const FmmGuard guard)
{
    int* target = status + 40;
    if (FMM_GUARD(guard, target, sizeof(int), 1901)) *target = 1;
}

fmm_status_t fmm_launch_guard_selftest(int* status, cudaStream_t st)
{
    const FmmGuard guard = fmm_make_guard(status + 32, 8 * sizeof(int), nullptr, 0, status + FMM_GUARD_WORD);
    guard_selftest_kernel<<<1, 1, 0, st>>>(status, guard);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_stats_guard_read(int* code)
{
    *code = 0;
#ifdef FMM_DEBUG
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (cudaMemcpyFromSymbol(code, g_stats_guard_code, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
#endif
    return FMM_OK;
}

extern "C" {

size_t fmm_error_stats_scratch_bytes(void) { return sizeof(double) * 3 * STAT_BLOCKS; }

fmm_status_t fmm_error_stats(const float* C, const double* Cref, int64_t M, int64_t N, double* out3,
                             void* scratch, size_t scratch_bytes, void* stream)
{
    if (!C || !Cref || !out3 || !scratch) return FMM_ERR_INVALID_ARG;
    // bound each factor before forming the product (signed overflow otherwise)
    if (M <= 0 || N <= 0 || M > STATS_MAX_DIM || N > STATS_MAX_DIM || ((M * N) & 1)) return FMM_ERR_SHAPE;
    if (scratch_bytes < fmm_error_stats_scratch_bytes() || ((uintptr_t)scratch & 15)) return FMM_ERR_WORKSPACE;
    if (((uintptr_t)C & 7) || ((uintptr_t)Cref & 15)) return FMM_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    double* partial = static_cast<double*>(scratch);
    const FmmGuard guard = fmm_make_guard(partial, sizeof(double) * 3 * STAT_BLOCKS, out3, sizeof(double) * 3, stats_guard_word());
    error_partial_kernel<<<STAT_BLOCKS, STAT_THREADS, 0, st>>>(C, Cref, M * N, partial, guard);
    error_final_kernel<<<1, STAT_THREADS, 0, st>>>(partial, STAT_BLOCKS, out3, guard);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

fmm_status_t fmm_ref_gemm_fp64(const float* A, const float* B, double* Cref, int64_t M, int64_t N, int64_t K,
                               void* stream)
{
    if (!A || !B || !Cref) return FMM_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || (M % 64) || (N % 64) || (K % 16)) return FMM_ERR_SHAPE;
    if ((uintptr_t)Cref & 15) return FMM_ERR_INVALID_ARG;
    dim3 grid((unsigned)(N / 64), (unsigned)(M / 64));
    const FmmGuard guard = fmm_make_guard(Cref, sizeof(double) * (size_t)M * (size_t)N, nullptr, 0, stats_guard_word());
    ref_gemm_fp64_kernel<<<grid, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(A, B, Cref, M, N, K, guard);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

// ---- variant of fmm_error_stats for callers that cannot allocate device memory ----------------
namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
constexpr int64_t NOALLOC_MAX_ELEMS = (int64_t)1 << 28;    // a constant of the interface, not of the array: the kernels handle any count
std::mutex g_noalloc_mutex;
double* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {nullptr};

// Device address of the static scratch on the current device, resolved once per device.
fmm_status_t noalloc_scratch(double** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return FMM_ERR_CUDA; }
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return FMM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        double* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_partials) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return FMM_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return FMM_OK;
}
}  // namespace

fmm_status_t fmm_error_stats_noalloc(const float* C, const double* Cref, int64_t M, int64_t N, double* out3,
                                     void* stream)
{
    if (!C || !Cref || !out3) return FMM_ERR_INVALID_ARG;
    if (M <= 0 || N <= 0 || M > NOALLOC_MAX_ELEMS || N > NOALLOC_MAX_ELEMS) return FMM_ERR_SHAPE;
    if (M * N > NOALLOC_MAX_ELEMS || ((M * N) & 1)) return FMM_ERR_SHAPE;
    if (((uintptr_t)C & 7) || ((uintptr_t)Cref & 15)) return FMM_ERR_INVALID_ARG;
    double* partial = nullptr;
    fmm_status_t s = noalloc_scratch(&partial);
    if (s != FMM_OK) return s;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // every one of the STAT_BLOCKS slots is rewritten by the first kernel, so nothing left behind by
    // an earlier call is ever read and no clearing is needed
    const FmmGuard guard = fmm_make_guard(partial, sizeof(double) * 3 * STAT_BLOCKS, out3, sizeof(double) * 3, stats_guard_word());
    error_partial_kernel<<<STAT_BLOCKS, STAT_THREADS, 0, st>>>(C, Cref, M * N, partial, guard);
    error_final_kernel<<<1, STAT_THREADS, 0, st>>>(partial, STAT_BLOCKS, out3, guard);
    return cudaGetLastError() == cudaSuccess ? FMM_OK : FMM_ERR_CUDA;
}

int64_t fmm_error_stats_noalloc_max_elements(void) { return NOALLOC_MAX_ELEMS; }

}  // extern "C"
