// Fallback, cross-check and scaling kernels: plain CUDA-core code that accepts any storage type, layout,
// pitch and alignment.  The fallback is the paper's naive one-thread-per-output kernel (section 2.2)
// after thread-block tiling and thread tiling (64x64 block tile staged through shared memory, 4x4
// outputs per thread); the cross-check kernel is the naive kernel itself with an fp64 accumulator.
#include "common.cuh"

namespace peak {
namespace {

constexpr int FB_TILE = 64;  // block tile is FB_TILE x FB_TILE
constexpr int FB_BK = 16;
constexpr int FB_THREADS = 256;  // 16 x 16 threads, 4 x 4 outputs each

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(FB_THREADS)
fallback_gemm_kernel(int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const TIn *__restrict__ A,
                     int64_t lda, const TIn *__restrict__ B, int64_t ldb, float beta, TOut *__restrict__ C,
                     int64_t ldc, const float *__restrict__ bias, int act, const TOut *__restrict__ R, int64_t ldr) {
    __shared__ float As[FB_BK][FB_TILE + 1];  // As[k][m]
    __shared__ float Bs[FB_BK][FB_TILE + 1];  // Bs[k][n]
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t m0 = (int64_t)blockIdx.y * FB_TILE, n0 = (int64_t)blockIdx.x * FB_TILE;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    for (int64_t k0 = 0; k0 < K; k0 += FB_BK) {
        // stage op(A)[m0.., k0..] and op(B)[k0.., n0..]; the fast-running index follows the storage order
        for (int e = tid; e < FB_TILE * FB_BK; e += FB_THREADS) {
            int mm, kk;
            if (transA) { mm = e % FB_TILE; kk = e / FB_TILE; } else { kk = e % FB_BK; mm = e / FB_BK; }
            const int64_t m = m0 + mm, k = k0 + kk;
            float v = 0.0f;
            if (m < M && k < K) v = to_f32(transA ? A[k * lda + m] : A[m * lda + k]);
            As[kk][mm] = v;
        }
        for (int e = tid; e < FB_TILE * FB_BK; e += FB_THREADS) {
            int nn, kk;
            if (transB) { kk = e % FB_BK; nn = e / FB_BK; } else { nn = e % FB_TILE; kk = e / FB_TILE; }
            const int64_t n = n0 + nn, k = k0 + kk;
            float v = 0.0f;
            if (n < N && k < K) v = to_f32(transB ? B[n * ldb + k] : B[k * ldb + n]);
            Bs[kk][nn] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < FB_BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty + 16 * i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx + 16 * j;
            if (n >= N) continue;
            TOut *p = C + m * ldc + n;
            const float c_old = (beta != 0.0f) ? to_f32(*p) : 0.0f;
            *p = from_f32<TOut>(add_residual(finish_f32(epilogue_f32(alpha, acc[i][j], beta, c_old), bias, n, act), R,
                                             m * ldr + n));
        }
    }
}

// One thread per output element, fp64 accumulation with k ascending; result left unrounded in fp64.
template <typename TIn, typename TOut>
__global__ void xcheck_f64_kernel(int transA, int transB, int64_t M, int64_t N, int64_t K, double alpha,
                                  const TIn *__restrict__ A, int64_t lda, const TIn *__restrict__ B, int64_t ldb,
                                  double beta, const TOut *__restrict__ C0, int64_t ldc, double *__restrict__ Cref,
                                  int64_t ldcref) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = (int64_t)blockIdx.y * blockDim.y + threadIdx.y;
    if (i >= M || j >= N) return;
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        const double a = (double)to_f32(transA ? A[k * lda + i] : A[i * lda + k]);
        const double b = (double)to_f32(transB ? B[j * ldb + k] : B[k * ldb + j]);
        acc = fma(a, b, acc);
    }
    double r = alpha * acc;
    if (beta != 0.0) r += beta * (double)to_f32(C0[i * ldc + j]);
    Cref[i * ldcref + j] = r;
}

// C = beta * C (beta == 0 stores zeros without reading C).
template <typename TOut>
__global__ void scale_kernel(int64_t M, int64_t N, float beta, TOut *__restrict__ C, int64_t ldc,
                             const float *__restrict__ bias, int act, const TOut *__restrict__ R, int64_t ldr) {
    const int64_t total = M * N;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        TOut *p = C + (e / N) * ldc + (e % N);
        const float x = (beta == 0.0f) ? 0.0f : beta * to_f32(*p);
        *p = from_f32<TOut>(add_residual(finish_f32(x, bias, e % N, act), R, (e / N) * ldr + (e % N)));
    }
}

template <typename TIn, typename TOut> int run_fallback(const GemmArgs &g) {
    dim3 grid((unsigned)((g.N + FB_TILE - 1) / FB_TILE), (unsigned)((g.M + FB_TILE - 1) / FB_TILE));
    if (grid.y > 65535u) return PEAK_ERR_UNSUPPORTED;
    fallback_gemm_kernel<TIn, TOut><<<grid, FB_THREADS, 0, g.stream>>>(
        g.transA, g.transB, g.M, g.N, g.K, g.alpha, (const TIn *)g.A, g.lda, (const TIn *)g.B, g.ldb, g.beta,
        (TOut *)g.C, g.ldc, g.bias, g.act, (const TOut *)g.R, g.ldr);
    count_launch();
    note_kernel("fallback_gemm_kernel grid=%ux%u", grid.x, grid.y);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <typename TIn, typename TOut>
int run_xcheck(const GemmArgs &g, const void *C0, double *Cref, int64_t ldcref) {
    dim3 block(32, 8);
    dim3 grid((unsigned)((g.N + 31) / 32), (unsigned)((g.M + 7) / 8));
    if (grid.y > 65535u) return PEAK_ERR_UNSUPPORTED;
    xcheck_f64_kernel<TIn, TOut><<<grid, block, 0, g.stream>>>(g.transA, g.transB, g.M, g.N, g.K, (double)g.alpha,
                                                               (const TIn *)g.A, g.lda, (const TIn *)g.B, g.ldb,
                                                               (double)g.beta, (const TOut *)C0, g.ldc, Cref, ldcref);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <typename TOut> int run_scale(const GemmArgs &g) {
    const int64_t total = g.M * g.N;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    scale_kernel<TOut><<<(unsigned)blocks, 256, 0, g.stream>>>(g.M, g.N, g.beta, (TOut *)g.C, g.ldc, g.bias, g.act,
                                                               (const TOut *)g.R, g.ldr);
    count_launch();
    note_kernel("scale_kernel grid=%u", (unsigned)blocks);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

}  // namespace

int launch_fallback(const GemmArgs &g) {
    switch (g.dtype) {
        case PEAK_F16_F32: return run_fallback<__half, float>(g);
        case PEAK_BF16_BF16: return run_fallback<__nv_bfloat16, __nv_bfloat16>(g);
        case PEAK_F32_F32: return run_fallback<float, float>(g);
        case PEAK_F16_F16: return run_fallback<__half, __half>(g);
        case PEAK_BF16_F32: return run_fallback<__nv_bfloat16, float>(g);
        case PEAK_E4M3_BF16: return run_fallback<__nv_fp8_e4m3, __nv_bfloat16>(g);
        case PEAK_E4M3_F32: return run_fallback<__nv_fp8_e4m3, float>(g);
        case PEAK_E5M2_BF16: return run_fallback<__nv_fp8_e5m2, __nv_bfloat16>(g);
        case PEAK_E5M2_F32: return run_fallback<__nv_fp8_e5m2, float>(g);
    }
    return PEAK_ERR_INVALID_VALUE;
}

int launch_xcheck_f64(const GemmArgs &g, const void *C0, double *Cref, int64_t ldcref) {
    switch (g.dtype) {
        case PEAK_F16_F32: return run_xcheck<__half, float>(g, C0, Cref, ldcref);
        case PEAK_BF16_BF16: return run_xcheck<__nv_bfloat16, __nv_bfloat16>(g, C0, Cref, ldcref);
        case PEAK_F32_F32: return run_xcheck<float, float>(g, C0, Cref, ldcref);
        case PEAK_F16_F16: return run_xcheck<__half, __half>(g, C0, Cref, ldcref);
        case PEAK_BF16_F32: return run_xcheck<__nv_bfloat16, float>(g, C0, Cref, ldcref);
        case PEAK_E4M3_BF16: return run_xcheck<__nv_fp8_e4m3, __nv_bfloat16>(g, C0, Cref, ldcref);
        case PEAK_E4M3_F32: return run_xcheck<__nv_fp8_e4m3, float>(g, C0, Cref, ldcref);
        case PEAK_E5M2_BF16: return run_xcheck<__nv_fp8_e5m2, __nv_bfloat16>(g, C0, Cref, ldcref);
        case PEAK_E5M2_F32: return run_xcheck<__nv_fp8_e5m2, float>(g, C0, Cref, ldcref);
    }
    return PEAK_ERR_INVALID_VALUE;
}

int launch_scale(const GemmArgs &g) {
    switch (out_elem(g.dtype)) {
        case Elem::F32: return run_scale<float>(g);
        case Elem::F16: return run_scale<__half>(g);
        case Elem::BF16: return run_scale<__nv_bfloat16>(g);
        default: break;  // outputs are never 8-bit
    }
    return PEAK_ERR_INVALID_VALUE;
}

}  // namespace peak
