// The C ABI: argument validation, quick returns, variant selection, the host-buffer entry point and the
// small amount of process state (launch counter, last CUDA error, per-device status word, staging buffers).
#include <atomic>
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace peak {

namespace {
std::atomic<int64_t> g_launches{0};
thread_local int t_last_cuda_error = 0;

// One status word per device, living in the module's own global memory (no allocation).  Kernels OR
// a code into it when a bounded wait gives up; peak_check() reads and clears it.
__device__ uint32_t g_status_word[4];

uint32_t *g_status_ptr[kMaxDevices] = {};
std::mutex g_status_mutex;
}  // namespace

namespace {
std::atomic<int> g_tuning[PEAK_TUNE_COUNT_];
}
int tuning(int key) {
    if (key < 0 || key >= PEAK_TUNE_COUNT_) return 0;
    const int v = g_tuning[key].load(std::memory_order_relaxed);
    return v != 0 ? v : tuned_knob(key);  // what the caller set wins; else the tuning table's entry, if any
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
namespace {
thread_local char t_last_kernel[256] = "";
}
void note_kernel(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_last_kernel, sizeof(t_last_kernel), fmt, ap);
    va_end(ap);
}
void set_cuda_error(cudaError_t e) { t_last_cuda_error = (int)e; }

uint32_t *device_status_word() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_status_word);
        if (e != cudaSuccess) { set_cuda_error(e); return nullptr; }
        g_status_ptr[dev] = static_cast<uint32_t *>(p);
    }
    return g_status_ptr[dev];
}

namespace {

bool valid_dtype(int d) { return d >= PEAK_F16_F32 && d <= PEAK_E5M2_F32; }

// Returns PEAK_OK or PEAK_ERR_INVALID_VALUE; checks only the arguments, touches no device.
int validate(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, const void *A, int64_t lda,
             const void *B, int64_t ldb, float alpha, float beta, const void *C, int64_t ldc) {
    if (!valid_dtype(dtype)) return PEAK_ERR_INVALID_VALUE;
    if ((transA != 0 && transA != 1) || (transB != 0 && transB != 1)) return PEAK_ERR_INVALID_VALUE;
    if (M < 0 || N < 0 || K < 0) return PEAK_ERR_INVALID_VALUE;
    if (lda < 1 || ldb < 1 || ldc < 1) return PEAK_ERR_INVALID_VALUE;
    if (lda < (transA ? M : K) || ldb < (transB ? K : N) || ldc < N) return PEAK_ERR_INVALID_VALUE;
    if (M == 0 || N == 0) return PEAK_OK;
    if (!C) return PEAK_ERR_INVALID_VALUE;
    if (K > 0 && alpha != 0.0f && (!A || !B)) return PEAK_ERR_INVALID_VALUE;
    (void)beta;
    return PEAK_OK;
}

// The dispatcher's choice, as a peak_variant_t (arguments already validated).
int choose_variant(const GemmArgs &g) {
    if (g.M == 0 || g.N == 0) return PEAK_VARIANT_NONE;
    const bool fused = g.bias != nullptr || g.act != PEAK_ACT_NONE || g.R != nullptr;
    if (g.K == 0 || g.alpha == 0.0f) return (g.beta == 1.0f && !fused) ? PEAK_VARIANT_NONE : PEAK_VARIANT_SCALE;
    if (in_elem(g.dtype) == Elem::F32) return sgemm_supports(g) ? PEAK_VARIANT_SGEMM : PEAK_VARIANT_FALLBACK;
    // CTA pairs (256-row tiles, B shared between the two SMs) win whenever there is more than one
    // 128-row block of C (a single block of rows would leave the second CTA of each pair idle) and enough
    // tiles: a problem whose 256 x 256 pair tiles would occupy at most half of the SM pairs runs as
    // single-CTA tiles instead, which spread it over up to four times as many SMs (measured 6-13 % faster
    // from 512^3 to 1536^3, 1024x2048x1024, 256x4096x4096).
    const int tv = tuned_variant();  // the tuning table's preference, honoured when that family can run the problem
    if ((tv == PEAK_VARIANT_UMMA_1CTA || tv == PEAK_VARIANT_UMMA_2CTA) && umma_supports(g, tv == PEAK_VARIANT_UMMA_2CTA ? 2 : 1) &&
        (tv == PEAK_VARIANT_UMMA_1CTA || g.M > 128))
        return tv;
    // More than a wave of tiles with at most four k-blocks each (eight when the epilogue also reads C): the epilogue
    // bounds the launch, and single-CTA tiles -- CTA-local barriers between the epilogue warps and the MMA issuer, two
    // accumulator slots -- drain faster than pairs, whose smaller operand traffic buys nothing there (bf16, us, single /
    // pair tiles / cuBLAS: 8192x8192x64 26.0 / 33.5 / 26.7, x128 29.1 / 36.6 / 31.8, x256 41.2 / 46.1 / 40.9;
    // x512 72 / 63 with beta = 0 but 91 / 100 with beta = 1).
    if (umma_supports(g, 1) && g.M > 128) {
        const int64_t pair_tiles = ((g.M + 255) / 256) * ((g.N + 255) / 256) * g.nbatch();
        const int64_t num_kb = (g.K + (is_fp8(in_elem(g.dtype)) ? 127 : 63)) / (is_fp8(in_elem(g.dtype)) ? 128 : 64);
        if (pair_tiles > umma_units(2) && (num_kb <= 4 || (num_kb <= 8 && g.beta != 0.0f))) return PEAK_VARIANT_UMMA_1CTA;
    }
    if (umma_supports(g, 2) && g.M > 128) {
        const int64_t pair_tiles = ((g.M + 255) / 256) * ((g.N + 255) / 256) * g.nbatch();
        if (2 * pair_tiles > umma_units(2) || !umma_supports(g, 1)) return PEAK_VARIANT_UMMA_2CTA;
    }
    if (umma_supports(g, 1)) return PEAK_VARIANT_UMMA_1CTA;
    return PEAK_VARIANT_FALLBACK;
}

int check_arch() {
    static int result[kMaxDevices];
    static bool init = false;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return PEAK_ERR_ARCH;
    static std::mutex m;
    std::lock_guard<std::mutex> lock(m);
    if (!init) { for (int i = 0; i < kMaxDevices; ++i) result[i] = -1; init = true; }
    if (result[dev] < 0) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
        result[dev] = (major == 10) ? PEAK_OK : PEAK_ERR_ARCH;
    }
    return result[dev];
}

int run_variant(int variant, const GemmArgs &g) {
    switch (variant) {
        case PEAK_VARIANT_NONE: return PEAK_OK;
        case PEAK_VARIANT_SCALE: return launch_scale(g);
        case PEAK_VARIANT_FALLBACK: return launch_fallback(g);
        case PEAK_VARIANT_SGEMM: return launch_sgemm(g);
        case PEAK_VARIANT_UMMA_1CTA: return launch_umma(g, 1);
        case PEAK_VARIANT_UMMA_2CTA: return launch_umma(g, 2);
    }
    return PEAK_ERR_INVALID_VALUE;
}

int gemm_impl(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
              const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, void *stream,
              const float *bias = nullptr, int act = PEAK_ACT_NONE, const void *R = nullptr, int64_t ldr = 0) {
    t_last_cuda_error = 0;
    int rc = validate(dtype, transA, transB, M, N, K, A, lda, B, ldb, alpha, beta, C, ldc);
    if (rc != PEAK_OK) return rc;
    if (variant < PEAK_VARIANT_AUTO || variant > PEAK_VARIANT_NONE) return PEAK_ERR_INVALID_VALUE;
    if (act < PEAK_ACT_NONE || act > PEAK_ACT_GELU) return PEAK_ERR_INVALID_VALUE;
    if (R && ldr < N) return PEAK_ERR_INVALID_VALUE;
    GemmArgs g{dtype, transA, transB, M, N, K, alpha, beta, A, B, C, lda, ldb, ldc, (cudaStream_t)stream, bias, act};
    g.R = R;
    g.ldr = ldr;
    TunedScope tuned(g);
    const int chosen = choose_variant(g);
    int v = chosen;
    if (variant != PEAK_VARIANT_AUTO && chosen != PEAK_VARIANT_NONE && chosen != PEAK_VARIANT_SCALE) {
        if (variant == PEAK_VARIANT_NONE || variant == PEAK_VARIANT_SCALE) return PEAK_ERR_UNSUPPORTED;
        v = variant;
    }
    if (v == PEAK_VARIANT_NONE) return PEAK_OK;
    rc = check_arch();
    if (rc != PEAK_OK) return rc;
    return run_variant(v, g);
}

// ---- staging buffers for the host-buffer entry point ------------------------------------------------
struct Staging {
    void *ptr = nullptr;
    size_t bytes = 0;
    int device = -1;  // the device the buffer lives on
};
Staging g_stage_of[kMaxDevices][3];  // per device: a process may call from several GPUs in turn

// Streams and events of the host-buffer entry point's copy / compute pipeline (created on first use, for the
// device that is current then; guarded by g_stage_mutex like the staging buffers).
constexpr int kHostPanels = 8;
struct HostPipeline {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, out_done = nullptr, in_done[kHostPanels] = {}, mm_done[kHostPanels] = {};
    int device = -1;
};
HostPipeline g_pipe_of[kMaxDevices];
std::mutex g_stage_mutex;

int ensure(Staging &s, size_t need) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (need <= s.bytes && (s.device == dev || s.bytes == 0)) return PEAK_OK;
    if (s.ptr) { cudaFree(s.ptr); s.ptr = nullptr; s.bytes = 0; }  // too small, or on another device
    if (need == 0) return PEAK_OK;
    e = cudaMalloc(&s.ptr, need);
    if (e != cudaSuccess) { set_cuda_error(e); s.ptr = nullptr; return PEAK_ERR_NO_MEMORY; }
    s.bytes = need;
    s.device = dev;
    return PEAK_OK;
}

void release_pipeline(HostPipeline &g_pipe) {
    if (g_pipe.in) cudaStreamDestroy(g_pipe.in);
    if (g_pipe.out) cudaStreamDestroy(g_pipe.out);
    if (g_pipe.start) cudaEventDestroy(g_pipe.start);
    if (g_pipe.out_done) cudaEventDestroy(g_pipe.out_done);
    for (int i = 0; i < kHostPanels; ++i) {
        if (g_pipe.in_done[i]) cudaEventDestroy(g_pipe.in_done[i]);
        if (g_pipe.mm_done[i]) cudaEventDestroy(g_pipe.mm_done[i]);
    }
    g_pipe = HostPipeline{};
}

int ensure_pipeline(HostPipeline &g_pipe, int dev) {
    cudaError_t e = cudaSuccess;
    if (g_pipe.in && g_pipe.device == dev) return PEAK_OK;
    release_pipeline(g_pipe);
    e = cudaStreamCreateWithFlags(&g_pipe.in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&g_pipe.out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g_pipe.start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g_pipe.out_done, cudaEventDisableTiming);
    for (int i = 0; i < kHostPanels && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&g_pipe.in_done[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g_pipe.mm_done[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) { set_cuda_error(e); release_pipeline(g_pipe); return PEAK_ERR_CUDA; }
    g_pipe.device = dev;
    return PEAK_OK;
}

size_t span_bytes(int64_t rows, int64_t cols, int64_t ld, int eb) {
    if (rows <= 0 || cols <= 0) return 0;
    return (size_t)((rows - 1) * ld + cols) * (size_t)eb;
}

}  // namespace
}  // namespace peak

using namespace peak;

extern "C" {

int peak_gemm(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
              int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, void *stream) {
    return gemm_impl(PEAK_VARIANT_AUTO, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream);
}

int peak_gemm_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                      const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc,
                      void *stream) {
    return gemm_impl(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream);
}

int peak_gemm_fused(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                    int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, const float *bias,
                    int activation, void *stream) {
    return gemm_impl(PEAK_VARIANT_AUTO, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream, bias,
                     activation);
}

int peak_gemm_fused_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                            const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc,
                            const float *bias, int activation, void *stream) {
    return gemm_impl(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream, bias,
                     activation);
}

int peak_gemm_fused_residual(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                             int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, const float *bias,
                             int activation, const void *R, int64_t ldr, void *stream) {
    return gemm_impl(PEAK_VARIANT_AUTO, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream, bias,
                     activation, R, ldr);
}

int peak_gemm_fused_residual_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K,
                                     float alpha, const void *A, int64_t lda, const void *B, int64_t ldb, float beta,
                                     void *C, int64_t ldc, const float *bias, int activation, const void *R, int64_t ldr,
                                     void *stream) {
    return gemm_impl(variant, dtype, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, stream, bias,
                     activation, R, ldr);
}

int peak_gemm_strided_batched(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                              const void *A, int64_t lda, int64_t strideA, const void *B, int64_t ldb, int64_t strideB,
                              float beta, void *C, int64_t ldc, int64_t strideC, int64_t batch, void *stream) {
    t_last_cuda_error = 0;
    int rc = validate(dtype, transA, transB, M, N, K, A, lda, B, ldb, alpha, beta, C, ldc);
    if (rc != PEAK_OK) return rc;
    if (batch < 0 || strideA < 0 || strideB < 0 || strideC < 0) return PEAK_ERR_INVALID_VALUE;
    if (batch > 1 && M > 0 && N > 0 && strideC < (M - 1) * ldc + N) return PEAK_ERR_INVALID_VALUE;  // C matrices overlap
    if (batch == 0) return PEAK_OK;
    GemmArgs g{dtype, transA, transB, M, N, K, alpha, beta, A, B, C, lda, ldb, ldc, (cudaStream_t)stream, nullptr,
               PEAK_ACT_NONE, batch, strideA, strideB, strideC};
    const int v = choose_variant(g);
    if (v == PEAK_VARIANT_NONE) return PEAK_OK;
    rc = check_arch();
    if (rc != PEAK_OK) return rc;
    if (v == PEAK_VARIANT_UMMA_1CTA || v == PEAK_VARIANT_UMMA_2CTA) {
        rc = run_variant(v, g);  // one launch: the batch index is the third coordinate of the tensor maps
        if (rc != PEAK_ERR_UNSUPPORTED) return rc;
    }
    // every other kernel family: one launch per matrix
    const int ib = elem_bytes(in_elem(dtype)), ob = elem_bytes(out_elem(dtype));
    for (int64_t b = 0; b < batch; ++b) {
        GemmArgs gb = g;
        gb.batch = 0;
        gb.A = A ? static_cast<const char *>(A) + b * strideA * ib : nullptr;
        gb.B = B ? static_cast<const char *>(B) + b * strideB * ib : nullptr;
        gb.C = static_cast<char *>(C) + b * strideC * ob;
        rc = run_variant(choose_variant(gb), gb);
        if (rc != PEAK_OK) return rc;
    }
    return PEAK_OK;
}

int peak_gemm_host(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                   int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, void *stream) {
    t_last_cuda_error = 0;
    int rc = validate(dtype, transA, transB, M, N, K, A, lda, B, ldb, alpha, beta, C, ldc);
    if (rc != PEAK_OK) return rc;
    if (M == 0 || N == 0) return PEAK_OK;
    rc = check_arch();
    if (rc != PEAK_OK) return rc;
    const int ib = elem_bytes(in_elem(dtype)), ob = elem_bytes(out_elem(dtype));
    const bool need_ab = (K > 0 && alpha != 0.0f);
    const size_t a_bytes = need_ab ? span_bytes(transA ? K : M, transA ? M : K, lda, ib) : 0;
    const size_t b_bytes = need_ab ? span_bytes(transB ? N : K, transB ? K : N, ldb, ib) : 0;
    const size_t c_bytes = span_bytes(M, N, ldc, ob);
    cudaStream_t st = (cudaStream_t)stream;
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return PEAK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_stage_mutex);
    Staging *g_stage = g_stage_of[dev];
    HostPipeline &g_pipe = g_pipe_of[dev];
    if ((rc = ensure(g_stage[0], a_bytes)) || (rc = ensure(g_stage[1], b_bytes)) || (rc = ensure(g_stage[2], c_bytes)))
        return rc;
    // C travels to the device when its old values are needed, or when the pitch leaves gaps that the
    // copy back would otherwise overwrite with stale staging contents
    const bool c_in = beta != 0.0f || ldc != N;
    char *dA = static_cast<char *>(g_stage[0].ptr), *dB = static_cast<char *>(g_stage[1].ptr),
         *dC = static_cast<char *>(g_stage[2].ptr);
    const char *hA = static_cast<const char *>(A);
    char *hC = static_cast<char *>(C);
    cudaError_t e = cudaSuccess;
    auto fail = [&](cudaError_t err) { set_cuda_error(err); return (int)PEAK_ERR_CUDA; };

    // Row panels of op(A) and C: the copy engines bring panel i + 1 in and take panel i - 1 out while the SMs
    // multiply panel i.  Copies in run on one internal stream (B first, then the panels in order), the
    // products on the caller's stream, copies out on a second internal stream; events order them.
    const int64_t panels = need_ab ? std::max<int64_t>(1, std::min<int64_t>(kHostPanels, M / 512)) : 1;
    if (panels > 1 && (rc = ensure_pipeline(g_pipe, dev)) != PEAK_OK) return rc;
    if (panels == 1) {
        if (a_bytes) e = cudaMemcpyAsync(dA, A, a_bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && b_bytes) e = cudaMemcpyAsync(dB, B, b_bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess && c_in) e = cudaMemcpyAsync(dC, C, c_bytes, cudaMemcpyHostToDevice, st);
        // on any error the stream is still drained, so that no copy uses the caller's buffers after the return
        if (e == cudaSuccess)
            rc = gemm_impl(PEAK_VARIANT_AUTO, dtype, transA, transB, M, N, K, alpha, dA, lda, dB, ldb, beta, dC, ldc, stream);
        const int rc_cuda = peak_last_cuda_error();
        if (e == cudaSuccess && rc == PEAK_OK) e = cudaMemcpyAsync(C, dC, c_bytes, cudaMemcpyDeviceToHost, st);
        const cudaError_t es = cudaStreamSynchronize(st);
        if (rc != PEAK_OK) { t_last_cuda_error = rc_cuda; return rc; }
        if (e != cudaSuccess) return fail(e);
        if (es != cudaSuccess) return fail(es);
        return PEAK_OK;
    }
    cudaStream_t s_in = g_pipe.in, s_out = g_pipe.out;
    // the internal streams start after whatever the caller's stream already holds
    // Nothing is in flight on the internal streams yet, so a failure here may return at once; from the first
    // copy on, every failure leaves the loop into the common tail below, which drains all three streams.
    if ((e = cudaEventRecord(g_pipe.start, st)) != cudaSuccess) return fail(e);
    if ((e = cudaStreamWaitEvent(s_in, g_pipe.start, 0)) != cudaSuccess) return fail(e);
    if ((e = cudaStreamWaitEvent(s_out, g_pipe.start, 0)) != cudaSuccess) return fail(e);
    e = cudaMemcpyAsync(dB, B, b_bytes, cudaMemcpyHostToDevice, s_in);
    const int64_t rows_per = ((M + panels - 1) / panels + 127) / 128 * 128;  // whole 128-row tiles per panel
    int rc_cuda = 0;
    for (int64_t i = 0; i < panels && e == cudaSuccess; ++i) {
        const int64_t m0 = i * rows_per, mp = std::min(rows_per, M - m0);
        if (mp <= 0) break;
        const size_t c_off = (size_t)m0 * (size_t)ldc * (size_t)ob;
        const size_t c_len = span_bytes(mp, N, ldc, ob);
        if (!transA) {  // rows m0 .. m0 + mp of a row-major M x K matrix: one contiguous span
            const size_t off = (size_t)m0 * (size_t)lda * (size_t)ib;
            e = cudaMemcpyAsync(dA + off, hA + off, span_bytes(mp, K, lda, ib), cudaMemcpyHostToDevice, s_in);
        } else {        // columns m0 .. m0 + mp of the stored K x M matrix: a strided copy
            const size_t off = (size_t)m0 * (size_t)ib;
            e = cudaMemcpy2DAsync(dA + off, (size_t)lda * ib, hA + off, (size_t)lda * ib, (size_t)mp * ib, (size_t)K,
                                  cudaMemcpyHostToDevice, s_in);
        }
        if (e == cudaSuccess && c_in) e = cudaMemcpyAsync(dC + c_off, hC + c_off, c_len, cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaEventRecord(g_pipe.in_done[i], s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, g_pipe.in_done[i], 0);
        if (e != cudaSuccess) break;
        const char *a_panel = transA ? dA + (size_t)m0 * ib : dA + (size_t)m0 * (size_t)lda * ib;
        rc = gemm_impl(PEAK_VARIANT_AUTO, dtype, transA, transB, mp, N, K, alpha, a_panel, lda, dB, ldb, beta, dC + c_off,
                       ldc, stream);
        if (rc != PEAK_OK) { rc_cuda = peak_last_cuda_error(); break; }
        if ((e = cudaEventRecord(g_pipe.mm_done[i], st)) != cudaSuccess) break;
        if ((e = cudaStreamWaitEvent(s_out, g_pipe.mm_done[i], 0)) != cudaSuccess) break;
        e = cudaMemcpyAsync(hC + c_off, dC + c_off, c_len, cudaMemcpyDeviceToHost, s_out);
    }
    // everything rejoins the caller's stream, and all three streams are drained -- also after a refused product
    // or a failed CUDA call, so that no copy is still in flight when the caller gets its buffers back
    cudaError_t e1 = cudaEventRecord(g_pipe.out_done, s_out);
    if (e1 == cudaSuccess) e1 = cudaStreamWaitEvent(st, g_pipe.out_done, 0);
    cudaError_t e2 = cudaStreamSynchronize(s_in);
    cudaError_t e4 = cudaStreamSynchronize(s_out);
    cudaError_t e3 = cudaStreamSynchronize(st);
    if (rc != PEAK_OK) { t_last_cuda_error = rc_cuda; return rc; }
    if (e != cudaSuccess) return fail(e);
    if (e4 != cudaSuccess) return fail(e4);
    if (e1 != cudaSuccess) return fail(e1);
    if (e2 != cudaSuccess) return fail(e2);
    if (e3 != cudaSuccess) return fail(e3);
    return PEAK_OK;
}

int peak_release_staging(void) {
    std::lock_guard<std::mutex> lock(g_stage_mutex);
    int prev = -1;
    cudaGetDevice(&prev);
    for (int dev = 0; dev < kMaxDevices; ++dev) {
        bool any = g_pipe_of[dev].in != nullptr;
        for (auto &s : g_stage_of[dev]) any = any || s.ptr != nullptr;
        if (!any) continue;
        cudaSetDevice(dev);  // buffers, streams and events are released with their own device current
        for (auto &s : g_stage_of[dev]) {
            if (s.ptr) cudaFree(s.ptr);
            s.ptr = nullptr;
            s.bytes = 0;
        }
        release_pipeline(g_pipe_of[dev]);
    }
    if (prev >= 0) cudaSetDevice(prev);
    return PEAK_OK;
}

int peak_gemm_xcheck_f64(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                         const void *A, int64_t lda, const void *B, int64_t ldb, float beta, const void *C0,
                         int64_t ldc, double *Cref, int64_t ldcref, void *stream) {
    t_last_cuda_error = 0;
    int rc = validate(dtype, transA, transB, M, N, K, A, lda, B, ldb, 1.0f, beta, Cref, ldc);
    if (rc != PEAK_OK) return rc;
    if (ldcref < N || (K > 0 && (!A || !B) && M > 0 && N > 0)) return PEAK_ERR_INVALID_VALUE;
    if (beta != 0.0f && !C0 && M > 0 && N > 0) return PEAK_ERR_INVALID_VALUE;
    if (M == 0 || N == 0) return PEAK_OK;
    rc = check_arch();
    if (rc != PEAK_OK) return rc;
    GemmArgs g{dtype, transA, transB, M, N, K, alpha, beta, A, B, nullptr, lda, ldb, ldc, (cudaStream_t)stream};
    return launch_xcheck_f64(g, C0, Cref, ldcref);
}

int peak_query_variant(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                       const void *A, int64_t lda, const void *B, int64_t ldb, float beta, const void *C,
                       int64_t ldc) {
    int rc = validate(dtype, transA, transB, M, N, K, A, lda, B, ldb, alpha, beta, C, ldc);
    if (rc != PEAK_OK) return -rc;
    GemmArgs g{dtype, transA, transB, M, N, K, alpha, beta, A, B, const_cast<void *>(C), lda, ldb, ldc, nullptr};
    TunedScope tuned(g);
    return choose_variant(g);
}

int peak_tile_coord(int64_t tile, int64_t tiles_m, int64_t tiles_n, int64_t group, int64_t *tile_m,
                    int64_t *tile_n) {
    if (tiles_m < 1 || tiles_n < 1 || tile < 0 || tile >= tiles_m * tiles_n || !tile_m || !tile_n)
        return PEAK_ERR_INVALID_VALUE;
    tile_coord(tile, tiles_m, tiles_n, group, *tile_m, *tile_n);
    return PEAK_OK;
}

int peak_check(void *stream, uint32_t *detail) {
    t_last_cuda_error = 0;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    uint32_t *w = device_status_word();
    if (!w) return PEAK_ERR_CUDA;
    uint32_t host = 0, zero = 0;
    e = cudaMemcpy(&host, w, sizeof(host), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && host != 0) e = cudaMemcpy(w, &zero, sizeof(zero), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (detail) *detail = host;
    return (host & kStatusTimeout) ? PEAK_ERR_TIMEOUT : PEAK_OK;
}

int peak_set_tuning(int key, int value) {
    if (key < 0 || key >= PEAK_TUNE_COUNT_ || value < 0) return PEAK_ERR_INVALID_VALUE;
    g_tuning[key].store(value, std::memory_order_relaxed);
    return PEAK_OK;
}

int peak_multicast_available(void) { return umma_multicast_available() ? 1 : 0; }

int64_t peak_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int peak_last_cuda_error(void) { return t_last_cuda_error; }

int peak_last_kernel(char *buf, size_t len) {
    if (!buf || len == 0) return PEAK_ERR_INVALID_VALUE;
    strncpy(buf, t_last_kernel, len - 1);
    buf[len - 1] = '\0';
    return PEAK_OK;
}

int peak_selftest_per_device_once(void) {
    // host-only check of the once-per-device bookkeeping behind the kernels' context set-up
    PerDeviceOnce once;
    int calls[4] = {0, 0, 0, 0};
    auto run = [&](int dev, cudaError_t result) {
        return once.run(dev, [&] { ++calls[dev < 0 || dev > 2 ? 3 : dev]; return result; });
    };
    if (run(0, cudaSuccess) != cudaSuccess || run(0, cudaErrorUnknown) != cudaSuccess || calls[0] != 1) return 1;
    if (run(1, cudaErrorInvalidValue) != cudaErrorInvalidValue || calls[1] != 1) return 2;  // device 1 set up itself
    if (run(1, cudaSuccess) != cudaErrorInvalidValue || calls[1] != 1) return 3;            // and its result is kept
    if (run(2, cudaSuccess) != cudaSuccess || calls[2] != 1 || calls[0] != 1) return 4;
    if (run(kMaxDevices - 1, cudaSuccess) != cudaSuccess) return 5;
    run(-1, cudaSuccess); run(-1, cudaSuccess); run(kMaxDevices, cudaSuccess);  // outside the table: no memory
    if (calls[3] != 4) return 6;
    return 0;
}

const char *peak_status_string(int status) {
    switch (status) {
        case PEAK_OK: return "ok";
        case PEAK_ERR_INVALID_VALUE: return "invalid value";
        case PEAK_ERR_ARCH: return "device is not compute capability 10.x (B200)";
        case PEAK_ERR_CUDA: return "CUDA call failed";
        case PEAK_ERR_UNSUPPORTED: return "variant does not support this problem";
        case PEAK_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case PEAK_ERR_NO_MEMORY: return "out of device memory for staging or workspace";
        case PEAK_ERR_WORKSPACE_TOO_SMALL: return "partial tiles exceed the fixed workspace of peak_gemm_static_ws";
    }
    return "unknown status";
}

const char *peak_variant_string(int variant) {
    switch (variant) {
        case PEAK_VARIANT_AUTO: return "auto";
        case PEAK_VARIANT_FALLBACK: return "fallback";
        case PEAK_VARIANT_UMMA_1CTA: return "umma_1cta";
        case PEAK_VARIANT_UMMA_2CTA: return "umma_2cta";
        case PEAK_VARIANT_SGEMM: return "sgemm";
        case PEAK_VARIANT_SCALE: return "scale";
        case PEAK_VARIANT_NONE: return "none";
    }
    return "unknown variant";
}

int peak_version(void) { return 100; }

}  // extern "C"
