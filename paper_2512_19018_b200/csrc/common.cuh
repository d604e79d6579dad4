// Shared declarations of the CUDA library: storage types, epilogue arithmetic, launch bookkeeping.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/peak_gemm.h"

namespace peak {

// ---- storage types ---------------------------------------------------------------------------
enum class Elem : int { F16 = 0, BF16 = 1, F32 = 2, E4M3 = 3, E5M2 = 4 };

__host__ __device__ inline Elem in_elem(int dtype) {
    return (dtype == PEAK_F16_F32 || dtype == PEAK_F16_F16)     ? Elem::F16
           : (dtype == PEAK_F32_F32)                           ? Elem::F32
           : (dtype == PEAK_E4M3_BF16 || dtype == PEAK_E4M3_F32) ? Elem::E4M3
           : (dtype == PEAK_E5M2_BF16 || dtype == PEAK_E5M2_F32) ? Elem::E5M2
                                                               : Elem::BF16;
}
__host__ __device__ inline Elem out_elem(int dtype) {
    return (dtype == PEAK_BF16_BF16 || dtype == PEAK_E4M3_BF16 || dtype == PEAK_E5M2_BF16) ? Elem::BF16
           : (dtype == PEAK_F16_F16)                                                       ? Elem::F16
                                                                                           : Elem::F32;
}
__host__ __device__ inline int elem_bytes(Elem e) {
    return e == Elem::F32 ? 4 : (e == Elem::E4M3 || e == Elem::E5M2) ? 1 : 2;
}
__host__ __device__ inline bool is_fp8(Elem e) { return e == Elem::E4M3 || e == Elem::E5M2; }

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__nv_fp8_e4m3 v) { return float(v); }
__device__ __forceinline__ float to_f32(__nv_fp8_e5m2 v) { return float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// The epilogue's arithmetic, in one place: alpha*acc, plus beta*c_old only when beta != 0.
__device__ __forceinline__ float epilogue_f32(float alpha, float acc, float beta, float c_old) {
    float r = alpha * acc;
    if (beta != 0.0f) r = fmaf(beta, c_old, r);
    return r;
}

// Fused epilogue tail: x + bias (one fp32 value per column), then the activation (a peak_activation_t).
__device__ __forceinline__ float activate_f32(float x, int act) {
    if (act == PEAK_ACT_RELU) return fmaxf(x, 0.0f);
    if (act == PEAK_ACT_GELU) return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f));
    return x;
}
__device__ __forceinline__ float finish_f32(float x, const float *bias, int64_t col, int act) {
    if (bias) x += __ldg(bias + col);
    return activate_f32(x, act);
}
// ... and the residual operand, added after the activation (fp32, before the one output rounding)
template <typename T> __device__ __forceinline__ float add_residual(float x, const T *R, int64_t idx) {
    return R ? x + to_f32(R[idx]) : x;
}

// ---- host-side bookkeeping (api.cu owns the definitions) ---------------------------------------
void count_launch(int n = 1);
// Remembers, for this host thread, which kernel the entry point launched last and how (printf-style; the
// kernel's name is written the way profilers print it); read back through peak_last_kernel().
void note_kernel(const char *fmt, ...);
void set_cuda_error(cudaError_t e);
uint32_t *device_status_word();  // address of the per-device status word (nullptr on failure)
int tuning(int key);             // value set through peak_set_tuning (0 = library default)

struct GemmArgs {
    int dtype, transA, transB;
    int64_t M, N, K;
    float alpha, beta;
    const void *A, *B;
    void *C;
    int64_t lda, ldb, ldc;
    cudaStream_t stream;
    const float *bias;  // fused epilogue: one fp32 value per column of C (device), or nullptr
    int act;            // fused epilogue: a peak_activation_t
    int64_t batch;      // strided batch: number of independent problems (0 or 1: a single GEMM)
    int64_t strideA, strideB, strideC;  // elements between consecutive matrices of the batch
    // fused epilogue: residual matrix added after the activation (device, the output's storage type, M x N with
    // pitch ldr), or nullptr
    const void *R = nullptr;
    int64_t ldr = 0;
    int64_t nbatch() const { return batch > 1 ? batch : 1; }
};

// One-time set-up that belongs to a device's context rather than to the process (a kernel's
// cudaFuncAttributeMaxDynamicSharedMemorySize, an occupancy query): done the first time each device runs the
// code, with that device current, and remembered per device.  A process that drives several GPUs therefore
// gets every one of them set up, not just the first.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    std::mutex m;
    bool done[kMaxDevices] = {};
    cudaError_t err[kMaxDevices] = {};
    // Runs fn() once for device `dev` (its later callers get the remembered result).  A device index outside
    // the table is served without memory: fn() runs every time.
    template <typename Fn> cudaError_t run(int dev, Fn fn) {
        if (dev < 0 || dev >= kMaxDevices) return fn();
        std::lock_guard<std::mutex> lock(m);
        if (!done[dev]) {
            err[dev] = fn();
            done[dev] = true;
        }
        return err[dev];
    }
};
inline int current_device() {
    int dev = 0;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// Persisted tuning table (tuned_table.cu): while a TunedScope lives, tuning() answers knobs the caller left at
// 0 from the table entry that covers the problem, and tuned_variant() names the family that entry prefers.
struct TunedScope {
    explicit TunedScope(const GemmArgs &g);
    ~TunedScope();
    TunedScope(const TunedScope &) = delete;
    TunedScope &operator=(const TunedScope &) = delete;
};
int tuned_knob(int key);
int tuned_variant();

// kernel-family launchers; each returns a peak_status_t
int launch_fallback(const GemmArgs &g);
int launch_scale(const GemmArgs &g);
int launch_xcheck_f64(const GemmArgs &g, const void *C0, double *Cref, int64_t ldcref);
int launch_sgemm(const GemmArgs &g);
bool sgemm_supports(const GemmArgs &g);
int launch_sgemm_tma(const GemmArgs &g);        // TMA-fed SGEMM: any shape, 16-byte aligned operands
bool sgemm_tma_supports(const GemmArgs &g);
int launch_umma(const GemmArgs &g, int cta_group);
bool umma_supports(const GemmArgs &g, int cta_group);
int umma_units(int cta_group);  // CTAs (cta_group 1) or CTA pairs (2) a persistent launch can keep resident
bool umma_multicast_available();
cudaMemPool_t scratch_pool();  // per-device stream-ordered pool that keeps its memory (split-K partials, SGEMM transposes)

// status word layout: bit 31 = a bounded wait gave up; bits 0..7 = role, 8..15 = barrier index
constexpr uint32_t kStatusTimeout = 0x80000000u;

// Tile order of the persistent scheduler (also exported on the host as peak_tile_coord).
__host__ __device__ inline void tile_coord(int64_t tile, int64_t tiles_m, int64_t tiles_n, int64_t group,
                                           int64_t &tm, int64_t &tn) {
    if (group < 1) group = 1;
    const int64_t per_group = group * tiles_n;
    const int64_t g = tile / per_group;
    const int64_t first_m = g * group;
    const int64_t rows = (tiles_m - first_m < group) ? (tiles_m - first_m) : group;
    const int64_t r = tile - g * per_group;
    tm = first_m + r % rows;
    tn = r / rows;
}

}  // namespace peak
