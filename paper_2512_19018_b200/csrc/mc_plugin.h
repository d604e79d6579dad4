// Interface between the main library and its optional single-GPU accelerator plug-in
// (libpeak_gemm_mc.so): the tensor-core GEMM run by clusters of four CTAs that share B tiles, and single-CTA tiles
// in clusters that share A and / or B tiles (problems with few tiles).
// Plain C structs and one entry point, so that the two shared objects need nothing else from each other.
//
// Contract: the plug-in is for single-GPU processes.  Its tensor maps must cover memory of the GPU it runs on
// and nothing else; the entry point verifies that A and B are ordinary device allocations of the current
// device (first and last byte of each) and answers PEAK_ERR_UNSUPPORTED otherwise, in which case the main
// library runs its own kernel.  Multi-rank jobs switch the plug-in off (PEAK_TUNE_MULTICAST = 1) and do not
// ship it.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

extern "C" {

struct peak_mc_request {
    int dtype, transA, transB;
    int64_t M, N, K;
    float alpha, beta;
    const void *A, *B;
    void *C;
    int64_t lda, ldb, ldc;
    cudaStream_t stream;
    uint32_t *status;       // the main library's per-device status word
    int raster_group;       // 0 = default
    int epilogue;           // PEAK_TUNE_EPILOGUE value
    int wait_ms;            // PEAK_TUNE_WAIT_MS value
    int dependent_launch;   // PEAK_TUNE_DEPENDENT_LAUNCH value
    int inject_stall;       // PEAK_TUNE_INJECT_STALL value
    int balanced_grid;      // PEAK_TUNE_BALANCED_GRID value
    const float *bias;      // fused epilogue: fp32 value per column (device) or NULL
    int activation;         // fused epilogue: a peak_activation_t
    int epilogue_warps;     // PEAK_TUNE_EPILOGUE_WARPS value
    int tile_n;             // 256 (512 x 256 super-tiles) or 512 (512 x 512 super-tiles of two-half tiles)
    const void *R;          // fused epilogue: residual matrix (output type, device) or NULL
    int64_t ldr;
    int k_order;            // PEAK_TUNE_K_ORDER value
    int share_cm, share_cn; // both 0: CTA-pair tiles as described above; otherwise single-CTA 128 x tile_n tiles (tile_n
                            // 128 or 256) in clusters of share_cm x share_cn tiles that share their A / B tiles
    int cuda_error;         // out: cudaError_t of a failing CUDA call
};

// Returns a peak_status_t.  PEAK_ERR_UNSUPPORTED: the caller should run its own kernel instead.
typedef int (*peak_mc_gemm_fn)(peak_mc_request *req);
int peak_mc_gemm(peak_mc_request *req);
// Four-CTA clusters of the pair kernel (tile_n 256 or 512) the current device holds at once; 0 = unknown.
typedef int (*peak_mc_max_clusters_fn)(int tile_n);
int peak_mc_max_clusters(int tile_n);

}  // extern "C"
