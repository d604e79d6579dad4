// Single-GPU accelerator plug-in: the tensor-core GEMM with cluster-multicast B loads.
//
// Built into its own shared object (libpeak_gemm_mc.so) and loaded by the main library only when present.
// It is kept out of every multi-GPU run: this file is the only place in the repository that issues a
// multicast bulk-tensor copy, and it only ever reads this GPU's own memory (the caller's A and B).
//
// Clusters of four CTAs = two CTA pairs stacked in M work on a 512 x 256 super-tile.  Both pairs need the
// same 256-column B tile for every k-block; each CTA fetches one 64-column quarter of it and the copy engine
// delivers that quarter to the CTA itself and to the CTA of the same parity in the other pair.  L2 reads per
// super-tile k-block drop from 128 KiB to 96 KiB (512 x 512 super-tiles of two-half tiles: from 192 to 128).
// Motivation: one SM's L2 port sustains 40-57 bytes per cycle, a 256 x 256 pair tile asks for 64, and under
// the 1 kW power cap operand traffic is part of the energy budget (measured gains: a few per cent).
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace peak {
namespace umma {
template <int MC> struct McOps;
}
}  // namespace peak

#include "umma_device.cuh"
#include "umma_share_mc.cuh"
#include "umma_host.cuh"
#include "mc_plugin.h"

namespace peak {
namespace umma {

// 64 x 64-element box -> the same shared-memory offset in every CTA of `mask`; completion bytes are
// signalled on the full barrier of each destination's pair leader.
template <> struct McOps<1> {
    __device__ static void load_b_quarter(uint32_t dst, const CUtensorMap *tm, int x, int y, int /*batch: unused, the plug-in runs single GEMMs*/,
                                          uint32_t leader_bar, uint16_t mask) {
        asm volatile(
            "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
            ".multicast::cluster [%0], [%1, {%2, %3}], [%4], %5;"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(leader_bar), "h"(mask)
            : "memory");
    }
};

}  // namespace umma

// The plug-in does not use the main library's bookkeeping; these satisfy common.cuh's declarations.
void count_launch(int) {}
void note_kernel(const char *, ...) {}
void set_cuda_error(cudaError_t) {}
uint32_t *device_status_word() { return nullptr; }
int tuning(int) { return 0; }

namespace {
using namespace umma;

// True when `p` lies in an ordinary device allocation (cudaMalloc, a memory pool) of the CURRENT device.
bool local_device_memory(const void *p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeDevice && at.device == current_device();
}

template <typename TOut, bool G2, int BN = 256, bool IN8 = false> int launch_mc(peak_mc_request *r) {
    constexpr int CG = 2;
    constexpr int BKE = IN8 ? 2 * BK : BK;  // elements per k-block (8-bit inputs: 128 per 128-byte row)
    using C_ = Cfg<CG, BN>;
    auto kernel = umma_gemm_kernel<CG, BN, TOut, 1, false, IN8, G2>;
    const int dev = current_device();
    static PerDeviceOnce attr_once;  // once per device, not per process
    const cudaError_t attr_err = attr_once.run(dev, [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { r->cuda_error = (int)attr_err; return PEAK_ERR_CUDA; }

    const Elem ein = in_elem(r->dtype), eout = out_elem(r->dtype);
    const int a_mn = r->transA ? 1 : 0, b_mn = r->transB ? 0 : 1;
    CUtensorMap tmA, tmB, tmC;
    if (IN8 && (a_mn || b_mn)) return PEAK_ERR_UNSUPPORTED;  // 8-bit operands: K-major only
    bool ok = a_mn ? make_map(&tmA, ein, r->A, r->M, r->K, r->lda, 64, BK) : make_map(&tmA, ein, r->A, r->K, r->M, r->lda, BKE, 128);
    ok = ok && (b_mn ? make_map(&tmB, ein, r->B, r->N, r->K, r->ldb, 64, BK) : make_map(&tmB, ein, r->B, r->K, r->N, r->ldb, BKE, 64));
    if (!ok) return PEAK_ERR_CUDA;

    UmmaParams p;
    p.M = (int)r->M; p.N = (int)r->N; p.K = (int)r->K;
    p.num_kb = (int)((r->K + BKE - 1) / BKE);
    p.tiles_m = (int)((r->M + 4 * BM - 1) / (4 * BM));  // 512-row super-tiles
    p.tiles_n = (int)((r->N + BN - 1) / BN);
    p.group = r->raster_group > 0 ? r->raster_group : 2;  // super-tile rows per raster group (measured best)
    const int tiles = p.tiles_m * p.tiles_n;
    p.tiles_per_batch = tiles; p.stride_c = 0;
    p.full_tiles = tiles; p.tail_splits = 1; p.kb_per_split = p.num_kb; p.total_items = tiles;
    p.a_mn = a_mn; p.b_mn = b_mn;
    const uint32_t fmt = (ein == Elem::BF16 || ein == Elem::E5M2) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(C_::SLOT_N >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);
    p.alpha = r->alpha; p.beta = r->beta;
    p.C = r->C; p.ldc = r->ldc;
    p.bias = r->bias; p.act = r->activation;
    const int ob = elem_bytes(eout);
    p.R = r->R; p.ldr = r->ldr;
    p.r_vec = (r->R && reinterpret_cast<uintptr_t>(r->R) % 16 == 0 && (r->ldr * ob) % 16 == 0) ? 1 : 0;
    p.vec_ok = ((reinterpret_cast<uintptr_t>(r->C) % 16) == 0 && (r->ldc * ob) % 16 == 0) ? 1 : 0;
    p.tma_store = (p.vec_ok && (r->N * ob) % 16 == 0 && r->epilogue != 1) ? 1 : 0;
    tmC = tmA;
    p.c_prefetch = (p.tma_store && r->beta != 0.0f && r->epilogue != 3) ? 1 : 0;
    if (p.tma_store && !make_map(&tmC, eout, r->C, r->N, r->M, r->ldc, 128 / ob, 32)) return PEAK_ERR_CUDA;
    p.k_alternate = r->k_order == 2 ? 1 : 0;
    p.a_boxes = BM / 64; p.stage_tx = (uint32_t)(C_::STAGE_BYTES * CG);  // both CTAs' parts arrive at the leader's barrier
    p.bulk_exchange = 0;
    p.bn_eff = BN; p.slot_eff = C_::SLOT_N; p.hrows_eff = C_::HROWS;
    p.status = r->status;
    p.wait_cycles = r->wait_ms > 0 ? (long long)r->wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.inject_stall = r->inject_stall == 1 ? 1 : 0;

    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(C_::threads(G2));
    cfg.dynamicSmemBytes = C_::SMEM_BYTES;
    cfg.stream = r->stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // how many 4-CTA clusters the device can hold at once (GPC boundaries may leave some SMs out)
    static PerDeviceOnce occ_once;
    static int max_clusters_of[kMaxDevices] = {};
    int queried = 0;
    occ_once.run(dev, [&] {
        cfg.gridDim = dim3(4 * 37);
        int n = 0;
        cudaError_t oe = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
        queried = (oe == cudaSuccess && n > 0) ? n : 32;
        if (dev >= 0 && dev < kMaxDevices) max_clusters_of[dev] = queried;
        return cudaSuccess;
    });
    const int max_clusters = (dev >= 0 && dev < kMaxDevices) ? max_clusters_of[dev] : queried;
    int clusters = max_clusters < tiles ? max_clusters : tiles;
    if (r->balanced_grid != 1) {  // the fewest clusters that finish in the same number of waves
        const int waves = (tiles + clusters - 1) / clusters;
        clusters = (tiles + waves - 1) / waves;
    }
    cfg.gridDim = dim3((unsigned)(clusters * 4));
    cfg.numAttrs = r->dependent_launch == 1 ? 1 : 2;
    CUtensorMap tmW = tmA;
    float *ws = nullptr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, tmW, ws, p);
    if (e != cudaSuccess) { r->cuda_error = (int)e; return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

// Single-CTA tiles in clusters of CM x CN tiles with shared operand tiles (umma_share_mc.cuh).  16-bit inputs.
template <int BN, typename TOut, int CM, int CN> int launch_share(peak_mc_request *r) {
    using C_ = Cfg<1, BN>;
    using S_ = ShareCfg<BN, CM, CN>;
    auto kernel = umma_share_kernel<BN, TOut, CM, CN>;
    const int dev = current_device();
    static PerDeviceOnce attr_once;
    const cudaError_t attr_err = attr_once.run(dev, [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { r->cuda_error = (int)attr_err; return PEAK_ERR_CUDA; }
    const Elem ein = in_elem(r->dtype), eout = out_elem(r->dtype);
    const int a_mn = r->transA ? 1 : 0, b_mn = r->transB ? 0 : 1;
    CUtensorMap tmA, tmB, tmC;
    // one box per operand part: K-major `part` matrix rows of one k-block; MN-major 64 elements of M / N by up to
    // 64 k-rows
    constexpr int A_BOX_K = S_::A_PART < 64 ? S_::A_PART : 64, B_BOX_K = S_::B_PART < 64 ? S_::B_PART : 64;
    bool ok = a_mn ? make_map(&tmA, ein, r->A, r->M, r->K, r->lda, 64, A_BOX_K)
                   : make_map(&tmA, ein, r->A, r->K, r->M, r->lda, BK, S_::A_PART);
    ok = ok && (b_mn ? make_map(&tmB, ein, r->B, r->N, r->K, r->ldb, 64, B_BOX_K)
                     : make_map(&tmB, ein, r->B, r->K, r->N, r->ldb, BK, S_::B_PART));
    if (!ok) return PEAK_ERR_CUDA;

    UmmaParams p = {};
    p.M = (int)r->M; p.N = (int)r->N; p.K = (int)r->K;
    p.num_kb = (int)((r->K + BK - 1) / BK);
    p.tiles_m = (int)((r->M + CM * BM - 1) / (CM * BM));   // super-tiles
    p.tiles_n = (int)((r->N + CN * BN - 1) / (CN * BN));
    p.group = r->raster_group > 0 ? r->raster_group : 16;
    const int super_tiles = p.tiles_m * p.tiles_n;
    p.tiles_per_batch = super_tiles;
    p.full_tiles = super_tiles; p.tail_splits = 1; p.kb_per_split = p.num_kb; p.total_items = super_tiles;
    p.a_mn = a_mn; p.b_mn = b_mn;
    const uint32_t fmt = (ein == Elem::BF16) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    p.alpha = r->alpha; p.beta = r->beta;
    p.C = r->C; p.ldc = r->ldc;
    p.bias = r->bias; p.act = r->activation;
    const int ob = elem_bytes(eout);
    p.R = r->R; p.ldr = r->ldr;
    p.r_vec = (r->R && reinterpret_cast<uintptr_t>(r->R) % 16 == 0 && (r->ldr * ob) % 16 == 0) ? 1 : 0;
    p.vec_ok = ((reinterpret_cast<uintptr_t>(r->C) % 16) == 0 && (r->ldc * ob) % 16 == 0) ? 1 : 0;
    p.tma_store = (p.vec_ok && (r->N * ob) % 16 == 0 && r->epilogue != 1) ? 1 : 0;
    tmC = tmA;
    p.c_prefetch = (p.tma_store && r->beta != 0.0f && r->epilogue != 3) ? 1 : 0;
    if (p.tma_store && !make_map(&tmC, eout, r->C, r->N, r->M, r->ldc, 128 / ob, 32)) return PEAK_ERR_CUDA;
    p.a_boxes = BM / 64; p.stage_tx = (uint32_t)C_::STAGE_BYTES;
    p.status = r->status;
    p.wait_cycles = r->wait_ms > 0 ? (long long)r->wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.inject_stall = r->inject_stall == 1 ? 1 : 0;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(super_tiles * S_::CL));
    cfg.blockDim = dim3(S_::THREADS);
    cfg.dynamicSmemBytes = C_::SMEM_BYTES;
    cfg.stream = r->stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S_::CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = r->dependent_launch == 1 ? 1 : 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, p);
    if (e != cudaSuccess) { r->cuda_error = (int)e; return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <int BN, int CM, int CN> int launch_share_typed(peak_mc_request *r) {
    switch (out_elem(r->dtype)) {
        case Elem::F32: return launch_share<BN, float, CM, CN>(r);
        case Elem::F16: return launch_share<BN, __half, CM, CN>(r);
        case Elem::BF16: return launch_share<BN, __nv_bfloat16, CM, CN>(r);
        default: break;
    }
    return PEAK_ERR_INVALID_VALUE;
}

int run_share(peak_mc_request *r) {
    if (is_fp8(in_elem(r->dtype))) return PEAK_ERR_UNSUPPORTED;
    const int key = r->tile_n * 100 + r->share_cm * 10 + r->share_cn;
    switch (key) {
        case 12812: return launch_share_typed<128, 1, 2>(r);
        case 12814: return launch_share_typed<128, 1, 4>(r);
        case 12821: return launch_share_typed<128, 2, 1>(r);
        case 12822: return launch_share_typed<128, 2, 2>(r);
        case 12824: return launch_share_typed<128, 2, 4>(r);
        case 12841: return launch_share_typed<128, 4, 1>(r);
        case 12842: return launch_share_typed<128, 4, 2>(r);
        case 25612: return launch_share_typed<256, 1, 2>(r);
        case 25614: return launch_share_typed<256, 1, 4>(r);
        case 25621: return launch_share_typed<256, 2, 1>(r);
        case 25622: return launch_share_typed<256, 2, 2>(r);
        default: break;
    }
    return PEAK_ERR_UNSUPPORTED;
}

}  // namespace
}  // namespace peak

extern "C" int peak_mc_gemm(peak_mc_request *r) {
    using namespace peak;
    if (!r) return PEAK_ERR_INVALID_VALUE;
    r->cuda_error = 0;
    if (in_elem(r->dtype) == Elem::F32 || r->M < 1 || r->N < 1 || r->K < 1) return PEAK_ERR_UNSUPPORTED;
    // The multicast loads below may only ever read this GPU's own memory: both operands must be plain device
    // allocations of the current device over their whole extent (first and last byte are looked up); a peer
    // GPU's buffer, managed or host memory sends the caller back to its own kernel.
    {
        const int ib = elem_bytes(in_elem(r->dtype));
        const int64_t a_rows = r->transA ? r->K : r->M, a_cols = r->transA ? r->M : r->K;
        const int64_t b_rows = r->transB ? r->N : r->K, b_cols = r->transB ? r->K : r->N;
        const char *a0 = static_cast<const char *>(r->A), *b0 = static_cast<const char *>(r->B);
        if (!local_device_memory(a0) || !local_device_memory(a0 + ((a_rows - 1) * r->lda + a_cols) * ib - 1) ||
            !local_device_memory(b0) || !local_device_memory(b0 + ((b_rows - 1) * r->ldb + b_cols) * ib - 1))
            return PEAK_ERR_UNSUPPORTED;
    }
    if (r->share_cm > 0 || r->share_cn > 0) return run_share(r);
    // two groups of epilogue warps when the launch is at most two waves of 512 x 256 super-tiles long (the
    // last tile's epilogue is then a visible part of the run time)
    const int64_t super_tiles = ((r->M + 511) / 512) * ((r->N + 255) / 256);
    const bool g2 = r->epilogue_warps ? r->epilogue_warps == 2 : super_tiles <= 64;
    if (is_fp8(in_elem(r->dtype))) {  // 8-bit inputs: 256-wide tiles, bf16 or fp32 output
        switch (out_elem(r->dtype)) {
            case Elem::F32: return g2 ? launch_mc<float, true, 256, true>(r) : launch_mc<float, false, 256, true>(r);
            case Elem::BF16:
                return g2 ? launch_mc<__nv_bfloat16, true, 256, true>(r) : launch_mc<__nv_bfloat16, false, 256, true>(r);
            default: break;
        }
        return PEAK_ERR_INVALID_VALUE;
    }
    if (r->tile_n == 512) {  // two-half tiles: 512 x 512 super-tiles
        switch (out_elem(r->dtype)) {
            case Elem::F32: return launch_mc<float, false, 512>(r);
            case Elem::F16: return launch_mc<__half, false, 512>(r);
            case Elem::BF16: return launch_mc<__nv_bfloat16, false, 512>(r);
            default: break;
        }
        return PEAK_ERR_INVALID_VALUE;
    }
    switch (out_elem(r->dtype)) {
        case Elem::F32: return g2 ? launch_mc<float, true>(r) : launch_mc<float, false>(r);
        case Elem::F16: return g2 ? launch_mc<__half, true>(r) : launch_mc<__half, false>(r);
        case Elem::BF16: return g2 ? launch_mc<__nv_bfloat16, true>(r) : launch_mc<__nv_bfloat16, false>(r);
        default: break;  // outputs are never 8-bit
    }
    return PEAK_ERR_INVALID_VALUE;
}

// How many four-CTA clusters of the pair kernel the current device holds at once (tile_n 256 or 512; 8-bit inputs use
// the same shared-memory footprint as 16-bit ones at 256): the caller compares waves of super-tiles on that many
// clusters with waves of pair tiles on all pairs.  0 = unknown.
extern "C" int peak_mc_max_clusters(int tile_n) {
    using namespace peak;
    using namespace peak::umma;
    static int cached[kMaxDevices][2] = {};
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return 0;
    const int slot = tile_n == 512 ? 1 : 0;
    if (cached[dev][slot] != 0) return cached[dev][slot] > 0 ? cached[dev][slot] : 0;
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(4 * 37);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (slot == 1) {
        using C_ = Cfg<2, 512>;
        auto kernel = umma_gemm_kernel<2, 512, __nv_bfloat16, 1, false, false, false>;
        cfg.blockDim = dim3(C_::threads(false));
        cfg.dynamicSmemBytes = C_::SMEM_BYTES;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
    } else {
        using C_ = Cfg<2, 256>;
        auto kernel = umma_gemm_kernel<2, 256, __nv_bfloat16, 1, false, false, false>;
        cfg.blockDim = dim3(C_::threads(false));
        cfg.dynamicSmemBytes = C_::SMEM_BYTES;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
    }
    if (e != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    cached[dev][slot] = n > 0 ? n : -1;
    return n > 0 ? n : 0;
}
