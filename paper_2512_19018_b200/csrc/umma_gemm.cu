// Tensor-core GEMM for 16-bit inputs on sm_100a.
//
// One persistent CTA (or CTA pair) per SM walks output tiles in a grouped order (the paper's block
// swizzle).  Inside a CTA three roles run concurrently (warp specialisation):
//   warp 0      producer: TMA tile loads of A and B into a ring of 128-byte-swizzled shared-memory stages
//               (the paper's thread-block tiling + pipelining + bank-conflict offset, section 2.2),
//   warp 1      one thread issues tcgen05.mma; fp32 accumulators live in tensor memory (the paper's
//               warp tiling / tensor-core steps), two accumulator buffers so that the next tile's main
//               loop overlaps this tile's epilogue,
//   warps 2..5  epilogue: tcgen05.ld -> alpha/beta in fp32 -> one rounding -> vectorised global stores.
// mbarriers connect the roles (full/empty per stage, full/empty per accumulator).  Every wait is bounded.
//
// Tile: 128 x 256 x 64 per CTA (CTA_GROUP 1) or 256 x 256 x 64 per CTA pair (CTA_GROUP 2, each CTA stages
// its 128 rows of A and its 128-column half of B; the leader CTA issues MMAs for both).
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace peak {
namespace {

constexpr int BM = 128;   // rows of C per CTA
constexpr int BN = 256;   // columns of C per tile
constexpr int BK = 64;    // k-block: 64 16-bit elements = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;  // 16 KiB
constexpr int ATOM_BYTES = 64 * BK * 2;     // one 64-wide MN-major box: 64 k-rows of 128 bytes = 8 KiB
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;              // two 256-column fp32 accumulators

template <int CG> struct Cfg {
    static constexpr int B_ROWS = BN / CG;                 // rows of op(B)^T this CTA stages
    static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;  // 32 KiB or 16 KiB
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES = (CG == 1) ? 4 : 6;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct UmmaParams {
    int M, N, K;
    int num_kb;            // ceil(K / BK)
    int tiles_m, tiles_n;  // in units of (128*CG) x 256
    int group;             // tile-rows per raster group
    int a_mn, b_mn;        // 1: operand is MN-major in memory (transA == 1 / transB == 0)
    uint32_t idesc;
    float alpha, beta;
    void *C;
    int64_t ldc;
    int vec_ok;            // C base and pitch allow 16-byte vector access
    uint32_t *status;
};

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// descriptor version 1 (sm_100), 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void report_timeout(const UmmaParams &p, volatile uint32_t *abort_flag, uint32_t role,
                                               uint32_t which) {
    if (*abort_flag == 0) atomicOr(p.status, kStatusTimeout | (which << 8) | role);
    *abort_flag = 1;
}

template <typename TOut>
__device__ __forceinline__ void store_row_chunk(TOut *dst, const float (&v)[32], int valid, bool vec) {
    if (vec && valid == 32) {
        if constexpr (sizeof(TOut) == 4) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                reinterpret_cast<float4 *>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    TOut lo = from_f32<TOut>(v[8 * i + 2 * j]), hi = from_f32<TOut>(v[8 * i + 2 * j + 1]);
                    w[j] = (uint32_t)(*reinterpret_cast<uint16_t *>(&lo)) |
                           ((uint32_t)(*reinterpret_cast<uint16_t *>(&hi)) << 16);
                }
                reinterpret_cast<uint4 *>(dst)[i] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < valid) dst[i] = from_f32<TOut>(v[i]);
    }
}

template <typename TOut>
__device__ __forceinline__ void load_row_chunk(const TOut *src, float (&c)[32], int valid, bool vec) {
    if (vec && valid == 32) {
        if constexpr (sizeof(TOut) == 4) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 t = reinterpret_cast<const float4 *>(src)[i];
                c[4 * i] = t.x; c[4 * i + 1] = t.y; c[4 * i + 2] = t.z; c[4 * i + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 t = reinterpret_cast<const uint4 *>(src)[i];
                uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint16_t lo = (uint16_t)(w[j] & 0xffffu), hi = (uint16_t)(w[j] >> 16);
                    c[8 * i + 2 * j] = to_f32(*reinterpret_cast<TOut *>(&lo));
                    c[8 * i + 2 * j + 1] = to_f32(*reinterpret_cast<TOut *>(&hi));
                }
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) c[i] = (i < valid) ? to_f32(src[i]) : 0.0f;
    }
}

template <int CG, typename TOut>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const UmmaParams p) {
    using C_ = Cfg<CG>;
    constexpr int STAGES = C_::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t stage_base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    uint8_t *aux = smem_raw + (stage_base - raw) + STAGES * C_::STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aux);  // full[S], empty[S], acc_full[2], acc_empty[2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 8 * (2 * STAGES + 4));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const uint32_t full0 = ptx::smem_u32(bars);
    const uint32_t empty0 = full0 + 8 * STAGES;
    const uint32_t accfull0 = empty0 + 8 * STAGES;
    const uint32_t accempty0 = accfull0 + 16;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;
    const bool leader = (rank == 0);
    const int unit = blockIdx.x / CG;          // CTA (or CTA pair) index
    const int num_units = gridDim.x / CG;
    const int total_tiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(accfull0 + 8 * b, 1);
            ptx::mbar_init(accempty0 + 8 * b, 4 * CG);  // one arrival per epilogue warp of every CTA
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0 && lane == 0) {
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        ptx::tmem_alloc<CG>(ptx::smem_u32(tmem_slot), TMEM_COLS);
        ptx::tmem_relinquish<CG>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (CG == 2) ptx::cluster_sync();  // the peer's barriers must be initialised before anything signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
                int64_t tm, tn;
                tile_coord(tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
                const int m_cta = (int)tm * (BM * CG) + (int)rank * BM;
                const int n_cta = (int)tn * BN + (int)rank * C_::B_ROWS;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag)) {
                        report_timeout(p, abort_flag, 1, s);
                        ok = false;
                        break;
                    }
                    uint32_t bar = full0 + 8 * s;
                    if (leader) ptx::mbar_arrive_expect_tx(bar, (uint32_t)(C_::STAGE_BYTES * CG));
                    if (CG == 2) bar = ptx::map_to_cta(bar, 0);
                    const uint32_t a_dst = stage_base + s * C_::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + A_STAGE_BYTES;
                    const int k0 = kb * BK;
                    if (!p.a_mn) {
                        if (CG == 1) ptx::tma_load_2d(a_dst, &tmA, k0, m_cta, bar);
                        else ptx::tma_load_2d_pair(a_dst, &tmA, k0, m_cta, bar);
                    } else {
#pragma unroll
                        for (int h = 0; h < BM / 64; ++h) {
                            if (CG == 1) ptx::tma_load_2d(a_dst + h * ATOM_BYTES, &tmA, m_cta + 64 * h, k0, bar);
                            else ptx::tma_load_2d_pair(a_dst + h * ATOM_BYTES, &tmA, m_cta + 64 * h, k0, bar);
                        }
                    }
                    if (!p.b_mn) {
#pragma unroll
                        for (int h = 0; h < C_::B_ROWS / 128; ++h) {
                            if (CG == 1) ptx::tma_load_2d(b_dst + h * 128 * 128, &tmB, k0, n_cta + 128 * h, bar);
                            else ptx::tma_load_2d_pair(b_dst + h * 128 * 128, &tmB, k0, n_cta + 128 * h, bar);
                        }
                    } else {
#pragma unroll
                        for (int h = 0; h < C_::B_ROWS / 64; ++h) {
                            if (CG == 1) ptx::tma_load_2d(b_dst + h * ATOM_BYTES, &tmB, n_cta + 64 * h, k0, bar);
                            else ptx::tma_load_2d_pair(b_dst + h * ATOM_BYTES, &tmB, n_cta + 64 * h, k0, bar);
                        }
                    }
                }
            }
            // tail: every stage this CTA filled must have been released before the CTA may exit
            for (int j = 0; j < STAGES && ok; ++j, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                if (!ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag)) {
                    report_timeout(p, abort_flag, 2, s);
                    ok = false;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && leader) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            const uint32_t a_lbo = p.a_mn ? (uint32_t)ATOM_BYTES : 16u, b_lbo = p.b_mn ? (uint32_t)ATOM_BYTES : 16u;
            const uint32_t a_kstep = p.a_mn ? 2048u : 32u, b_kstep = p.b_mn ? 2048u : 32u;
            for (int tile = unit; tile < total_tiles && ok; tile += num_units, ++tl) {
                const uint32_t b = tl & 1u, aph = (tl >> 1) & 1u;
                if (!ptx::mbar_wait<CG == 2>(accempty0 + 8 * b, aph ^ 1u, abort_flag)) {
                    report_timeout(p, abort_flag, 3, b);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait<CG == 2>(full0 + 8 * s, ph, abort_flag)) {
                        report_timeout(p, abort_flag, 4, s);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_base = stage_base + s * C_::STAGE_BYTES;
                    const uint32_t b_base = a_base + A_STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t ad = smem_desc(a_base + k * a_kstep, a_lbo, 1024u);
                        const uint64_t bd = smem_desc(b_base + k * b_kstep, b_lbo, 1024u);
                        ptx::umma_f16<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb | k) != 0));
                    }
                    // release the stage (in both CTAs of a pair) once these MMAs have read it
                    if (CG == 1) ptx::umma_commit_1cta(empty0 + 8 * s);
                    else ptx::umma_commit_pair(empty0 + 8 * s, 3);
                }
                if (!ok) break;
                if (CG == 1) ptx::umma_commit_1cta(accfull0 + 8 * b);
                else ptx::umma_commit_pair(accfull0 + 8 * b, 3);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (4 warps)
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        TOut *Cout = reinterpret_cast<TOut *>(p.C);
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = unit; tile < total_tiles && ok; tile += num_units, ++tl) {
            int64_t tm, tn;
            tile_coord(tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
            const int row = (int)tm * (BM * CG) + (int)rank * BM + q * 32 + lane;
            const int n0 = (int)tn * BN;
            const uint32_t b = tl & 1u, aph = (tl >> 1) & 1u;
            // the outcome is made warp-uniform: tcgen05.ld below needs the whole warp
            const bool got = ptx::mbar_wait<CG == 2>(accfull0 + 8 * b, aph, abort_flag);
            if (!__all_sync(0xffffffffu, got)) {
                if (lane == 0) report_timeout(p, abort_flag, 5, b);
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + b * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col = n0 + c * 32;
                if (col >= p.N) break;  // warp-uniform
                uint32_t r[32];
                ptx::tmem_ld_32x32(t_addr + c * 32, r);
                ptx::tmem_ld_wait();
                if (row < p.M) {
                    const int valid = (p.N - col < 32) ? (p.N - col) : 32;
                    TOut *dst = Cout + (int64_t)row * p.ldc + col;
                    float v[32];
                    if (p.beta != 0.0f) {
                        float cold[32];
                        load_row_chunk<TOut>(dst, cold, valid, p.vec_ok != 0);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = fmaf(p.beta, cold[i], p.alpha * __uint_as_float(r[i]));
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = p.alpha * __uint_as_float(r[i]);
                    }
                    store_row_chunk<TOut>(dst, v, valid, p.vec_ok != 0);
                }
            }
            // hand the accumulator buffer back to the MMA issuer
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (CG == 1) ptx::mbar_arrive(accempty0 + 8 * b);
                else ptx::mbar_arrive_cluster(ptx::map_to_cta(accempty0 + 8 * b, 0));
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag != 0) {
        // a wait gave up: give copies that may still be in flight time to land before shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (CG == 2) ptx::cluster_sync();  // the peer may still signal this CTA's barriers or read its tiles
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc<CG>(tmem_base, TMEM_COLS);
    }
}

// ---- host side -------------------------------------------------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    });
    return fn;
}

// Tensor map over a row-major 2-D array of 16-bit elements: `inner` contiguous elements per row,
// `outer` rows, `pitch` elements between rows; box = box_inner x box_outer, 128-byte swizzle, zero fill.
bool make_map(CUtensorMap *tm, Elem e, const void *base, int64_t inner, int64_t outer, int64_t pitch, int box_inner,
              int box_outer) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, e == Elem::F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                    const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int CG, typename TOut> int run_umma(const GemmArgs &g) {
    using C_ = Cfg<CG>;
    auto kernel = umma_gemm_kernel<CG, TOut>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }

    const Elem ein = in_elem(g.dtype);
    const int a_mn = g.transA ? 1 : 0;  // A stored K x M: M is the contiguous index
    const int b_mn = g.transB ? 0 : 1;  // B stored K x N: N is the contiguous index
    CUtensorMap tmA, tmB;
    bool ok = a_mn ? make_map(&tmA, ein, g.A, g.M, g.K, g.lda, 64, BK) : make_map(&tmA, ein, g.A, g.K, g.M, g.lda, BK, 128);
    ok = ok && (b_mn ? make_map(&tmB, ein, g.B, g.N, g.K, g.ldb, 64, BK) : make_map(&tmB, ein, g.B, g.K, g.N, g.ldb, BK, 128));
    if (!ok) return PEAK_ERR_CUDA;

    UmmaParams p;
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.num_kb = (int)((g.K + BK - 1) / BK);
    p.tiles_m = (int)((g.M + BM * CG - 1) / (BM * CG));
    p.tiles_n = (int)((g.N + BN - 1) / BN);
    p.group = (CG == 1) ? 16 : 8;
    p.a_mn = a_mn; p.b_mn = b_mn;
    const uint32_t fmt = (ein == Elem::BF16) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.ldc = g.ldc;
    const int ob = elem_bytes(out_elem(g.dtype));
    p.vec_ok = ((reinterpret_cast<uintptr_t>(g.C) % 16) == 0 && (g.ldc * ob) % 16 == 0) ? 1 : 0;
    p.status = device_status_word();
    if (!p.status) return PEAK_ERR_CUDA;

    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t total = (int64_t)p.tiles_m * p.tiles_n;
    int units = sms / CG;
    if (total < units) units = (int)total;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * CG));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = C_::SMEM_BYTES;
    cfg.stream = g.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, p);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <int CG> int dispatch_out(const GemmArgs &g) {
    switch (out_elem(g.dtype)) {
        case Elem::F32: return run_umma<CG, float>(g);
        case Elem::F16: return run_umma<CG, __half>(g);
        case Elem::BF16: return run_umma<CG, __nv_bfloat16>(g);
    }
    return PEAK_ERR_INVALID_VALUE;
}

}  // namespace

bool umma_supports(const GemmArgs &g, int cta_group) {
    (void)cta_group;
    if (in_elem(g.dtype) == Elem::F32) return false;
    if (g.M < 1 || g.N < 1 || g.K < 1) return false;
    if (g.M >= (1ll << 31) - 512 || g.N >= (1ll << 31) - 512 || g.K >= (1ll << 31) - 512) return false;
    if (reinterpret_cast<uintptr_t>(g.A) % 16 || reinterpret_cast<uintptr_t>(g.B) % 16) return false;
    if (g.lda % 8 || g.ldb % 8) return false;  // TMA: row pitch must be a multiple of 16 bytes
    if (g.lda >= (1ll << 38) || g.ldb >= (1ll << 38)) return false;
    const int64_t tiles = ((g.M + 127) / 128) * ((g.N + 255) / 256);
    if (tiles >= (1ll << 31)) return false;
    return true;
}

int launch_umma(const GemmArgs &g, int cta_group) {
    if (!umma_supports(g, cta_group)) return PEAK_ERR_UNSUPPORTED;
    return cta_group == 2 ? dispatch_out<2>(g) : dispatch_out<1>(g);
}

}  // namespace peak
