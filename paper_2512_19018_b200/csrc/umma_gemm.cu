// Tensor-core GEMM for 16-bit inputs on sm_100a.
//
// One persistent CTA (or CTA pair) per SM walks work items -- output tiles, or (tile, k-slice) pairs when
// K is split -- in a grouped order (the paper's block swizzle).  Inside a CTA three roles run concurrently
// (warp specialisation):
//   warp 0      producer: TMA tile loads of A and B into a ring of 128-byte-swizzled shared-memory stages
//               (the paper's thread-block tiling + pipelining + bank-conflict offset, section 2.2),
//   warp 1      one thread issues tcgen05.mma; fp32 accumulators live in tensor memory (the paper's
//               warp tiling / tensor-core steps), two accumulator buffers so that the next tile's main
//               loop overlaps this tile's epilogue,
//   warps 2..5  epilogue: tcgen05.ld -> alpha/beta in fp32 -> one rounding -> swizzled shared-memory
//               staging -> TMA store (coalesced, clipped at the matrix edge); a direct vector / scalar
//               store path serves outputs whose base or pitch is not 16-byte aligned.
// mbarriers connect the roles (full/empty per stage, full/empty per accumulator).  Every wait is bounded.
//
// Tile: 128 x BN x 64 per CTA (CTA_GROUP 1) or 256 x BN x 64 per CTA pair (CTA_GROUP 2: each CTA stages its
// 128 rows of A and its BN/2-column half of B; the leader CTA issues MMAs for both).  BN is 256 or 128.
//
// Split-K (the paper's Split-K transformation, section 4.1).  The first `full_tiles` tiles are computed
// whole; each remaining tile has its k-blocks divided among `tail_splits` work items that store fp32 partial
// tiles to a workspace, and a second kernel adds a tile's slices in slice order and applies alpha/beta, so
// the result does not depend on scheduling.  Two uses: shapes with too few tiles to fill the GPU split every
// tile (full_tiles = 0); shapes whose tile count is not a multiple of the SM (pair) count split only the
// tiles of the last, partly filled wave, so that the wave finishes in a fraction of a tile time.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace peak {
namespace {

constexpr int BM = 128;   // rows of C per CTA
constexpr int BK = 64;    // k-block: 64 16-bit elements = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;  // 16 KiB
constexpr int ATOM_BYTES = 64 * BK * 2;     // one 64-wide MN-major box: 64 k-rows of 128 bytes = 8 KiB
constexpr int NUM_THREADS = 192;
constexpr int EPI_BUF_BYTES = 32 * 128;               // one staging buffer: 32 rows x 128 bytes
constexpr int EPI_BYTES = 4 * 2 * EPI_BUF_BYTES;      // 4 epilogue warps x 2 buffers = 32 KiB
constexpr int SMEM_LIMIT = 232448;                    // 227 KiB of dynamic shared memory per CTA

template <int CG, int BN> struct Cfg {
    static constexpr int B_ROWS = BN / CG;                 // rows of op(B)^T this CTA stages
    static constexpr int B_BOX_ROWS = B_ROWS < 128 ? B_ROWS : 128;
    static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int AUX_BYTES = 256;
    static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - EPI_BYTES - AUX_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + AUX_BYTES;
    static constexpr int TMEM_COLS = 2 * BN;               // two fp32 accumulators
    static_assert(STAGES >= 3, "pipeline too shallow");
    static_assert(8 * (2 * STAGES + 4) + 8 <= AUX_BYTES, "barrier area too small");
};

struct UmmaParams {
    int M, N, K;
    int num_kb;            // ceil(K / BK)
    int tiles_m, tiles_n;  // in units of (128*CG) x BN
    int group;             // tile-rows per raster group
    int full_tiles;        // tiles [0, full_tiles) are computed whole and stored to C
    int tail_splits;       // k-slices of every later tile (partials go to the workspace)
    int kb_per_split;
    int total_items;       // full_tiles + (tiles - full_tiles) * tail_splits
    int a_mn, b_mn;        // 1: operand is MN-major in memory (transA == 1 / transB == 0)
    uint32_t idesc;
    float alpha, beta;
    void *C;
    int64_t ldc;
    int vec_ok;            // C base and pitch allow 16-byte vector access
    int tma_store;         // epilogue stores through TMA
    long long wait_cycles; // budget of every mbarrier wait
    int inject_stall;      // test hook: CTA (pair) 0 never fills the stage of its last k-block
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

template <typename TOut> __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    TOut a = from_f32<TOut>(lo), b = from_f32<TOut>(hi);
    return (uint32_t)(*reinterpret_cast<uint16_t *>(&a)) | ((uint32_t)(*reinterpret_cast<uint16_t *>(&b)) << 16);
}

// 32 consecutive outputs of one row -> global memory (vector path when aligned and whole)
template <typename TOut>
__device__ __forceinline__ void store_row32(TOut *dst, const float (&v)[32], int valid, bool vec) {
    if (vec && valid == 32) {
        if constexpr (sizeof(TOut) == 4) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                reinterpret_cast<float4 *>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                reinterpret_cast<uint4 *>(dst)[i] =
                    make_uint4(pack2<TOut>(v[8 * i], v[8 * i + 1]), pack2<TOut>(v[8 * i + 2], v[8 * i + 3]),
                               pack2<TOut>(v[8 * i + 4], v[8 * i + 5]), pack2<TOut>(v[8 * i + 6], v[8 * i + 7]));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < valid) dst[i] = from_f32<TOut>(v[i]);
    }
}

// 32 consecutive old values of one row <- global memory
template <typename TOut>
__device__ __forceinline__ void load_row32(const TOut *src, float (&c)[32], int valid, bool vec) {
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

// 32 consecutive outputs of row `lane` -> staging buffer laid out as the 128-byte-swizzled box a TMA
// store expects: 16-byte piece j of row r sits at piece (j ^ (r & 7)).  `h` selects which 32-column
// half of a 64-column (16-bit) chunk is written; fp32 chunks are 32 columns wide and use h = 0.
template <typename TOut>
__device__ __forceinline__ void stage_row32(uint32_t buf, int lane, int h, const float (&v)[32]) {
    constexpr int PIECES = 32 * (int)sizeof(TOut) / 16;  // 8 (fp32) or 4 (16-bit)
    const uint32_t row = buf + (uint32_t)lane * 128u;
#pragma unroll
    for (int j = 0; j < PIECES; ++j) {
        uint32_t w0, w1, w2, w3;
        if constexpr (sizeof(TOut) == 4) {
            w0 = __float_as_uint(v[4 * j]); w1 = __float_as_uint(v[4 * j + 1]);
            w2 = __float_as_uint(v[4 * j + 2]); w3 = __float_as_uint(v[4 * j + 3]);
        } else {
            w0 = pack2<TOut>(v[8 * j], v[8 * j + 1]); w1 = pack2<TOut>(v[8 * j + 2], v[8 * j + 3]);
            w2 = pack2<TOut>(v[8 * j + 4], v[8 * j + 5]); w3 = pack2<TOut>(v[8 * j + 6], v[8 * j + 7]);
        }
        const uint32_t piece = (uint32_t)((h * PIECES + j) ^ (lane & 7));
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + piece * 16u), "r"(w0), "r"(w1), "r"(w2),
                     "r"(w3)
                     : "memory");
    }
}

// Work item -> tile, k-block range and destination (ws_block < 0: the tile is whole and goes to C;
// otherwise the index of the (tile, slice) block of the partial-tile workspace).
struct Item {
    int tile, kb0, kb1, ws_block;
};
__device__ __forceinline__ Item decode_item(const UmmaParams &p, int item) {
    Item w;
    if (item < p.full_tiles) {
        w.tile = item; w.kb0 = 0; w.kb1 = p.num_kb; w.ws_block = -1;
    } else {
        const int j = item - p.full_tiles;
        const int t = j / p.tail_splits, slice = j - t * p.tail_splits;
        w.tile = p.full_tiles + t;
        w.kb0 = slice * p.kb_per_split;
        w.kb1 = min(w.kb0 + p.kb_per_split, p.num_kb);
        w.ws_block = j;
    }
    return w;
}

// Epilogue of one accumulator tile for one warp: TMEM -> registers -> alpha/beta -> T -> staging + TMA
// store (or direct stores).  `cbase` is the column of chunk 0 used for bounds and addressing, `ncols` the
// column limit, `nrows` the row limit for `row`; (x0, y0) is where chunk 0 of this warp lands in `tm`.
template <typename T, int BN>
__device__ __forceinline__ void epilogue_tile(uint32_t t_addr, uint32_t my_stage, uint32_t &chunk_no, int lane,
                                              T *base, int64_t ld, int row, int row0, int nrows, int cbase,
                                              int ncols, const CUtensorMap *tm, int x0, int y0, bool tma, bool vec,
                                              float alpha, float beta) {
    constexpr int CHUNK_COLS = 128 / (int)sizeof(T);  // columns per staged chunk: 32 (fp32) or 64 (16-bit)
#pragma unroll 1
    for (int c = 0; c < BN / CHUNK_COLS; ++c) {
        const int col0 = cbase + c * CHUNK_COLS;
        if (col0 >= ncols) break;  // warp-uniform
        uint32_t buf = 0;
        if (tma) {
            // the store that last read this buffer (two chunks ago) must have drained it
            buf = my_stage + (chunk_no & 1u) * EPI_BUF_BYTES;
            if (lane == 0) ptx::tma_store_wait_read<1>();
            __syncwarp();
        }
#pragma unroll
        for (int h = 0; h < CHUNK_COLS / 32; ++h) {
            const int col = col0 + h * 32;
            uint32_t r[32];
            ptx::tmem_ld_32x32(t_addr + c * CHUNK_COLS + h * 32, r);
            ptx::tmem_ld_wait();
            const int valid = (ncols - col >= 32) ? 32 : (ncols - col > 0 ? ncols - col : 0);
            T *dst = base + (int64_t)row * ld + col;
            float v[32];
            if (beta != 0.0f) {
                float cold[32];
                if (row < nrows && valid > 0) load_row32<T>(dst, cold, valid, vec);
                else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) cold[i] = 0.0f;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = fmaf(beta, cold[i], alpha * __uint_as_float(r[i]));
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = alpha * __uint_as_float(r[i]);
            }
            if (tma) stage_row32<T>(buf, lane, h, v);
            else if (row < nrows && valid > 0) store_row32<T>(dst, v, valid, vec);
        }
        if (tma) {
            ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the TMA engine
            __syncwarp();
            if (lane == 0 && row0 < nrows) {
                ptx::tma_store_2d(tm, x0 + c * CHUNK_COLS, y0, buf);
                ptx::tma_store_commit();
            }
            ++chunk_no;
        }
    }
}

template <int CG, int BN, typename TOut>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmW,
                 float *__restrict__ ws, const UmmaParams p) {
    using C_ = Cfg<CG, BN>;
    constexpr int STAGES = C_::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t stage_base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    const uint32_t epi_base = stage_base + STAGES * C_::STAGE_BYTES;
    uint8_t *aux = smem_raw + (epi_base - raw) + EPI_BYTES;
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
    const int total_items = p.total_items;

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
        if (p.tma_store) ptx::prefetch_tensormap(&tmC);
        if (p.total_items > p.full_tiles) ptx::prefetch_tensormap(&tmW);
    }
    if (warp == 1) {
        ptx::tmem_alloc<CG>(ptx::smem_u32(tmem_slot), C_::TMEM_COLS);
        ptx::tmem_relinquish<CG>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (CG == 2) ptx::cluster_sync();  // the peer's barriers must be initialised before anything signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: everything above touched only this CTA's shared and tensor memory, so
    // it may overlap the tail of the previous kernel in the stream; global memory is touched only after
    // that kernel has completed.  The next kernel in the stream may start its own prologue as soon as
    // SMs free up.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int item = unit; item < total_items && ok; item += num_units) {
                const Item w = decode_item(p, item);
                int64_t tm, tn;
                tile_coord(w.tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
                const int m_cta = (int)tm * (BM * CG) + (int)rank * BM;
                const int n_cta = (int)tn * BN + (int)rank * C_::B_ROWS;
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles)) {
                        report_timeout(p, abort_flag, 1, s);
                        ok = false;
                        break;
                    }
                    if (p.inject_stall && unit == 0 && leader && item + num_units >= total_items && kb == w.kb1 - 1)
                        continue;  // test hook: leave this stage empty so that the waits downstream run out
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
                        for (int h = 0; h < C_::B_ROWS / C_::B_BOX_ROWS; ++h) {
                            const uint32_t d = b_dst + h * C_::B_BOX_ROWS * 128;
                            if (CG == 1) ptx::tma_load_2d(d, &tmB, k0, n_cta + C_::B_BOX_ROWS * h, bar);
                            else ptx::tma_load_2d_pair(d, &tmB, k0, n_cta + C_::B_BOX_ROWS * h, bar);
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
                if (!ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles)) {
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
            for (int item = unit; item < total_items && ok; item += num_units, ++tl) {
                const Item w = decode_item(p, item);
                const int kb0 = w.kb0, kb1 = w.kb1;
                const uint32_t b = tl & 1u, aph = (tl >> 1) & 1u;
                if (!ptx::mbar_wait<CG == 2>(accempty0 + 8 * b, aph ^ 1u, abort_flag, p.wait_cycles)) {
                    report_timeout(p, abort_flag, 3, b);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + b * BN;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait<CG == 2>(full0 + 8 * s, ph, abort_flag, p.wait_cycles)) {
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
                        ptx::umma_f16<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > kb0) | (k != 0)));
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
        const uint32_t my_stage = epi_base + (uint32_t)(warp - 2) * 2u * EPI_BUF_BYTES;
        const bool vec = p.vec_ok != 0;
        uint32_t tl = 0, chunk_no = 0;
        bool ok = true;
        for (int item = unit; item < total_items && ok; item += num_units, ++tl) {
            const Item w = decode_item(p, item);
            int64_t tm, tn;
            tile_coord(w.tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
            const int row0 = (int)tm * (BM * CG) + (int)rank * BM + q * 32;  // first row of this warp
            const int n0 = (int)tn * BN;
            const uint32_t b = tl & 1u, aph = (tl >> 1) & 1u;
            // the outcome is made warp-uniform: tcgen05.ld below needs the whole warp
            const bool got = ptx::mbar_wait<CG == 2>(accfull0 + 8 * b, aph, abort_flag, p.wait_cycles);
            if (!__all_sync(0xffffffffu, got)) {
                if (lane == 0) report_timeout(p, abort_flag, 5, b);
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + b * BN;
            if (w.ws_block < 0) {
                // whole tile: alpha/beta epilogue straight to C
                epilogue_tile<TOut, BN>(t_addr, my_stage, chunk_no, lane, reinterpret_cast<TOut *>(p.C), p.ldc,
                                        row0 + lane, row0, p.M, n0, p.N, &tmC, n0, row0, p.tma_store != 0, vec,
                                        p.alpha, p.beta);
            } else {
                // k-slice: raw fp32 partial tile to its dense (BM*CG) x BN block of the workspace
                const int wrow0 = w.ws_block * (BM * CG) + (int)rank * BM + q * 32;
                epilogue_tile<float, BN>(t_addr, my_stage, chunk_no, lane, ws, (int64_t)BN, wrow0 + lane, wrow0,
                                         0x7fffffff, 0, BN, &tmW, 0, wrow0, true, true, 1.0f, 0.0f);
            }
            // hand the accumulator buffer back to the MMA issuer
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (CG == 1) ptx::mbar_arrive(accempty0 + 8 * b);
                else ptx::mbar_arrive_cluster(ptx::map_to_cta(accempty0 + 8 * b, 0));
            }
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();  // staging memory must outlive the stores
        __syncwarp();
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
        ptx::tmem_dealloc<CG>(tmem_base, C_::TMEM_COLS);
    }
}

// Adds the k-slices of every split tile in slice order and applies the epilogue:
// C = alpha * (ws[tile][0] + ws[tile][1] + ...) + beta * C, one rounding.  The workspace holds, for split tile
// t (counted from full_tiles) and slice s, a dense rows_t x bn fp32 block at index t * splits + s.
// One block of 256 threads handles a quarter of a tile's float4 columns groups at a time.
template <typename TOut>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ ws, int splits, int full_tiles, int tiles_m, int tiles_n, int group,
                     int rows_t, int bn, int M, int N, float alpha, float beta, TOut *__restrict__ C, int64_t ldc,
                     int vec_ok) {
    const int blocks_per_tile = gridDim.y;
    const int t = blockIdx.x;  // split tile number
    int64_t tm, tn;
    tile_coord(full_tiles + t, tiles_m, tiles_n, group, tm, tn);
    const int vec_per_row = bn / 4;
    const int total_vec = rows_t * vec_per_row;
    const int64_t block_elems = (int64_t)rows_t * bn;
    const float *base = ws + (int64_t)t * splits * block_elems;
    for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < total_vec; e += blocks_per_tile * blockDim.x) {
        const int r = e / vec_per_row, c4 = e - r * vec_per_row;
        const int64_t i = tm * rows_t + r;
        const int64_t j = tn * bn + c4 * 4;
        if (i >= M || j >= N) continue;
        const float *src = base + (int64_t)r * bn + c4 * 4;
        float4 acc = *reinterpret_cast<const float4 *>(src);
        for (int sl = 1; sl < splits; ++sl) {
            const float4 v = *reinterpret_cast<const float4 *>(src + sl * block_elems);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
        TOut *dst = C + i * ldc + j;
        if (vec_ok && j + 4 <= N) {
            float o[4] = {0.f, 0.f, 0.f, 0.f};
            if (beta != 0.0f) {
                if constexpr (sizeof(TOut) == 4) {
                    const float4 t4 = *reinterpret_cast<const float4 *>(dst);
                    o[0] = t4.x; o[1] = t4.y; o[2] = t4.z; o[3] = t4.w;
                } else {
                    const uint2 t2 = *reinterpret_cast<const uint2 *>(dst);
                    uint16_t h[4] = {(uint16_t)(t2.x & 0xffffu), (uint16_t)(t2.x >> 16), (uint16_t)(t2.y & 0xffffu),
                                     (uint16_t)(t2.y >> 16)};
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[k] = to_f32(*reinterpret_cast<TOut *>(&h[k]));
                }
            }
            float rr[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) rr[k] = epilogue_f32(alpha, a4[k], beta, o[k]);
            if constexpr (sizeof(TOut) == 4) {
                *reinterpret_cast<float4 *>(dst) = make_float4(rr[0], rr[1], rr[2], rr[3]);
            } else {
                *reinterpret_cast<uint2 *>(dst) = make_uint2(pack2<TOut>(rr[0], rr[1]), pack2<TOut>(rr[2], rr[3]));
            }
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (j + k < N) {
                    const float c_old = (beta != 0.0f) ? to_f32(dst[k]) : 0.0f;
                    dst[k] = from_f32<TOut>(epilogue_f32(alpha, a4[k], beta, c_old));
                }
            }
        }
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

// Tensor map over a row-major 2-D array: `inner` contiguous elements per row, `outer` rows, `pitch`
// elements between rows; box = box_inner x box_outer, 128-byte swizzle, zero fill.
bool make_map(CUtensorMap *tm, Elem e, const void *base, int64_t inner, int64_t outer, int64_t pitch, int box_inner,
              int box_outer) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const CUtensorMapDataType dt = e == Elem::F16    ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                   : e == Elem::BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                     : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch * (cuuint64_t)elem_bytes(e)};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int sm_count() {
    static int sms[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return 148;
    if (sms[dev] == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        sms[dev] = n > 0 ? n : 148;
    }
    return sms[dev];
}

constexpr double kL2BytesPerClk = 64.0;      // assumed L2 -> shared-memory bandwidth per SM
constexpr double kSplitFixedCycles = 20000.0;  // workspace allocation + second launch of a split (~12 us)

struct Plan {
    int bn;           // tile width: 256 or 128
    int full_tiles;   // tiles computed whole
    int tail_splits;  // k-slices of each remaining tile (1 when nothing is split)
};

int64_t tiles_of(const GemmArgs &g, int cg, int bn) {
    return ((g.M + BM * cg - 1) / (BM * cg)) * ((g.N + bn - 1) / bn);
}

// Tile width and k-splitting from a small cost model (cycles): an item costs its k-blocks times the slower
// of the tensor pipe (2*BN cycles per k-block per SM) and the operand stream (bytes per k-block over an
// assumed 64 bytes/cycle/SM of L2->shared bandwidth), plus a fixed per-item overhead; items are spread over
// the units in waves.  Splitting additionally pays for writing and re-reading fp32 partials and for the
// second launch.  Candidates: no split; every tile split s ways (few tiles); only the last wave split.
Plan choose_plan(const GemmArgs &g, int cg, int units) {
    const int64_t num_kb = (g.K + BK - 1) / BK;
    Plan best{256, 0, 1};
    double best_cost = 1e300;
    const int force_bn = tuning(PEAK_TUNE_TILE_N), force_split = tuning(PEAK_TUNE_SPLIT_K);
    const int tail_mode = tuning(PEAK_TUNE_TAIL_SPLIT);  // 2 = split the last wave whenever possible
    for (int bn : {256, 128}) {
        if (force_bn && bn != force_bn) continue;
        const int64_t tiles = tiles_of(g, cg, bn);
        const double kb_cycles = fmax(2.0 * bn, (128.0 + bn / cg) * 128.0 / kL2BytesPerClk);
        const double item_ovh = 1500.0;
        const double tile_bytes = (double)BM * bn * 4.0;  // fp32 partial tile per SM
        auto consider = [&](int64_t full, int s, double cost) {
            if (cost < best_cost) { best_cost = cost; best = Plan{bn, (int)full, s}; }
        };
        // (a) every tile whole, or every tile split s ways
        for (int s = 1; s <= 16; ++s) {
            if (force_split && s != force_split) continue;
            if (s > num_kb) break;
            if (s > 1 && !force_split && tiles * s > 2 * units) break;
            const int64_t kbps = (num_kb + s - 1) / s;
            if (s > 1 && kbps * (s - 1) >= num_kb) continue;  // an empty last slice
            const int64_t waves = (tiles * s + units - 1) / units;
            double cost = (double)waves * (kbps * kb_cycles + item_ovh);
            if (s > 1) cost += 2.0 * waves * tile_bytes / 24.0 + kSplitFixedCycles;
            if (s > 1 && tail_mode == 2 && !force_split) cost *= 4.0;  // forced tail mode prefers (b)
            consider(s == 1 ? tiles : 0, s, cost);
        }
        // (b) whole tiles for the full waves, the last partly filled wave split s ways
        const int64_t full = (tiles / units) * units, rest = tiles - full;
        // (measured on B200: under the power cap the busy SMs of a partly filled wave clock higher, so this
        // split gains nothing at 4096^3 or 5000x3000x2500; it stays opt-in through PEAK_TUNE_TAIL_SPLIT = 2)
        if (!force_split && tail_mode == 2 && full > 0 && rest > 0) {
            for (int s = 2; s <= 8; ++s) {
                if (rest * s > units || s > num_kb) break;
                const int64_t kbps = (num_kb + s - 1) / s;
                if (kbps * (s - 1) >= num_kb || kbps < 4) continue;
                double cost = (double)(full / units) * (num_kb * kb_cycles + item_ovh) + (kbps * kb_cycles + item_ovh) +
                              2.0 * tile_bytes / 24.0 + kSplitFixedCycles;
                cost *= 0.01;
                consider(full, s, cost);
            }
        }
    }
    return best;
}

template <int CG, int BN, typename TOut>
int launch_kernel(const GemmArgs &g, const Plan &plan, int units_max, float *ws) {
    using C_ = Cfg<CG, BN>;
    auto kernel = umma_gemm_kernel<CG, BN, TOut>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }

    const Elem ein = in_elem(g.dtype), eout = out_elem(g.dtype);
    const int a_mn = g.transA ? 1 : 0;  // A stored K x M: M is the contiguous index
    const int b_mn = g.transB ? 0 : 1;  // B stored K x N: N is the contiguous index
    CUtensorMap tmA, tmB, tmC, tmW;
    bool ok = a_mn ? make_map(&tmA, ein, g.A, g.M, g.K, g.lda, 64, BK) : make_map(&tmA, ein, g.A, g.K, g.M, g.lda, BK, 128);
    ok = ok && (b_mn ? make_map(&tmB, ein, g.B, g.N, g.K, g.ldb, 64, BK)
                     : make_map(&tmB, ein, g.B, g.K, g.N, g.ldb, BK, C_::B_BOX_ROWS));
    if (!ok) return PEAK_ERR_CUDA;

    UmmaParams p;
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.num_kb = (int)((g.K + BK - 1) / BK);
    p.tiles_m = (int)((g.M + BM * CG - 1) / (BM * CG));
    p.tiles_n = (int)((g.N + BN - 1) / BN);
    p.group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : ((CG == 1) ? 16 : 8);
    const int tiles = p.tiles_m * p.tiles_n;
    p.full_tiles = plan.full_tiles;
    p.tail_splits = plan.tail_splits;
    p.kb_per_split = (p.num_kb + plan.tail_splits - 1) / plan.tail_splits;
    p.total_items = plan.full_tiles + (tiles - plan.full_tiles) * plan.tail_splits;
    p.a_mn = a_mn; p.b_mn = b_mn;
    const uint32_t fmt = (ein == Elem::BF16) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.ldc = g.ldc;
    const int ob = elem_bytes(eout);
    p.vec_ok = ((reinterpret_cast<uintptr_t>(g.C) % 16) == 0 && (g.ldc * ob) % 16 == 0) ? 1 : 0;
    const int epi = tuning(PEAK_TUNE_EPILOGUE);  // 0 auto, 1 direct stores, 2 TMA stores
    // TMA stores clip rows exactly but clip the contiguous index only at 16-byte granularity, so they are
    // used when a row of C is a whole number of 16-byte pieces; other widths take the direct-store path
    p.tma_store = (p.vec_ok && (g.N * ob) % 16 == 0 && epi != 1) ? 1 : 0;
    tmC = tmA;  // placeholders when unused
    tmW = tmA;
    if (p.tma_store && plan.full_tiles > 0 && !make_map(&tmC, eout, g.C, g.N, g.M, g.ldc, 128 / ob, 32))
        return PEAK_ERR_CUDA;
    if (plan.full_tiles < tiles) {
        // the workspace as one tall matrix of dense (BM*CG) x BN blocks, one per (split tile, slice)
        const int64_t rows = (int64_t)(tiles - plan.full_tiles) * plan.tail_splits * (BM * CG);
        if (!ws || !make_map(&tmW, Elem::F32, ws, BN, rows, BN, 32, 32)) return PEAK_ERR_CUDA;
    }
    p.status = device_status_word();
    if (!p.status) return PEAK_ERR_CUDA;
    const int wait_ms = tuning(PEAK_TUNE_WAIT_MS);
    p.wait_cycles = wait_ms > 0 ? (long long)wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.inject_stall = tuning(PEAK_TUNE_INJECT_STALL) == 1 ? 1 : 0;

    int units = units_max;
    if (p.total_items < units) units = p.total_items;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * CG));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = C_::SMEM_BYTES;
    cfg.stream = g.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = tuning(PEAK_TUNE_DEPENDENT_LAUNCH) == 1 ? 1 : 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, tmW, ws, p);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (plan.full_tiles == tiles) return PEAK_OK;

    // second kernel: add the slices of the split tiles in order, apply alpha/beta
    const int split_tiles = tiles - plan.full_tiles;
    dim3 rgrid((unsigned)split_tiles, split_tiles >= 64 ? 2u : 8u);
    splitk_reduce_kernel<TOut><<<rgrid, 256, 0, g.stream>>>(ws, plan.tail_splits, plan.full_tiles, p.tiles_m, p.tiles_n,
                                                            p.group, BM * CG, BN, p.M, p.N, g.alpha, g.beta, (TOut *)g.C,
                                                            g.ldc, p.vec_ok);
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <int CG, int BN> int launch_typed(const GemmArgs &g, const Plan &plan, int units, float *ws) {
    switch (out_elem(g.dtype)) {
        case Elem::F32: return launch_kernel<CG, BN, float>(g, plan, units, ws);
        case Elem::F16: return launch_kernel<CG, BN, __half>(g, plan, units, ws);
        case Elem::BF16: return launch_kernel<CG, BN, __nv_bfloat16>(g, plan, units, ws);
    }
    return PEAK_ERR_INVALID_VALUE;
}

// Bytes of fp32 partial tiles a plan needs (0 when nothing is split).
size_t workspace_bytes(const GemmArgs &g, int cg, const Plan &plan) {
    const int64_t split_tiles = tiles_of(g, cg, plan.bn) - plan.full_tiles;
    return (size_t)split_tiles * plan.tail_splits * (size_t)(BM * cg) * plan.bn * sizeof(float);
}

// Stream-ordered workspace for split-K partials: one memory pool per device that keeps what it has been
// given (release threshold = max), so that steady-state calls neither touch the OS allocator nor share a
// buffer between streams.
cudaMemPool_t workspace_pool() {
    static cudaMemPool_t pools[64] = {};
    static std::mutex m;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(m);
    if (!pools[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t pool = nullptr;
        cudaError_t e = cudaMemPoolCreate(&pool, &props);
        if (e != cudaSuccess) { set_cuda_error(e); return nullptr; }
        uint64_t keep = UINT64_MAX;
        cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        pools[dev] = pool;
    }
    return pools[dev];
}

template <int CG, int BN> int run_umma(const GemmArgs &g, const Plan &plan, int units) {
    const size_t need = workspace_bytes(g, CG, plan);
    if (need == 0) return launch_typed<CG, BN>(g, plan, units, nullptr);
    float *ws = nullptr;
    cudaMemPool_t pool = workspace_pool();
    if (!pool) return PEAK_ERR_CUDA;
    cudaError_t e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&ws), need, pool, g.stream);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_NO_MEMORY; }
    int rc = launch_typed<CG, BN>(g, plan, units, ws);
    e = cudaFreeAsync(ws, g.stream);
    if (e != cudaSuccess && rc == PEAK_OK) { set_cuda_error(e); rc = PEAK_ERR_CUDA; }
    return rc;
}

// ---- split-K with a fixed, library-owned workspace (no allocation at call time) --------------------------
// The partial tiles of peak_gemm_static_ws live in this array instead of in pool memory.  It is part of
// the loaded module, so every GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticWsBytes = 32u << 20;  // 32 MiB
static __device__ __align__(256) float g_static_ws[kStaticWsBytes / sizeof(float)];

// Device address of g_static_ws on the current device.  In host code the array's name is only a handle
// for the runtime, not a device address, so the address is asked for once per device (with that device
// current) and cached.
float *static_ws_address() {
    static float *addr[64] = {};
    static std::mutex m;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e); return nullptr; }
    if (dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(m);
    if (!addr[dev]) {
        float *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_ws);
        if (e != cudaSuccess) { set_cuda_error(e); return nullptr; }
        addr[dev] = ptr;
    }
    return addr[dev];
}

// Every tile split `splits` ways with the workspace passed in; 128 x 128 tiles, one CTA per tile slice.
int run_umma_static_ws(const GemmArgs &g, int splits, float *ws) {
    const Plan plan{128, 0, splits};
    return launch_typed<1, 128>(g, plan, sm_count(), ws);
}

}  // namespace

bool umma_supports(const GemmArgs &g, int cta_group) {
    (void)cta_group;
    if (in_elem(g.dtype) == Elem::F32) return false;
    if (g.M < 1 || g.N < 1 || g.K < 1) return false;
    if (g.M >= (1ll << 31) - 512 || g.N >= (1ll << 31) - 512 || g.K >= (1ll << 31) - 512) return false;
    if (reinterpret_cast<uintptr_t>(g.A) % 16 || reinterpret_cast<uintptr_t>(g.B) % 16) return false;
    if (g.lda % 8 || g.ldb % 8) return false;  // TMA: row pitch must be a multiple of 16 bytes
    if (g.lda >= (1ll << 38) || g.ldb >= (1ll << 38) || g.ldc >= (1ll << 38)) return false;
    const int64_t tiles = ((g.M + 127) / 128) * ((g.N + 127) / 128);
    if (tiles * 16 >= (1ll << 31)) return false;
    return true;
}

int launch_umma(const GemmArgs &g, int cta_group) {
    if (!umma_supports(g, cta_group)) return PEAK_ERR_UNSUPPORTED;
    const int units = sm_count() / cta_group;
    const Plan plan = choose_plan(g, cta_group, units);
    if (cta_group == 2) return plan.bn == 256 ? run_umma<2, 256>(g, plan, units) : run_umma<2, 128>(g, plan, units);
    return plan.bn == 256 ? run_umma<1, 256>(g, plan, units) : run_umma<1, 128>(g, plan, units);
}

}  // namespace peak

extern "C" {

size_t peak_static_ws_bytes(void) { return peak::kStaticWsBytes; }

int peak_gemm_static_ws(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                        int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, int splits,
                        void *stream) {
    using namespace peak;
    set_cuda_error(cudaSuccess);
    // arguments first: nothing is launched or written on an error
    if (dtype != PEAK_F16_F32 && dtype != PEAK_BF16_BF16 && dtype != PEAK_F16_F16 && dtype != PEAK_BF16_F32)
        return PEAK_ERR_INVALID_VALUE;  // 16-bit inputs only: this is the tensor-core path
    if ((transA != 0 && transA != 1) || (transB != 0 && transB != 1)) return PEAK_ERR_INVALID_VALUE;
    if (M < 1 || N < 1 || K < 1 || !A || !B || !C) return PEAK_ERR_INVALID_VALUE;
    if (lda < (transA ? M : K) || ldb < (transB ? K : N) || ldc < N) return PEAK_ERR_INVALID_VALUE;
    const int64_t num_kb = (K + BK - 1) / BK;
    if (splits < 2 || splits > 64) return PEAK_ERR_INVALID_VALUE;
    const int64_t kbps = (num_kb + splits - 1) / splits;
    if (splits > num_kb || kbps * (splits - 1) >= num_kb) return PEAK_ERR_INVALID_VALUE;  // a slice would be empty
    GemmArgs g{dtype, transA, transB, M, N, K, alpha, beta, A, B, C, lda, ldb, ldc, (cudaStream_t)stream};
    if (!umma_supports(g, 1)) return PEAK_ERR_UNSUPPORTED;
    const int64_t rows_pad = ((M + 127) / 128) * 128, cols_pad = ((N + 127) / 128) * 128;
    if ((double)rows_pad * (double)cols_pad * (double)splits * sizeof(float) > (double)kStaticWsBytes)
        return PEAK_ERR_WORKSPACE_TOO_SMALL;  // 128 x 128 fp32 blocks: one per (tile, slice)
    int major = 0, dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (major != 10) return PEAK_ERR_ARCH;
    float *ws = static_ws_address();
    if (!ws) return PEAK_ERR_CUDA;
    return run_umma_static_ws(g, splits, ws);
}

}  // extern "C"
