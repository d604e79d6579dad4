// Tensor-core GEMM for 16-bit (and 8-bit float) inputs on sm_100a: device code (kernel, epilogue, split-K
// reduction).
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
//   (or 2..9)   staging -> TMA store (coalesced, clipped at the matrix edge); with beta != 0 old C comes in by
//               TMA through the same buffers; a direct vector / scalar path serves outputs whose base or
//               pitch is not 16-byte aligned.  Two-half tiles, and one-slot tiles of short launches, have a
//               second group of four epilogue warps.
// mbarriers connect the roles (full/empty per stage, full/empty per accumulator).  Every wait is bounded.
//
// Tile: 128 x BN x 64 per CTA (CTA_GROUP 1) or 256 x BN x 64 per CTA pair (CTA_GROUP 2: each CTA stages its
// 128 rows of A and its BN/2-column half of B; the leader CTA issues MMAs for both).  BN is 128, 256, or --
// CTA pairs only -- 512: a 256 x 512 tile is computed as two 256-column halves that occupy both accumulator
// slots, so a quarter fewer operand bytes reach each SM per flop (what limits the sustained rate under the
// power cap) at the price of an epilogue that is exposed once per tile: the two halves are drained at the
// same time by the two warp groups, and the last k-blocks of the tile are issued half by half so that half 0
// reaches its warps early.
//
// Split-K (the paper's Split-K transformation, section 4.1).  The first `full_tiles` tiles are computed
// whole; each remaining tile has its k-blocks divided among `tail_splits` work items that store fp32 partial
// tiles to a workspace, and a second kernel adds a tile's slices in slice order and applies alpha/beta, so
// the result does not depend on scheduling.  Two uses: shapes with too few tiles to fill the GPU split every
// tile (full_tiles = 0); shapes whose tile count is not a multiple of the SM (pair) count split only the
// tiles of the last, partly filled wave, so that the wave finishes in a fraction of a tile time (opt-in: it
// measured no gain under the power cap).
#pragma once
#include <type_traits>
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace peak {
namespace umma {

constexpr int BM = 128;   // rows of C per CTA
constexpr int BK = 64;    // k-block: 64 16-bit elements = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;  // 16 KiB
constexpr int ATOM_BYTES = 64 * BK * 2;     // one 64-wide MN-major box: 64 k-rows of 128 bytes = 8 KiB
// Warp 0 loads, warp 1 issues the MMAs, the others run the epilogue.  A warp may only read the 32 TMEM lanes
// of quadrant (warp % 4), so epilogue warps come in groups of four that cover all 128 rows.  A one-slot tile
// has one group (its epilogue hides behind the next tile's main loop); a two-half tile, whose epilogue is
// exposed because the tile fills the whole tensor memory, has two groups that drain one half each at the
// same time.
constexpr int MAX_EPI_WARPS = 8;
constexpr int EPI_BUF_BYTES = 32 * 128;                    // one staging buffer: 32 rows x 128 bytes
constexpr int EPI_BYTES = MAX_EPI_WARPS * EPI_BUF_BYTES;   // 32 KiB: two buffers per warp (one group) or one
constexpr int SMEM_LIMIT = 232448;                    // 227 KiB of dynamic shared memory per CTA

template <int CG, int BN> struct Cfg {
    // A tile wider than one MMA (BN = 512) is computed as two 256-column halves, one per accumulator slot.
    static constexpr int SLOT_N = BN > 256 ? 256 : BN;     // MMA N = width of one accumulator slot
    static constexpr int HALVES = BN / SLOT_N;
    // groups of four epilogue warps: a two-half tile always has two; a one-slot tile may get two as well (G2)
    static constexpr int threads(bool g2) { return 64 + 128 * ((HALVES == 2 || g2) ? 2 : 1); }
    static constexpr int HROWS = SLOT_N / CG;              // rows of op(B)^T this CTA stages per half
    static constexpr int B_ROWS = HALVES * HROWS;
    static constexpr int B_BOX_ROWS = HROWS < 128 ? HROWS : 128;
    static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int AUX_BYTES = 256;
    static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - EPI_BYTES - AUX_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + AUX_BYTES;
    static constexpr int TMEM_COLS = 2 * SLOT_N;           // two fp32 accumulator slots
    static_assert(HALVES == 1 || CG == 2, "512-wide tiles are for CTA pairs");
    static_assert(STAGES >= 3, "pipeline too shallow");
    // full[S], empty[S], acc_full[2], acc_empty[2], two old-C barriers for each of four epilogue warps, TMEM
    // slot, abort flag
    static_assert(8 * (2 * STAGES + 4 + 8) + 8 <= AUX_BYTES, "barrier area too small");
};

struct UmmaParams {
    int M, N, K;
    int num_kb;            // k-blocks: ceil(K / 64) for 16-bit inputs, ceil(K / 128) for 8-bit ones
    int tiles_m, tiles_n;  // in units of (128*CG) x BN
    int group;             // tile-rows per raster group
    int full_tiles;        // tiles [0, full_tiles) are computed whole and stored to C
    int tail_splits;       // k-slices of every later tile (partials go to the workspace)
    int kb_per_split;
    int total_items;       // full_tiles + (tiles - full_tiles) * tail_splits
    int tiles_per_batch;   // tiles_m * tiles_n: tile numbers run over all matrices of a strided batch
    int64_t stride_c;      // elements between the C matrices of a batch
    int a_mn, b_mn;        // 1: operand is MN-major in memory (transA == 1 / transB == 0)
    uint32_t idesc;
    float alpha, beta;
    void *C;
    int64_t ldc;
    int vec_ok;            // C base and pitch allow 16-byte vector access
    int tma_store;         // epilogue stores through TMA
    int c_prefetch;        // beta != 0: old C chunks arrive by TMA in the staging buffers (one-slot tiles only)
    const float *bias;     // fused epilogue: fp32 value per column of C, or nullptr
    int act;               // fused epilogue: a peak_activation_t
    const void *R;         // fused epilogue: residual (output type, M x N, pitch ldr) added after the activation
    int64_t ldr;
    int r_vec;             // R base and pitch allow 16-byte vector loads
    int k_alternate;       // 1: every other item of a CTA walks its k-blocks downwards (L2 reuse across waves)
    // Single-CTA tiles of a problem with fewer than 128 rows load only the rows of A that exist (rounded up to
    // the copy's granularity): every box row is one request to the copy engine, whose request rate -- not bytes --
    // bounds these kernels.  What the unloaded rows of the stage hold only reaches accumulator rows that are never
    // stored.  a_boxes: MN-major A, how many 64-row (8-bit: 128-row) boxes are fetched; stage_tx: bytes per stage.
    int a_boxes;
    uint32_t stage_tx;
    // Narrower tiles on the same kernel (CTA pairs, B with k contiguous, whole tiles): the tile is bn_eff <= BN columns
    // wide -- slot_eff = bn_eff / HALVES per accumulator slot, a multiple of the 128-byte store chunk -- so that a
    // problem's tiles can fill one wave where the next power of two would leave most of a second wave empty.  Shared
    // and tensor memory keep the layout of the full width; each CTA fetches hrows_eff = slot_eff / 2 rows of B per
    // half, and the MMA's N comes from the instruction descriptor.  bn_eff = BN everywhere else.
    int bn_eff, slot_eff, hrows_eff;
    int bulk_exchange;     // one-tile-per-CTA kernel: 1 = k-slices always travel by bulk copies (also for tiles of <= 32 rows)
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

// Two fp32 values -> one 32-bit word of two 16-bit outputs (lo in the low half), round to nearest even.
// The packed conversion is one instruction; converting the halves one by one and merging them made the
// staging of a 32 x 32 chunk three times as long (about 540 instead of 190 cycles per warp).
template <typename TOut> __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    static_assert(sizeof(TOut) == 2, "pack2 packs 16-bit outputs");
    uint32_t d;
    if constexpr (std::is_same<TOut, __nv_bfloat16>::value)
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    else
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
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

// The reverse of stage_row32: 32 consecutive stored values of row `lane` out of a 128-byte-swizzled box that a
// TMA load has filled.
template <typename TOut>
__device__ __forceinline__ void unstage_row32(uint32_t buf, int lane, int h, float (&c)[32]) {
    constexpr int PIECES = 32 * (int)sizeof(TOut) / 16;
    const uint32_t row = buf + (uint32_t)lane * 128u;
#pragma unroll
    for (int j = 0; j < PIECES; ++j) {
        const uint32_t piece = (uint32_t)((h * PIECES + j) ^ (lane & 7));
        uint32_t w[4];
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
                     : "r"(row + piece * 16u)
                     : "memory");
        if constexpr (sizeof(TOut) == 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) c[4 * j + i] = __uint_as_float(w[i]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint16_t lo = (uint16_t)(w[i] & 0xffffu), hi = (uint16_t)(w[i] >> 16);
                c[8 * j + 2 * i] = to_f32(*reinterpret_cast<TOut *>(&lo));
                c[8 * j + 2 * i + 1] = to_f32(*reinterpret_cast<TOut *>(&hi));
            }
        }
    }
}

// Old-C prefetch of one epilogue warp (beta != 0 with TMA stores): chunk c of a tile is loaded by TMA into
// staging buffer c & 1, where the result later overwrites it in place and leaves by a TMA store.
// With two staging buffers per warp (one-group kernels) chunk c uses buffer and barrier c & 1 and the load of
// chunk c + 1 overlaps the work on chunk c; with one buffer per warp (two-group kernels: `single`) the next
// chunk is requested as soon as the store of the current one has read the buffer.
struct CFetch {
    uint32_t bar0;    // mbarrier(s) of this warp, 8 bytes apart
    uint32_t phases;  // bit b: parity the next wait on barrier b uses
    bool on;
    bool single;
};
template <typename T, bool MAP3D>
__device__ __forceinline__ void cfetch_issue(const CFetch &cf, uint32_t my_stage, int c, const CUtensorMap *tm, int x0,
                                             int y0, int z0) {
    constexpr int CHUNK_COLS = 128 / (int)sizeof(T);
    const uint32_t slot = cf.single ? 0u : (uint32_t)(c & 1);
    const uint32_t bar = cf.bar0 + 8u * slot;
    ptx::mbar_arrive_expect_tx(bar, (uint32_t)EPI_BUF_BYTES);
    const uint32_t dst = my_stage + slot * EPI_BUF_BYTES;
    if (MAP3D) ptx::tma_load_3d(dst, tm, x0 + c * CHUNK_COLS, y0, z0, bar);
    else ptx::tma_load_2d(dst, tm, x0 + c * CHUNK_COLS, y0, bar);
}

// tile_coord() in 32-bit arithmetic for the kernels (the host checks that tile counts fit): the 64-bit divisions of the
// general form cost a lone thread about 2700 cycles per tile, which sat between the epilogues of consecutive tiles.
__device__ __forceinline__ void tile_coord32(int tile, int tiles_m, int tiles_n, int group, int &tm, int &tn) {
    const uint32_t grp = (uint32_t)(group < 1 ? 1 : (group > tiles_m ? tiles_m : group));
    const uint32_t per_group = grp * (uint32_t)tiles_n;
    const uint32_t g = (uint32_t)tile / per_group;
    const uint32_t first_m = g * grp;
    const uint32_t left = (uint32_t)tiles_m - first_m;
    const uint32_t rows = left < grp ? left : grp;
    const uint32_t r = (uint32_t)tile - g * per_group;
    const uint32_t q = r / rows;
    tn = (int)q;
    tm = (int)(first_m + (r - q * rows));
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

// The case the plain-store loop of epilogue_tile() handles: C = alpha * acc, TMA stores, nothing fused, no old C.
__device__ __forceinline__ bool plain_store_case(bool tma, bool c_prefetch, float beta, const float *bias, int act,
                                                 const void *rbase) {
    return tma && !c_prefetch && beta == 0.0f && bias == nullptr && act == 0 && rbase == nullptr;
}

// Epilogue of one accumulator tile for one warp: TMEM -> registers -> alpha/beta -> T -> staging + TMA
// store (or direct stores).  `cbase` is the column of chunk 0 used for bounds and addressing, `ncols` the
// column limit, `nrows` the row limit for `row`; (x0, y0[, z0]) is where chunk 0 of this warp lands in `tm`
// (z0 is used when MAP3D says that `tm` is three-dimensional).
// ACC2: the tile's sums are split over two accumulators (t_addr and, when nonzero, t_addr2: two MMA issuers that
// took the k-blocks in turn); they are added as they are read.
// FUSED = false compiles the bias / activation / residual code out: the loop of a plain alpha / beta epilogue then is a
// fraction of the size, which matters to a warp that walks it once per 64 columns.
template <typename T, int BN, bool MAP3D, bool ACC2, bool FUSED>
__device__ __forceinline__ bool epilogue_tile_impl(uint32_t t_addr, uint32_t my_stage, int lane,
                                              T *base, int64_t ld, int row, int row0, int nrows, int cbase,
                                              int ncols, const CUtensorMap *tm, int x0, int y0, int z0, bool tma,
                                              bool vec, float alpha, float beta, const float *bias, int act,
                                              const T *rbase, int64_t ldr, bool rvec, CFetch &cf,
                                              volatile uint32_t *abort_flag, long long wait_cycles,
                                              uint32_t t_addr2, uint32_t release_bar, bool release_remote) {
    constexpr int CHUNK_COLS = 128 / (int)sizeof(T);  // columns per staged chunk: 32 (fp32) or 64 (16-bit)
    if (!FUSED && plain_store_case(tma, cf.on, beta, bias, act, rbase)) {
        // Plain C = alpha * acc through TMA stores, the case that bounds problems with few k-blocks: a loop of its own,
        // small enough to stay in the instruction cache, in which the tensor-memory load of the next chunk is in
        // flight while the current one is fenced and stored.
        constexpr int H = CHUNK_COLS / 32;
        const int left = ncols - cbase;
        const int nchunks = left <= 0 ? 0 : min(BN / CHUNK_COLS, (left + CHUNK_COLS - 1) / CHUNK_COLS);
        // `release_bar` (plain-store case only): the accumulator is handed back to the MMA issuer as soon as its last
        // chunk is in registers, so that the next tile's MMAs run under this tile's last stores
        auto release = [&]() {
            if (release_bar == 0u) return;
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (release_remote) ptx::mbar_arrive_cluster(release_bar);
                else ptx::mbar_arrive(release_bar);
            }
        };
        if (nchunks == 0) { release(); return true; }
        uint32_t r[H][32];
#pragma unroll
        for (int h = 0; h < H; ++h) ptx::tmem_ld_32x32(t_addr + h * 32, r[h]);
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
            const uint32_t buf = my_stage + (!cf.single ? (uint32_t)(c & 1) * EPI_BUF_BYTES : 0u);
            if (lane == 0) {  // the last store out of this buffer has read it (see below for c == 0)
                if (cf.single || c == 0) ptx::tma_store_wait_read<0>();
                else ptx::tma_store_wait_read<1>();
            }
            ptx::tmem_ld_wait();
            if constexpr (ACC2) {
                if (t_addr2 != 0u) {  // the sums of the second MMA issuer
#pragma unroll
                    for (int h = 0; h < H; ++h) {
                        uint32_t r2[32];
                        ptx::tmem_ld_32x32(t_addr2 + c * CHUNK_COLS + h * 32, r2);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[h][i] = __float_as_uint(__uint_as_float(r[h][i]) + __uint_as_float(r2[i]));
                    }
                }
            }
            if (c + 1 == nchunks) release();
            __syncwarp();
#pragma unroll
            for (int h = 0; h < H; ++h) {
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = alpha * __uint_as_float(r[h][i]);
                stage_row32<T>(buf, lane, h, v);
            }
            if (c + 1 < nchunks) {
#pragma unroll
                for (int h = 0; h < H; ++h) ptx::tmem_ld_32x32(t_addr + (c + 1) * CHUNK_COLS + h * 32, r[h]);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && row0 < nrows) {
                if (MAP3D) ptx::tma_store_3d(tm, x0 + c * CHUNK_COLS, y0, z0, buf);
                else ptx::tma_store_2d(tm, x0 + c * CHUNK_COLS, y0, buf);
                ptx::tma_store_commit();
            }
        }
        return true;
    }
#pragma unroll 1
    for (int c = 0; c < BN / CHUNK_COLS; ++c) {
        const int col0 = cbase + c * CHUNK_COLS;
        if (col0 >= ncols) break;  // warp-uniform
        // a warp with two staging buffers alternates between them (with and without prefetched old C)
        const uint32_t buf = my_stage + (!cf.single ? (uint32_t)(c & 1) * EPI_BUF_BYTES : 0u);
        // the whole chunk is requested from tensor memory before the first wait
        uint32_t r[CHUNK_COLS / 32][32];
#pragma unroll
        for (int h = 0; h < CHUNK_COLS / 32; ++h) ptx::tmem_ld_32x32(t_addr + c * CHUNK_COLS + h * 32, r[h]);
        ptx::tmem_ld_wait();
        if constexpr (ACC2) {
            if (t_addr2 != 0u) {
#pragma unroll
                for (int h = 0; h < CHUNK_COLS / 32; ++h) {
                    uint32_t r2[32];
                    ptx::tmem_ld_32x32(t_addr2 + c * CHUNK_COLS + h * 32, r2);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[h][i] = __float_as_uint(__uint_as_float(r[h][i]) + __uint_as_float(r2[i]));
                }
            }
        }
        if (cf.on) {
            // chunks 0 and 1 were requested before the accumulator was waited for; chunk c + 1 (c >= 1) goes
            // into the buffer chunk c - 1 left by a store, which has had this chunk's tensor-memory load to
            // finish reading it
            if (!cf.single && c >= 1 && c + 1 < BN / CHUNK_COLS && cbase + (c + 1) * CHUNK_COLS < ncols) {
                if (lane == 0) {
                    ptx::tma_store_wait_read<0>();
                    cfetch_issue<T, MAP3D>(cf, my_stage, c + 1, tm, x0, y0, z0);
                }
            }
            const uint32_t b = cf.single ? 0u : (uint32_t)(c & 1);
            const bool got = ptx::mbar_wait<false>(cf.bar0 + 8u * b, (cf.phases >> b) & 1u, abort_flag, wait_cycles);
            cf.phases ^= 1u << b;
            if (!__all_sync(0xffffffffu, got)) return false;
        }
#pragma unroll
        for (int h = 0; h < CHUNK_COLS / 32; ++h) {
            const int col = col0 + h * 32;
            const int valid = (ncols - col >= 32) ? 32 : (ncols - col > 0 ? ncols - col : 0);
            T *dst = base + (int64_t)row * ld + col;
            float v[32];
            if (beta != 0.0f) {
                float cold[32];
                if (cf.on) unstage_row32<T>(buf, lane, h, cold);  // out-of-range elements were zero-filled
                else if (row < nrows && valid > 0) load_row32<T>(dst, cold, valid, vec);
                else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) cold[i] = 0.0f;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = fmaf(beta, cold[i], alpha * __uint_as_float(r[h][i]));
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = alpha * __uint_as_float(r[h][i]);
            }
            if (FUSED && bias != nullptr) {  // fused tail: every thread of the warp adds the same 32 bias values
                if (valid == 32 && (reinterpret_cast<uintptr_t>(bias + col) & 15u) == 0) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 b4 = __ldg(reinterpret_cast<const float4 *>(bias + col) + i);
                        v[4 * i] += b4.x; v[4 * i + 1] += b4.y; v[4 * i + 2] += b4.z; v[4 * i + 3] += b4.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < valid) v[i] += __ldg(bias + col + i);
                }
            }
            if (FUSED && act == PEAK_ACT_RELU) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = fmaxf(v[i], 0.0f);
            } else if (FUSED && act == PEAK_ACT_GELU) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = activate_f32(v[i], PEAK_ACT_GELU);
            }
            if (FUSED && rbase != nullptr && row < nrows && valid > 0) {
                // residual: each thread reads its own row's contiguous run (the same access as old C without TMA)
                float rr[32];
                load_row32<T>(rbase + (int64_t)row * ldr + col, rr, valid, rvec);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] += rr[i];
            }
            if (tma) {
                if (h == 0 && !cf.on) {
                    // the last store out of this staging buffer must have read it: with one buffer that is the
                    // previous chunk's, with two the one before (a tile starts with every store read, so that an odd
                    // number of chunks in the previous tile cannot leave this buffer busy)
                    if (lane == 0) {
                        if (cf.single || c == 0) ptx::tma_store_wait_read<0>();
                        else ptx::tma_store_wait_read<1>();
                    }
                    __syncwarp();
                }
                stage_row32<T>(buf, lane, h, v);  // with prefetched C: in place, over this thread's own row
            } else if (row < nrows && valid > 0) store_row32<T>(dst, v, valid, vec);
        }
        if (tma) {
            ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the TMA engine
            __syncwarp();
            if (lane == 0 && row0 < nrows) {
                if (MAP3D) ptx::tma_store_3d(tm, x0 + c * CHUNK_COLS, y0, z0, buf);
                else ptx::tma_store_2d(tm, x0 + c * CHUNK_COLS, y0, buf);
                ptx::tma_store_commit();
                if (cf.on && cf.single && c + 1 < BN / CHUNK_COLS && cbase + (c + 1) * CHUNK_COLS < ncols) {
                    ptx::tma_store_wait_read<0>();  // the one buffer: its store must have read it
                    cfetch_issue<T, MAP3D>(cf, my_stage, c + 1, tm, x0, y0, z0);
                }
            }
        }
    }
    return true;
}

template <typename T, int BN, bool MAP3D = false, bool ACC2 = false>
__device__ __forceinline__ bool epilogue_tile(uint32_t t_addr, uint32_t my_stage, int lane, T *base, int64_t ld, int row,
                                              int row0, int nrows, int cbase, int ncols, const CUtensorMap *tm, int x0,
                                              int y0, int z0, bool tma, bool vec, float alpha, float beta,
                                              const float *bias, int act, const T *rbase, int64_t ldr, bool rvec,
                                              CFetch &cf, volatile uint32_t *abort_flag, long long wait_cycles,
                                              uint32_t t_addr2 = 0u, uint32_t release_bar = 0u,
                                              bool release_remote = false) {
    if (bias != nullptr || act != 0 || rbase != nullptr)
        return epilogue_tile_impl<T, BN, MAP3D, ACC2, true>(t_addr, my_stage, lane, base, ld, row, row0, nrows, cbase, ncols,
                                                            tm, x0, y0, z0, tma, vec, alpha, beta, bias, act, rbase, ldr,
                                                            rvec, cf, abort_flag, wait_cycles, t_addr2, release_bar,
                                                            release_remote);
    return epilogue_tile_impl<T, BN, MAP3D, ACC2, false>(t_addr, my_stage, lane, base, ld, row, row0, nrows, cbase, ncols, tm,
                                                         x0, y0, z0, tma, vec, alpha, beta, nullptr, 0, nullptr, ldr, rvec,
                                                         cf, abort_flag, wait_cycles, t_addr2, release_bar, release_remote);
}

// Epilogue of a tile computed with the operands exchanged (C^T = op(B)^T op(A)^T: the accumulator's rows are
// columns n of C, its columns are rows m): each thread owns one n and walks the m of the tile, so for a fixed m
// the 32 lanes of a warp touch 32 consecutive elements of a row of C -- coalesced without staging.  Bias is
// per column of C, i.e. one value per thread; the residual is read the same way as old C.
template <typename T, int W>
__device__ __forceinline__ void epilogue_tile_swapped(uint32_t t_addr, T *C, int64_t ldc, int n, int n_limit, int m0,
                                                      int m_limit, float alpha, float beta, const float *bias, int act,
                                                      const T *R, int64_t ldr) {
#pragma unroll 1
    for (int c = 0; c < W / 32; ++c) {
        const int mc = m0 + c * 32;
        if (mc >= m_limit) break;  // warp-uniform
        uint32_t r[32];
        ptx::tmem_ld_32x32(t_addr + c * 32, r);
        ptx::tmem_ld_wait();
        if (n < n_limit) {
            const float b = bias ? __ldg(bias + n) : 0.0f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int m = mc + i;
                if (m < m_limit) {
                    T *dst = C + (int64_t)m * ldc + n;
                    float x = alpha * __uint_as_float(r[i]);
                    if (beta != 0.0f) x = fmaf(beta, to_f32(*dst), x);
                    x = activate_f32(x + b, act);
                    if (R) x += to_f32(R[(int64_t)m * ldr + n]);
                    *dst = from_f32<T>(x);
                }
            }
        }
    }
}

// Tile copies: a single GEMM uses two-dimensional descriptors, a strided batch three-dimensional ones.  The
// choice is a template parameter of the kernel: the single-GEMM instantiation carries no trace of the batch
// (three-dimensional descriptors with a batch of one, or a run-time choice, measured 1-10 % slower).
template <int CG, bool BATCHED>
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar) {
    if (BATCHED) {
        if (CG == 1) ptx::tma_load_3d(dst, tm, x, y, z, bar);
        else ptx::tma_load_3d_pair(dst, tm, x, y, z, bar);
    } else {
        if (CG == 1) ptx::tma_load_2d(dst, tm, x, y, bar);
        else ptx::tma_load_2d_pair(dst, tm, x, y, bar);
    }
}

// Hook for the cluster-multicast build (a separate, single-GPU-only translation unit specialises
// McOps<1>; nothing in this header issues a multicast copy).  MC = 1 runs clusters of four CTAs = two CTA
// pairs stacked in M that share every B tile: each CTA fetches one quarter of the pair-wide B tile and
// delivers it to the CTA of the same rank parity in the other pair as well.
template <int MC> struct McOps;
template <> struct McOps<0> {
    __device__ static void load_b_quarter(uint32_t, const CUtensorMap *, int, int, int, uint32_t, uint16_t) {}
};

// IN8: the inputs are 8-bit floats.  A k-block is still one 128-byte swizzle row per matrix row, so it holds
// 128 elements instead of 64, every byte count and descriptor of a K-major operand stays as it is, and the MMA
// is the f8f6f4 kind with K = 32 per instruction.  An MN-major 8-bit operand (A transposed, B not transposed)
// is described to the MMA exactly like a 16-bit one -- major bit in the instruction descriptor, 128-byte
// swizzle, 8-row groups 1 KiB apart -- with every count taken in bytes: a swizzle row holds 128 elements of
// M (or N), a k-block has 128 k-rows, so one box is 128 x 128 bytes = 16 KiB, the boxes of a tile lie 16 KiB
// apart (leading-dimension offset) and one K = 32 instruction advances 32 rows = 4 KiB.
// G2: a one-slot tile is drained by two groups of four epilogue warps, each taking half of the columns.  The
// epilogue of such a tile hides behind the next tile's main loop, so the second group only pays when there is
// no next tile: problems of at most two waves, where it shortens the exposed tail of the launch.
// SWAP: the caller exchanged the operands (the kernel's M is the problem's N and the other way round, see
// launch_swapped): whole tiles are written transposed, straight from registers.
template <int CG, int BN, typename TOut, int MC = 0, bool BATCHED = false, bool IN8 = false, bool G2 = false,
          bool SWAP = false>
__global__ void __launch_bounds__((Cfg<CG, BN>::threads(G2)), 1)
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
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 8 * (2 * STAGES + 4 + 8));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const uint32_t full0 = ptx::smem_u32(bars);
    const uint32_t empty0 = full0 + 8 * STAGES;
    const uint32_t accfull0 = empty0 + 8 * STAGES;
    const uint32_t accempty0 = accfull0 + 16;
    const uint32_t cbar0 = accempty0 + 16;  // old-C barriers: two per epilogue warp of a one-group kernel

    // MN-major operands: elements of M / N per 128-byte swizzle row, and bytes of one box (all k-rows of a
    // k-block under that row)
    constexpr int MN_ELEMS = IN8 ? 128 : 64;
    constexpr int MN_ATOM = IN8 ? 2 * ATOM_BYTES : ATOM_BYTES;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    static_assert(MC == 0 || (CG == 2 && BN >= 256), "the multicast build pairs CTAs and uses 256- or 512-wide tiles");
    constexpr int CLUSTER = MC ? 4 : CG;       // CTAs that work on one (super-)tile together
    const uint32_t crank = (CG == 2) ? ptx::cluster_ctarank() : 0u;
    const uint32_t rank = crank & 1u;          // position inside the CTA pair
    const uint32_t pair = crank >> 1;          // which pair of the cluster (always 0 without multicast)
    const uint32_t leader_crank = crank & ~1u; // cluster rank of this pair's leader
    const bool leader = (rank == 0);
    const int unit = blockIdx.x / CLUSTER;     // cluster index
    const int num_units = gridDim.x / CLUSTER;
    const int total_items = p.total_items;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, MC ? 2 : 1);  // with multicast both pairs must release a stage
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(accfull0 + 8 * b, 1);
            // one arrival per epilogue warp that drains the slot, in every CTA
            ptx::mbar_init(accempty0 + 8 * b, ((C_::HALVES == 1 && G2) ? 8 : 4) * CG);
        }
        for (int b = 0; b < 8; ++b) ptx::mbar_init(cbar0 + 8 * b, 1);
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
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int item = unit; item < total_items && ok; item += num_units, ++tl) {
                const Item w = decode_item(p, item);
                // Every other item walks k downwards.  All CTAs are at about the same k at any time, so what L2
                // holds when a wave of tiles ends is the k-range that was read last; a next wave that starts there
                // (instead of at k = 0, whose panels were read longest ago and are gone) finds the panels it shares
                // with the previous wave still cached.  The order in which k-blocks are accumulated changes
                // with it, but it is a fixed function of the launch, so results stay run-to-run identical.
                const bool rev = p.k_alternate && (tl & 1u);
                const int bz = BATCHED ? w.tile / p.tiles_per_batch : 0;  // matrix of the batch
                int tm, tn;
                tile_coord32(w.tile - bz * p.tiles_per_batch, p.tiles_m, p.tiles_n, p.group, tm, tn);
                const int m_cta = (int)tm * (BM * CLUSTER) + (int)crank * BM;
                const int n_cta = (int)tn * p.bn_eff + (int)rank * p.hrows_eff;  // first B row of this CTA (half 0)
                for (int j = 0, nk = w.kb1 - w.kb0; j < nk; ++j, ++it) {
                    const int kb = rev ? w.kb1 - 1 - j : w.kb0 + j;
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles)) {
                        report_timeout(p, abort_flag, 1, s);
                        ok = false;
                        break;
                    }
                    if (p.inject_stall && unit == 0 && leader && item + num_units >= total_items && j == nk - 1)
                        continue;  // test hook: leave this stage empty so that the waits downstream run out
                    uint32_t bar = full0 + 8 * s;
                    if (leader) ptx::mbar_arrive_expect_tx(bar, p.stage_tx);
                    if (CG == 2) bar = ptx::map_to_cta(bar, leader_crank);
                    const uint32_t a_dst = stage_base + s * C_::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + A_STAGE_BYTES;
                    const int k0 = kb * (IN8 ? 2 * BK : BK);  // element coordinate of the k-block
                    if (!p.a_mn) {
                        load_tile<CG, BATCHED>(a_dst, &tmA, k0, m_cta, bz, bar);
                    } else {
#pragma unroll
                        for (int h = 0; h < BM / MN_ELEMS; ++h) {
                            if (CG == 1 && h >= p.a_boxes) break;
                            load_tile<CG, BATCHED>(a_dst + h * MN_ATOM, &tmA, m_cta + MN_ELEMS * h, k0, bz, bar);
                        }
                    }
                    if (MC) {
                        // this CTA's quarter (64 of the pair-wide tile's 256 columns) goes to itself and to the
                        // CTA of the same parity in the other pair; both layouts use 64 x 64 boxes of 8 KiB
                        const uint16_t mask = (uint16_t)((1u << crank) | (1u << (crank ^ 2u)));
#pragma unroll
                        for (int hf = 0; hf < C_::HALVES; ++hf) {
                            const int n_q = n_cta + hf * p.slot_eff + 64 * (int)pair;
                            McOps<MC>::load_b_quarter(b_dst + hf * C_::HROWS * 128 + pair * ATOM_BYTES, &tmB,
                                                      p.b_mn ? n_q : k0, p.b_mn ? k0 : n_q, bz, bar, mask);
                        }
                    } else if (!p.b_mn) {
#pragma unroll
                        for (int hf = 0; hf < C_::HALVES; ++hf) {
#pragma unroll
                            for (int h = 0; h < C_::HROWS / C_::B_BOX_ROWS; ++h) {
                                const uint32_t d = b_dst + (hf * C_::HROWS + h * C_::B_BOX_ROWS) * 128;
                                const int n = n_cta + hf * p.slot_eff + C_::B_BOX_ROWS * h;
                                load_tile<CG, BATCHED>(d, &tmB, k0, n, bz, bar);
                            }
                        }
                    } else {
#pragma unroll
                        for (int hf = 0; hf < C_::HALVES; ++hf) {
#pragma unroll
                            for (int h = 0; h < C_::HROWS / MN_ELEMS; ++h) {  // (8-bit: HROWS >= 128, host-checked)
                                const uint32_t d = b_dst + hf * C_::HROWS * 128 + h * MN_ATOM;
                                const int n = n_cta + hf * p.slot_eff + MN_ELEMS * h;
                                load_tile<CG, BATCHED>(d, &tmB, n, k0, bz, bar);
                            }
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
            const uint32_t a_lbo = p.a_mn ? (uint32_t)MN_ATOM : 16u, b_lbo = p.b_mn ? (uint32_t)MN_ATOM : 16u;
            // one instruction's K: 32 bytes along a K-major row, or 16 (8-bit: 32) k-rows of 128 bytes
            constexpr uint32_t MN_KSTEP = IN8 ? 4096u : 2048u;
            const uint32_t a_kstep = p.a_mn ? MN_KSTEP : 32u, b_kstep = p.b_mn ? MN_KSTEP : 32u;
            for (int item = unit; item < total_items && ok; item += num_units, ++tl) {
                const Item w = decode_item(p, item);
                const int kb0 = w.kb0, kb1 = w.kb1;
                // one-slot tiles alternate between the two accumulator slots; a two-half tile uses both
                const uint32_t b = (C_::HALVES == 1) ? (tl & 1u) : 0u;
                const uint32_t aph = (C_::HALVES == 1) ? ((tl >> 1) & 1u) : (tl & 1u);
                if (C_::HALVES == 1) {
                    if (!ptx::mbar_wait<CG == 2>(accempty0 + 8 * b, aph ^ 1u, abort_flag, p.wait_cycles)) {
                        report_timeout(p, abort_flag, 3, b);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                }
                // A two-half tile ends with its last k-blocks taken apart: half 0 finishes them first and is
                // handed to its epilogue warps while the tensor cores still work on half 1, which shortens the
                // exposed epilogue by that much.  The stages involved stay unreleased until half 1 has read them,
                // so at most STAGES - 1 k-blocks can be treated this way.
                const int kb_tail = (C_::HALVES == 2) ? max(kb0 + 1, kb1 - (STAGES - 1)) : kb1;
                for (int kb = kb0; kb < kb_tail; ++kb, ++it) {
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
                    for (int hf = 0; hf < C_::HALVES; ++hf) {
                        const uint32_t slot = (C_::HALVES == 1) ? b : (uint32_t)hf;
                        if (C_::HALVES == 2 && kb == kb0) {
                            // the epilogue hands the halves of the previous tile back one after the other
                            if (!ptx::mbar_wait<CG == 2>(accempty0 + 8 * slot, aph ^ 1u, abort_flag, p.wait_cycles)) {
                                report_timeout(p, abort_flag, 3, slot);
                                ok = false;
                                break;
                            }
                            ptx::tc_fence_after_sync();
                        }
                        const uint32_t d_tmem = tmem_base + slot * C_::SLOT_N;
                        const uint32_t bh_base = b_base + hf * C_::HROWS * 128;
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            const uint64_t ad = smem_desc(a_base + k * a_kstep, a_lbo, 1024u);
                            const uint64_t bd = smem_desc(bh_base + k * b_kstep, b_lbo, 1024u);
                            if (IN8) ptx::umma_f8<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > kb0) | (k != 0)));
                            else ptx::umma_f16<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > kb0) | (k != 0)));
                        }
                    }
                    if (!ok) break;
                    // release the stage (in both CTAs of a pair) once these MMAs have read it
                    if (CG == 1) ptx::umma_commit_1cta(empty0 + 8 * s);
                    else ptx::umma_commit_pair(empty0 + 8 * s, MC ? 0xF : 3);
                }
                if (!ok) break;
                if (C_::HALVES == 2) {
#pragma unroll 1
                    for (int hf = 0; hf < 2 && ok; ++hf) {
                        uint32_t jt = it;
                        for (int kb = kb_tail; kb < kb1; ++kb, ++jt) {
                            const uint32_t s = jt % STAGES, ph = (jt / STAGES) & 1u;
                            if (hf == 0) {
                                if (!ptx::mbar_wait<CG == 2>(full0 + 8 * s, ph, abort_flag, p.wait_cycles)) {
                                    report_timeout(p, abort_flag, 4, s);
                                    ok = false;
                                    break;
                                }
                                ptx::tc_fence_after_sync();
                            }
                            const uint32_t a_base = stage_base + s * C_::STAGE_BYTES;
                            const uint32_t bh_base = a_base + A_STAGE_BYTES + hf * C_::HROWS * 128;
                            const uint32_t d_tmem = tmem_base + (uint32_t)hf * C_::SLOT_N;
#pragma unroll
                            for (int k = 0; k < BK / UMMA_K; ++k) {
                                const uint64_t ad = smem_desc(a_base + k * a_kstep, a_lbo, 1024u);
                                const uint64_t bd = smem_desc(bh_base + k * b_kstep, b_lbo, 1024u);
                                if (IN8) ptx::umma_f8<CG>(d_tmem, ad, bd, p.idesc, 1u);
                                else ptx::umma_f16<CG>(d_tmem, ad, bd, p.idesc, 1u);
                            }
                            if (hf == 1) ptx::umma_commit_pair(empty0 + 8 * s, MC ? 0xF : 3);  // two-half tiles are pairs
                        }
                        if (ok) ptx::umma_commit_pair(accfull0 + 8 * hf, (uint16_t)(3u << leader_crank));
                    }
                    if (!ok) break;
                    it += (uint32_t)(kb1 - kb_tail);
                } else {
                    if (CG == 1) ptx::umma_commit_1cta(accfull0 + 8 * b);
                    else ptx::umma_commit_pair(accfull0 + 8 * b, (uint16_t)(3u << leader_crank));
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (4 or 8 warps)
        const int q = warp & 3;          // TMEM lane quadrant this warp may read
        const int grp = (warp - 2) >> 2; // group of four warps: drains half `grp` of a two-half tile
        constexpr bool SPLIT_COLS = C_::HALVES == 1 && G2;             // two groups share one slot
        constexpr int W = SPLIT_COLS ? C_::SLOT_N / 2 : C_::SLOT_N;    // columns a warp drains per tile
        // staging: two buffers per warp in a one-group kernel (old C of chunk c + 1 arrives while chunk c is
        // worked on), one per warp with two groups
        constexpr bool ONE_GROUP = C_::HALVES == 1 && !G2;
        const uint32_t my_stage = epi_base + (uint32_t)(warp - 2) * (ONE_GROUP ? 2u : 1u) * EPI_BUF_BYTES;
        const bool vec = p.vec_ok != 0;
        CFetch cf{ONE_GROUP ? cbar0 + 16u * (uint32_t)(warp - 2) : cbar0 + 8u * (uint32_t)(warp - 2), 0u,
                  p.c_prefetch != 0, !ONE_GROUP};
        CFetch no_cf{0u, 0u, false, !ONE_GROUP};
        uint32_t tl = 0;
        bool ok = true;
        for (int item = unit; item < total_items && ok; item += num_units, ++tl) {
            const Item w = decode_item(p, item);
            const int bz = BATCHED ? w.tile / p.tiles_per_batch : 0;
            int tm, tn;
            tile_coord32(w.tile - bz * p.tiles_per_batch, p.tiles_m, p.tiles_n, p.group, tm, tn);
            const int row0 = (int)tm * (BM * CLUSTER) + (int)crank * BM + q * 32;  // first row of this warp
            const int n0 = (int)tn * p.bn_eff;
            const bool live = row0 < p.M;  // none of this warp's 32 rows exists otherwise: nothing to drain
            {
                const int hf = (C_::HALVES == 2) ? grp : 0;
                const uint32_t b = (C_::HALVES == 1) ? (tl & 1u) : (uint32_t)hf;
                const uint32_t aph = (C_::HALVES == 1) ? ((tl >> 1) & 1u) : (tl & 1u);
                if (cf.on && live && w.ws_block < 0) {
                    // old C of the first two chunks is requested while the main loop still runs
                    constexpr int CC = 128 / (int)sizeof(TOut);
                    const int c0 = n0 + ((C_::HALVES == 2) ? hf * p.slot_eff : (SPLIT_COLS ? grp * W : 0));
                    const int c_end = min(p.N, n0 + ((C_::HALVES == 2) ? (hf + 1) * p.slot_eff : p.bn_eff));  // end of this warp's columns
                    // (a group whose columns start beyond N has no chunk in this tile: nothing to request, or the
                    // barrier would be armed for a wait that never comes)
                    if (lane == 0 && c0 < c_end) {
                        ptx::tma_store_wait_read<0>();  // the previous tile's stores have read the buffer(s)
                        cfetch_issue<TOut, BATCHED>(cf, my_stage, 0, &tmC, c0, row0, bz);
                        if (!cf.single && c0 + CC < c_end && CC < W) cfetch_issue<TOut, BATCHED>(cf, my_stage, 1, &tmC, c0, row0, bz);
                    }
                    if (cf.single) {
                        // the later chunks are fetched one by one between stores: have them wait in L2
                        const int r = row0 + lane;
                        if (r < p.M) {
                            const TOut *row_ptr = reinterpret_cast<const TOut *>(p.C) +
                                                  (BATCHED ? (int64_t)bz * p.stride_c : 0) + (int64_t)r * p.ldc + c0;
#pragma unroll
                            for (int c = CC; c < W; c += CC)
                                if (c0 + c < c_end) ptx::prefetch_l2(row_ptr + c);
                        }
                    }
                    __syncwarp();
                }
                // the outcome is made warp-uniform: tcgen05.ld below needs the whole warp
                const bool got = ptx::mbar_wait<CG == 2>(accfull0 + 8 * b, aph, abort_flag, p.wait_cycles);
                if (!__all_sync(0xffffffffu, got)) {
                    if (lane == 0) report_timeout(p, abort_flag, 5, b);
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const int co = SPLIT_COLS ? grp * W : hf * C_::SLOT_N;  // first accumulator column of this warp's slot
                const int cn = SPLIT_COLS ? grp * W : hf * p.slot_eff;  // ... and the tile column it belongs to
                const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + b * C_::SLOT_N +
                                        (SPLIT_COLS ? (uint32_t)(grp * W) : 0u);
                const int nh = n0 + cn;
                const int n_end = min(p.N, n0 + ((C_::HALVES == 2) ? (hf + 1) * p.slot_eff : p.bn_eff));
                bool released = false;  // the epilogue handed the accumulator back itself
                if (!live) {
                    // rows beyond M: the partial-tile reduction and C never look at them
                } else if (SWAP && w.ws_block < 0) {
                    // whole tile of C^T: this thread's accumulator row is column n = row0 + lane of C
                    epilogue_tile_swapped<TOut, W>(t_addr, reinterpret_cast<TOut *>(p.C), p.ldc, row0 + lane, p.M, nh,
                                                   p.N, p.alpha, p.beta, p.bias, p.act,
                                                   reinterpret_cast<const TOut *>(p.R), p.ldr);
                } else if (w.ws_block < 0) {
                    // whole tile: alpha/beta epilogue straight to C
                    TOut *c_base = reinterpret_cast<TOut *>(p.C);
                    if (BATCHED) c_base += (int64_t)bz * p.stride_c;
                    const uint32_t rel = CG == 1 ? accempty0 + 8 * b : ptx::map_to_cta(accempty0 + 8 * b, leader_crank);
                    released = plain_store_case(p.tma_store != 0, cf.on, p.beta, p.bias, p.act, p.R);
                    if (!epilogue_tile<TOut, W, BATCHED>(t_addr, my_stage, lane, c_base, p.ldc, row0 + lane, row0, p.M,
                                                         nh, n_end, &tmC, nh, row0, bz, p.tma_store != 0, vec, p.alpha,
                                                         p.beta, p.bias, p.act, reinterpret_cast<const TOut *>(p.R),
                                                         p.ldr, p.r_vec != 0, cf, abort_flag, p.wait_cycles, 0u,
                                                         released ? rel : 0u, CG == 2)) {
                        if (lane == 0) report_timeout(p, abort_flag, 6, b);
                        ok = false;
                        break;
                    }
                } else {
                    // k-slice: raw fp32 partial tile to its dense (BM*CG) x BN block of the workspace
                    const int wrow0 = w.ws_block * (BM * CG) + (int)rank * BM + q * 32;
                    epilogue_tile<float, W>(t_addr, my_stage, lane, ws, (int64_t)BN, wrow0 + lane, wrow0,
                                            0x7fffffff, co, BN, &tmW, co, wrow0, 0, true, true, 1.0f, 0.0f, nullptr, 0,
                                            nullptr, 0, false, no_cf, abort_flag, p.wait_cycles);
                }
                // hand the accumulator slot back to the MMA issuer
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !released) {
                    if (CG == 1) ptx::mbar_arrive(accempty0 + 8 * b);
                    else ptx::mbar_arrive_cluster(ptx::map_to_cta(accempty0 + 8 * b, leader_crank));
                }
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
                     int64_t stride_c, int vec_ok, const float *__restrict__ bias, int act,
                     const TOut *__restrict__ R, int64_t ldr, int trans) {
    // trans: the tiles are tiles of C^T (operands exchanged): element (i, j) of the tile grid is C[j][i], the bias
    // belongs to i, and nothing is vectorised
    const int blocks_per_tile = gridDim.y;
    const int t = blockIdx.x;  // split tile number
    const int tiles_per_batch = tiles_m * tiles_n;
    const int gt = full_tiles + t;           // tile number over the whole batch
    const int bz = gt / tiles_per_batch;
    C += (int64_t)bz * stride_c;
    int tm, tn;
    tile_coord32(gt - bz * tiles_per_batch, tiles_m, tiles_n, group, tm, tn);
    const int vec_per_row = bn / 4;
    const int64_t rows_left = (int64_t)M - tm * rows_t;  // rows of this tile that exist
    const int total_vec = (int)(rows_left < rows_t ? rows_left : rows_t) * vec_per_row;
    const int64_t block_elems = (int64_t)rows_t * bn;
    const float *base = ws + (int64_t)t * splits * block_elems;
    // launched as a programmatic dependent of the GEMM kernel: everything above overlapped its tail; the
    // partial tiles may be read only once that kernel has completed
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
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
        if (trans) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (j + k < N) {
                    TOut *d = C + (j + k) * ldc + i;
                    const float c_old = (beta != 0.0f) ? to_f32(*d) : 0.0f;
                    *d = from_f32<TOut>(add_residual(finish_f32(epilogue_f32(alpha, a4[k], beta, c_old), bias, i, act), R,
                                                     (j + k) * ldr + i));
                }
            }
            continue;
        }
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
            for (int k = 0; k < 4; ++k)
                rr[k] = add_residual(finish_f32(epilogue_f32(alpha, a4[k], beta, o[k]), bias, j + k, act), R, i * ldr + j + k);
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
                    dst[k] = from_f32<TOut>(add_residual(finish_f32(epilogue_f32(alpha, a4[k], beta, c_old), bias, j + k, act),
                                                         R, i * ldr + j + k));
                }
            }
        }
    }
}

}  // namespace umma
}  // namespace peak
