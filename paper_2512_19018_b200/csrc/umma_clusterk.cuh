// Split-K inside one launch (the paper's Split-K transformation, section 4.1, for problems with too few tiles
// to fill the GPU): the KC k-slices of an output tile run on the KC CTAs of a thread-block cluster, each with
// its own fp32 accumulator in tensor memory, and are added through distributed shared memory instead of through
// a workspace and a second kernel.
//
//   main loop   as in umma_gemm_kernel with single-CTA tiles: warp 0 feeds a ring of 128-byte-swizzled stages by
//               TMA, one thread of warp 1 issues tcgen05.mma over this CTA's k-blocks;
//   exchange    the tile's BN columns are divided into KC column slices, one per CTA.  When every CTA of the
//               cluster has finished its main loop (cluster barrier 1: the stage ring is free everywhere), each
//               epilogue thread copies, for every other CTA d, its row of slice d from tensor memory into a
//               receive area in CTA d's ring (st.shared::cluster, swizzled like the staging buffers so that the
//               32 lanes of a warp hit different banks);
//   reduction   after cluster barrier 2 each CTA adds the KC partials of its own slice in slice order 0..KC-1
//               (its own from tensor memory at its position in that order), writes the sums back to tensor
//               memory and runs the ordinary tile epilogue (alpha/beta, bias, activation, residual, TMA or
//               direct stores) over its slice.
// The order of the additions is fixed by the launch, so results are run-to-run identical.  Every mbarrier wait
// is bounded; the two cluster barriers are reached by every thread whether or not a wait gave up, so a CTA
// whose wait ran out cannot leave its peers waiting.
#pragma once
#include "umma_device.cuh"

namespace peak {
namespace umma {

template <int BN, int KC> struct ClusterKCfg {
    using C_ = Cfg<1, BN>;
    static constexpr int SW = BN / KC;            // columns each CTA finalises
    static constexpr int CHUNKS = SW / 32;        // 32-column chunks per slice
    static constexpr int RECV_BYTES = KC * CHUNKS * BM * 128;  // [source CTA][chunk][row][128 bytes]
    static constexpr int TMEM_COLS = 256;         // BN accumulator columns (+ slack for a 64-wide chunk read)
    static constexpr int THREADS = 192;
    static_assert(SW % 32 == 0 && SW >= 32, "a slice is a whole number of 32-column chunks");
    static_assert(RECV_BYTES <= C_::STAGES * C_::STAGE_BYTES, "the receive area lives in the stage ring");
    static_assert(BN + 32 <= TMEM_COLS || SW >= 64, "a 16-bit chunk read may look 32 columns past the slice");
};

template <int BN, typename TOut, int KC, bool IN8>
__global__ void __launch_bounds__(192, 1)
umma_clusterk_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
    using C_ = Cfg<1, BN>;
    using K_ = ClusterKCfg<BN, KC>;
    constexpr int STAGES = C_::STAGES;
    constexpr int SW = K_::SW;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t stage_base = (raw + 1023u) & ~1023u;
    const uint32_t epi_base = stage_base + STAGES * C_::STAGE_BYTES;
    uint8_t *aux = smem_raw + (epi_base - raw) + EPI_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aux);  // full[S], empty[S], acc_full, (unused), old-C barriers
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 8 * (2 * STAGES + 4 + 8));
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const uint32_t full0 = ptx::smem_u32(bars);
    const uint32_t empty0 = full0 + 8 * STAGES;
    const uint32_t accfull = empty0 + 8 * STAGES;
    const uint32_t cbar0 = accfull + 32;

    constexpr int MN_ELEMS = IN8 ? 128 : 64;
    constexpr int MN_ATOM = IN8 ? 2 * ATOM_BYTES : ATOM_BYTES;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t me = ptx::cluster_ctarank();  // k-slice of this CTA, and the column slice it finalises
    const int tile = blockIdx.x / KC;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        ptx::mbar_init(accfull, 1);
        for (int b = 0; b < 8; ++b) ptx::mbar_init(cbar0 + 8 * b, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0 && lane == 0) {
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
        if (p.tma_store) ptx::prefetch_tensormap(&tmC);
    }
    if (warp == 1) {
        ptx::tmem_alloc<1>(ptx::smem_u32(tmem_slot), K_::TMEM_COLS);
        ptx::tmem_relinquish<1>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's shared and tensor memory and may overlap the previous kernel
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    int64_t tm, tn;
    tile_coord(tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
    const int m0 = (int)tm * BM, n0 = (int)tn * BN;
    const int kb0 = (int)me * p.kb_per_split;
    const int kb1 = min(kb0 + p.kb_per_split, p.num_kb);  // the host guarantees kb0 < kb1
    bool ok = true;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                if (!ptx::mbar_wait<false>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles)) {
                    report_timeout(p, abort_flag, 1, s);
                    break;
                }
                if (p.inject_stall && blockIdx.x == 0 && kb == kb1 - 1)
                    continue;  // test hook: leave this stage empty so that the waits downstream run out
                const uint32_t bar = full0 + 8 * s;
                ptx::mbar_arrive_expect_tx(bar, p.stage_tx);
                const uint32_t a_dst = stage_base + s * C_::STAGE_BYTES;
                const uint32_t b_dst = a_dst + A_STAGE_BYTES;
                const int k0 = kb * (IN8 ? 2 * BK : BK);
                if (!p.a_mn) {
                    ptx::tma_load_2d(a_dst, &tmA, k0, m0, bar);
                } else {
#pragma unroll
                    for (int h = 0; h < BM / MN_ELEMS; ++h) {
                        if (h >= p.a_boxes) break;
                        ptx::tma_load_2d(a_dst + h * MN_ATOM, &tmA, m0 + MN_ELEMS * h, k0, bar);
                    }
                }
                if (!p.b_mn) {
#pragma unroll
                    for (int h = 0; h < C_::HROWS / C_::B_BOX_ROWS; ++h)
                        ptx::tma_load_2d(b_dst + h * C_::B_BOX_ROWS * 128, &tmB, k0, n0 + C_::B_BOX_ROWS * h, bar);
                } else {
#pragma unroll
                    for (int h = 0; h < C_::HROWS / MN_ELEMS; ++h)
                        ptx::tma_load_2d(b_dst + h * MN_ATOM, &tmB, n0 + MN_ELEMS * h, k0, bar);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t a_lbo = p.a_mn ? (uint32_t)MN_ATOM : 16u, b_lbo = p.b_mn ? (uint32_t)MN_ATOM : 16u;
            constexpr uint32_t MN_KSTEP = IN8 ? 4096u : 2048u;
            const uint32_t a_kstep = p.a_mn ? MN_KSTEP : 32u, b_kstep = p.b_mn ? MN_KSTEP : 32u;
            uint32_t it = 0;
            bool mma_ok = true;
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                if (!ptx::mbar_wait<false>(full0 + 8 * s, ph, abort_flag, p.wait_cycles)) {
                    report_timeout(p, abort_flag, 4, s);
                    mma_ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t a_base = stage_base + s * C_::STAGE_BYTES;
                const uint32_t b_base = a_base + A_STAGE_BYTES;
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    const uint64_t ad = smem_desc(a_base + k * a_kstep, a_lbo, 1024u);
                    const uint64_t bd = smem_desc(b_base + k * b_kstep, b_lbo, 1024u);
                    if (IN8) ptx::umma_f8<1>(tmem_base, ad, bd, p.idesc, (uint32_t)((kb > kb0) | (k != 0)));
                    else ptx::umma_f16<1>(tmem_base, ad, bd, p.idesc, (uint32_t)((kb > kb0) | (k != 0)));
                }
                ptx::umma_commit_1cta(empty0 + 8 * s);
            }
            if (mma_ok) ptx::umma_commit_1cta(accfull);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps: wait for the accumulator
        const bool got = ptx::mbar_wait<false>(accfull, 0u, abort_flag, p.wait_cycles);
        ok = __all_sync(0xffffffffu, got);
        if (!ok && lane == 0) report_timeout(p, abort_flag, 5, 0);
        ptx::tc_fence_after_sync();
    }

    // cluster barrier 1: every CTA's main loop is over (or has given up), so every stage ring may be overwritten
    ptx::cluster_sync();

    const int q = warp & 3;                       // TMEM lane quadrant of an epilogue warp
    const int row0 = m0 + q * 32;                 // first row of this warp
    const bool live = warp >= 2 && ok && row0 < p.M;
    const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
    const int trow = q * 32 + lane;               // row inside the tile
    if (live) {
        // ------------------------------------------------------------------ exchange
#pragma unroll 1
        for (int dd = 1; dd < KC; ++dd) {
            const uint32_t d = (me + (uint32_t)dd) % KC;  // start with the neighbour: the CTAs write to different peers
#pragma unroll 1
            for (int c = 0; c < K_::CHUNKS; ++c) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(t_row + d * SW + c * 32, r);
                ptx::tmem_ld_wait();
                if (m0 + trow < p.M) {
                    const uint32_t local = stage_base + (uint32_t)(((int)me * K_::CHUNKS + c) * BM + trow) * 128u;
                    const uint32_t remote = ptx::map_to_cta(local, d);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        ptx::st_cluster_v4(remote + (uint32_t)((j ^ (trow & 7)) * 16), r[4 * j], r[4 * j + 1], r[4 * j + 2],
                                           r[4 * j + 3]);
                }
            }
        }
    }

    // cluster barrier 2: all partials have arrived (release / acquire at cluster scope)
    ptx::cluster_sync();

    if (live) {
        // ------------------------------------------------------------------ reduction of this CTA's slice
#pragma unroll 1
        for (int c = 0; c < K_::CHUNKS; ++c) {
            uint32_t own[32];
            const uint32_t t_addr = t_row + me * SW + c * 32;
            ptx::tmem_ld_32x32(t_addr, own);
            ptx::tmem_ld_wait();
            float acc[32];
#pragma unroll 1
            for (uint32_t src = 0; src < (uint32_t)KC; ++src) {
                float v[32];
                if (src == me) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(own[i]);
                } else {
                    const uint32_t rowaddr = stage_base + (uint32_t)(((int)src * K_::CHUNKS + c) * BM + trow) * 128u;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t w0, w1, w2, w3;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                                     : "r"(rowaddr + (uint32_t)((j ^ (trow & 7)) * 16))
                                     : "memory");
                        v[4 * j] = __uint_as_float(w0); v[4 * j + 1] = __uint_as_float(w1);
                        v[4 * j + 2] = __uint_as_float(w2); v[4 * j + 3] = __uint_as_float(w3);
                    }
                }
                if (src == 0) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] = v[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] += v[i];
                }
            }
            uint32_t out[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) out[i] = __float_as_uint(acc[i]);
            ptx::tmem_st_32x32(t_addr, out);
        }
        ptx::tmem_st_wait();
        // ------------------------------------------------------------------ tile epilogue over the slice
        constexpr int CC = 128 / (int)sizeof(TOut);        // columns per staged chunk
        constexpr int W = SW < CC ? CC : SW;               // a slice narrower than a chunk takes the direct stores
        const bool tma = p.tma_store != 0 && SW >= CC;
        const int c_first = n0 + (int)me * SW;
        const int c_limit = min(p.N, c_first + SW);
        const uint32_t my_stage = epi_base + (uint32_t)(warp - 2) * 2u * EPI_BUF_BYTES;
        CFetch cf{cbar0 + 16u * (uint32_t)(warp - 2), 0u, tma && p.c_prefetch != 0, false};
        if (c_first < p.N) {
            if (cf.on && lane == 0) {
                cfetch_issue<TOut, false>(cf, my_stage, 0, &tmC, c_first, row0, 0);
                if (c_first + CC < c_limit) cfetch_issue<TOut, false>(cf, my_stage, 1, &tmC, c_first, row0, 0);
            }
            __syncwarp();
            if (!epilogue_tile<TOut, W, false>(t_row + me * SW, my_stage, lane, reinterpret_cast<TOut *>(p.C), p.ldc,
                                               row0 + lane, row0, p.M, c_first, c_limit, &tmC, c_first, row0, 0, tma,
                                               p.vec_ok != 0, p.alpha, p.beta, p.bias, p.act,
                                               reinterpret_cast<const TOut *>(p.R), p.ldr, p.r_vec != 0, cf, abort_flag,
                                               p.wait_cycles)) {
                if (lane == 0) report_timeout(p, abort_flag, 6, 0);
            }
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();  // staging memory must outlive the stores
        __syncwarp();
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc<1>(tmem_base, K_::TMEM_COLS);
    }
}

}  // namespace umma
}  // namespace peak
