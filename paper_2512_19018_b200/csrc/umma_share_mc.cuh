// Single-CTA tiles whose operand tiles are shared inside a thread-block cluster by multicast copies.
// Only the single-GPU plug-in includes this file (it issues multicast bulk-tensor copies and reads nothing but
// this GPU's own memory).
//
// A cluster of CM x CN CTAs computes a (CM*128) x (CN*BN) super-tile, one 128 x BN tile per CTA, one launch, no
// k-split.  The CN CTAs of a cluster row need the same A tile for every k-block and the CM CTAs of a cluster
// column the same B tile: each CTA fetches 1/CN of its row's A tile and 1/CM of its column's B tile and the copy
// engine delivers every piece to all CTAs that need it.  What one SM has to request per k-block drops from
// 16 KiB + BN*128 bytes to 16/CN KiB + BN*128/CM bytes -- the request stream of one SM's copy engine, about
// 40 bytes per clock when the data comes from DRAM, is what bounds problems with few tiles (the paper's
// section 2.2 tiling, with the thread-block tile's operands loaded once per cluster instead of once per block).
//
// Barriers: full[s] of a CTA counts the bytes of a whole stage whoever sends them; empty[s] of a CTA needs one
// arrival from every CTA its copies write to (its row and column peers, itself included), delivered by
// tcgen05.commit with a CTA mask when that CTA's MMAs have read the stage.  Every wait is bounded; a cluster
// barrier at the start makes the peers' barriers valid before anything signals them and one at the end keeps a
// CTA's shared memory alive until no peer can write to it.
#pragma once
#include "umma_device.cuh"

namespace peak {
namespace umma {

__device__ __forceinline__ void tma_load_2d_mc(uint32_t dst, const CUtensorMap *tm, int32_t x, int32_t y, uint32_t bar,
                                               uint16_t mask) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.multicast::cluster"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar), "h"(mask)
        : "memory");
}
// one arrival on the barrier at the same offset in every CTA of `mask` once this thread's MMAs so far are done
__device__ __forceinline__ void umma_commit_1cta_mc(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask)
                 : "memory");
}

template <int BN, int CM, int CN> struct ShareCfg {
    using C_ = Cfg<1, BN>;
    static constexpr int CL = CM * CN;
    static constexpr int A_PART = BM / CN;   // 128-byte rows of the A stage this CTA fetches (for its whole cluster row)
    static constexpr int B_PART = BN / CM;   // rows of the B stage this CTA fetches (for its whole cluster column)
    // warps: 0 producer, 1 MMA issuer, 2..9 two groups of four epilogue warps, 10 second producer, 11 second issuer
    static constexpr int THREADS = 384;
    static constexpr int PRODUCER2 = 10, ISSUER2 = 11;
    // two issuers with an accumulator each take the k-blocks in turn (see umma_clusterk.cuh); 128-wide tiles only
    static constexpr bool DUAL = BN == 128;
    static_assert(CL <= 8 && A_PART >= 32 && B_PART >= 32 && B_PART <= 256, "cluster shape");
};

// One operand part: `part` consecutive 128-byte rows of a stage starting at row `unit0`.  K-major: rows are
// matrix rows (one box).  MN-major: the stage is a sequence of 64-row atoms (64 k-rows under one 128-byte line
// of 64 elements of M / N); a part is a whole number of atoms or a fraction of one.
template <int PART>
__device__ __forceinline__ void load_part(uint32_t stage, const CUtensorMap *tm, bool mn, int mn0, int k0, int unit0,
                                          uint32_t bar, uint16_t mask, bool multicast) {
    if (!mn) {
        const uint32_t dst = stage + (uint32_t)unit0 * 128u;
        if (multicast) tma_load_2d_mc(dst, tm, k0, mn0 + unit0, bar, mask);
        else ptx::tma_load_2d(dst, tm, k0, mn0 + unit0, bar);
    } else {
        constexpr int BOX_K = PART < 64 ? PART : 64;
#pragma unroll
        for (int u = 0; u < PART; u += BOX_K) {
            const int unit = unit0 + u;
            const uint32_t dst = stage + (uint32_t)unit * 128u;
            const int x = mn0 + 64 * (unit / 64), y = k0 + unit % 64;
            if (multicast) tma_load_2d_mc(dst, tm, x, y, bar, mask);
            else ptx::tma_load_2d(dst, tm, x, y, bar);
        }
    }
}

template <int BN, typename TOut, int CM, int CN>
__global__ void __launch_bounds__(384, 1)
umma_share_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
    using C_ = Cfg<1, BN>;
    using S_ = ShareCfg<BN, CM, CN>;
    constexpr int STAGES = C_::STAGES;
    extern __shared__ uint8_t smem_raw[];

    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t stage_base = (raw + 1023u) & ~1023u;
    const uint32_t epi_base = stage_base + STAGES * C_::STAGE_BYTES;
    uint8_t *aux = smem_raw + (epi_base - raw) + EPI_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aux);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 8 * (2 * STAGES + 4 + 8));
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const uint32_t full0 = ptx::smem_u32(bars);
    const uint32_t empty0 = full0 + 8 * STAGES;
    const uint32_t accfull = empty0 + 8 * STAGES;
    const uint32_t cbar0 = accfull + 32;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t crank = ptx::cluster_ctarank();
    const int rm = (int)crank / CN, rn = (int)crank % CN;  // position inside the cluster's CM x CN grid of tiles
    uint16_t row_mask = 0, col_mask = 0;
#pragma unroll
    for (int j = 0; j < CN; ++j) row_mask |= (uint16_t)(1u << (rm * CN + j));
#pragma unroll
    for (int i = 0; i < CM; ++i) col_mask |= (uint16_t)(1u << (i * CN + rn));

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, CM + CN - 1);
        }
        ptx::mbar_init(accfull, S_::DUAL ? 2 : 1);
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
        ptx::tmem_alloc<1>(ptx::smem_u32(tmem_slot), S_::DUAL ? 2 * BN : BN);
        ptx::tmem_relinquish<1>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // the peers' barriers exist before anything signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    // p.tiles_m / p.tiles_n count super-tiles
    int64_t sm_, sn_;
    tile_coord(blockIdx.x / S_::CL, p.tiles_m, p.tiles_n, p.group, sm_, sn_);
    const int m0 = ((int)sm_ * CM + rm) * BM, n0 = ((int)sn_ * CN + rn) * BN;
    const int num_kb = p.num_kb;

    if (warp == 0 || warp == S_::PRODUCER2) {
        // ------------------------------------------------------------------ producers: two warps take the k-blocks in
        // turn; lane 0 fetches this CTA's part of A, lane 1 its part of B, in the same instruction
        const int pw = warp == 0 ? 0 : 1;
        uint32_t it = (uint32_t)pw;
        bool ok = true;
        for (int kb = pw; kb < num_kb && ok; kb += 2, it += 2) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            const uint32_t bar = full0 + 8 * s;
            if (lane == 0) {
                ok = ptx::mbar_wait<true>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles);
                if (!ok) report_timeout(p, abort_flag, 1, s);
                else if (!(p.inject_stall && blockIdx.x == 0 && kb == num_kb - 1))
                    ptx::mbar_arrive_expect_tx(bar, (uint32_t)C_::STAGE_BYTES);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            if (p.inject_stall && blockIdx.x == 0 && kb == num_kb - 1)
                continue;  // test hook: this CTA's parts of the last stage never arrive anywhere
            const uint32_t a_dst = stage_base + s * C_::STAGE_BYTES;
            const int k0 = kb * BK;
            if (lane == 0) load_part<S_::A_PART>(a_dst, &tmA, p.a_mn != 0, m0, k0, rn * S_::A_PART, bar, row_mask, CN > 1);
            else if (lane == 1)
                load_part<S_::B_PART>(a_dst + A_STAGE_BYTES, &tmB, p.b_mn != 0, n0, k0, rm * S_::B_PART, bar, col_mask, CM > 1);
            __syncwarp();
        }
        // every stage this CTA wrote to (here and in its peers) must have been released before it may leave
        if (lane == 0) {
            for (int j = 0; j < STAGES && ok; ++j) {
                // stages whose last use was one of this warp's k-blocks
                const int last = num_kb - 1 - j;
                if (last < 0 || (last & 1) != pw) continue;
                const uint32_t itl = (uint32_t)last + (uint32_t)STAGES, s = itl % STAGES, ph = (itl / STAGES) & 1u;
                if (!ptx::mbar_wait<true>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles)) {
                    report_timeout(p, abort_flag, 2, s);
                    ok = false;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == S_::ISSUER2) {
        // ------------------------------------------------------------------ MMA issuers
        constexpr int NI = S_::DUAL ? 2 : 1;
        const int iw = warp == 1 ? 0 : 1;
        if (lane == 0 && iw < NI) {
            const uint32_t a_lbo = p.a_mn ? (uint32_t)ATOM_BYTES : 16u, b_lbo = p.b_mn ? (uint32_t)ATOM_BYTES : 16u;
            const uint32_t a_kstep = p.a_mn ? 2048u : 32u, b_kstep = p.b_mn ? 2048u : 32u;
            const uint16_t release_mask = (uint16_t)(row_mask | col_mask);
            const uint32_t d_tmem = tmem_base + (uint32_t)(iw * BN);
            uint32_t it = (uint32_t)iw;
            bool ok = true;
            for (int kb = iw; kb < num_kb; kb += NI, it += NI) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                if (!ptx::mbar_wait<true>(full0 + 8 * s, ph, abort_flag, p.wait_cycles)) {
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
                    ptx::umma_f16<1>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > iw) | (k != 0)));
                }
                // release the stage in every CTA whose copies write into it
                umma_commit_1cta_mc(empty0 + 8 * s, release_mask);
            }
            if (ok) ptx::umma_commit_1cta(accfull);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: two groups, half of the columns each
        const int q = warp & 3;
        const int grp = (warp - 2) >> 2;  // warps 2..9
        constexpr int W = BN / 2;
        const uint32_t my_stage = epi_base + (uint32_t)(warp - 2) * EPI_BUF_BYTES;
        const int row0 = m0 + q * 32;
        const int c0 = n0 + grp * W;
        const bool live = row0 < p.M && c0 < p.N;
        CFetch cf{cbar0 + 8u * (uint32_t)(warp - 2), 0u, p.c_prefetch != 0, true};
        if (cf.on && live) {
            if (lane == 0) cfetch_issue<TOut, false>(cf, my_stage, 0, &tmC, c0, row0, 0);
            __syncwarp();
        }
        const bool got = ptx::mbar_wait<false>(accfull, 0u, abort_flag, p.wait_cycles);
        if (!__all_sync(0xffffffffu, got)) {
            if (lane == 0) report_timeout(p, abort_flag, 5, 0);
        } else if (live) {
            ptx::tc_fence_after_sync();
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(grp * W);
            if (S_::DUAL && num_kb >= 2) {
                // add the second issuer's accumulator to the first's
#pragma unroll 1
                for (int c = 0; c < W / 32; ++c) {
                    uint32_t r0[32], r1[32];
                    ptx::tmem_ld_32x32(t_addr + c * 32, r0);
                    ptx::tmem_ld_32x32(t_addr + BN + c * 32, r1);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r0[i] = __float_as_uint(__uint_as_float(r0[i]) + __uint_as_float(r1[i]));
                    ptx::tmem_st_32x32(t_addr + c * 32, r0);
                }
                ptx::tmem_st_wait();
            }
            if (!epilogue_tile<TOut, W, false>(t_addr, my_stage, lane, reinterpret_cast<TOut *>(p.C), p.ldc, row0 + lane,
                                               row0, p.M, c0, p.N, &tmC, c0, row0, 0, p.tma_store != 0, p.vec_ok != 0,
                                               p.alpha, p.beta, p.bias, p.act, reinterpret_cast<const TOut *>(p.R), p.ldr,
                                               p.r_vec != 0, cf, abort_flag, p.wait_cycles)) {
                if (lane == 0) report_timeout(p, abort_flag, 6, 0);
            }
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
        __syncwarp();
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // no peer writes to this CTA's shared memory or barriers after this
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc<1>(tmem_base, S_::DUAL ? 2 * BN : BN);
    }
}

}  // namespace umma
}  // namespace peak
