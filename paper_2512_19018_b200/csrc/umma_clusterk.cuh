// One-tile-per-CTA tensor-core kernel for problems whose tiles all run at once (single-CTA 128 x BN tiles, single
// matrices), with split-K inside the launch (the paper's Split-K transformation, section 4.1, for problems with
// too few tiles to fill the GPU): the KC k-slices of an output tile run on the KC CTAs of a thread-block cluster,
// each with its own fp32 accumulators in tensor memory, and are added through distributed shared memory instead
// of through a workspace and a second kernel.  KC = 1 is the same kernel without a cluster: whole tiles.
//
//   main loop   a ring of 128-byte-swizzled stages fed by TMA and consumed by tcgen05.mma, with the issuing work
//               spread over more threads than in umma_gemm_kernel: two producer warps take the k-blocks in turn
//               and issue the copies of a stage from several lanes in one instruction; with 128-wide tiles two
//               MMA issuers take the k-blocks in turn as well, each accumulating into its own half of tensor
//               memory.  (A 128 x 128 x 64 k-block is 256 tensor cycles, while one thread needs about 540 cycles
//               per k-block for barrier wait, fence, descriptors, four MMAs and commit: measured, the main loop
//               of 512x4096x4096 went from 540 to 413 cycles per k-block, where the operand stream takes over.)
//   exchange    (KC > 1) the tile's BN columns are divided into KC column slices, one per CTA.  When every CTA of
//               the cluster has finished its main loop (a cluster barrier: the stage ring is free everywhere), each
//               epilogue warp stages its 32 rows of every other CTA's slice (both accumulators added) in its own
//               ring, swizzled against bank conflicts, and sends them with one 4 KiB bulk copy per 32-column chunk
//               into a receive area in that CTA's ring; the receiver's mbarrier counts the bytes.  Tiles of at most
//               32 rows skip the staging: plain remote stores into the peers' idle staging buffers and one cluster
//               barrier;
//   reduction   (KC > 1) when all bytes are in, each CTA adds the KC partials of its own slice in slice order
//               0..KC-1 (its own at its position in that order) and writes the sums back to tensor memory;
//   epilogue    the ordinary tile epilogue (alpha/beta, bias, activation, residual, TMA or direct stores) over the
//               slice -- or, for KC = 1, over the whole tile by two groups of four warps that read and add both
//               accumulators.
// The order of the additions is fixed by the launch, so results are run-to-run identical.  Every mbarrier wait
// is bounded; the cluster barriers (after the main loop and before exit) are reached by every thread whether or
// not a wait gave up, so a CTA whose wait ran out cannot leave its peers waiting.
#pragma once
#include "umma_device.cuh"

namespace peak {
namespace umma {

template <int BN, int KC, int CG = 1> struct ClusterKCfg {
    using C_ = Cfg<CG, BN>;
    static constexpr int SW = BN / KC;            // columns each CTA finalises
    static constexpr int CHUNKS = SW / 32;        // 32-column chunks per slice
    // receive area [peer 0..KC-2][chunk][row][128 bytes] and, behind it, a send area of the same shape, both in the ring
    static constexpr int AREA_BYTES = (KC - 1) * CHUNKS * BM * 128;
    static constexpr int RECV_BYTES = 2 * AREA_BYTES;
    // Two MMA issuers, each with an accumulator of its own, take the k-blocks in turn (128-wide tiles: both
    // accumulators fit 256 columns of tensor memory; 256-wide tiles keep one issuer -- a second one, with all of
    // tensor memory for the two accumulators, measured no gain: 512x4096x4096 in two slices 24.2 us against 20.8
    // for whole 128-wide tiles).
    static constexpr bool DUAL = BN == 128;
    static constexpr int TMEM_COLS = 256;         // accumulator columns (+ slack for a 64-wide chunk read)
    // warps: 0 producer, 1 MMA issuer, then GROUPS groups of four epilogue warps, second producer, second issuer.  Whole
    // tiles (KC = 1) are drained by two groups, half of the columns each; a column slice of a split tile by one.
    static constexpr int GROUPS = KC == 1 ? 2 : 1;
    static constexpr int PRODUCER2 = 2 + 4 * GROUPS;
    static constexpr int ISSUER2 = PRODUCER2 + 1;
    static constexpr int THREADS = 32 * (ISSUER2 + 1);
    static_assert(KC == 1 || KC == 2 || KC == 4, "cluster sizes");
    static_assert(CG == 1 || (CG == 2 && KC <= 2 && BN == 128) || (CG == 2 && KC == 1 && BN == 256),
                  "CTA pairs: 256 x 128 tiles, whole or in two k-slices; whole 256 x 256 tiles");
    static_assert(SW % 32 == 0 && SW >= 32, "a slice is a whole number of 32-column chunks");
    static_assert(RECV_BYTES <= C_::STAGES * C_::STAGE_BYTES, "the receive area lives in the stage ring");
    static_assert((DUAL ? 2 : 1) * BN <= TMEM_COLS, "accumulators fit the allocation");
};

// CG = 2: the tile is 256 x BN, computed by a CTA pair (cta_group::2 MMAs issued by the pair's leader; each CTA stages
// its 128 rows of A and its half of the B tile).  BN = 128: a quarter less per SM than two 128 x 128 tiles, which is
// what bounds one-wave problems once the issuing threads are out of the way; whole tiles, or two k-slices on the two
// pairs of a four-CTA cluster (each CTA exchanges its partial sums with the CTA of the same position in the other
// pair).  BN = 256: whole tiles of a problem with at most one tile per pair (one issuer), also p.bn_eff = 192 columns
// wide when B is stored with k contiguous.
template <int BN, typename TOut, int KC, bool IN8, int CG = 1>
__global__ void __launch_bounds__((ClusterKCfg<BN, KC, CG>::THREADS), 1)
umma_clusterk_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmC, const UmmaParams p) {
    using C_ = Cfg<CG, BN>;
    using K_ = ClusterKCfg<BN, KC, CG>;
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
    const uint32_t recvbar = accfull + 8;  // the peers' partial sums of this CTA's slice have arrived
    const uint32_t ackbar = accfull + 16;  // the peers have received what this CTA sent them (bulk copies)
    const uint32_t cbar0 = accfull + 32;

    constexpr int MN_ELEMS = IN8 ? 128 : 64;
    constexpr int MN_ATOM = IN8 ? 2 * ATOM_BYTES : ATOM_BYTES;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t crank = (KC > 1 || CG > 1) ? ptx::cluster_ctarank() : 0u;
    const uint32_t me = crank / CG;            // k-slice of this CTA, and the column slice it finalises
    const uint32_t rank = crank % CG;          // position inside a CTA pair (always 0 for single-CTA tiles)
    const uint32_t leader_crank = crank - rank;
    const bool leader = rank == 0;
    const int tile = blockIdx.x / (KC * CG);
    int64_t tm, tn;
    tile_coord(tile, p.tiles_m, p.tiles_n, p.group, tm, tn);
    // (p.bn_eff < BN: narrower whole tiles of a pair, see UmmaParams; bn_eff = BN otherwise)
    const int m0 = (int)tm * (BM * CG) + (int)rank * BM, n0 = (int)tn * p.bn_eff;
    const int kb0 = (int)me * p.kb_per_split;
    const int kb1 = min(kb0 + p.kb_per_split, p.num_kb);  // the host guarantees kb0 < kb1
    // How the k-slices travel (KC > 1).  A tile with at most 32 rows: the one warp that owns them writes its few
    // values straight into the peers' staging buffers (unused there: only one epilogue warp works), followed by
    // one cluster barrier (measured at 16x4096x4096: 11.8 us, against 12.5 with a remote mbarrier arrival in place
    // of the barrier and 12.9 with bulk copies).  Taller tiles: bulk copies into the peers' rings, which must be
    // free first (cluster barrier after the main loop); the receiver's mbarrier counts the bytes and the senders
    // are told when their staging may go away (256x4096x4096: 17.0 us with per-thread remote stores between two
    // cluster barriers, 16.4 this way).
    const int live_warps = max(0, min(4, (p.M - m0 + 31) / 32));  // (the second CTA of a pair may lie wholly beyond M)
    const bool direct = CG == 1 && KC > 1 && live_warps == 1 && !p.bulk_exchange;  // (pairs: every CTA of a cluster must agree)

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        ptx::mbar_init(accfull, K_::DUAL ? 2 : 1);
        ptx::mbar_init(recvbar, 1);
        ptx::mbar_init(ackbar, KC > 1 ? KC - 1 : 1);
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
        ptx::tmem_alloc<CG>(ptx::smem_u32(tmem_slot), K_::TMEM_COLS);
        ptx::tmem_relinquish<CG>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    // this CTA's barriers exist: tell the peers (k-slices wait for it only when the main loop is over; the CTAs of a
    // pair signal each other's barriers from the first copy on and wait here)
    if (CG == 2) ptx::cluster_sync();
    else if (KC > 1) ptx::cluster_arrive();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's shared and tensor memory and may overlap the previous kernel
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    bool ok = true;
    if (KC > 1 && !direct && live_warps > 0 && threadIdx.x == 0) {
        // what the peers will send: from each of them, for every 32-row block of the tile that exists, one 4 KiB
        // piece per 32-column chunk of this CTA's slice
        ptx::mbar_arrive_expect_tx(recvbar, (uint32_t)((KC - 1) * K_::CHUNKS * live_warps * 4096));
    }

    // epilogue parameters of this warp (meaningful for warps 2 .. PRODUCER2 - 1)
    constexpr int CC = 128 / (int)sizeof(TOut);        // columns per staged chunk
    constexpr int GW = SW / K_::GROUPS;                // columns this warp's group drains
    constexpr int W = GW < CC ? CC : GW;               // a slice narrower than a chunk takes the direct stores
    const int q = warp & 3;                            // TMEM lane quadrant of an epilogue warp
    const int row0 = m0 + q * 32;                      // first row of this warp
    const int grp = (warp - 2) >> 2;
    const bool tma = p.tma_store != 0 && GW >= CC;
    const int c_first = n0 + (int)me * SW + grp * GW;
    const int c_limit = min(min(p.N, n0 + p.bn_eff), c_first + GW);
    // staging: two buffers per warp with one group, one per warp with two
    const uint32_t my_stage = epi_base + (uint32_t)(warp - 2) * (K_::GROUPS == 1 ? 2u : 1u) * EPI_BUF_BYTES;
    CFetch cf{K_::GROUPS == 1 ? cbar0 + 16u * (uint32_t)(warp - 2) : cbar0 + 8u * (uint32_t)(warp - 2), 0u,
              tma && p.c_prefetch != 0, K_::GROUPS == 2};

    if (warp == 0 || warp == K_::PRODUCER2) {
        // ------------------------------------------------------------------ producers
        // Two warps take the k-blocks in turn, and inside a warp every copy of a stage is issued by a lane of its
        // own in one instruction: a copy instruction occupies its thread for a few hundred cycles, and with a
        // 128 x BN tile a k-block is only 2 * BN tensor cycles long, so one thread issuing everything is what
        // bounds the main loop (measured on a copy-only kernel: 1100 cycles per k-block with one thread, 420 with
        // two warps of two lanes).
        const int pw = warp == 0 ? 0 : 1;
        // this lane's copy within a stage: A boxes first, then B boxes
        const int a_ops = p.a_mn ? p.a_boxes : 1;
        const int b_ops = p.b_mn ? C_::HROWS / MN_ELEMS : C_::HROWS / C_::B_BOX_ROWS;
        const bool mine = lane < a_ops + b_ops;
        const bool is_a = lane < a_ops;
        const int h = is_a ? lane : lane - a_ops;
        const CUtensorMap *tmap = is_a ? &tmA : &tmB;
        const bool mn = is_a ? p.a_mn != 0 : p.b_mn != 0;
        const int mn0 = (is_a ? m0 : n0 + (int)rank * p.hrows_eff) + h * (mn ? MN_ELEMS : (is_a ? 0 : C_::B_BOX_ROWS));
        const uint32_t off = (is_a ? 0u : (uint32_t)A_STAGE_BYTES) +
                             (uint32_t)h * (mn ? (uint32_t)MN_ATOM : (uint32_t)(C_::B_BOX_ROWS * 128));
        uint32_t it = (uint32_t)pw;
        for (int kb = kb0 + pw; kb < kb1; kb += 2, it += 2) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            // the bytes of a stage are counted by the barrier of the pair's leader (its own, for single-CTA tiles)
            const uint32_t bar = CG == 2 ? ptx::map_to_cta(full0 + 8 * s, leader_crank) : full0 + 8 * s;
            bool go = true;
            if (lane == 0) {
                go = ptx::mbar_wait<CG == 2>(empty0 + 8 * s, ph ^ 1u, abort_flag, p.wait_cycles);
                if (!go) report_timeout(p, abort_flag, 1, s);
                else if (leader && !(p.inject_stall && blockIdx.x == 0 && kb == kb1 - 1))
                    ptx::mbar_arrive_expect_tx(full0 + 8 * s, p.stage_tx);
            }
            go = __shfl_sync(0xffffffffu, go, 0);
            if (!go) break;
            if (p.inject_stall && blockIdx.x == 0 && kb == kb1 - 1)
                continue;  // test hook: leave this stage empty so that the waits downstream run out
            if (mine) {
                const int k0 = kb * (IN8 ? 2 * BK : BK);
                const uint32_t dst = stage_base + s * C_::STAGE_BYTES + off;
                if (CG == 2) ptx::tma_load_2d_pair(dst, tmap, mn ? mn0 : k0, mn ? k0 : mn0, bar);
                else ptx::tma_load_2d(dst, tmap, mn ? mn0 : k0, mn ? k0 : mn0, bar);  // one instruction for all lanes
            }
            __syncwarp();
        }
    } else if (warp == 1 || warp == K_::ISSUER2) {
        // ------------------------------------------------------------------ MMA issuers
        // With 128-wide tiles the four MMAs of a k-block keep the tensor pipe busy for about 380 cycles while the
        // issuing thread needs about 540 per k-block (barrier wait, fence, descriptors, commit), so two threads
        // take the k-blocks in turn, each accumulating into its own half of tensor memory; the halves are added
        // when the accumulators are read.
        constexpr int NI = K_::DUAL ? 2 : 1;
        const int iw = warp == 1 ? 0 : 1;
        if (lane == 0 && iw < NI && leader) {
            const uint32_t a_lbo = p.a_mn ? (uint32_t)MN_ATOM : 16u, b_lbo = p.b_mn ? (uint32_t)MN_ATOM : 16u;
            constexpr uint32_t MN_KSTEP = IN8 ? 4096u : 2048u;
            const uint32_t a_kstep = p.a_mn ? MN_KSTEP : 32u, b_kstep = p.b_mn ? MN_KSTEP : 32u;
            const uint32_t d_tmem = tmem_base + (uint32_t)(iw * BN);
            uint32_t it = (uint32_t)iw;
            bool mma_ok = true;
            for (int kb = kb0 + iw; kb < kb1; kb += NI, it += NI) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                if (!ptx::mbar_wait<CG == 2>(full0 + 8 * s, ph, abort_flag, p.wait_cycles)) {
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
                    if (IN8) ptx::umma_f8<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > kb0 + iw) | (k != 0)));
                    else ptx::umma_f16<CG>(d_tmem, ad, bd, p.idesc, (uint32_t)((kb > kb0 + iw) | (k != 0)));
                }
                // release the stage (in both CTAs of a pair) once these MMAs have read it
                if (CG == 1) ptx::umma_commit_1cta(empty0 + 8 * s);
                else ptx::umma_commit_pair(empty0 + 8 * s, (uint16_t)(3u << leader_crank));
            }
            // (an issuer without k-blocks arrives at once)
            if (mma_ok) {
                if (CG == 1) ptx::umma_commit_1cta(accfull);
                else ptx::umma_commit_pair(accfull, (uint16_t)(3u << leader_crank));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue warps: old C of the first chunk(s)
        // is requested while the main loop runs (beta != 0 with TMA stores); then wait for the accumulator
        if (cf.on && row0 < p.M && c_first < p.N && lane == 0) {
            cfetch_issue<TOut, false>(cf, my_stage, 0, &tmC, c_first, row0, 0);
            if (!cf.single && c_first + CC < c_limit) cfetch_issue<TOut, false>(cf, my_stage, 1, &tmC, c_first, row0, 0);
        }
        __syncwarp();
        const bool got = ptx::mbar_wait<CG == 2>(accfull, 0u, abort_flag, p.wait_cycles);
        ok = __all_sync(0xffffffffu, got);
        if (!ok && lane == 0) report_timeout(p, abort_flag, 5, 0);
        ptx::tc_fence_after_sync();
    }

    if (KC > 1) {
        if (CG == 1) ptx::cluster_wait(); // the peers' barriers exist (they arrived long ago; pairs waited at the start)
        if (!direct) ptx::cluster_sync(); // every CTA's main loop is over (or has given up): every ring may be overwritten
    }

    const bool live = warp >= 2 && warp < K_::PRODUCER2 && ok && row0 < p.M;
    const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
    const int trow = q * 32 + lane;               // row inside the tile
    // this CTA's partial sums of 32 columns: the first issuer's accumulator plus, when the second issuer had
    // k-blocks of its own, the second's
    const bool two_acc = K_::DUAL && kb1 - kb0 >= 2;
    auto load_partial = [&](int col, uint32_t (&r)[32]) {
        ptx::tmem_ld_32x32(t_row + (uint32_t)col, r);
        if (two_acc) {
            uint32_t r2[32];
            ptx::tmem_ld_32x32(t_row + (uint32_t)(BN + col), r2);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
        } else {
            ptx::tmem_ld_wait();
        }
    };
    bool exchange_ok = true;
    if (live && KC > 1) {
        // ------------------------------------------------------------------ exchange
        if (direct) {
            // slot i of the receive area: 4 KiB pieces in the staging buffers the idle epilogue warps do not use
            // (the one working warp, quadrant 0, owns bytes 16..24 KiB of the 32 KiB)
#pragma unroll 1
            for (int dd = 1; dd < KC; ++dd) {
                const uint32_t d = (me + (uint32_t)dd) % KC;
                const int ord_there = KC - 1 - dd;
#pragma unroll 1
                for (int c = 0; c < K_::CHUNKS; ++c) {
                    uint32_t r[32];
                    load_partial((int)d * SW + c * 32, r);
                    if (m0 + trow < p.M) {
                        const int slot = ord_there * K_::CHUNKS + c;
                        const uint32_t local = epi_base + (uint32_t)((slot < 4 ? slot : slot + 2) * 4096 + lane * 128);
                        const uint32_t remote = ptx::map_to_cta(local, d * CG + rank);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            ptx::st_cluster_v4(remote + (uint32_t)((j ^ (lane & 7)) * 16), r[4 * j], r[4 * j + 1], r[4 * j + 2],
                                               r[4 * j + 3]);
                    }
                }
            }
        } else {
        // Each warp stages its 32 rows of a peer's slice in this CTA's own ring (free since its accumulators are
        // complete) and sends them with one bulk copy per 32-column chunk; the peer's barrier counts the bytes.
#pragma unroll 1
        for (int dd = 1; dd < KC; ++dd) {
            const uint32_t d = (me + (uint32_t)dd) % KC;  // start with the neighbour: the CTAs write to different peers
            const int ord_there = KC - 1 - dd;            // this CTA's place among d's peers: (me - d - 1) mod KC
#pragma unroll 1
            for (int c = 0; c < K_::CHUNKS; ++c) {
                uint32_t r[32];
                load_partial((int)d * SW + c * 32, r);
                const uint32_t row = stage_base + (uint32_t)K_::AREA_BYTES +
                                     (uint32_t)((((dd - 1) * K_::CHUNKS + c) * BM + trow) * 128);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (uint32_t)((j ^ (trow & 7)) * 16)),
                                 "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3])
                                 : "memory");
            }
            ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the bulk copy
            __syncwarp();
            if (lane == 0) {
                const uint32_t bar_there = ptx::map_to_cta(recvbar, d * CG + rank);
#pragma unroll 1
                for (int c = 0; c < K_::CHUNKS; ++c) {
                    const uint32_t src = stage_base + (uint32_t)K_::AREA_BYTES +
                                         (uint32_t)((((dd - 1) * K_::CHUNKS + c) * BM + q * 32) * 128);
                    const uint32_t dst = stage_base + (uint32_t)(((ord_there * K_::CHUNKS + c) * BM + q * 32) * 128);
                    ptx::bulk_copy_to_cluster(ptx::map_to_cta(dst, d * CG + rank), src, 4096u, bar_there);
                }
            }
        }
        }
        // the peers' partial sums of this CTA's slice: all bytes in (bounded wait)
        const bool arrived = direct || ptx::mbar_wait<true>(recvbar, 0u, abort_flag, p.wait_cycles);
        if (!__all_sync(0xffffffffu, arrived)) {
            if (lane == 0) report_timeout(p, abort_flag, 7, 0);
            exchange_ok = false;
        } else if (!direct && q == 0 && lane == 0) {
            // everything the peers sent has been written here, so their send areas are no longer read: tell them
            for (int dd = 1; dd < KC; ++dd)
                ptx::mbar_arrive_cluster(ptx::map_to_cta(ackbar, ((me + (uint32_t)dd) % KC) * CG + rank));
        }
    }

    if (direct) ptx::cluster_sync();  // the few values of a short tile have been stored everywhere (release / acquire)
    if (live && exchange_ok) {
        // ------------------------------------------------------------------ reduction of this CTA's slice
#pragma unroll 1
        for (int c = 0; c < K_::CHUNKS && KC > 1; ++c) {
            uint32_t own[32];
            const uint32_t t_addr = t_row + me * SW + c * 32;
            load_partial((int)me * SW + c * 32, own);
            float acc[32];
#pragma unroll 1
            for (uint32_t src = 0; src < (uint32_t)KC; ++src) {
                float v[32];
                if (src == me) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(own[i]);
                } else {
                    const int ord = ((int)src - (int)me - 1 + KC) % KC;  // src's place among this CTA's peers
                    const int slot = ord * K_::CHUNKS + c;
                    const uint32_t rowaddr = direct ? epi_base + (uint32_t)((slot < 4 ? slot : slot + 2) * 4096 + lane * 128)
                                                    : stage_base + (uint32_t)((ord * K_::CHUNKS + c) * BM + trow) * 128u;
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
        if (c_first < p.N) {
            const uint32_t t_first = t_row + me * SW + (uint32_t)(grp * GW);
            // a whole tile (KC = 1) is read from both issuers' accumulators; a slice's sums were written back above
            const uint32_t t_second = (KC == 1 && two_acc) ? t_first + BN : 0u;
            if (!epilogue_tile<TOut, W, false, KC == 1>(t_first, my_stage, lane, reinterpret_cast<TOut *>(p.C), p.ldc,
                                                        row0 + lane, row0, p.M, c_first, c_limit, &tmC, c_first, row0, 0, tma,
                                                        p.vec_ok != 0, p.alpha, p.beta, p.bias, p.act,
                                                        reinterpret_cast<const TOut *>(p.R), p.ldr, p.r_vec != 0, cf,
                                                        abort_flag, p.wait_cycles, t_second)) {
                if (lane == 0) report_timeout(p, abort_flag, 6, 0);
            }
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();  // staging memory must outlive the stores
        __syncwarp();
    }

    // ---------------------------------------------------------------------- teardown
    if (KC > 1 && !direct && warp >= 2 && warp < K_::PRODUCER2 && (warp & 3) == 0 && lane == 0) {
        // this CTA's send area must outlive the bulk copies that read it: every peer has acknowledged receipt
        // (a CTA whose rows all lie beyond M sent nothing and is owed nothing)
        if (ok && exchange_ok && m0 < p.M && !ptx::mbar_wait<true>(ackbar, 0u, abort_flag, p.wait_cycles))
            report_timeout(p, abort_flag, 8, 0);
    }
    __syncwarp();
    if (*abort_flag != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (CG == 2) ptx::cluster_sync();  // the peer may still signal this CTA's barriers or read its tiles
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc<CG>(tmem_base, K_::TMEM_COLS);
    }
}

}  // namespace umma
}  // namespace peak
