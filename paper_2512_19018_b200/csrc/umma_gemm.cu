// Tensor-core GEMM for 16-bit (and 8-bit float) inputs on sm_100a: host side (plan, dispatch rules, launch,
// workspace, entry points).
// The kernels are in umma_device.cuh.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_device.cuh"
#include "umma_clusterk.cuh"
#include "umma_host.cuh"
#include "mc_plugin.h"

#include <dlfcn.h>

#include <string>

namespace peak {
namespace {

using namespace umma;

// ---- optional single-GPU plug-in (cluster-multicast B loads), loaded from beside this library ------------
peak_mc_max_clusters_fn g_mc_max_clusters = nullptr;
peak_mc_gemm_fn mc_entry() {
    static peak_mc_gemm_fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        Dl_info info;
        if (!dladdr(reinterpret_cast<void *>(&mc_entry), &info) || !info.dli_fname) return;
        std::string path(info.dli_fname);
        const size_t slash = path.find_last_of('/');
        path = (slash == std::string::npos ? std::string(".") : path.substr(0, slash)) + "/libpeak_gemm_mc.so";
        void *h = dlopen(path.c_str(), RTLD_NOW | RTLD_LOCAL);
        if (!h) return;
        fn = reinterpret_cast<peak_mc_gemm_fn>(dlsym(h, "peak_mc_gemm"));
        g_mc_max_clusters = reinterpret_cast<peak_mc_max_clusters_fn>(dlsym(h, "peak_mc_max_clusters"));
    });
    return fn;
}
int mc_max_clusters(int tile_n) {
    return (mc_entry() && g_mc_max_clusters) ? g_mc_max_clusters(tile_n) : 0;
}

constexpr double kL2BytesPerClk = 40.0;        // L2 -> shared-memory bytes per cycle one SM sustains (measured ~39)
constexpr double kSplitFixedCycles = 20000.0;  // workspace allocation + second launch of a split (~12 us)

struct Plan {
    int bn;           // tile width the kernel is instantiated for: 512, 256 or 128
    int full_tiles;   // tiles computed whole
    int tail_splits;  // k-slices of each remaining tile (1 when nothing is split)
    int bn_eff = 0;   // columns of a tile actually computed (0 = bn): 192 on the 256-wide kernel, 384 on the 512-wide one
};

// Tiles of the whole call (all matrices of a strided batch).
int64_t tiles_of(const GemmArgs &g, int cg, int bn) {
    return ((g.M + BM * cg - 1) / (BM * cg)) * ((g.N + bn - 1) / bn) * g.nbatch();
}

// Clusters of KC single-CTA tiles of width bn that can be resident at once on the current device (umma_clusterk.cuh).
int clusterk_max_clusters(int bn, int kc);

// Tile width and k-splitting from a small cost model (cycles): an item costs its k-blocks times the slower
// of the tensor pipe (2*BN cycles per k-block per SM) and the operand stream (bytes per k-block over an
// about 40 bytes/cycle/SM of L2->shared bandwidth), plus a fixed per-item overhead; items are spread over
// the units in waves.  Splitting additionally pays for writing and re-reading fp32 partials and for the
// second launch.  Candidates: no split; every tile split s ways (few tiles); only the last wave split.
Plan choose_plan(const GemmArgs &g, int cg, int units) {
    const int bke = is_fp8(in_elem(g.dtype)) ? 2 * BK : BK;  // elements per k-block (one 128-byte row)
    const int64_t num_kb = (g.K + bke - 1) / bke;
    Plan best{256, 0, 1};
    double best_cost = 1e300;
    const int force_bn = tuning(PEAK_TUNE_TILE_N), force_split = tuning(PEAK_TUNE_SPLIT_K);
    const int tail_mode = tuning(PEAK_TUNE_TAIL_SPLIT);  // 2 = split the last wave whenever possible
    // Single matrices whose 128 x 128 tiles fill between an eighth and all of the SMs: k-slices on the CTAs of a
    // cluster cost one launch and no workspace, so the rule is simply the most CTAs that still run at once --
    // measured (NT, us; best other plan in brackets): 128x7168x4096 two slices 18.6 (20.4), 256x4096x4096 two slices
    // 17.8 (20.2), 128x4096x8192 four slices 20.0 (21.8), 64x4096x4096 four slices 12.6 (14.8), 128x14336x4096
    // whole tiles 29.3 (30.9).  Each slice keeps at least eight k-blocks.
    if (cg == 1 && g.nbatch() == 1 && !force_bn && !force_split && tail_mode != 2 && tuning(PEAK_TUNE_CLUSTER_K) != 1) {
        const int64_t t128 = tiles_of(g, 1, 128);
        if (t128 <= units && t128 * 8 > units) {
            // a split must shorten the main loop (about 0.22 us per k-block) by more than the exchange costs: about
            // 1 us for tiles of at most 32 rows, 4-5 us otherwise (fp16 1024^3 -> fp32, 16 k-blocks: whole tiles 7.7 us,
            // two slices 8.6; bf16 1024x1024x2048, 32 k-blocks: 9.8 against 10.3; 256x4096x4096, 64: 20.7 against 16.3)
            const int64_t need_saved = g.M <= 32 ? 6 : 24;
            for (int s : {4, 2}) {
                const int64_t kbps = (num_kb + s - 1) / s;
                if (t128 * s > units || kbps < 8 || kbps * (s - 1) >= num_kb || num_kb - kbps < need_saved) continue;
                if (t128 > clusterk_max_clusters(128, s)) continue;
                return Plan{128, 0, s};
            }
            return Plan{128, (int)t128, 1};
        }
        // Fewer tiles than an eighth of the SMs: four slices in a cluster beat both whole tiles and the two-launch
        // split with a workspace while a slice stays short -- measured (NT, us; whole tiles / workspace split /
        // four slices): 256x256x2048 9.4 / - / 7.2, 128x512x4096 13.8 / 12.0 / 8.6, 512x512x8192 26.8 / 15.1 / 13.5;
        // from 256 k-blocks the sixteen-way workspace split wins (512x512x16384: 19.5 against 21.6).
        if (t128 * 8 <= units && num_kb >= 16 && num_kb <= 160 && t128 <= clusterk_max_clusters(128, 4))
            return Plan{128, 0, 4};
    }
    for (int bn : {512, 256, 128}) {
        if (force_bn ? bn != force_bn : bn == 512) continue;  // 512-wide tiles only on request (see launch_umma)
        if (bn == 512 && cg != 2) continue;
        // an 8-bit B stored K x N is fetched 128 columns at a time: a pair's 128-wide tile (64 per CTA) is out
        if (bn == 128 && cg == 2 && is_fp8(in_elem(g.dtype)) && !g.transB) continue;
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
            if (s > num_kb || (bn == 512 && s > 1)) break;
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
        if (!force_split && tail_mode == 2 && full > 0 && rest > 0 && bn != 512) {
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
    if (best_cost == 1e300) best = Plan{256, (int)tiles_of(g, cg, 256), 1};  // a forced width nothing above accepts
    return best;
}

// SWAP: `g` already has its operands exchanged (see launch_swapped); g.C / g.ldc / g.R / g.bias are the caller's.
template <int CG, int BN, typename TOut, bool BATCHED, bool IN8 = false, bool G2 = false, bool SWAP = false>
int launch_kernel(const GemmArgs &g, const Plan &plan, int units_max, float *ws) {
    using C_ = Cfg<CG, BN>;
    constexpr int BKE = IN8 ? 2 * BK : BK;  // elements per k-block
    auto kernel = umma_gemm_kernel<CG, BN, TOut, 0, BATCHED, IN8, G2, SWAP>;
    static PerDeviceOnce attr_once;  // the attribute belongs to the device's context: once per device
    const cudaError_t attr_err = attr_once.run(current_device(), [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }

    const Elem ein = in_elem(g.dtype), eout = out_elem(g.dtype);
    const int a_mn = g.transA ? 1 : 0;  // A stored K x M: M is the contiguous index
    const int b_mn = g.transB ? 0 : 1;  // B stored K x N: N is the contiguous index
    CUtensorMap tmA, tmB, tmC, tmW;
    const int64_t nb = g.nbatch();
    // An MN-major operand is fetched in boxes of one 128-byte swizzle row of M / N (64 16-bit or 128 8-bit
    // elements) by all k-rows of a k-block; an 8-bit B of that kind needs at least 128 columns per CTA.
    constexpr int MNE = IN8 ? 128 : 64;
    if (IN8 && b_mn && C_::HROWS < MNE) return PEAK_ERR_UNSUPPORTED;
    // rows of A a single-CTA tile fetches: all 128, or, when the whole problem has fewer, only those that exist
    // (K-major: rounded up to 8; MN-major: whole boxes of MNE rows)
    const int bn_eff = plan.bn_eff > 0 ? plan.bn_eff : BN;
    const int slot_eff = bn_eff / C_::HALVES, hrows_eff = slot_eff / CG;
    if (bn_eff != BN && (CG != 2 || b_mn || nb > 1 || plan.tail_splits != 1 || SWAP || slot_eff % 64 || bn_eff > BN))
        return PEAK_ERR_UNSUPPORTED;  // narrower tiles: CTA pairs, B with k contiguous, whole tiles of a single matrix
    const bool short_a = CG == 1 && g.M < 128 && tuning(PEAK_TUNE_SHORT_A) != 1;
    const int a_rows = short_a ? (int)((g.M + 7) / 8 * 8) : 128;
    const int a_boxes = short_a ? (int)((g.M + MNE - 1) / MNE) : 128 / MNE;
    bool ok = a_mn ? make_map(&tmA, ein, g.A, g.M, g.K, g.lda, MNE, BKE, nb, g.strideA)
                   : make_map(&tmA, ein, g.A, g.K, g.M, g.lda, BKE, a_rows, nb, g.strideA);
    ok = ok && (b_mn ? make_map(&tmB, ein, g.B, g.N, g.K, g.ldb, MNE, BKE, nb, g.strideB)
                     : make_map(&tmB, ein, g.B, g.K, g.N, g.ldb, BKE, bn_eff != BN ? hrows_eff : C_::B_BOX_ROWS, nb, g.strideB));
    if (!ok) return nb > 1 ? PEAK_ERR_UNSUPPORTED : PEAK_ERR_CUDA;  // e.g. a batch stride TMA cannot express

    UmmaParams p;
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.num_kb = (int)((g.K + BKE - 1) / BKE);
    p.tiles_m = (int)((g.M + BM * CG - 1) / (BM * CG));
    p.tiles_n = (int)((g.N + bn_eff - 1) / bn_eff);
    p.bn_eff = bn_eff; p.slot_eff = slot_eff; p.hrows_eff = hrows_eff;
    // tile-rows per raster group (measured: 16 rows of 256 x 512 tiles are 1 % faster than 8 at 8192^3)
    p.group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : ((CG == 1 || BN == 512) ? 16 : 8);
    if (tuning(PEAK_TUNE_RASTER_GROUP) == 0 && nb == 1 && p.tiles_m * (int64_t)p.tiles_n > 2 * units_max) {
        // An operand that fits L2 with room to spare is best kept there for the whole launch: walk the tiles so
        // that every wave needs all of it and only streams the other operand (measured: 16384x4096x4096 NT, B =
        // 32 MiB, row by row 1287 against 1254 TFLOP/s with groups of eight rows).
        const int64_t a_bytes = g.M * g.K * elem_bytes(ein), b_bytes = g.K * g.N * elem_bytes(ein);
        const int64_t keep = 40ll << 20;
        if (b_bytes <= keep && b_bytes <= a_bytes) p.group = 1;                 // row by row: B stays
        else if (a_bytes <= keep) p.group = p.tiles_m;                          // column by column: A stays
    }
    p.tiles_per_batch = p.tiles_m * p.tiles_n;
    p.stride_c = g.strideC;
    const int tiles = p.tiles_per_batch * (int)nb;
    p.bulk_exchange = 0;
    p.full_tiles = plan.full_tiles;
    p.tail_splits = plan.tail_splits;
    p.kb_per_split = (p.num_kb + plan.tail_splits - 1) / plan.tail_splits;
    p.total_items = plan.full_tiles + (tiles - plan.full_tiles) * plan.tail_splits;
    p.a_mn = a_mn; p.b_mn = b_mn;
    p.a_boxes = a_boxes;
    // bytes a stage's barrier counts: a single CTA's A rows and B tile, or both CTAs' parts of a pair
    p.stage_tx = CG == 1 ? (uint32_t)(C_::B_STAGE_BYTES + (a_mn ? a_boxes * MNE * 128 : a_rows * 128))
                         : (uint32_t)(CG * (A_STAGE_BYTES + C_::HALVES * hrows_eff * 128));
    // operand format field: f16 kind: 0 = fp16, 1 = bf16; f8f6f4 kind: 0 = E4M3, 1 = E5M2
    const uint32_t fmt = (ein == Elem::BF16 || ein == Elem::E5M2) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(slot_eff >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.ldc = g.ldc;
    p.bias = g.bias; p.act = g.act;
    const int ob = elem_bytes(eout);
    if (g.R && nb > 1) return PEAK_ERR_UNSUPPORTED;  // no residual on the batched path
    p.R = g.R; p.ldr = g.ldr;
    p.r_vec = (g.R && reinterpret_cast<uintptr_t>(g.R) % 16 == 0 && (g.ldr * ob) % 16 == 0) ? 1 : 0;
    p.vec_ok = ((reinterpret_cast<uintptr_t>(g.C) % 16) == 0 && (g.ldc * ob) % 16 == 0 &&
                (nb == 1 || (g.strideC * ob) % 16 == 0)) ? 1 : 0;
    const int epi = tuning(PEAK_TUNE_EPILOGUE);  // 0 auto, 1 direct stores, 2 TMA stores
    // TMA stores clip rows exactly but clip the contiguous index only at 16-byte granularity, so they are
    // used when a row of C is a whole number of 16-byte pieces; other widths take the direct-store path
    p.tma_store = (p.vec_ok && (g.N * ob) % 16 == 0 && epi != 1 && !SWAP) ? 1 : 0;
    tmC = tmA;  // placeholders when unused
    tmW = tmA;
    if (nb > 1 && (g.strideC * ob) % 16 != 0) p.tma_store = 0;  // the batch stride must suit the store map too
    // beta != 0 with TMA stores on one-slot tiles: old C comes in by TMA as well (PEAK_TUNE_EPILOGUE 3 keeps the
    // per-thread loads)
    p.c_prefetch = (p.tma_store && g.beta != 0.0f && epi != 3) ? 1 : 0;
    if (p.tma_store && plan.full_tiles > 0 && !make_map(&tmC, eout, g.C, g.N, g.M, g.ldc, 128 / ob, 32, nb, g.strideC))
        return PEAK_ERR_CUDA;
    if (plan.full_tiles < tiles) {
        // the workspace as one tall matrix of dense (BM*CG) x BN blocks, one per (split tile, slice)
        const int64_t rows = (int64_t)(tiles - plan.full_tiles) * plan.tail_splits * (BM * CG);
        if (!ws || !make_map(&tmW, Elem::F32, ws, BN, rows, BN, 32, 32)) return PEAK_ERR_CUDA;
    }
    // every other tile walks k downwards: on by default for the 512-wide tiles (8192^3: DRAM reads 0.85 -> 0.72 GB,
    // +1..2 %); with 256-wide tiles and a good tile order it measured within +-0.5 %, so those keep ascending k
    const int ko = tuning(PEAK_TUNE_K_ORDER);
    p.k_alternate = ko == 1 ? 0 : (ko == 2 ? 1 : (BN == 512 ? 1 : 0));
    p.status = device_status_word();
    if (!p.status) return PEAK_ERR_CUDA;
    const int wait_ms = tuning(PEAK_TUNE_WAIT_MS);
    p.wait_cycles = wait_ms > 0 ? (long long)wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.inject_stall = tuning(PEAK_TUNE_INJECT_STALL) == 1 ? 1 : 0;

    // Balanced grid: the fewest CTAs (pairs) that still finish in the same number of waves, so that every
    // unit gets the same number of items and the SMs left out draw no power (under the power cap the busy
    // ones then clock higher: 256 tiles run faster on 64 pairs x 4 tiles than on 74 pairs x 3.46).
    int units = units_max;
    if (p.total_items < units) units = p.total_items;
    if (tuning(PEAK_TUNE_BALANCED_GRID) != 1) {
        const int waves = (p.total_items + units - 1) / units;
        units = (p.total_items + waves - 1) / waves;
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * CG));
    cfg.blockDim = dim3(C_::threads(G2));
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
    note_kernel("umma_gemm_kernel<%d, %d, %s, 0, %d, %d, %d, %d> grid=%d items=%d splits=%d%s", CG, BN,
                sizeof(TOut) == 4 ? "float" : (std::is_same<TOut, __half>::value ? "__half" : "__nv_bfloat16"),
                (int)BATCHED, (int)IN8, (int)G2, (int)SWAP, units * CG, p.total_items, plan.tail_splits,
                bn_eff == BN ? "" : (bn_eff == 192 ? " width=192" : " width=384"));
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    if (plan.full_tiles == tiles) return PEAK_OK;

    // second kernel: add the slices of the split tiles in order, apply alpha/beta
    const int split_tiles = tiles - plan.full_tiles;
    cudaLaunchConfig_t rcfg = {};
    rcfg.gridDim = dim3((unsigned)split_tiles, split_tiles >= 64 ? 2u : 8u);
    rcfg.blockDim = dim3(256);
    rcfg.dynamicSmemBytes = 0;
    rcfg.stream = g.stream;
    cudaLaunchAttribute rattr[1];
    rattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    rattr[0].val.programmaticStreamSerializationAllowed = 1;
    rcfg.attrs = rattr;
    rcfg.numAttrs = tuning(PEAK_TUNE_DEPENDENT_LAUNCH) == 1 ? 0 : 1;
    const float *ws_c = ws;
    e = cudaLaunchKernelEx(&rcfg, splitk_reduce_kernel<TOut>, ws_c, plan.tail_splits, plan.full_tiles, p.tiles_m, p.tiles_n,
                           p.group, BM * CG, BN, p.M, p.N, g.alpha, g.beta, (TOut *)g.C, g.ldc, g.strideC, p.vec_ok,
                           g.bias, g.act, (const TOut *)g.R, g.ldr, SWAP ? 1 : 0);
    count_launch();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

// Two groups of epilogue warps on a one-slot tile (G2): measured on problems of one or two waves, where the
// last tile's epilogue is an exposed tail of the launch (fp16 2048^3 -> fp32: see the A/B notes); on longer
// runs the extra warps cost about 1 %.  16-bit inputs, single matrices.
template <int BN> bool want_two_groups(const GemmArgs &g, const Plan &plan, int units) {
    if (BN == 512 || is_fp8(in_elem(g.dtype))) return false;
    // batches: instantiated for the single-CTA 256-wide tiles of epilogue-bound problems only (launch_typed)
    if (g.nbatch() > 1) return BN == 256 && plan.tail_splits == 1 && (g.K + BK - 1) / BK <= 8 && tuning(PEAK_TUNE_EPILOGUE_WARPS) != 1;
    const int mode = tuning(PEAK_TUNE_EPILOGUE_WARPS);  // 1 = four warps, 2 = eight warps
    if (mode) return mode == 2;
    // (also up to eight k-blocks, where the epilogue bounds every tile: 8192x8192x512 70 -> 64 us)
    if (plan.tail_splits == 1 && (g.K + BK - 1) / BK <= 8) return true;
    return plan.tail_splits == 1 && (int64_t)plan.full_tiles <= 2 * (int64_t)units;
}

template <int CG, int BN> int launch_typed(const GemmArgs &g, const Plan &plan, int units, float *ws) {
    const bool g2 = want_two_groups<BN>(g, plan, units);
    switch (out_elem(g.dtype)) {
        case Elem::F32:
            if (is_fp8(in_elem(g.dtype)))
                return g.nbatch() > 1 ? launch_kernel<CG, BN, float, true, true>(g, plan, units, ws)
                                      : launch_kernel<CG, BN, float, false, true>(g, plan, units, ws);
            if (g.nbatch() > 1) {
                if constexpr (CG == 1 && BN == 256)
                    if (g2) return launch_kernel<CG, BN, float, true, false, true>(g, plan, units, ws);
                return launch_kernel<CG, BN, float, true>(g, plan, units, ws);
            }
            if constexpr (BN != 512)
                if (g2) return launch_kernel<CG, BN, float, false, false, true>(g, plan, units, ws);
            return launch_kernel<CG, BN, float, false>(g, plan, units, ws);
        case Elem::F16:
            if (g.nbatch() > 1) {
                if constexpr (CG == 1 && BN == 256)
                    if (g2) return launch_kernel<CG, BN, __half, true, false, true>(g, plan, units, ws);
                return launch_kernel<CG, BN, __half, true>(g, plan, units, ws);
            }
            if constexpr (BN != 512)
                if (g2) return launch_kernel<CG, BN, __half, false, false, true>(g, plan, units, ws);
            return launch_kernel<CG, BN, __half, false>(g, plan, units, ws);
        case Elem::BF16:
            if (is_fp8(in_elem(g.dtype)))
                return g.nbatch() > 1 ? launch_kernel<CG, BN, __nv_bfloat16, true, true>(g, plan, units, ws)
                                      : launch_kernel<CG, BN, __nv_bfloat16, false, true>(g, plan, units, ws);
            if (g.nbatch() > 1) {
                if constexpr (CG == 1 && BN == 256)
                    if (g2) return launch_kernel<CG, BN, __nv_bfloat16, true, false, true>(g, plan, units, ws);
                return launch_kernel<CG, BN, __nv_bfloat16, true>(g, plan, units, ws);
            }
            if constexpr (BN != 512)
                if (g2) return launch_kernel<CG, BN, __nv_bfloat16, false, false, true>(g, plan, units, ws);
            return launch_kernel<CG, BN, __nv_bfloat16, false>(g, plan, units, ws);
        default: break;  // outputs are never 8-bit
    }
    return PEAK_ERR_INVALID_VALUE;
}

// Bytes of fp32 partial tiles a plan needs (0 when nothing is split).
size_t workspace_bytes(const GemmArgs &g, int cg, const Plan &plan) {
    if (plan.tail_splits <= 1) return 0;
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

// ---- k-slices on the CTAs of a cluster, added through distributed shared memory (umma_clusterk.cuh) -------
// One launch instead of tile kernel + reduction kernel, no workspace.  Single matrices, single-CTA tiles,
// every tile split KC = 2 or 4 ways.
template <int BN, typename TOut, int KC, bool IN8, int CG = 1> int launch_clusterk(const GemmArgs &g, const Plan &plan) {
    using C_ = Cfg<CG, BN>;
    constexpr int BKE = IN8 ? 2 * BK : BK;
    constexpr int MNE = IN8 ? 128 : 64;
    auto kernel = umma_clusterk_kernel<BN, TOut, KC, IN8, CG>;
    static PerDeviceOnce attr_once;
    const cudaError_t attr_err = attr_once.run(current_device(), [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }
    const Elem ein = in_elem(g.dtype), eout = out_elem(g.dtype);
    const int a_mn = g.transA ? 1 : 0, b_mn = g.transB ? 0 : 1;
    if (IN8 && b_mn && C_::HROWS < MNE) return PEAK_ERR_UNSUPPORTED;
    // narrower whole tiles of a pair (plan.bn_eff, e.g. 192 on the 256-wide instantiation): B with k contiguous only
    const int bn_eff = plan.bn_eff > 0 ? plan.bn_eff : BN;
    const int hrows_eff = bn_eff / CG;
    if (bn_eff != BN && (CG != 2 || KC != 1 || b_mn || bn_eff % 64 || bn_eff > BN)) return PEAK_ERR_UNSUPPORTED;
    const bool short_a = CG == 1 && g.M < 128 && tuning(PEAK_TUNE_SHORT_A) != 1;
    const int a_rows = short_a ? (int)((g.M + 7) / 8 * 8) : 128;
    const int a_boxes = short_a ? (int)((g.M + MNE - 1) / MNE) : 128 / MNE;
    CUtensorMap tmA, tmB, tmC;
    bool ok = a_mn ? make_map(&tmA, ein, g.A, g.M, g.K, g.lda, MNE, BKE) : make_map(&tmA, ein, g.A, g.K, g.M, g.lda, BKE, a_rows);
    ok = ok && (b_mn ? make_map(&tmB, ein, g.B, g.N, g.K, g.ldb, MNE, BKE)
                     : make_map(&tmB, ein, g.B, g.K, g.N, g.ldb, BKE, bn_eff != BN ? hrows_eff : C_::B_BOX_ROWS));
    if (!ok) return PEAK_ERR_CUDA;
    UmmaParams p = {};
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.num_kb = (int)((g.K + BKE - 1) / BKE);
    p.tiles_m = (int)((g.M + BM * CG - 1) / (BM * CG));
    p.tiles_n = (int)((g.N + bn_eff - 1) / bn_eff);
    p.group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : 16;
    p.tiles_per_batch = p.tiles_m * p.tiles_n;
    p.full_tiles = 0;
    p.tail_splits = KC;
    p.kb_per_split = (p.num_kb + KC - 1) / KC;
    p.total_items = p.tiles_per_batch * KC * CG;  // CTAs
    p.a_mn = a_mn; p.b_mn = b_mn;
    p.a_boxes = a_boxes;
    p.stage_tx = CG == 1 ? (uint32_t)(C_::B_STAGE_BYTES + (a_mn ? a_boxes * MNE * 128 : a_rows * 128))
                         : (uint32_t)(CG * (A_STAGE_BYTES + hrows_eff * 128));  // both CTAs' parts arrive at the leader's barrier
    p.bulk_exchange = tuning(PEAK_TUNE_CLUSTER_K) == 2 ? 1 : 0;
    p.bn_eff = bn_eff; p.slot_eff = bn_eff; p.hrows_eff = hrows_eff;
    const uint32_t fmt = (ein == Elem::BF16 || ein == Elem::E5M2) ? 1u : 0u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
              ((uint32_t)(bn_eff >> 3) << 17) | ((uint32_t)((BM * CG) >> 4) << 24);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = g.C; p.ldc = g.ldc;
    p.bias = g.bias; p.act = g.act;
    const int ob = elem_bytes(eout);
    p.R = g.R; p.ldr = g.ldr;
    p.r_vec = (g.R && reinterpret_cast<uintptr_t>(g.R) % 16 == 0 && (g.ldr * ob) % 16 == 0) ? 1 : 0;
    p.vec_ok = ((reinterpret_cast<uintptr_t>(g.C) % 16) == 0 && (g.ldc * ob) % 16 == 0) ? 1 : 0;
    const int epi = tuning(PEAK_TUNE_EPILOGUE);
    p.tma_store = (p.vec_ok && (g.N * ob) % 16 == 0 && epi != 1) ? 1 : 0;
    p.c_prefetch = (p.tma_store && g.beta != 0.0f && epi != 3) ? 1 : 0;
    tmC = tmA;
    if (p.tma_store && !make_map(&tmC, eout, g.C, g.N, g.M, g.ldc, 128 / ob, 32)) return PEAK_ERR_CUDA;
    p.status = device_status_word();
    if (!p.status) return PEAK_ERR_CUDA;
    const int wait_ms = tuning(PEAK_TUNE_WAIT_MS);
    p.wait_cycles = wait_ms > 0 ? (long long)wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.inject_stall = tuning(PEAK_TUNE_INJECT_STALL) == 1 ? 1 : 0;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.total_items);
    cfg.blockDim = dim3(ClusterKCfg<BN, KC, CG>::THREADS);
    cfg.dynamicSmemBytes = C_::SMEM_BYTES;
    cfg.stream = g.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KC * CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = tuning(PEAK_TUNE_DEPENDENT_LAUNCH) == 1 ? 1 : 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmC, p);
    if (e == cudaErrorInvalidClusterSize || e == cudaErrorLaunchOutOfResources || e == cudaErrorInvalidConfiguration) {
        // a device (or partition) that cannot place this cluster shape: nothing was launched, the caller takes the
        // workspace path
        (void)cudaGetLastError();
        return PEAK_ERR_UNSUPPORTED;
    }
    count_launch();
    note_kernel("umma_clusterk_kernel<%d, %s, %d, %d%s> grid=%d clusters=%d", BN,
                sizeof(TOut) == 4 ? "float" : (std::is_same<TOut, __half>::value ? "__half" : "__nv_bfloat16"), KC, (int)IN8,
                CG == 2 ? ", 2" : "", p.total_items, p.tiles_per_batch);
    if (bn_eff != BN) note_kernel("umma_clusterk_kernel<%d, %s, %d, %d, 2> grid=%d clusters=%d width=%d", BN,
                                  sizeof(TOut) == 4 ? "float" : (std::is_same<TOut, __half>::value ? "__half" : "__nv_bfloat16"),
                                  KC, (int)IN8, p.total_items, p.tiles_per_batch, bn_eff);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

// PEAK_TUNE_CLUSTER_K: 1 = never (workspace + reduction kernel), otherwise whenever the plan splits every tile of
// a single matrix 2 or 4 ways on single-CTA tiles.
bool clusterk_applies(const GemmArgs &g, int cta_group, const Plan &plan) {
    if (tuning(PEAK_TUNE_CLUSTER_K) == 1) return false;
    if (cta_group != 1 || g.nbatch() > 1) return false;
    if (plan.bn != 128 && plan.bn != 256) return false;
    // whole tiles that all run at once: the same kernel without a cluster (one tile per CTA, two MMA issuers)
    if (plan.tail_splits == 1) return plan.bn == 128 && plan.full_tiles <= sm_count();
    if (plan.full_tiles != 0) return false;
    return plan.tail_splits == 2 || plan.tail_splits == 4;
}

template <int BN, int KC> int launch_clusterk_typed(const GemmArgs &g, const Plan &plan) {
    const bool in8 = is_fp8(in_elem(g.dtype));
    switch (out_elem(g.dtype)) {
        case Elem::F32:
            return in8 ? launch_clusterk<BN, float, KC, true>(g, plan) : launch_clusterk<BN, float, KC, false>(g, plan);
        case Elem::F16: return launch_clusterk<BN, __half, KC, false>(g, plan);
        case Elem::BF16:
            return in8 ? launch_clusterk<BN, __nv_bfloat16, KC, true>(g, plan)
                       : launch_clusterk<BN, __nv_bfloat16, KC, false>(g, plan);
        default: break;
    }
    return PEAK_ERR_INVALID_VALUE;
}

template <int BN, int KC> int max_clusters_of() {
    static int cached[kMaxDevices] = {};
    static std::mutex m;
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(m);
    if (cached[dev] == 0) {
        using C_ = Cfg<1, BN>;
        auto kernel = umma_clusterk_kernel<BN, __nv_bfloat16, KC, false>;
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(KC * 64);
        cfg.blockDim = dim3(ClusterKCfg<BN, KC>::THREADS);
        cfg.dynamicSmemBytes = C_::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = KC; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::SMEM_BYTES);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
        if (e != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
        cached[dev] = n > 0 ? n : -1;
    }
    return cached[dev] > 0 ? cached[dev] : 0;
}

int clusterk_max_clusters(int bn, int kc) {
    if (bn == 128) return kc == 2 ? max_clusters_of<128, 2>() : max_clusters_of<128, 4>();
    return kc == 2 ? max_clusters_of<256, 2>() : max_clusters_of<256, 4>();
}

// Whole tiles as 256 x 128 pair tiles (a quarter fewer operand bytes per SM) when the problem has at least two
// 128-row blocks and its pair tiles still run at once; 16-bit inputs, or 8-bit ones with B stored N x K.
// PEAK_TUNE_CLUSTER_K = 3 keeps single-CTA tiles.
template <typename TOut, bool IN8> int launch_pair_tiles(const GemmArgs &g, const Plan &plan) {
    return launch_clusterk<128, TOut, 1, IN8, 2>(g, plan);
}
bool pair_tiles_apply(const GemmArgs &g) {
    if (tuning(PEAK_TUNE_CLUSTER_K) == 3 || g.M <= 128) return false;
    if (is_fp8(in_elem(g.dtype)) && !g.transB) return false;  // an 8-bit B stored K x N needs 128 columns per CTA
    // (from 32 k-blocks on: measured, us, pair against single tiles: 512x4096x4096 18.8 / 21.6, 2048x1024x4096
    // 18.8 / 22.1, 1024x2048x2048 11.1 / 11.6, but 1536^3 10.9 / 9.8 and 1024^3 7.5 / 7.2)
    const int bke = is_fp8(in_elem(g.dtype)) ? 2 * BK : BK;
    if ((g.K + bke - 1) / bke < 32 && tuning(PEAK_TUNE_CLUSTER_K) != 4) return false;  // 4 = pairs whenever possible
    const int64_t pair_tiles = ((g.M + 255) / 256) * ((g.N + 127) / 128);
    return 2 * pair_tiles <= (int64_t)sm_count();
}

int run_clusterk(const GemmArgs &g, const Plan &plan) {
    if (plan.tail_splits == 1 && pair_tiles_apply(g)) {
        const bool in8 = is_fp8(in_elem(g.dtype));
        switch (out_elem(g.dtype)) {
            case Elem::F32: return in8 ? launch_pair_tiles<float, true>(g, plan) : launch_pair_tiles<float, false>(g, plan);
            case Elem::F16: return launch_pair_tiles<__half, false>(g, plan);
            case Elem::BF16:
                return in8 ? launch_pair_tiles<__nv_bfloat16, true>(g, plan) : launch_pair_tiles<__nv_bfloat16, false>(g, plan);
            default: break;
        }
        return PEAK_ERR_INVALID_VALUE;
    }
    if (plan.tail_splits == 1) return launch_clusterk_typed<128, 1>(g, plan);
    // (... when all of the four-CTA clusters are resident at once: 33 on this device, like those of four k-slices)
    if (plan.tail_splits == 2 && plan.bn == 128 && pair_tiles_apply(g) && !is_fp8(in_elem(g.dtype)) &&
        ((g.M + 255) / 256) * ((g.N + 127) / 128) <= (int64_t)clusterk_max_clusters(128, 4)) {
        // two k-slices of 256 x 128 pair tiles on the two pairs of a four-CTA cluster
        switch (out_elem(g.dtype)) {
            case Elem::F32: return launch_clusterk<128, float, 2, false, 2>(g, plan);
            case Elem::F16: return launch_clusterk<128, __half, 2, false, 2>(g, plan);
            case Elem::BF16: return launch_clusterk<128, __nv_bfloat16, 2, false, 2>(g, plan);
            default: break;
        }
        return PEAK_ERR_INVALID_VALUE;
    }
    if (plan.bn == 128)
        return plan.tail_splits == 2 ? launch_clusterk_typed<128, 2>(g, plan) : launch_clusterk_typed<128, 4>(g, plan);
    return plan.tail_splits == 2 ? launch_clusterk_typed<256, 2>(g, plan) : launch_clusterk_typed<256, 4>(g, plan);
}

// One wave of whole 256 x 256 pair tiles (at most one tile per CTA pair) on the one-tile kernel: two producer warps per
// CTA and no persistent-loop bookkeeping (measured, us, against the persistent kernel / the multicast plug-in: 2048^3
// 16.9 / 17.5 / 18.0, 1792^3 15.5 / 16.2, 1024x4096x1024 11.7 / 12.2 / 12.5; cuBLAS 16.5 / 12.9 / 11.4).
bool one_wave_pair_tiles_apply(const GemmArgs &g, int cta_group, const Plan &plan, int units) {
    const int mode = tuning(PEAK_TUNE_CLUSTER_K);
    if (mode == 1 || mode == 3 || cta_group != 2 || g.nbatch() > 1) return false;
    const int forced = tuning(PEAK_TUNE_TILE_N);
    if ((forced != 0 && forced != 256) || plan.bn != 256 || plan.tail_splits != 1) return false;
    return tiles_of(g, 2, 256) <= units;
}
int run_one_wave_pair_tiles(const GemmArgs &g, const Plan &plan) {
    const bool in8 = is_fp8(in_elem(g.dtype));
    switch (out_elem(g.dtype)) {
        case Elem::F32:
            return in8 ? launch_clusterk<256, float, 1, true, 2>(g, plan) : launch_clusterk<256, float, 1, false, 2>(g, plan);
        case Elem::F16: return launch_clusterk<256, __half, 1, false, 2>(g, plan);
        case Elem::BF16:
            return in8 ? launch_clusterk<256, __nv_bfloat16, 1, true, 2>(g, plan)
                       : launch_clusterk<256, __nv_bfloat16, 1, false, 2>(g, plan);
        default: break;
    }
    return PEAK_ERR_INVALID_VALUE;
}

// ---- exchanged operands for very skinny problems (M <= 64) -----------------------------------------------
// C^T = op(B)^T op(A)^T: N takes the role of the MMA's M (128-row tiles over N) and M that of its N (one 64-wide
// tile), so the small operand costs 8 KiB of shared memory and a few hundred bytes of traffic per k-block
// instead of a 16 KiB box of which all but M rows are padding.  (The paper's Split-K row of its transformation
// table covers the k-slices; the exchange is the same product written for the other operand order.)
template <typename TOut> int run_swapped(const GemmArgs &gs, const Plan &plan, int units) {
    const size_t need = workspace_bytes(gs, 1, plan);
    if (need == 0) return launch_kernel<1, 64, TOut, false, false, false, true>(gs, plan, units, nullptr);
    float *ws = nullptr;
    cudaMemPool_t pool = workspace_pool();
    if (!pool) return PEAK_ERR_CUDA;
    cudaError_t e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&ws), need, pool, gs.stream);
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_NO_MEMORY; }
    int rc = launch_kernel<1, 64, TOut, false, false, false, true>(gs, plan, units, ws);
    e = cudaFreeAsync(ws, gs.stream);
    if (e != cudaSuccess && rc == PEAK_OK) { set_cuda_error(e); rc = PEAK_ERR_CUDA; }
    return rc;
}

bool swap_applies(const GemmArgs &g) {
    // Opt-in (PEAK_TUNE_SWAP_AB = 2, or a tuning-table entry): measured on B200 it is slower than the plain
    // single-CTA tiles on every skinny shape tried -- 16x4096x4096 TN 15.3 against 14.1 us, NT 13.7 against 13.4,
    // 8x8192x8192 33.3 against 29.4, 64x8192x8192 35.6 against 33.0, 32x14336x4096 25.7 against 25.1 -- although
    // each SM receives little more than half the bytes: these launches are bound by their fixed costs and the
    // latency of a short pipeline, not by operand traffic.
    const int mode = tuning(PEAK_TUNE_SWAP_AB);
    if (mode != 2 || g.nbatch() > 1 || is_fp8(in_elem(g.dtype)) || g.M > 64 || g.N < 128) return false;
    return true;
}

// Shared-operand clusters of single-CTA tiles (plug-in).  PEAK_TUNE_SHARE: 1 = never; 100 * w + 10 * CM + CN with
// w = 1 (128-wide tiles) or 2 (256-wide) forces a cluster shape; 0 = the built-in rule.
bool share_applies(const GemmArgs &g, int &bn, int &cm, int &cn) {
    const int mode = tuning(PEAK_TUNE_SHARE);
    if (mode == 1 || tuning(PEAK_TUNE_MULTICAST) == 1 || g.nbatch() > 1 || is_fp8(in_elem(g.dtype)) || !mc_entry())
        return false;
    if (mode >= 100) {
        bn = mode / 100 == 2 ? 256 : 128;
        cm = mode / 10 % 10;
        cn = mode % 10;
        return true;
    }
    return false;
}

int launch_swapped(const GemmArgs &g) {
    GemmArgs gs = g;
    gs.A = g.B; gs.lda = g.ldb; gs.B = g.A; gs.ldb = g.lda;
    gs.M = g.N; gs.N = g.M;
    gs.transA = g.transB ? 0 : 1;
    gs.transB = g.transA ? 0 : 1;
    const int units = sm_count();
    const int64_t num_kb = (g.K + BK - 1) / BK;
    const int64_t tiles = (gs.M + BM - 1) / BM;
    // k-slices: fill the SMs once, at least four k-blocks per slice
    int64_t s = tuning(PEAK_TUNE_SPLIT_K) > 0 ? tuning(PEAK_TUNE_SPLIT_K) : std::min<int64_t>(units / tiles, num_kb / 4);
    s = std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(s, 16), num_kb));
    while (s > 1 && ((num_kb + s - 1) / s) * (s - 1) >= num_kb) --s;  // no empty last slice
    const Plan plan{64, s == 1 ? (int)tiles : 0, (int)s};
    switch (out_elem(g.dtype)) {
        case Elem::F32: return run_swapped<float>(gs, plan, units);
        case Elem::F16: return run_swapped<__half>(gs, plan, units);
        case Elem::BF16: return run_swapped<__nv_bfloat16>(gs, plan, units);
        default: break;
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
    const bool in8 = is_fp8(in_elem(g.dtype));
    const int pitch_unit = in8 ? 16 : 8;               // TMA: row pitch must be a multiple of 16 bytes
    if (g.lda % pitch_unit || g.ldb % pitch_unit) return false;
    if (g.lda >= (1ll << 38) || g.ldb >= (1ll << 38) || g.ldc >= (1ll << 38)) return false;
    const int64_t tiles = ((g.M + 127) / 128) * ((g.N + 127) / 128) * g.nbatch();
    if (tiles * 16 >= (1ll << 31)) return false;
    if (g.nbatch() > 1) {  // the batch is the third dimension of the tensor maps: strides in 16-byte units
        if (g.strideA % pitch_unit || g.strideB % pitch_unit || g.strideA < 1 || g.strideB < 1) return false;
        if (g.strideA >= (1ll << 38) || g.strideB >= (1ll << 38) || g.strideC >= (1ll << 38)) return false;
    }
    return true;
}

bool umma_multicast_available() { return mc_entry() != nullptr; }

cudaMemPool_t scratch_pool() { return workspace_pool(); }

int umma_units(int cta_group) { return sm_count() / (cta_group == 2 ? 2 : 1); }

int launch_umma(const GemmArgs &g, int cta_group) {
    if (!umma_supports(g, cta_group)) return PEAK_ERR_UNSUPPORTED;
    if (cta_group == 1 && swap_applies(g)) return launch_swapped(g);
    {
        // Single-CTA tiles in clusters that share operand tiles by multicast (single-GPU plug-in).
        int bn = 0, cm = 0, cn = 0;
        if (share_applies(g, bn, cm, cn)) {
            peak_mc_request r{g.dtype, g.transA, g.transB, g.M, g.N, g.K, g.alpha, g.beta, g.A, g.B, g.C, g.lda, g.ldb,
                              g.ldc, g.stream, device_status_word(), tuning(PEAK_TUNE_RASTER_GROUP),
                              tuning(PEAK_TUNE_EPILOGUE), tuning(PEAK_TUNE_WAIT_MS), tuning(PEAK_TUNE_DEPENDENT_LAUNCH),
                              tuning(PEAK_TUNE_INJECT_STALL), tuning(PEAK_TUNE_BALANCED_GRID), g.bias, g.act,
                              tuning(PEAK_TUNE_EPILOGUE_WARPS), bn, g.R, g.ldr, tuning(PEAK_TUNE_K_ORDER), cm, cn, 0};
            if (!r.status) return PEAK_ERR_CUDA;
            const int rc = mc_entry()(&r);
            if (rc == PEAK_OK) {
                count_launch();
                const Elem eo = out_elem(g.dtype);
                note_kernel("umma_share_kernel<%d, %s, %d, %d> (cluster-multicast plug-in)", bn,
                            eo == Elem::F32 ? "float" : (eo == Elem::F16 ? "__half" : "__nv_bfloat16"), cm, cn);
                return rc;
            }
            if (rc == PEAK_ERR_CUDA) { set_cuda_error((cudaError_t)r.cuda_error); return rc; }
            if (rc != PEAK_ERR_UNSUPPORTED) return rc;
        }
    }
    const int units = sm_count() / cta_group;
    Plan plan = choose_plan(g, cta_group, units);
    const bool in8 = is_fp8(in_elem(g.dtype));
    const bool whole256 = cta_group == 2 && plan.bn == 256 && plan.tail_splits == 1;
    // 256 x 512 pair tiles move a third less operand data per flop, but the tile fills the tensor memory, so
    // its epilogue (two groups of warps, one per half) is exposed once per tile.  Measured under the power
    // cap (sustained, random inputs): with 16-bit inputs and beta = 0 they win from 48 k-blocks on (+1..2 % at
    // 8192x8192x3072, +2 % at 8192x8192x4096, +5 % at 8192^3, +9 % at fp16 8192^3 TN), with beta != 0 (the epilogue also reads C)
    // only from 128 k-blocks on (-7 % at 16384x14336x4096, +3 % at 16384x4096x14336); 8-bit inputs, whose
    // k-blocks take the same time but hold twice the K, from 96 k-blocks (K = 12288) on (a tie at 64 k-blocks,
    // +2.6 % at 96, +3..5 % at 128).  They must fill the grid as well as the 256-wide tiles do (4096x8192x4096: 3.46 waves
    // against 6.9, -3 %).
    bool wide = false, short_k = false;
    if (whole256 && !tuning(PEAK_TUNE_TILE_N)) {
        const int bke = in8 ? 2 * BK : BK;
        const int64_t num_kb = (g.K + bke - 1) / bke;
        const bool light_tail = g.beta == 0.0f && g.act != PEAK_ACT_GELU;
        const int64_t min_kb = !light_tail ? 128 : (in8 ? 96 : 48);
        auto fill = [&](int64_t tiles) { return (double)tiles / (double)(((tiles + units - 1) / units) * units); };
        const int64_t t512 = tiles_of(g, 2, 512), t256 = tiles_of(g, 2, 256);
        // (3072^3: 72 wide tiles on 74 pairs, one wave: 40.0 us against 41.3 for two waves of 256-wide tiles)
        wide = num_kb >= min_kb && t512 * 10 >= (int64_t)units * 9 && fill(t512) >= fill(t256) - 0.02;
        // ... and from 32 k-blocks on where the wide tiles make one wave of what would be two waves of 256-wide ones
        // (sustained, 16-bit output, beta = 0: 3000^3 1109 against 962 TFLOP/s; ties at 2304^3 and 2560^3)
        if (!wide && light_tail && !in8 && elem_bytes(out_elem(g.dtype)) == 2 && num_kb >= 32 && t512 <= units &&
            t256 > units && t512 * 10 >= (int64_t)units * 6)
            wide = true;
        // Up to four k-blocks the epilogue, not the main loop, bounds a tile, and the wide tile's eight epilogue warps
        // drain it faster than four (8192x8192x64: 58 -> 41 us, 8192x8192x256: 61 -> 53, 4096x4096x128: 20 -> 15.5);
        // the multicast plug-in has nothing to share there.
        // (taken where the wide tiles waste no more columns than the 256-wide ones: 128 matrices of 256 x 256 x 128
        // ran 13.6 us on 256-wide tiles and 15.3 on half-empty wide ones)
        if (!wide && num_kb <= 4 && t256 > units && t512 * 16 <= t256 * 9) wide = true;
        if (num_kb <= 8) short_k = true;
    }
    // Whole 256-wide pair tiles, at least two pairs tall: the multicast plug-in can run it, if it is there.
    // Measured (sustained, random inputs, interleaved): fp16 4096^3 -> fp32 1162 against 1132 (512-wide) and
    // 1108 (256-wide); +12 % at 5000x3000x2500; but with 16-bit output, where the exposed epilogue of the wide
    // tile is half as long, the wide tile wins (bf16 4096^3: 1231 against 1244-1249), and from 2.7e11 flop on
    // the plug-in loses 3-6 % (8192x8192x2048, 4096x8192x4096, 16384x4096x4096).
    {
        // ... 192 columns wide where that still is one wave (B with k contiguous): more pairs at work, an eighth fewer
        // operand bytes per k-block and CTA
        Plan p1 = plan;
        const int forced = tuning(PEAK_TUNE_TILE_N);
        const int64_t t192 = ((g.M + 255) / 256) * ((g.N + 191) / 192);
        const bool can192 = cta_group == 2 && g.transB && g.nbatch() == 1 && !in8 && plan.tail_splits == 1 &&
                            (plan.bn == 256 || forced == 192) && t192 <= units && tuning(PEAK_TUNE_CLUSTER_K) != 1 &&
                            tuning(PEAK_TUNE_CLUSTER_K) != 3 && tuning(PEAK_TUNE_MULTICAST) != 2;
        if (can192 && (forced == 192 || (forced == 0 && tuning(PEAK_TUNE_NARROW) != 1 && t192 > tiles_of(g, 2, 256)))) {
            p1.bn = 256; p1.bn_eff = 192;
            const int rc = run_one_wave_pair_tiles(g, p1);
            if (rc != PEAK_ERR_UNSUPPORTED) return rc;
        }
    }
    if (one_wave_pair_tiles_apply(g, cta_group, plan, units) && tuning(PEAK_TUNE_MULTICAST) != 2) {
        const int rc = run_one_wave_pair_tiles(g, plan);
        if (rc != PEAK_ERR_UNSUPPORTED) return rc;
    }
    // Narrower tiles on the 256- / 512-wide pair kernels (192 / 384 columns; B with k contiguous, whole tiles): taken
    // when a cycle estimate -- waves x k-blocks x the slower of the tensor pipe (2 cycles per column) and the operand
    // stream (56 bytes per clock per SM), plus the exposed epilogue of a two-half tile -- says they beat the plan
    // above by 15 %, which happens when they fill a single wave much better (measured, us, bf16 NT: 2304^3 32.1 -> 28.2,
    // 2560^3 34.6 -> 30.4 with 384-wide tiles; cuBLAS 21.0 / 26.7; at an estimated 10 % the gains were 0-4 %).
    // PEAK_TUNE_TILE_N = 192 / 384 forces them, PEAK_TUNE_NARROW = 1 switches the rule off.
    if (cta_group == 2 && g.transB && g.nbatch() == 1 && plan.tail_splits == 1) {
        const int forced = tuning(PEAK_TUNE_TILE_N);
        const int bke = in8 ? 2 * BK : BK;
        const int64_t num_kb = (g.K + bke - 1) / bke;
        const int64_t rows = (g.M + 255) / 256;
        auto estimate = [&](int w) {
            const int64_t tiles = rows * ((g.N + w - 1) / w);
            const int64_t waves = (tiles + units - 1) / units;
            const double per_kb = fmax(2.0 * w, (16384.0 + 64.0 * w) / 56.0);
            const double tail = w > 256 ? (g.beta != 0.0f ? 14000.0 : (elem_bytes(out_elem(g.dtype)) == 4 ? 11000.0 : 8000.0)) : 3000.0;
            return (double)waves * ((double)num_kb * per_kb + (w > 256 ? tail : 0.0)) + (w > 256 ? 0.0 : tail);
        };
        int narrow = 0;
        if (forced == 192 || forced == 384) narrow = forced;
        else if (forced == 0 && tuning(PEAK_TUNE_NARROW) != 1 && g.M > 128 && !short_k) {  // (the estimate knows no epilogue-bound tiles)
            const double now = estimate(wide ? 512 : plan.bn);
            const double e192 = estimate(192), e384 = estimate(384);
            if (plan.bn >= 256 && e192 < 0.85 * now && e192 <= e384) narrow = 192;
            else if (plan.bn >= 256 && e384 < 0.85 * now) narrow = 384;
        }
        if (narrow) {
            Plan pn{narrow == 192 ? 256 : 512, (int)(rows * ((g.N + narrow - 1) / narrow)), 1, narrow};
            const int rc = narrow == 192 ? run_umma<2, 256>(g, pn, units) : run_umma<2, 512>(g, pn, units);
            if (rc != PEAK_ERR_UNSUPPORTED) return rc;
        }
    }
    const int mc_mode = tuning(PEAK_TUNE_MULTICAST);  // 1 = never, 2 = whenever possible
    // With a 16-bit output the wide tile is preferred, and the plug-in then shares its 512-wide B tile between
    // the two pairs of a cluster (512 x 512 super-tiles): bf16 4096^3 1222 -> 1248 in the bench protocol; at
    // 8192^3, beyond the plug-in's size limit, it would lose (1251 against 1327: only 33 clusters fit).
    // (8-bit inputs, 256-wide tiles only: 2048^3 1295 -> 1415, 4096^3 unchanged, larger problems excluded as above)
    const bool wide_first = wide && elem_bytes(out_elem(g.dtype)) == 2;
    const bool whole512 = cta_group == 2 && plan.bn == 512 && plan.tail_splits == 1 && mc_mode == 2;  // forced
    if ((whole256 || whole512) && mc_mode != 1 && g.M > 256 && g.nbatch() == 1 && (!short_k || mc_mode == 2) && mc_entry()) {
        const int mc_tile_n = ((whole512 || wide_first) && !in8) ? 512 : 256;
        const int64_t super_tiles = ((g.M + 511) / 512) * ((g.N + mc_tile_n - 1) / mc_tile_n);
        const double flops = 2.0 * (double)g.M * (double)g.N * (double)g.K;
        // A cluster works on two pair tiles at once, but fewer clusters fit the device than half its pairs (33 of 37
        // here): the plug-in only runs when its super-tiles need no more waves than the pair tiles would on all pairs
        // (3072^3: 72 super-tiles = 3 waves against 2 -- 56.7 us through the plug-in, 40.0 without).
        const int maxc = mc_max_clusters(mc_tile_n);
        const int64_t pair_tiles = tiles_of(g, 2, mc_tile_n);
        const bool waves_ok = maxc <= 0 || (super_tiles + maxc - 1) / maxc <= (pair_tiles + units - 1) / units;
        if (mc_mode == 2 || (super_tiles >= 32 && flops <= 2e11 && waves_ok)) {
            peak_mc_request r{g.dtype, g.transA, g.transB, g.M, g.N, g.K, g.alpha, g.beta, g.A, g.B, g.C, g.lda, g.ldb,
                              g.ldc, g.stream, device_status_word(), tuning(PEAK_TUNE_RASTER_GROUP),
                              tuning(PEAK_TUNE_EPILOGUE), tuning(PEAK_TUNE_WAIT_MS), tuning(PEAK_TUNE_DEPENDENT_LAUNCH),
                              tuning(PEAK_TUNE_INJECT_STALL), tuning(PEAK_TUNE_BALANCED_GRID), g.bias, g.act,
                              tuning(PEAK_TUNE_EPILOGUE_WARPS), mc_tile_n, g.R, g.ldr, tuning(PEAK_TUNE_K_ORDER), 0};
            if (!r.status) return PEAK_ERR_CUDA;
            const int rc = mc_entry()(&r);
            if (rc == PEAK_OK) {
                count_launch();
                const Elem eo = out_elem(g.dtype);
                note_kernel("umma_gemm_kernel<2, %d, %s, 1, 0, %d, *> (cluster-multicast plug-in)", mc_tile_n,
                            eo == Elem::F32 ? "float" : (eo == Elem::F16 ? "__half" : "__nv_bfloat16"), (int)in8);
                return rc;
            }
            if (rc == PEAK_ERR_CUDA) { set_cuda_error((cudaError_t)r.cuda_error); return rc; }
            if (rc != PEAK_ERR_UNSUPPORTED) return rc;
        }
    }
    if (wide) plan = Plan{512, (int)tiles_of(g, 2, 512), 1};
    if (clusterk_applies(g, cta_group, plan)) {
        const int rc = run_clusterk(g, plan);
        if (rc != PEAK_ERR_UNSUPPORTED) return rc;  // otherwise: the persistent kernel, with a workspace for k-slices
    }
    if (cta_group == 2) {
        if (plan.bn == 512) return run_umma<2, 512>(g, plan, units);
        return plan.bn == 256 ? run_umma<2, 256>(g, plan, units) : run_umma<2, 128>(g, plan, units);
    }
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
