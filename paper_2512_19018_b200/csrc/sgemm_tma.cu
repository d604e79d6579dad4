// fp32 GEMM on the CUDA cores (plain fp32 FMA, never TF32), fed by TMA through an mbarrier ring.
//
// The arithmetic is the paper's CUDA-core sequence (sections 2.2 and 4.3): thread-block tiling (128 x 128 x 16),
// thread tiling (8 x 8 outputs per thread in registers), operands cached in registers, a grouped block order.
// What differs from the paper's kernels is how tiles reach shared memory and how the stages are handed over:
//   * one elected thread issues two TMA tile copies per k-block (the paper's Pipelining step, six stages); no
//     thread spends instructions on address arithmetic or copies, and the copy engine zero-fills whatever lies
//     beyond M, N or K, so any shape runs here (edges are only predicated in the epilogue);
//   * an operand whose contiguous index is m / n lands as a dense S[k][128] tile and is read with 16-byte loads
//     as before; an operand whose contiguous index is k lands as S[128][16] with the 64-byte swizzle of the
//     copy engine (the paper's Transpose and Offset steps: no transposing copy, no padding) and is read along
//     k, four (or two) k at a time;
//   * per-stage full / empty mbarriers replace the block-wide barrier: a warp that is ahead keeps going for up
//     to two k-blocks instead of waiting for the slowest warp at every step.  Every wait is bounded.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_host.cuh"

namespace peak {
namespace {

constexpr int ST_BM = 128, ST_BN = 128, ST_BK = 16;
constexpr int ST_THREADS = 256;
constexpr int ST_STAGES = 6;
constexpr int ST_AHEAD = ST_STAGES - 2;            // k-blocks in flight ahead of the one being multiplied
constexpr int ST_TILE_BYTES = ST_BM * ST_BK * 4;   // 8 KiB per operand tile
constexpr int ST_STAGE_BYTES = 2 * ST_TILE_BYTES;
constexpr int ST_SMEM_BYTES = ST_STAGES * ST_STAGE_BYTES + 1024 /*alignment slack*/ + 128 /*barriers, flag*/;

struct SgemmParams {
    int M, N, K, nkb;
    float alpha, beta;
    float *C;
    int64_t ldc;
    int tiles_m, tiles_n, group;
    const float *bias;
    int act;
    const float *R;  // residual added after the activation, or nullptr
    int64_t ldr;
    int vec_ok;  // C (and R) base and pitch allow 16-byte accesses
    // k-slices (gridDim.y > 1): block (x, y) multiplies k-blocks [y * kb_per_split, ...) of tile x and stores the
    // raw sums to ws[y][M][ldw]; sgemm_splitk_reduce_kernel adds the slices in order and applies the epilogue
    int kb_per_split;
    float *ws;
    int64_t ldw;
    long long wait_cycles;
    uint32_t *status;
};

__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float2 lds64(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}

// A_KC / B_KC: the operand's contiguous index in memory is k (A not transposed / B transposed).
// KG: how many k one shared-memory load of a k-contiguous operand covers (4: 16-byte loads, 2: 8-byte loads;
// two k-contiguous operands at 4 k each would not fit the register budget of two blocks per SM).
// WIDE: the same 128 x 128 x 16 block tile worked on by 128 threads, each with an 8 x 16 register tile (128
// accumulators, up to 255 registers, still two blocks per SM): six shared-memory loads per 64 two-wide FMAs
// instead of four per 32, and the operands of the next k are fetched into a second set of registers while the
// current k is multiplied, so that two warps per scheduler are enough to keep the FMA pipe fed.  B must land
// dense.
template <bool A_KC, bool B_KC, int KG, bool WIDE = false>
__global__ void __launch_bounds__(WIDE ? 128 : ST_THREADS, 2)
sgemm_tma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const SgemmParams p) {
    static_assert(!WIDE || !B_KC, "the wide register tile needs B dense");
    constexpr int THREADS = WIDE ? 128 : ST_THREADS, NWARPS = THREADS / 32;
    constexpr int NT = WIDE ? 16 : 8;            // columns of C per thread
    constexpr int TXN = WIDE ? 8 : 16;           // threads along n; each takes groups of 4 columns TXN*4 apart
    extern __shared__ uint8_t st_smem_raw[];
    const uint32_t raw = ptx::smem_u32(st_smem_raw);
    const uint32_t stage0 = (raw + 1023u) & ~1023u;
    const uint32_t full0 = stage0 + ST_STAGES * ST_STAGE_BYTES;
    const uint32_t empty0 = full0 + 8 * ST_STAGES;
    volatile uint32_t *abort_flag =
        reinterpret_cast<volatile uint32_t *>(st_smem_raw + (empty0 + 8 * ST_STAGES - raw));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tx = tid % TXN, ty = tid / TXN;
    int64_t tm, tn;
    tile_coord(blockIdx.x, p.tiles_m, p.tiles_n, p.group, tm, tn);
    const int m0 = (int)tm * ST_BM, n0 = (int)tn * ST_BN;

    if (tid == 0) {
        for (int s = 0; s < ST_STAGES; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, NWARPS);  // one arrival per warp
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    __syncthreads();
    ptx::grid_launch_dependents();  // a reduction kernel that follows may be scheduled; it waits for this grid to end

    const bool sliced = gridDim.y > 1;
    const int koff = sliced ? (int)blockIdx.y * p.kb_per_split : 0;  // first k-block of this block's slice
    auto issue = [&](int kb) {  // one thread: both tiles of k-block kb (of the slice) into stage kb % STAGES
        const uint32_t s = (uint32_t)kb % ST_STAGES;
        const uint32_t bar = full0 + 8 * s;
        const uint32_t a_dst = stage0 + s * ST_STAGE_BYTES, b_dst = a_dst + ST_TILE_BYTES;
        const int k0 = (koff + kb) * ST_BK;
        ptx::mbar_arrive_expect_tx(bar, (uint32_t)ST_STAGE_BYTES);
        if (A_KC) ptx::tma_load_2d(a_dst, &tmA, k0, m0, bar);
        else ptx::tma_load_2d(a_dst, &tmA, m0, k0, bar);
        if (B_KC) ptx::tma_load_2d(b_dst, &tmB, k0, n0, bar);
        else ptx::tma_load_2d(b_dst, &tmB, n0, k0, bar);
    };

    const int nkb = sliced ? min(p.kb_per_split, p.nkb - koff) : p.nkb;
    if (tid == 0)
        for (int kb = 0; kb < ST_AHEAD && kb < nkb; ++kb) issue(kb);

    float acc[8][NT];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j) acc[i][j] = 0.0f;

    // Row i of this thread's 8 x 8 tile is m0 + ty*4 + (i & 3) + 64*(i >> 2).  Column j is n0 + tx*4 + (j & 3) +
    // 64*(j >> 2) when B lands dense, n0 + tx + 16*j when B is k-contiguous: with the 64-byte swizzle the sixteen
    // tx of a warp then read sixteen different 16-byte pieces spread over all banks.
    // Byte offset inside a swizzled S[row][16 k] tile: row*64 + ((chunk ^ ((row >> 1) & 3)) * 16).  For A the
    // swizzle term of row i is a compile-time part ((i & 3) >> 1) XOR a per-thread part (ty & 1) * 2, so every
    // address is one of two per-thread bases (+32 or -32 bytes for the per-thread part) plus a constant; for B
    // the term (tx >> 1) & 3 is the same for all eight rows, so four per-thread offsets (one per chunk) serve.
    const uint32_t a_t = A_KC ? (uint32_t)(ty & 1) * 32u : 0u;
    const uint32_t a_base = (uint32_t)ty * 256u;
    uint32_t b_off[4] = {0u, 0u, 0u, 0u};
    if (B_KC) {
#pragma unroll
        for (int c = 0; c < 4; ++c) b_off[c] = (uint32_t)tx * 64u + ((((uint32_t)c) ^ ((uint32_t)(tx >> 1) & 3u)) << 4);
    }

    bool ok = true;
    for (int kb = 0; kb < nkb; ++kb) {
        const uint32_t s = (uint32_t)kb % ST_STAGES, ph = ((uint32_t)kb / ST_STAGES) & 1u;
        // the warps take turns at refilling the ring: stage (kb + AHEAD) % STAGES was last read two k-blocks ago
        if (warp == (kb % NWARPS) && lane == 0 && kb + ST_AHEAD < nkb) {
            const int kl = kb + ST_AHEAD;
            const uint32_t sl = (uint32_t)kl % ST_STAGES, pl = ((uint32_t)kl / ST_STAGES) & 1u;
            if (ptx::mbar_wait<false>(empty0 + 8 * sl, pl ^ 1u, abort_flag, p.wait_cycles)) issue(kl);
            else {
                if (*abort_flag == 0) atomicOr(p.status, kStatusTimeout | (sl << 8) | 0x11u);
                *abort_flag = 1;
            }
        }
        __syncwarp();
        const bool got = ptx::mbar_wait<false>(full0 + 8 * s, ph, abort_flag, p.wait_cycles);
        if (!__all_sync(0xffffffffu, got)) {
            if (lane == 0) {
                if (*abort_flag == 0) atomicOr(p.status, kStatusTimeout | (s << 8) | 0x12u);
                *abort_flag = 1;
            }
            ok = false;
            break;
        }
        const uint32_t As = stage0 + s * ST_STAGE_BYTES, Bs = As + ST_TILE_BYTES;
        if constexpr (WIDE) {
            // operand fragments of one k: a[8] (rows) and b[16] (columns: four groups of 4, 32 columns apart, so
            // that the eight tx of a warp read 128 contiguous bytes per load and the four ty share them)
            auto load_b = [&](int k, float (&b)[16]) {
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 v = lds128(Bs + (uint32_t)(k * ST_BN + tx * 4 + 32 * h) * 4u);
                    b[4 * h] = v.x; b[4 * h + 1] = v.y; b[4 * h + 2] = v.z; b[4 * h + 3] = v.w;
                }
            };
            auto load_a_dense = [&](int k, float (&a)[8]) {
                const float4 v0 = lds128(As + (uint32_t)(k * ST_BM + ty * 4) * 4u);
                const float4 v1 = lds128(As + (uint32_t)(k * ST_BM + ty * 4 + 64) * 4u);
                a[0] = v0.x; a[1] = v0.y; a[2] = v0.z; a[3] = v0.w; a[4] = v1.x; a[5] = v1.y; a[6] = v1.z; a[7] = v1.w;
            };
            auto load_a_pair = [&](int k2, float (&a0)[8], float (&a1)[8]) {  // k-contiguous A: k = 2*k2 and 2*k2 + 1
                const uint32_t a_plus = As + a_base + a_t, a_minus = As + a_base - a_t;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t q = ((uint32_t)k2 >> 1) ^ (uint32_t)((i & 3) >> 1);
                    const uint32_t off = (uint32_t)((i & 3) + 64 * (i >> 2)) * 64u + (q << 4) + ((uint32_t)k2 & 1u) * 8u;
                    const float2 v = lds64(((q & 2u) ? a_minus : a_plus) + off);
                    a0[i] = v.x; a1[i] = v.y;
                }
            };
            auto fma_k = [&](const float (&a)[8], const float (&b)[16]) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float2 aa = make_float2(a[i], a[i]);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float2 c = make_float2(acc[i][2 * j], acc[i][2 * j + 1]);
                        c = __ffma2_rn(aa, make_float2(b[2 * j], b[2 * j + 1]), c);
                        acc[i][2 * j] = c.x;
                        acc[i][2 * j + 1] = c.y;
                    }
                }
            };
            if constexpr (A_KC && KG == 4) {
                // k-contiguous A, four k per 16-byte load: eight loads fetch this thread's rows for four k (the same
                // two loads per k as a dense tile); the next four k are fetched while these are multiplied
                auto load_a_quad = [&](int k4, float (&aq)[8][4]) {
                    const uint32_t a_plus = As + a_base + a_t, a_minus = As + a_base - a_t;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t q = (uint32_t)k4 ^ (uint32_t)((i & 3) >> 1);
                        const uint32_t off = (uint32_t)((i & 3) + 64 * (i >> 2)) * 64u + (q << 4);
                        const float4 v = lds128(((q & 2u) ? a_minus : a_plus) + off);
                        aq[i][0] = v.x; aq[i][1] = v.y; aq[i][2] = v.z; aq[i][3] = v.w;
                    }
                };
                float aq[2][8][4], bq[2][16];
                load_a_quad(0, aq[0]);
                load_b(0, bq[0]);
#pragma unroll
                for (int k4 = 0; k4 < ST_BK / 4; ++k4) {
                    const int ca = k4 & 1;
                    if (k4 + 1 < ST_BK / 4) load_a_quad(k4 + 1, aq[ca ^ 1]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int kg = 4 * k4 + k, cb = kg & 1;
                        if (kg + 1 < ST_BK) load_b(kg + 1, bq[cb ^ 1]);
                        float a[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) a[i] = aq[ca][i][k];
                        fma_k(a, bq[cb]);
                    }
                }
            } else {
            // two k per step, fragments of the next step fetched before this step's FMAs are issued
            float a0[2][8], a1[2][8], b0[2][16], b1[2][16];
            if (A_KC) load_a_pair(0, a0[0], a1[0]);
            else { load_a_dense(0, a0[0]); load_a_dense(1, a1[0]); }
            load_b(0, b0[0]);
            load_b(1, b1[0]);
#pragma unroll
            for (int k2 = 0; k2 < ST_BK / 2; ++k2) {
                const int cur = k2 & 1, nxt = cur ^ 1;
                if (k2 + 1 < ST_BK / 2) {
                    if (A_KC) load_a_pair(k2 + 1, a0[nxt], a1[nxt]);
                    else { load_a_dense(2 * k2 + 2, a0[nxt]); load_a_dense(2 * k2 + 3, a1[nxt]); }
                    load_b(2 * k2 + 2, b0[nxt]);
                }
                fma_k(a0[cur], b0[cur]);
                if (k2 + 1 < ST_BK / 2) load_b(2 * k2 + 3, b1[nxt]);
                fma_k(a1[cur], b1[cur]);
            }
            }
        } else {
#pragma unroll
        for (int kk = 0; kk < ST_BK; kk += KG) {
            float ak[8][KG], bk[8][KG];
            if (A_KC) {
                const uint32_t a_plus = As + a_base + a_t, a_minus = As + a_base - a_t;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    // chunk ^ const part, then ^ (ty & 1) * 2: adds 32 bytes when bit 1 is clear, else subtracts
                    const uint32_t q = ((uint32_t)kk >> 2) ^ (uint32_t)((i & 3) >> 1);
                    const uint32_t off = (uint32_t)((i & 3) + 64 * (i >> 2)) * 64u + (q << 4) +
                                         (KG == 2 ? (((uint32_t)kk >> 1) & 1u) * 8u : 0u);
                    const uint32_t addr = ((q & 2u) ? a_minus : a_plus) + off;
                    if (KG == 4) {
                        const float4 v = lds128(addr);
                        ak[i][0] = v.x; ak[i][1] = v.y; ak[i][KG - 2] = v.z; ak[i][KG - 1] = v.w;
                    } else {
                        const float2 v = lds64(addr);
                        ak[i][0] = v.x; ak[i][1] = v.y;
                    }
                }
            }
            if (B_KC) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t addr = Bs + b_off[(kk >> 2) & 3] + (uint32_t)j * 1024u +
                                          (KG == 2 ? (((uint32_t)kk >> 1) & 1u) * 8u : 0u);
                    if (KG == 4) {
                        const float4 v = lds128(addr);
                        bk[j][0] = v.x; bk[j][1] = v.y; bk[j][KG - 2] = v.z; bk[j][KG - 1] = v.w;
                    } else {
                        const float2 v = lds64(addr);
                        bk[j][0] = v.x; bk[j][1] = v.y;
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < KG; ++k) {
                float a[8], b[8];
                if (A_KC) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) a[i] = ak[i][k];
                } else {
                    const float4 v0 = lds128(As + (uint32_t)((kk + k) * ST_BM + ty * 4) * 4u);
                    const float4 v1 = lds128(As + (uint32_t)((kk + k) * ST_BM + ty * 4 + 64) * 4u);
                    a[0] = v0.x; a[1] = v0.y; a[2] = v0.z; a[3] = v0.w; a[4] = v1.x; a[5] = v1.y; a[6] = v1.z; a[7] = v1.w;
                }
                if (B_KC) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) b[j] = bk[j][k];
                } else {
                    const float4 v0 = lds128(Bs + (uint32_t)((kk + k) * ST_BN + tx * 4) * 4u);
                    const float4 v1 = lds128(Bs + (uint32_t)((kk + k) * ST_BN + tx * 4 + 64) * 4u);
                    b[0] = v0.x; b[1] = v0.y; b[2] = v0.z; b[3] = v0.w; b[4] = v1.x; b[5] = v1.y; b[6] = v1.z; b[7] = v1.w;
                }
                // two-wide fp32 FMA: two independent, individually rounded fp32 FMAs per instruction
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float2 aa = make_float2(a[i], a[i]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float2 c = make_float2(acc[i][2 * j], acc[i][2 * j + 1]);
                        c = __ffma2_rn(aa, make_float2(b[2 * j], b[2 * j + 1]), c);
                        acc[i][2 * j] = c.x;
                        acc[i][2 * j + 1] = c.y;
                    }
                }
            }
        }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(empty0 + 8 * s);  // this warp is done reading the stage
    }
    if (!ok || *abort_flag != 0) {
        // a wait gave up: let copies that may still be in flight land before shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
        return;
    }

    // ---- epilogue: alpha / beta (+ bias, activation) in fp32, predicated at the edges -------------------------
    // a k-slice stores its raw sums to the workspace: alpha = 1, beta = 0, nothing fused
    const float alpha = sliced ? 1.0f : p.alpha, beta = sliced ? 0.0f : p.beta;
    float *const c_base = sliced ? p.ws + (int64_t)blockIdx.y * p.M * p.ldw : p.C;
    const int64_t c_ld = sliced ? p.ldw : p.ldc;
    const float *const bias = sliced ? nullptr : bias;
    const int act = sliced ? 0 : act;
    const float *const res = sliced ? nullptr : p.R;
    const bool vec_ok = sliced ? true : p.vec_ok != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int m = m0 + ty * 4 + (i & 3) + 64 * (i >> 2);
        if (m >= p.M) continue;
        float *crow = c_base + (int64_t)m * c_ld;
        if (!B_KC) {
#pragma unroll
            for (int h = 0; h < NT / 4; ++h) {
                const int n = n0 + tx * 4 + TXN * 4 * h;
                if (n >= p.N) continue;
                if (vec_ok && n + 4 <= p.N) {
                    float4 *dst = reinterpret_cast<float4 *>(crow + n);
                    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (beta != 0.0f) o = *dst;
                    float4 r;
                    r.x = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 0], beta, o.x), bias, n + 0, act);
                    r.y = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 1], beta, o.y), bias, n + 1, act);
                    r.z = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 2], beta, o.z), bias, n + 2, act);
                    r.w = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 3], beta, o.w), bias, n + 3, act);
                    if (res) {
                        const float4 q = *reinterpret_cast<const float4 *>(res + (int64_t)m * p.ldr + n);
                        r.x += q.x; r.y += q.y; r.z += q.z; r.w += q.w;
                    }
                    *dst = r;
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (n + q < p.N) {
                            const float o = (beta != 0.0f) ? crow[n + q] : 0.0f;
                            crow[n + q] = add_residual(finish_f32(epilogue_f32(alpha, acc[i][4 * h + q], beta, o), bias, n + q, act),
                                                       res, (int64_t)m * p.ldr + n + q);
                        }
                    }
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int n = n0 + tx + 16 * j;
                if (n < p.N) {
                    const float o = (beta != 0.0f) ? crow[n] : 0.0f;
                    crow[n] = add_residual(finish_f32(epilogue_f32(alpha, acc[i][j], beta, o), bias, n, act), res,
                                           (int64_t)m * p.ldr + n);
                }
            }
        }
    }
}

// Adds the k-slices of a sliced launch in slice order and applies the epilogue: C = alpha * (ws[0] + ws[1] + ...) +
// beta * C (+ bias, activation, residual), four columns per thread.
__global__ void __launch_bounds__(256)
sgemm_splitk_reduce_kernel(const float *__restrict__ ws, int splits, int M, int N, int64_t ldw, float alpha, float beta,
                           float *__restrict__ C, int64_t ldc, const float *__restrict__ bias, int act,
                           const float *__restrict__ R, int64_t ldr, int vec_ok) {
    const int n4 = (N + 3) / 4;
    const int64_t total = (int64_t)M * n4;
    const int64_t slice = (int64_t)M * ldw;
    // launched as a programmatic dependent of the slice kernel: the slices may be read once that kernel has completed
    ptx::grid_dependency_wait();
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int m = (int)(e / n4), n = (int)(e - (int64_t)m * n4) * 4;
        const float *src = ws + (int64_t)m * ldw + n;
        float4 a = *reinterpret_cast<const float4 *>(src);
        for (int sl = 1; sl < splits; ++sl) {
            const float4 v = *reinterpret_cast<const float4 *>(src + sl * slice);
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        const float av[4] = {a.x, a.y, a.z, a.w};
        float *crow = C + (int64_t)m * ldc;
        if (vec_ok && n + 4 <= N) {
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (beta != 0.0f) o = *reinterpret_cast<const float4 *>(crow + n);
            const float ov[4] = {o.x, o.y, o.z, o.w};
            float r[4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
                r[q] = add_residual(finish_f32(epilogue_f32(alpha, av[q], beta, ov[q]), bias, n + q, act), R, (int64_t)m * ldr + n + q);
            *reinterpret_cast<float4 *>(crow + n) = make_float4(r[0], r[1], r[2], r[3]);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (n + q < N) {
                    const float o = (beta != 0.0f) ? crow[n + q] : 0.0f;
                    crow[n + q] = add_residual(finish_f32(epilogue_f32(alpha, av[q], beta, o), bias, n + q, act), R,
                                               (int64_t)m * ldr + n + q);
                }
            }
        }
    }
}

// dst[c][r] = src[r][c] for an r x c row-major matrix: 32 x 32 tiles through padded shared memory, both sides
// coalesced.  The paper's Transpose step as a pass of its own.
__global__ void __launch_bounds__(256)
transpose_f32_kernel(const float *__restrict__ src, int64_t ld_src, int rows, int cols, float *__restrict__ dst,
                     int64_t ld_dst) {
    __shared__ float tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
        const int r = r0 + ty + i, c = c0 + tx;
        if (r < rows && c < cols) tile[ty + i][tx] = src[(int64_t)r * ld_src + c];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
        const int c = c0 + ty + i, r = r0 + tx;
        if (r < rows && c < cols) dst[(int64_t)c * ld_dst + r] = tile[tx][ty + i];
    }
}

int launch_transpose(const float *src, int64_t ld_src, int64_t rows, int64_t cols, float *dst, int64_t ld_dst,
                     cudaStream_t stream) {
    dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32));
    if (grid.y > 65535u) return PEAK_ERR_UNSUPPORTED;
    transpose_f32_kernel<<<grid, 256, 0, stream>>>(src, ld_src, (int)rows, (int)cols, dst, ld_dst);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <bool A_KC, bool B_KC, int KG, bool WIDE = false> int run_sgemm_tma(const GemmArgs &g) {
    auto kernel = sgemm_tma_kernel<A_KC, B_KC, KG, WIDE>;
    static PerDeviceOnce attr_once;
    const cudaError_t attr_err = attr_once.run(current_device(), [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }

    CUtensorMap tmA, tmB;
    // k-contiguous operand: rows of the stored matrix are rows of the tile, 16 k wide, 64-byte swizzle;
    // otherwise the stored matrix is [k][mn]: dense boxes of 128 contiguous elements by 16 k-rows
    bool ok = A_KC ? umma::make_map(&tmA, Elem::F32, g.A, g.K, g.M, g.lda, ST_BK, ST_BM, 1, 0, 64)
                   : umma::make_map(&tmA, Elem::F32, g.A, g.M, g.K, g.lda, ST_BM, ST_BK, 1, 0, 0);
    ok = ok && (B_KC ? umma::make_map(&tmB, Elem::F32, g.B, g.K, g.N, g.ldb, ST_BK, ST_BN, 1, 0, 64)
                     : umma::make_map(&tmB, Elem::F32, g.B, g.N, g.K, g.ldb, ST_BN, ST_BK, 1, 0, 0));
    if (!ok) return PEAK_ERR_CUDA;

    SgemmParams p;
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.nkb = (int)((g.K + ST_BK - 1) / ST_BK);
    p.alpha = g.alpha; p.beta = g.beta;
    p.C = (float *)g.C; p.ldc = g.ldc;
    p.tiles_m = (int)((g.M + ST_BM - 1) / ST_BM);
    p.tiles_n = (int)((g.N + ST_BN - 1) / ST_BN);
    p.group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : 8;
    p.bias = g.bias; p.act = g.act;
    p.R = (const float *)g.R; p.ldr = g.ldr;
    p.vec_ok = (reinterpret_cast<uintptr_t>(g.C) % 16 == 0 && g.ldc % 4 == 0 &&
                (!g.R || (reinterpret_cast<uintptr_t>(g.R) % 16 == 0 && g.ldr % 4 == 0))) ? 1 : 0;
    const int wait_ms = tuning(PEAK_TUNE_WAIT_MS);
    p.wait_cycles = wait_ms > 0 ? (long long)wait_ms * 2000000LL : ptx::kWaitBudgetCycles;
    p.status = device_status_word();
    if (!p.status) return PEAK_ERR_CUDA;
    const unsigned grid = (unsigned)(p.tiles_m * p.tiles_n);
    // k-slices for small grids.  The kernel needs two blocks per SM to keep the FMA pipe fed (four warps of a lone
    // block reach about 40 % of it), so a problem with fewer tiles than that is cut along k until it has them, down
    // to four k-blocks per slice and never beyond one full wave of two blocks per SM (measured, us, NN: 256^3 47 ->
    // 15.6, 512^3 69 -> 18.4, 1024^3 113 -> 55.6, 1536^3 159 -> 142, 128x4096x4096 381 -> 92.6; cuBLAS 8.2 / 13.2 /
    // 45.1 / 121 / 104.7).  PEAK_TUNE_SPLIT_K forces the number of slices (1 = none).
    int splits = 1;
    {
        const int want_blocks = 2 * umma::sm_count();
        const int forced = tuning(PEAK_TUNE_SPLIT_K);
        if (forced > 0) splits = forced;
        else if ((int)grid < want_blocks) splits = std::max(1, want_blocks / (int)grid);  // one full wave of two blocks per SM
        splits = std::min(splits, std::max(1, p.nkb / 4));
        splits = std::min(splits, 64);
        while (splits > 1 && (size_t)splits * (size_t)g.M * (size_t)((g.N + 3) / 4 * 4) * 4 > (256ull << 20)) --splits;
        p.kb_per_split = (p.nkb + splits - 1) / splits;
        splits = (p.nkb + p.kb_per_split - 1) / p.kb_per_split;  // no empty slice
    }
    p.ws = nullptr; p.ldw = (g.N + 3) / 4 * 4;
    if (splits > 1) {
        cudaMemPool_t pool = scratch_pool();
        if (!pool) return PEAK_ERR_CUDA;
        cudaError_t me = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&p.ws), (size_t)splits * g.M * p.ldw * sizeof(float),
                                                 pool, g.stream);
        if (me != cudaSuccess) { set_cuda_error(me); return PEAK_ERR_NO_MEMORY; }
    }
    kernel<<<dim3(grid, (unsigned)splits), WIDE ? 128 : ST_THREADS, ST_SMEM_BYTES, g.stream>>>(tmA, tmB, p);
    count_launch();
    note_kernel("sgemm_tma_kernel<%d, %d, %d, %d> grid=%u slices=%d", (int)A_KC, (int)B_KC, KG, (int)WIDE, grid, splits);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && splits > 1) {
        const int64_t work = (int64_t)g.M * ((g.N + 3) / 4);
        const unsigned rgrid = (unsigned)std::min<int64_t>((work + 255) / 256, 4 * (int64_t)umma::sm_count());
        cudaLaunchConfig_t rcfg = {};
        rcfg.gridDim = dim3(rgrid);
        rcfg.blockDim = dim3(256);
        rcfg.stream = g.stream;
        cudaLaunchAttribute rattr[1];
        rattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        rattr[0].val.programmaticStreamSerializationAllowed = 1;
        rcfg.attrs = rattr;
        rcfg.numAttrs = tuning(PEAK_TUNE_DEPENDENT_LAUNCH) == 1 ? 0 : 1;
        const float *ws_c = p.ws;
        e = cudaLaunchKernelEx(&rcfg, sgemm_splitk_reduce_kernel, ws_c, splits, p.M, p.N, p.ldw, g.alpha, g.beta, (float *)g.C,
                               g.ldc, g.bias, g.act, (const float *)g.R, g.ldr, p.vec_ok);
        count_launch();
    }
    if (p.ws) {
        const cudaError_t fe = cudaFreeAsync(p.ws, g.stream);
        if (e == cudaSuccess) e = fe;
    }
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

}  // namespace

// Any shape and layout; the copy engine needs 16-byte aligned operand bases and pitches.
bool sgemm_tma_supports(const GemmArgs &g) {
    if (g.dtype != PEAK_F32_F32) return false;
    if (g.M < 1 || g.N < 1 || g.K < 1) return false;
    if (g.M >= (1ll << 31) - 256 || g.N >= (1ll << 31) - 256 || g.K >= (1ll << 31) - 256) return false;
    if (((g.M + ST_BM - 1) / ST_BM) * ((g.N + ST_BN - 1) / ST_BN) >= (1ll << 31)) return false;
    if (g.lda % 4 || g.ldb % 4 || g.lda >= (1ll << 38) || g.ldb >= (1ll << 38)) return false;
    if (reinterpret_cast<uintptr_t>(g.A) % 16 || reinterpret_cast<uintptr_t>(g.B) % 16) return false;
    if (reinterpret_cast<uintptr_t>(g.C) % 4) return false;
    return true;
}

// A k-contiguous operand costs the kernel 7 points of FMA-pipe time (A) or far more (B); a copy of it with m / n
// contiguous costs one pass over that operand.  Where the product is large against the operand -- the other
// dimension at least 2048, so the pass is under about 2 % -- and the copy fits a bounded workspace, the operand
// is transposed into pool memory first and the dense-dense kernel runs (4096^3 NN: 58.8 -> 63+ TFLOP/s).
int launch_with_transposes(const GemmArgs &g, bool tr_a, bool tr_b) {
    GemmArgs d = g;
    float *wa = nullptr, *wb = nullptr;
    cudaMemPool_t pool = scratch_pool();
    if (!pool) return PEAK_ERR_CUDA;
    int rc = PEAK_OK;
    cudaError_t e = cudaSuccess;
    if (tr_a) {  // A stored M x K  ->  K x M
        const int64_t ld = (g.M + 3) / 4 * 4;
        e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&wa), (size_t)g.K * ld * sizeof(float), pool, g.stream);
        if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_NO_MEMORY; }
        rc = launch_transpose((const float *)g.A, g.lda, g.M, g.K, wa, ld, g.stream);
        d.A = wa; d.lda = ld; d.transA = 1;
    }
    if (rc == PEAK_OK && tr_b) {  // B stored N x K  ->  K x N
        const int64_t ld = (g.N + 3) / 4 * 4;
        e = cudaMallocFromPoolAsync(reinterpret_cast<void **>(&wb), (size_t)g.K * ld * sizeof(float), pool, g.stream);
        if (e != cudaSuccess) { set_cuda_error(e); rc = PEAK_ERR_NO_MEMORY; }
        else {
            rc = launch_transpose((const float *)g.B, g.ldb, g.N, g.K, wb, ld, g.stream);
            d.B = wb; d.ldb = ld; d.transB = 0;
        }
    }
    if (rc == PEAK_OK) {
        const bool a_kc = !d.transA, b_kc = d.transB != 0;  // what is still k-contiguous
        if (a_kc && b_kc) rc = run_sgemm_tma<true, true, 2>(d);
        else if (b_kc) rc = run_sgemm_tma<false, true, 4>(d);
        else if (a_kc) rc = run_sgemm_tma<true, false, 4, true>(d);
        else rc = run_sgemm_tma<false, false, 2, true>(d);
    }
    if (wa) cudaFreeAsync(wa, g.stream);
    if (wb) cudaFreeAsync(wb, g.stream);
    return rc;
}

int launch_sgemm_tma(const GemmArgs &g) {
    if (!sgemm_tma_supports(g)) return PEAK_ERR_UNSUPPORTED;
    const bool a_kc = !g.transA, b_kc = g.transB != 0;
    {
        const int mode = tuning(PEAK_TUNE_SGEMM_TRANSPOSE);  // 1 = never, 2 = whenever an operand is k-contiguous
        const int64_t limit = 512ll << 20;                   // bytes of one transposed copy
        const bool fits_a = g.M * g.K * 4 <= limit && g.M <= 65535ll * 32, fits_b = g.N * g.K * 4 <= limit && g.N <= 65535ll * 32;
        const bool tr_a = a_kc && fits_a && (mode == 2 || (mode == 0 && g.N >= 2048 && g.M >= 512));
        // (a B with k contiguous is also transposed first when the grid is small: the problem is then cut along k by
        // the dense kernel, which beats the k-contiguous kernel's 60 % of the FMA rate by more than the extra pass costs)
        const bool small_grid = ((g.M + ST_BM - 1) / ST_BM) * ((g.N + ST_BN - 1) / ST_BN) < 2 * (int64_t)umma::sm_count();
        const bool tr_b = b_kc && fits_b && (mode == 2 || (mode == 0 && ((g.M >= 2048 && g.N >= 512) || small_grid)));
        if (mode != 1 && (tr_a || tr_b)) return launch_with_transposes(g, tr_a, tr_b);
    }
    // k per load of a k-contiguous operand, measured at 4096^3 / 8192^3 NN: two (58.8 / 59.3 TFLOP/s) beats four
    // (58.1 / 58.7): the sixteen fewer live registers leave the scheduler more room
    if (a_kc && b_kc) return run_sgemm_tma<true, true, 2>(g);
    if (b_kc) return run_sgemm_tma<false, true, 4>(g);
    const bool wide = tuning(PEAK_TUNE_SGEMM_FMA) != 3;  // 3 = the 8 x 8 register tile (A/B measurements)
    if (wide && a_kc) return tuning(PEAK_TUNE_SGEMM_FMA) == 4 ? run_sgemm_tma<true, false, 2, true>(g) : run_sgemm_tma<true, false, 4, true>(g);
    if (wide) return run_sgemm_tma<false, false, 2, true>(g);
    if (a_kc) return run_sgemm_tma<true, false, 2>(g);
    return run_sgemm_tma<false, false, 4>(g);
}

}  // namespace peak
