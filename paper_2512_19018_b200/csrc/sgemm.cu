// fp32 GEMM on the CUDA cores (plain fp32 FMA; TF32 is never used).
//
// The structure follows the paper's CUDA-core sequence (sections 2.2 and 4.3): thread-block tiling
// (128 x 128 x 16 tile staged in shared memory), thread tiling (8 x 8 outputs per thread held in
// registers, operands cached in registers per k), vectorised float4 global and shared accesses,
// register staging of the next k-block while the current one is multiplied (two shared-memory buffers),
// a transposing store for the operand whose contiguous index is k, padding against bank conflicts, and a
// grouped block order for L2 reuse.
#include "common.cuh"

namespace peak {
namespace {

constexpr int SG_BM = 128, SG_BN = 128, SG_BK = 16;
constexpr int SG_THREADS = 256;
constexpr int SG_PAD = 4;  // floats of padding per shared-memory row
constexpr int SG_LD = SG_BM + SG_PAD;

// Stage a (128 x 16) operand tile as S[k][mn].  KCONTIG: memory is [mn][k] (k contiguous), so the float4
// read along k is scattered into four rows; otherwise memory is [k][mn] and the float4 is stored as is.
template <bool KCONTIG> struct Loader {
    const float *base;  // tile origin
    int64_t pitch;
    int r0, c0;  // this thread's first float4: KCONTIG: row mn=r0 (+64), k=c0 ; else: row k=r0 (+8), mn=c0
    __device__ __forceinline__ Loader(const float *origin, int64_t pitch_, int tid) : base(origin), pitch(pitch_) {
        if (KCONTIG) { r0 = tid / 4; c0 = (tid % 4) * 4; } else { r0 = tid / 32; c0 = (tid % 32) * 4; }
    }
    __device__ __forceinline__ void load(float4 (&g)[2], int64_t k0) const {
        if (KCONTIG) {
            g[0] = *reinterpret_cast<const float4 *>(base + (int64_t)r0 * pitch + k0 + c0);
            g[1] = *reinterpret_cast<const float4 *>(base + (int64_t)(r0 + 64) * pitch + k0 + c0);
        } else {
            g[0] = *reinterpret_cast<const float4 *>(base + (k0 + r0) * pitch + c0);
            g[1] = *reinterpret_cast<const float4 *>(base + (k0 + r0 + 8) * pitch + c0);
        }
    }
    __device__ __forceinline__ void store(float (*S)[SG_LD], const float4 (&g)[2]) const {
        if (KCONTIG) {
            S[c0 + 0][r0] = g[0].x; S[c0 + 1][r0] = g[0].y; S[c0 + 2][r0] = g[0].z; S[c0 + 3][r0] = g[0].w;
            S[c0 + 0][r0 + 64] = g[1].x; S[c0 + 1][r0 + 64] = g[1].y; S[c0 + 2][r0 + 64] = g[1].z; S[c0 + 3][r0 + 64] = g[1].w;
        } else {
            *reinterpret_cast<float4 *>(&S[r0][c0]) = g[0];
            *reinterpret_cast<float4 *>(&S[r0 + 8][c0]) = g[1];
        }
    }
};

// PACKED selects the two-wide fp32 FMA of sm_100 (two independent fp32 FMAs per instruction, same rounding
// as two scalar FMAs): half the issue slots for the same arithmetic.
template <bool TA, bool TB, bool PACKED>
__global__ void __launch_bounds__(SG_THREADS, 2)
sgemm_kernel(int M, int N, int K, float alpha, const float *__restrict__ A, int64_t lda, const float *__restrict__ B,
             int64_t ldb, float beta, float *__restrict__ C, int64_t ldc, int tiles_m, int tiles_n, int group,
             const float *__restrict__ bias, int act, const float *__restrict__ R, int64_t ldr) {
    __shared__ __align__(16) float As[2][SG_BK][SG_LD];
    __shared__ __align__(16) float Bs[2][SG_BK][SG_LD];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    int64_t tm, tn;
    tile_coord(blockIdx.x, tiles_m, tiles_n, group, tm, tn);
    const int64_t m0 = tm * SG_BM, n0 = tn * SG_BN;

    // A: not transposed -> stored [m][k] (k contiguous); transposed -> stored [k][m]
    // B: not transposed -> stored [k][n];               transposed -> stored [n][k] (k contiguous)
    Loader<!TA> la(TA ? A + m0 : A + m0 * lda, lda, tid);
    Loader<TB> lb(TB ? B + n0 * ldb : B + n0, ldb, tid);

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    float4 ga[2], gb[2];
    la.load(ga, 0);
    lb.load(gb, 0);
    la.store(As[0], ga);
    lb.store(Bs[0], gb);
    __syncthreads();

    const int nkb = K / SG_BK;
    for (int kb = 0; kb < nkb; ++kb) {
        const int cur = kb & 1;
        if (kb + 1 < nkb) {  // register staging of the next k-block
            la.load(ga, (int64_t)(kb + 1) * SG_BK);
            lb.load(gb, (int64_t)(kb + 1) * SG_BK);
        }
#pragma unroll
        for (int k = 0; k < SG_BK; ++k) {
            float a[8], b[8];
            *reinterpret_cast<float4 *>(&a[0]) = *reinterpret_cast<const float4 *>(&As[cur][k][ty * 4]);
            *reinterpret_cast<float4 *>(&a[4]) = *reinterpret_cast<const float4 *>(&As[cur][k][ty * 4 + 64]);
            *reinterpret_cast<float4 *>(&b[0]) = *reinterpret_cast<const float4 *>(&Bs[cur][k][tx * 4]);
            *reinterpret_cast<float4 *>(&b[4]) = *reinterpret_cast<const float4 *>(&Bs[cur][k][tx * 4 + 64]);
            if (PACKED) {
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
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
        }
        if (kb + 1 < nkb) {
            la.store(As[cur ^ 1], ga);
            lb.store(Bs[cur ^ 1], gb);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t m = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float4 *dst = reinterpret_cast<float4 *>(C + m * ldc + n0 + tx * 4 + h * 64);
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (beta != 0.0f) o = *dst;
            float4 r;
            const int64_t n = n0 + tx * 4 + h * 64;
            r.x = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 0], beta, o.x), bias, n + 0, act);
            r.y = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 1], beta, o.y), bias, n + 1, act);
            r.z = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 2], beta, o.z), bias, n + 2, act);
            r.w = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 3], beta, o.w), bias, n + 3, act);
            if (R) {
                const float4 q = *reinterpret_cast<const float4 *>(R + m * ldr + n);
                r.x += q.x; r.y += q.y; r.z += q.z; r.w += q.w;
            }
            *dst = r;
        }
    }
}

// ---- second SGEMM kernel: asynchronous copies into a 4-stage shared-memory ring --------------------------
// Same 128 x 128 x 16 block tile and 8 x 8 register tile, but global -> shared copies are cp.async
// operations that bypass the register file, and four stages are in flight (the paper's Pipelining step with
// NUM_STAGES = 4).  Both operand tiles are kept as S[k][mn] (rows padded by 4 floats): an operand whose
// contiguous index is mn is copied in 16-byte pieces; an operand whose contiguous index is k is transposed on
// the way in by 4-byte copies (the paper's Transpose step without a register round trip).
constexpr int SA_STAGES = 4;
constexpr int SA_PITCH = SG_BM + 4;  // floats per row of a [k][mn] tile
constexpr int SA_TILE_FLOATS = SG_BK * SA_PITCH;
constexpr int SA_SMEM_BYTES = SA_STAGES * 2 * SA_TILE_FLOATS * 4;

__device__ __forceinline__ void cp_async16(float *dst_smem, const float *src) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(float *dst_smem, const float *src) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Copy one 128 (mn) x 16 (k) operand tile into S[k][mn].  KCONTIG: memory is [mn][k].
template <bool KCONTIG>
__device__ __forceinline__ void async_tile(float *S, const float *origin, int64_t pitch, int64_t k0, int tid) {
    if (KCONTIG) {
        const int k = tid % 16, r0 = tid / 16;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = r0 + 16 * i;
            cp_async4(S + k * SA_PITCH + r, origin + (int64_t)r * pitch + k0 + k);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int id = tid + SG_THREADS * i;
            const int r = id / 32, c = (id % 32) * 4;
            cp_async16(S + r * SA_PITCH + c, origin + (k0 + r) * pitch + c);
        }
    }
}

template <bool TA, bool TB, bool PACKED>
__global__ void __launch_bounds__(SG_THREADS, 2)
sgemm_async_kernel(int M, int N, int K, float alpha, const float *__restrict__ A, int64_t lda,
                   const float *__restrict__ B, int64_t ldb, float beta, float *__restrict__ C, int64_t ldc, int tiles_m,
                   int tiles_n, int group, const float *__restrict__ bias, int act, const float *__restrict__ R,
                   int64_t ldr) {
    extern __shared__ __align__(16) float sg_smem[];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    int64_t tm, tn;
    tile_coord(blockIdx.x, tiles_m, tiles_n, group, tm, tn);
    const int64_t m0 = tm * SG_BM, n0 = tn * SG_BN;
    const float *Ag = TA ? A + m0 : A + m0 * lda;   // A stored [k][m] when transposed, else [m][k]
    const float *Bg = TB ? B + n0 * ldb : B + n0;   // B stored [n][k] when transposed, else [k][n]

    auto issue = [&](int kb) {
        float *As = sg_smem + (kb % SA_STAGES) * 2 * SA_TILE_FLOATS;
        float *Bs = As + SA_TILE_FLOATS;
        const int64_t k0 = (int64_t)kb * SG_BK;
        async_tile<!TA>(As, Ag, lda, k0, tid);
        async_tile<TB>(Bs, Bg, ldb, k0, tid);
    };

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    const int nkb = K / SG_BK;
#pragma unroll
    for (int s = 0; s < SA_STAGES - 1; ++s) {
        if (s < nkb) issue(s);
        cp_async_commit();
    }
    for (int kb = 0; kb < nkb; ++kb) {
        cp_async_wait<SA_STAGES - 2>();  // this thread's copies of stage kb have landed
        __syncthreads();                 // everyone's have, and everyone is done with stage kb-1
        if (kb + SA_STAGES - 1 < nkb) issue(kb + SA_STAGES - 1);
        cp_async_commit();
        const float *As = sg_smem + (kb % SA_STAGES) * 2 * SA_TILE_FLOATS;
        const float *Bs = As + SA_TILE_FLOATS;
#pragma unroll
        for (int k = 0; k < SG_BK; ++k) {
            float a[8], b[8];
            *reinterpret_cast<float4 *>(&a[0]) = *reinterpret_cast<const float4 *>(As + k * SA_PITCH + ty * 4);
            *reinterpret_cast<float4 *>(&a[4]) = *reinterpret_cast<const float4 *>(As + k * SA_PITCH + ty * 4 + 64);
            *reinterpret_cast<float4 *>(&b[0]) = *reinterpret_cast<const float4 *>(Bs + k * SA_PITCH + tx * 4);
            *reinterpret_cast<float4 *>(&b[4]) = *reinterpret_cast<const float4 *>(Bs + k * SA_PITCH + tx * 4 + 64);
            if (PACKED) {
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
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
        }
    }
    cp_async_wait<0>();

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t m = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float4 *dst = reinterpret_cast<float4 *>(C + m * ldc + n0 + tx * 4 + h * 64);
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (beta != 0.0f) o = *dst;
            float4 r;
            const int64_t n = n0 + tx * 4 + h * 64;
            r.x = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 0], beta, o.x), bias, n + 0, act);
            r.y = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 1], beta, o.y), bias, n + 1, act);
            r.z = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 2], beta, o.z), bias, n + 2, act);
            r.w = finish_f32(epilogue_f32(alpha, acc[i][4 * h + 3], beta, o.w), bias, n + 3, act);
            if (R) {
                const float4 q = *reinterpret_cast<const float4 *>(R + m * ldr + n);
                r.x += q.x; r.y += q.y; r.z += q.z; r.w += q.w;
            }
            *dst = r;
        }
    }
}

template <bool TA, bool TB, bool PACKED> int run_sgemm_async(const GemmArgs &g) {
    auto kernel = sgemm_async_kernel<TA, TB, PACKED>;
    static PerDeviceOnce attr_once;  // once per device, not per process
    const cudaError_t attr_err = attr_once.run(current_device(), [&] {
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SA_SMEM_BYTES);
    });
    if (attr_err != cudaSuccess) { set_cuda_error(attr_err); return PEAK_ERR_CUDA; }
    const int tiles_m = (int)(g.M / SG_BM), tiles_n = (int)(g.N / SG_BN);
    const int group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : 8;
    kernel<<<(unsigned)(tiles_m * tiles_n), SG_THREADS, SA_SMEM_BYTES, g.stream>>>(
        (int)g.M, (int)g.N, (int)g.K, g.alpha, (const float *)g.A, g.lda, (const float *)g.B, g.ldb, g.beta,
        (float *)g.C, g.ldc, tiles_m, tiles_n, group, g.bias, g.act, (const float *)g.R, g.ldr);
    count_launch();
    note_kernel("sgemm_async_kernel<%d, %d, %d> grid=%d", (int)TA, (int)TB, (int)PACKED, tiles_m * tiles_n);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

template <bool PACKED> int dispatch_sgemm_async(const GemmArgs &g) {
    if (g.transA) return g.transB ? run_sgemm_async<true, true, PACKED>(g) : run_sgemm_async<true, false, PACKED>(g);
    return g.transB ? run_sgemm_async<false, true, PACKED>(g) : run_sgemm_async<false, false, PACKED>(g);
}

template <bool TA, bool TB> int run_sgemm(const GemmArgs &g) {
    const int tiles_m = (int)(g.M / SG_BM), tiles_n = (int)(g.N / SG_BN);
    const int group = tuning(PEAK_TUNE_RASTER_GROUP) > 0 ? tuning(PEAK_TUNE_RASTER_GROUP) : 8;
    if (tuning(PEAK_TUNE_SGEMM_FMA) == 1)
        sgemm_kernel<TA, TB, false><<<(unsigned)(tiles_m * tiles_n), SG_THREADS, 0, g.stream>>>(
            (int)g.M, (int)g.N, (int)g.K, g.alpha, (const float *)g.A, g.lda, (const float *)g.B, g.ldb, g.beta,
            (float *)g.C, g.ldc, tiles_m, tiles_n, group, g.bias, g.act, (const float *)g.R, g.ldr);
    else
        sgemm_kernel<TA, TB, true><<<(unsigned)(tiles_m * tiles_n), SG_THREADS, 0, g.stream>>>(
            (int)g.M, (int)g.N, (int)g.K, g.alpha, (const float *)g.A, g.lda, (const float *)g.B, g.ldb, g.beta,
            (float *)g.C, g.ldc, tiles_m, tiles_n, group, g.bias, g.act, (const float *)g.R, g.ldr);
    count_launch();
    note_kernel("sgemm_kernel<%d, %d, %d> grid=%d", (int)TA, (int)TB, (int)(tuning(PEAK_TUNE_SGEMM_FMA) != 1),
                tiles_m * tiles_n);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_cuda_error(e); return PEAK_ERR_CUDA; }
    return PEAK_OK;
}

}  // namespace

// The earlier kernels (block-wide barriers, no edge handling): whole 128 x 128 x 16 tiles only.
static bool sgemm_aligned_supports(const GemmArgs &g) {
    if (g.dtype != PEAK_F32_F32) return false;
    if (g.M < SG_BM || g.N < SG_BN || g.K < SG_BK) return false;
    if (g.M % SG_BM || g.N % SG_BN || g.K % SG_BK) return false;
    if (g.M >= (1ll << 31) || g.N >= (1ll << 31) || g.K >= (1ll << 31)) return false;
    if ((g.M / SG_BM) * (g.N / SG_BN) >= (1ll << 31)) return false;
    if (g.lda % 4 || g.ldb % 4 || g.ldc % 4) return false;
    if (reinterpret_cast<uintptr_t>(g.A) % 16 || reinterpret_cast<uintptr_t>(g.B) % 16 ||
        reinterpret_cast<uintptr_t>(g.C) % 16)
        return false;
    if (g.R && (reinterpret_cast<uintptr_t>(g.R) % 16 || g.ldr % 4)) return false;  // read in 16-byte pieces
    return true;
}

bool sgemm_supports(const GemmArgs &g) { return sgemm_tma_supports(g) || sgemm_aligned_supports(g); }

int launch_sgemm(const GemmArgs &g) {
    if (!sgemm_supports(g)) return PEAK_ERR_UNSUPPORTED;
    // Default: the TMA-fed kernel (any shape).  PEAK_TUNE_SGEMM_COPY = 1 / 2 selects the earlier kernels for
    // A/B measurements, on shapes made of whole tiles: 1 = tiles staged through registers, 2 = cp.async ring.
    // With B transposed (k-contiguous rows of B, sixteen different ones per warp) the TMA-fed kernel is slower
    // than the earlier kernels (4096^3: NT 34 against 53, TT 43 against 57 TFLOP/s), so whole-tile shapes of
    // those layouts stay on them; PEAK_TUNE_SGEMM_COPY = 3 forces the TMA-fed kernel.
    const int copy = tuning(PEAK_TUNE_SGEMM_COPY);
    const bool aligned = sgemm_aligned_supports(g);
    // (... unless B is large enough against M to be transposed first, after which the TMA-fed kernel reads dense
    // tiles and is the fastest for every layout)
    const bool b_gets_transposed = g.transB && tuning(PEAK_TUNE_SGEMM_TRANSPOSE) != 1 &&
                                   (tuning(PEAK_TUNE_SGEMM_TRANSPOSE) == 2 || (g.M >= 2048 && g.N >= 512)) &&
                                   g.N * g.K * 4 <= (512ll << 20);
    // (... or the grid is too small for whole tiles: the TMA-fed path cuts such problems along k, after transposing B)
    const int64_t tiles = ((g.M + 127) / 128) * ((g.N + 127) / 128);
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool small_grid = tiles < 2 * (int64_t)sms && tuning(PEAK_TUNE_SGEMM_TRANSPOSE) != 1;
    const bool want_tma = copy == 3 || !aligned || (copy == 0 && (!g.transB || b_gets_transposed || small_grid));
    if (want_tma && sgemm_tma_supports(g)) return launch_sgemm_tma(g);
    if (!aligned) return PEAK_ERR_UNSUPPORTED;
    const bool both_k_contiguous = !g.transA && g.transB;
    if (copy == 2 || (copy == 0 && !both_k_contiguous))
        return tuning(PEAK_TUNE_SGEMM_FMA) != 1 ? dispatch_sgemm_async<true>(g) : dispatch_sgemm_async<false>(g);
    if (g.transA) return g.transB ? run_sgemm<true, true>(g) : run_sgemm<true, false>(g);
    return g.transB ? run_sgemm<false, true>(g) : run_sgemm<false, false>(g);
}

}  // namespace peak
