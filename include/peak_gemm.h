/*
 * peak_gemm.h -- C ABI of the B200 (sm_100a) dense GEMM library.
 *
 * The operation is the matrix multiplication the PEAK paper optimises
 * (section 2.2, "Matrix Multiplication": A is m x k, B is k x n, C = A x B,
 * all matrices row-major, elements stored as fp32 or fp16), widened to the
 * BLAS form
 *
 *     C = alpha * op(A) * op(B) + beta * C
 *
 * over ROW-MAJOR storage.  alpha, beta, op(), leading dimensions and bfloat16
 * are additions with the reference-BLAS meaning; the paper has C = A x B only.
 *
 * Layout.  op(A) is M x K, op(B) is K x N, C is M x N.
 *     transA == 0 : A is stored M x K,  op(A)(i,k) = A[i*lda + k],  lda >= K
 *     transA == 1 : A is stored K x M,  op(A)(i,k) = A[k*lda + i],  lda >= M
 *     transB == 0 : B is stored K x N,  op(B)(k,j) = B[k*ldb + j],  ldb >= N
 *     transB == 1 : B is stored N x K,  op(B)(k,j) = B[j*ldb + k],  ldb >= K
 *     C(i,j) = C[i*ldc + j],  ldc >= N
 * Leading dimensions count elements, not bytes.  "NT" therefore means weights
 * stored N x K (the usual linear-layer layout), "TN" means A stored K x M.
 *
 * Arithmetic.  Products of the stored values are accumulated in fp32 (tensor
 * cores with fp32 accumulators for 16-bit inputs; fp32 FMA on the CUDA cores,
 * never TF32, for fp32 inputs), in an unspecified order.  The epilogue forms
 * alpha*acc (+ beta*C_old when beta != 0) in fp32 and rounds once, to nearest
 * even, to the output type.
 *
 * Ownership and asynchrony.  Unless stated otherwise A, B, C are DEVICE
 * pointers owned by the caller; the call enqueues work on `stream` (a
 * cudaStream_t passed as void*, NULL = the default stream) and returns without
 * synchronising.  C must not overlap A or B.  C is read only when beta != 0.
 *
 * Quick returns (reference-BLAS convention; the paper is silent):
 *     M == 0 or N == 0        -> nothing is touched
 *     K == 0 or alpha == 0    -> C = beta*C; A and B are not read
 *     beta == 0               -> C is not read (NaN in it does not propagate)
 *     alpha == 0 and beta == 1-> C is left bit-for-bit unchanged
 *
 * Errors.  Every entry point returns PEAK_OK or a positive peak_status_t.
 * Arguments are validated before anything is launched; on an error nothing is
 * written.  No entry point throws or aborts.
 */
#ifndef PEAK_GEMM_H
#define PEAK_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* (input, output) storage types.  Accumulation is always fp32. */
typedef enum peak_dtype {
    PEAK_F16_F32 = 0,   /* A, B binary16; C binary32 */
    PEAK_BF16_BF16 = 1, /* A, B bfloat16; C bfloat16 */
    PEAK_F32_F32 = 2,   /* A, B, C binary32 (CUDA-core SGEMM, no TF32) */
    PEAK_F16_F16 = 3,   /* A, B, C binary16 */
    PEAK_BF16_F32 = 4,  /* A, B bfloat16; C binary32 */
    /* 8-bit float inputs (the paper names fp8 only as an existing GPU type, section 2.1): E4M3 is the "fn"
       flavour (no infinities, one NaN pattern, largest value 448), E5M2 the IEEE-style one. */
    PEAK_E4M3_BF16 = 5, /* A, B E4M3; C bfloat16 */
    PEAK_E4M3_F32 = 6,  /* A, B E4M3; C binary32 */
    PEAK_E5M2_BF16 = 7, /* A, B E5M2; C bfloat16 */
    PEAK_E5M2_F32 = 8   /* A, B E5M2; C binary32 */
} peak_dtype_t;

typedef enum peak_status {
    PEAK_OK = 0,
    PEAK_ERR_INVALID_VALUE = 1, /* unknown dtype / trans, negative size, ld too small, null pointer */
    PEAK_ERR_ARCH = 2,          /* the current device is not compute capability 10.x */
    PEAK_ERR_CUDA = 3,          /* a CUDA runtime / driver call failed; see peak_last_cuda_error() */
    PEAK_ERR_UNSUPPORTED = 4,   /* the forced variant cannot run this problem */
    PEAK_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up; reported by peak_check() */
    PEAK_ERR_NO_MEMORY = 6,     /* staging or workspace memory could not be allocated */
    PEAK_ERR_WORKSPACE_TOO_SMALL = 7 /* peak_gemm_static_ws: the partial tiles do not fit the fixed workspace */
} peak_status_t;

/* Activation of the fused epilogue. */
typedef enum peak_activation {
    PEAK_ACT_NONE = 0,
    PEAK_ACT_RELU = 1, /* max(x, 0) */
    PEAK_ACT_GELU = 2  /* 0.5 x (1 + erf(x / sqrt 2)) */
} peak_activation_t;

/* Kernel families.  PEAK_VARIANT_AUTO lets the dispatcher choose. */
typedef enum peak_variant {
    PEAK_VARIANT_AUTO = 0,
    PEAK_VARIANT_FALLBACK = 1, /* plain tiled CUDA-core kernel: any dtype, layout, alignment (the paper's naive
                                  kernel of section 2.2 with thread-block tiling) */
    PEAK_VARIANT_UMMA_1CTA = 2, /* tcgen05.mma, 128 x (256|128) tile per CTA, TMA ring, persistent, optional
                                   split-K (16-bit inputs) */
    PEAK_VARIANT_UMMA_2CTA = 3, /* tcgen05.mma cta_group::2, 256 x (256|128) tile per CTA pair (16-bit inputs) */
    PEAK_VARIANT_SGEMM = 4,     /* register-tiled fp32 FMA kernel (fp32 inputs) */
    PEAK_VARIANT_SCALE = 5,     /* C = beta*C only (K == 0 or alpha == 0) */
    PEAK_VARIANT_NONE = 6       /* nothing to do (M == 0 or N == 0, or alpha == 0 and beta == 1) */
} peak_variant_t;

/*
 * peak_gemm: C = alpha*op(A)*op(B) + beta*C on the current device (paper section 2.2, widened as above).
 *   dtype          a peak_dtype_t
 *   transA/transB  0 or 1, meaning as in the layout table above
 *   M, N, K        >= 0
 *   alpha, beta    host fp32 scalars, by value
 *   A, B, C        device pointers (may be NULL only where the matrix is empty or not read)
 *   lda, ldb, ldc  row pitches in elements
 *   stream         cudaStream_t
 * The fastest variant whose preconditions hold is chosen: the tensor-core path needs 16-byte aligned
 * base pointers and row pitches that are multiples of 16 bytes (all four layouts, for 16-bit and 8-bit
 * inputs alike); anything else runs on the fallback kernel with the same result contract.  Returns after
 * enqueueing; never synchronises.
 */
int peak_gemm(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
              int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, void *stream);

/*
 * peak_gemm_variant: as peak_gemm, but runs the named kernel family (a peak_variant_t) or fails with
 * PEAK_ERR_UNSUPPORTED when that family cannot run the problem.  Quick returns still apply.  For tests,
 * A/B measurements and tuning (the paper's "tuning parameters", section 3.1).
 */
int peak_gemm_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                      const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc,
                      void *stream);

/*
 * peak_gemm_fused: GEMM with a fused epilogue tail,
 *     C = act( alpha*op(A)*op(B) + beta*C + bias ),   bias broadcast down the rows (one value per column).
 * The paper builds its kernels incrementally so that neighbouring operations can be fused into them
 * (sections 1 and 3.2); this is that fusion for the two operations that follow a linear layer.
 *   bias        device pointer to N fp32 values, or NULL for none
 *   activation  a peak_activation_t
 * Everything else is as for peak_gemm: same kernels, layouts, quick returns (with K == 0 or alpha == 0 the
 * result is act(beta*C + bias)), asynchrony and errors.  The sum alpha*acc + beta*C + bias and the activation
 * are evaluated in fp32 (erff for GELU) and rounded once to the output type.
 * peak_gemm_fused_variant additionally names the kernel family, like peak_gemm_variant.
 */
int peak_gemm_fused(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                    int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, const float *bias,
                    int activation, void *stream);
int peak_gemm_fused_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K,
                            float alpha, const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C,
                            int64_t ldc, const float *bias, int activation, void *stream);

/*
 * peak_gemm_fused_residual: the fused tail with a residual operand,
 *     C = act( alpha*op(A)*op(B) + beta*C + bias ) + R,
 * the third operation that commonly follows a linear layer (a skip connection); like bias and activation it
 * is fused into the producing kernel's epilogue instead of costing another pass over C (paper sections 1 and
 * 3.2 on fusing neighbouring operations).
 *   R    device pointer to an M x N row-major matrix of the OUTPUT storage type of `dtype`, or NULL for none
 *   ldr  row pitch of R in elements, >= N when R is given
 * R is only read; it must not overlap C (with R == C the result is unspecified: use beta instead).  The
 * residual is converted to fp32 and added after the activation; the sum is rounded once to the output type.
 * R may have any alignment (16-byte aligned bases and pitches are read with vector loads).  Everything else
 * -- kernels, layouts, quick returns (K == 0 or alpha == 0: C = act(beta*C + bias) + R), asynchrony, errors --
 * is as for peak_gemm_fused.  The _variant form names the kernel family.
 */
int peak_gemm_fused_residual(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                             const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C,
                             int64_t ldc, const float *bias, int activation, const void *R, int64_t ldr,
                             void *stream);
int peak_gemm_fused_residual_variant(int variant, int dtype, int transA, int transB, int64_t M, int64_t N,
                                     int64_t K, float alpha, const void *A, int64_t lda, const void *B,
                                     int64_t ldb, float beta, void *C, int64_t ldc, const float *bias,
                                     int activation, const void *R, int64_t ldr, void *stream);

/*
 * peak_gemm_strided_batched: `batch` independent GEMMs of one shape,
 *     C_b = alpha * op(A_b) * op(B_b) + beta * C_b,   X_b = X + b * strideX   (strides in elements),
 * the second half of the paper's fusion / specialisation motive (sections 1, 3.1: kernels are specialised
 * to the shapes of a workload, and attention-style workloads are batches of small GEMMs).
 * Arguments are those of peak_gemm plus the three strides and the batch count.  strideA and strideB may be 0
 * (the same matrix for every b); the C matrices must not overlap (strideC >= (M-1)*ldc + N, else
 * PEAK_ERR_INVALID_VALUE).  batch == 0 does nothing.  On the tensor-core path the whole batch is ONE launch
 * of the persistent kernel (tiles are numbered across the batch; the batch index is the third coordinate of
 * the TMA descriptors), which needs strideA and strideB to be positive multiples of 8 elements; any other
 * case runs one launch per matrix with the kernel peak_gemm would choose.
 */
int peak_gemm_strided_batched(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                              const void *A, int64_t lda, int64_t strideA, const void *B, int64_t ldb,
                              int64_t strideB, float beta, void *C, int64_t ldc, int64_t strideC, int64_t batch,
                              void *stream);

/*
 * peak_gemm_host: the same operation on HOST buffers (the paper's "driver", section 3.1: allocate,
 * copy in, run, copy out).  A, B, C are host pointers (pinned memory makes the copies faster but is
 * not required).  Copies A and B (and C when beta != 0) to device staging buffers, runs peak_gemm,
 * copies C back, and synchronises `stream` before returning.  From 1024 rows on the work is cut into up to
 * eight row panels of op(A) and C: panel i + 1 is copied in and panel i - 1 copied out (two internal
 * streams, ordered against `stream` by events) while panel i is multiplied on `stream`.  The staging buffers are owned by the
 * library, grow on demand and are reused by later calls; peak_release_staging() frees them.
 * Not thread-safe with respect to other peak_gemm_host calls.
 */
int peak_gemm_host(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha, const void *A,
                   int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc, void *stream);
int peak_release_staging(void);

/*
 * peak_gemm_xcheck_f64: cross-check kernel.  Writes the UNROUNDED fp64 value
 *     alpha * sum_k op(A)(i,k)*op(B)(k,j) + beta * C0(i,j)       (fp64 accumulation, k ascending)
 * to Cref[i*ldcref + j] (device pointer, double).  C0 (device, output type of `dtype`) is read only when
 * beta != 0 and is never written.  One thread per output element, as in the paper's naive kernel
 * (section 2.2); slow, meant for full-matrix verification at sizes the CPU cannot cover.
 */
int peak_gemm_xcheck_f64(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                         const void *A, int64_t lda, const void *B, int64_t ldb, float beta, const void *C0,
                         int64_t ldc, double *Cref, int64_t ldcref, void *stream);

/*
 * peak_gemm_static_ws: split-K GEMM that allocates nothing.  (The paper has no counterpart: this entry
 * point exists for callers, not for the method.)
 *
 * Who needs it: code that must not, or cannot, allocate device memory when it calls a GEMM -- a serving loop
 * that has handed all free HBM to its own pools, a process whose memory is accounted for up front, a
 * latency-critical path where an allocator call (which may take a lock or synchronise) is not acceptable.
 * The ordinary split-K path of peak_gemm takes its fp32 partial tiles from a stream-ordered memory pool;
 * this one keeps them in a fixed array that is part of the library image: peak_static_ws_bytes() bytes
 * (32 MiB), held by every GPU that loads the library for as long as the process lives.
 *
 * Same operation, arguments, layout rules and epilogue as peak_gemm, for 16-bit inputs only, with K cut
 * into `splits` slices (2 <= splits <= 64; every slice must get at least one 64-wide k-block) computed by
 * 128 x 128 tensor-core tiles; the slices are added in slice order by a second kernel, so results are
 * reproducible run to run.  A, B, C are device pointers; A and B need 16-byte aligned bases and pitches
 * that are multiples of 8 elements (else PEAK_ERR_UNSUPPORTED).  Enqueues two kernels on `stream` and
 * returns without synchronising.
 *
 * Limit: roundup(M,128) * roundup(N,128) * splits * 4 bytes must not exceed peak_static_ws_bytes();
 * otherwise PEAK_ERR_WORKSPACE_TOO_SMALL is returned and nothing is launched.
 *
 * Makes no cudaMalloc / cudaFree / pool call and calls no allocating library routine.  The first call on
 * each device looks up the array's device address (cudaGetSymbolAddress, cached per device); make that first
 * call outside any stream capture.  All calls share the one array, and it keeps whatever the previous call
 * left there; nothing in it needs clearing, because every cell the reduction reads is written by the
 * tile kernel of the same call first.  Two calls that overlap on the GPU (different streams, no ordering
 * between them) would overwrite each other's partial tiles: order them.
 */
int peak_gemm_static_ws(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                        const void *A, int64_t lda, const void *B, int64_t ldb, float beta, void *C, int64_t ldc,
                        int splits, void *stream);
size_t peak_static_ws_bytes(void);

/*
 * peak_query_variant: which kernel family peak_gemm would run for these arguments (a peak_variant_t),
 * or a negative peak_status_t when they are invalid.  Pure host logic: touches no device.
 */
int peak_query_variant(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float alpha,
                       const void *A, int64_t lda, const void *B, int64_t ldb, float beta, const void *C,
                       int64_t ldc);

/*
 * peak_tile_coord: the persistent scheduler's map from a linear tile index to tile coordinates
 * (block swizzle of the paper's optimisation sequences, section 4.3): tiles are visited in groups of
 * `group` tile-rows, walking down the rows of a group before moving to the next tile-column, so that
 * CTAs running at the same time share A and B panels in L2.  Host copy of the device function, for
 * tests.  Returns PEAK_ERR_INVALID_VALUE if tile is outside [0, tiles_m*tiles_n).
 */
int peak_tile_coord(int64_t tile, int64_t tiles_m, int64_t tiles_n, int64_t group, int64_t *tile_m,
                    int64_t *tile_n);

/*
 * peak_check: synchronises `stream`, then reads and clears the device status word that kernels set
 * when a bounded wait (on an mbarrier) gives up.  Returns PEAK_OK, PEAK_ERR_TIMEOUT or PEAK_ERR_CUDA.
 * `detail`, if not NULL, receives the raw status word (role and barrier that gave up).
 * There is ONE status word per device, not one per stream: a wait that gave up in a kernel on any stream of
 * the current device is reported to whichever caller checks first, and the read clears it.  A process that
 * runs GEMMs on several streams and wants to attribute a timeout should check after each stream's work, or
 * treat a report as "some call on this device since the last check".  (The paper's validators, section 3.3,
 * check results after a run; this is the run-time half: a stuck pipeline is reported, never a hang.)
 */
int peak_check(void *stream, uint32_t *detail);

/*
 * peak_set_tuning: performance knobs that never change results (the paper's "tuning parameters",
 * section 3.1).  value 0 restores the library default.  Process-wide; returns PEAK_ERR_INVALID_VALUE for an
 * unknown key or a negative value.
 */
typedef enum peak_tuning_key {
    PEAK_TUNE_RASTER_GROUP = 0, /* tile-rows per raster group of the persistent scheduler */
    PEAK_TUNE_TILE_N = 1,       /* tensor-core tile width: 128, 256, or (CTA pairs only) 512 */
    PEAK_TUNE_SPLIT_K = 2,      /* k-slices per tile (1 = never split; capped by the number of k-blocks) */
    PEAK_TUNE_EPILOGUE = 3,     /* 1 = direct global stores, 2 = shared-memory staging + TMA stores (with beta != 0
                                   old C arrives by TMA too), 3 = TMA stores but per-thread loads of old C */
    PEAK_TUNE_SGEMM_FMA = 4,    /* SGEMM inner product: 1 = scalar fp32 FMA, 2 = two-wide fp32 FMA (default) */
    PEAK_TUNE_TAIL_SPLIT = 5,   /* 2 = split the tiles of the last, partly filled wave whenever possible (off by default) */
    PEAK_TUNE_DEPENDENT_LAUNCH = 6, /* 1 = launch the tensor-core kernel without programmatic dependent launch */
    PEAK_TUNE_SGEMM_COPY = 7,   /* SGEMM tile loads: 1 = staged through registers, 2 = cp.async ring (both: whole
                                   128 x 128 x 16 tiles only), 3 = TMA + mbarrier ring (any shape; the default
                                   except for whole-tile problems with B transposed) */
    PEAK_TUNE_WAIT_MS = 8,      /* budget of each device-side barrier wait in ms at 2 GHz (default 2000) */
    PEAK_TUNE_INJECT_STALL = 9, /* test hook, 1 = one CTA leaves one pipeline stage unfilled so that the bounded
                                   waits run out: the call's result is then wrong by design and peak_check()
                                   reports PEAK_ERR_TIMEOUT; nothing hangs and the context stays usable */
    PEAK_TUNE_MULTICAST = 10,   /* cluster-multicast plug-in: 1 = never use it, 2 = use it whenever it can run */
    PEAK_TUNE_BALANCED_GRID = 11, /* 1 = always launch one CTA (pair) per SM instead of the fewest that give the
                                     same number of waves */
    PEAK_TUNE_EPILOGUE_WARPS = 12, /* one-slot (128- / 256-wide) tiles: 1 = one group of four epilogue warps, 2 = two
                                      groups that drain half of the columns each (default: two for problems of at
                                      most two waves and for tiles of at most eight k-blocks; in a strided batch only
                                      the single-CTA 256-wide tiles of such short-k problems have the second form) */
    PEAK_TUNE_K_ORDER = 13,     /* tensor-core kernels: 1 = every tile walks its k-blocks upwards, 2 = every other tile
                                   of a CTA walks them downwards, so that a wave of tiles starts in the k-range the
                                   previous wave left in L2 (default: 2 for 512-wide tiles, 1 otherwise) */
    PEAK_TUNE_SWAP_AB = 14,     /* problems with M <= 64 (single-CTA tiles, 16-bit inputs): computed as C^T = op(B)^T
                                   op(A)^T, so that M is the narrow side of the tensor-core tile, when set to 2
                                   (default: off -- it measured slower than the plain tiles on B200) */
    PEAK_TUNE_SGEMM_TRANSPOSE = 15, /* SGEMM: an operand whose contiguous index is k (A not transposed, B transposed) is
                                       first copied, transposed, into pool memory so that the kernel reads dense tiles;
                                       1 = never, 2 = always (default: when the other dimension is at least 2048 and
                                       the copy is at most 512 MiB) */
    PEAK_TUNE_SHORT_A = 16,     /* single-CTA tiles of problems with M < 128: 1 = always fetch all 128 rows of the A tile
                                   (default: only the rows that exist, which saves copy-engine requests) */
    PEAK_TUNE_CLUSTER_K = 17,   /* a single matrix on single-CTA tiles whose every tile is split 2 or 4 ways: 1 = partial tiles
                                   through the workspace and a reduction kernel (default: the slices run on the CTAs of
                                   a cluster and are added through distributed shared memory, one launch; one-wave problems
                                   of whole 128-wide tiles run the same one-tile-per-CTA kernel); 2 = as default, but
                                   the slices always travel by bulk copies (default: plain remote stores for tiles of
                                   at most 32 rows); 3 = whole tiles never as CTA-pair tiles on the one-tile kernel (256 x 128, or one wave of 256 x 256); 4 = as pair tiles
                                   whenever possible (default: from 32 k-blocks on) */
    PEAK_TUNE_SHARE = 18,       /* single-GPU plug-in, 16-bit inputs: single-CTA tiles in clusters of CM x CN tiles that share
                                   their A / B tiles by multicast copies: 1 = never, 100 * w + 10 * CM + CN (w = 1: 128-wide
                                   tiles, 2: 256-wide) = that cluster shape whenever the plug-in is present */
    PEAK_TUNE_NARROW = 19,      /* CTA-pair tiles of 192 / 384 columns on the 256- / 512-wide kernels (B transposed, whole tiles),
                                   chosen where they fill one wave instead of starting a nearly empty second one: 1 = never.
                                   PEAK_TUNE_TILE_N = 192 / 384 forces them */
    PEAK_TUNE_COUNT_ = 20
} peak_tuning_key_t;
int peak_set_tuning(int key, int value);

/*
 * Persisted tuning table (the paper's performance evaluator, section 3.3 -- enumerate the tuning-parameter
 * combinations, prune, keep the best -- with its result kept in a file).  `python -m paper_2512_19018_b200.tune
 * --sweep` times the candidates for each benchmark shape class and writes tuned_sm100.json; the library reads
 * that file (beside the shared object, or the file named by the environment variable PEAK_TUNED_TABLE; the
 * values "off", "0" and "none" disable the table) on first use.  For a problem of the same types, layout and
 * beta class (zero / non-zero) whose M, N and K each lie within a factor sqrt(2) of an entry's, the entry's
 * kernel family and knob values replace the dispatcher's built-in rules; knobs set through peak_set_tuning
 * still win, and results never depend on any of this.
 *   peak_tuned_table_load     replaces the table with the file at `path` (host string); NULL or "" empties it.
 *                             Returns the number of entries, -1 if the file is not understood, -2 if it
 *                             cannot be opened (the current table then stays).
 *   peak_tuned_table_entries  entries in the table now (loads the default file on first use).
 *   peak_tuned_lookup         1 and the entry's family (`variant`, 0 = none named) and knob values (`knobs`,
 *                             PEAK_TUNE_COUNT_ ints) when an entry covers the problem, else 0.  Host only.
 */
int peak_tuned_table_load(const char *path);
int peak_tuned_table_entries(void);
int peak_tuned_lookup(int dtype, int transA, int transB, int64_t M, int64_t N, int64_t K, float beta, int *variant,
                      int *knobs);

/*
 * peak_multicast_available: 1 when the optional single-GPU plug-in (libpeak_gemm_mc.so, beside the main
 * library) is present and loaded.  It runs large 16-bit GEMMs with clusters of four CTAs that share B tiles
 * through TMA multicast (the paper's thread-block tiling taken one level up: a cluster-level tile); results
 * and the call contract are the same with and without it.
 */
int peak_multicast_available(void);

/* Number of kernels this library has launched in this process (all entry points). */
int64_t peak_kernel_launches(void);

/* The cudaError_t of the most recent failing CUDA call made by this thread's last entry-point call. */
int peak_last_cuda_error(void);

/*
 * peak_last_kernel: which kernel this host thread's most recent GEMM call launched, and with which launch
 * configuration, as text: the kernel's name with its template arguments, written the way profilers print
 * it, followed by key=value pairs (grid, work items, k-slices, ...).  The paper's performance evaluator
 * (section 3.3) records which candidate produced a measurement; this is that record for a dispatcher that
 * chooses among kernels by shape.  `buf` (host) receives at most len - 1 characters and a terminator; the
 * text is empty before the first launch.  Returns PEAK_OK, or PEAK_ERR_INVALID_VALUE for a null buffer.
 */
int peak_last_kernel(char *buf, size_t len);

/*
 * peak_selftest_per_device_once: host-only self-check of the library's once-per-device bookkeeping (a
 * kernel's shared-memory attribute and similar context state are set the first time EACH device runs a
 * kernel, not once per process).  Touches no device.  Returns 0, or the number of the failed check.  (No
 * counterpart in the paper: test support.)
 */
int peak_selftest_per_device_once(void);

const char *peak_status_string(int status);
const char *peak_variant_string(int variant);
int peak_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PEAK_GEMM_H */
